"""B200-native PAMM hot path (compress / contract / weight-grad) behind a C ABI.

``paper_2506_02939_b200.pamm`` is the binding to the CUDA library and raises at
import when the library has not been built; ``paper_2506_02939_b200.synth``
makes seeded synthetic inputs and needs numpy only.
"""
__all__ = ["pamm", "synth", "autograd"]
