"""Host-side checks of the C ABI: the library loads, exports what the header
declares, validates arguments before touching a GPU, and samples generator
indices uniformly without replacement.  No GPU is used."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest
import torch

from paper_2506_02939_b200 import build as pamm_build

pamm_build.build()
from paper_2506_02939_b200 import pamm  # noqa: E402

HEADER = Path(__file__).resolve().parent.parent / "include" / "pamm.h"


def test_library_exports_every_declared_symbol():
    text = HEADER.read_text()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(pamm_[a-z_0-9]+)\s*\(", text))
    assert len(declared) >= 12
    lib = ctypes.CDLL(str(pamm._LIB_PATH))
    for name in declared:
        assert hasattr(lib, name), f"{name} declared in pamm.h but not exported"
    assert declared == set(pamm.EXPORTED)


def test_version_and_status_strings():
    assert pamm.version() >= 100
    seen = {pamm.status_string(c) for c in range(7)}
    assert len(seen) == 7 and "ok" in seen


def test_saved_bytes_follow_the_papers_count():
    # appendix "Complexity Analysis": k n + 2 b scalars instead of b n
    s = pamm.saved_bytes(65536, 2048, 128, pamm.BF16)
    assert s["scalars_full"] == 65536 * 2048 and s["scalars_pamm"] == 128 * 2048 + 2 * 65536
    assert s["full"] == 65536 * 2048 * 2 and s["pamm"] == 128 * 2048 * 2 + 8 * 65536
    assert abs(s["ratio"] - 256.0) < 1e-9
    narrow = pamm.saved_bytes(65536, 2048, 128, pamm.BF16, pamm.IDX_U8)
    assert narrow["pamm"] == 128 * 2048 * 2 + 5 * 65536
    with pytest.raises(pamm.PammError):
        pamm.saved_bytes(65536, 2048, 300, pamm.BF16, pamm.IDX_U8)      # 300 generators do not fit a byte


def test_workspace_sizes():
    w = pamm.workspace_bytes(pamm.WS_CONTRACT, 65536, 2048, 6144, 128, pamm.BF16)
    assert w % 256 == 0 and 0 < w < 64 << 20
    # grows with k and with m
    assert pamm.workspace_bytes(pamm.WS_CONTRACT, 65536, 2048, 6144, 256, pamm.BF16) > w
    assert pamm.workspace_bytes(pamm.WS_CONTRACT, 65536, 2048, 12288, 128, pamm.BF16) > w
    assert pamm.workspace_bytes(pamm.WS_STEP_HOST, 2048, 512, 1536, 4, pamm.F32) > 2048 * (512 + 1536) * 4
    # the sort products: one count per generator and block of rows, at most one block per SM
    p = pamm.workspace_bytes(pamm.WS_COMPRESS, 65536, 2048, 6144, 128, pamm.BF16)
    assert p % 256 == 0 and 128 * 4 <= p <= 256 * 128 * 4
    with pytest.raises(pamm.PammError):
        pamm.workspace_bytes(pamm.WS_CONTRACT, 16, 8, 8, 17, pamm.F32)     # k > b
    with pytest.raises(pamm.PammError):
        pamm.workspace_bytes(pamm.WS_CONTRACT, 0, 8, 8, 1, pamm.F32)


def _call(fn, *args):
    return getattr(pamm._lib, fn)(*args)


def test_argument_errors_are_synchronous_and_launch_nothing():
    fake = ctypes.c_void_p(0x1000)       # aligned, never dereferenced: checks come first
    odd = ctypes.c_void_p(0x1004)
    null = None
    i = pamm._lib
    # NULL pointers
    assert i.pamm_select_generators(null, 8, 16, 8, pamm.F32, 2, 0, null, fake, fake, 8, fake, null) == pamm.ERR_INVALID_ARG
    # k > b, k < 1
    assert i.pamm_select_generators(fake, 8, 16, 8, pamm.F32, 17, 0, null, fake, fake, 8, fake, null) == pamm.ERR_INVALID_ARG
    assert i.pamm_select_generators(fake, 8, 16, 8, pamm.F32, 0, 0, null, fake, fake, 8, fake, null) == pamm.ERR_INVALID_ARG
    I32, U8 = pamm.IDX_I32, pamm.IDX_U8
    # ld < n and ld not a multiple of 16 bytes
    assert i.pamm_compress(fake, 4, 16, 8, pamm.F32, fake, 8, 2, fake, fake, I32, fake, null, 0, null) == pamm.ERR_INVALID_ARG
    assert i.pamm_compress(fake, 9, 16, 8, pamm.F32, fake, 8, 2, fake, fake, I32, fake, null, 0, null) == pamm.ERR_INVALID_ARG
    assert i.pamm_compress(fake, 12, 16, 8, pamm.BF16, fake, 8, 2, fake, fake, I32, fake, null, 0, null) == pamm.ERR_INVALID_ARG
    # misaligned base pointer
    assert i.pamm_compress(odd, 8, 16, 8, pamm.F32, fake, 8, 2, fake, fake, I32, fake, null, 0, null) == pamm.ERR_INVALID_ARG
    # unknown dtype, unknown storage type of f
    assert i.pamm_compress(fake, 8, 16, 8, 7, fake, 8, 2, fake, fake, I32, fake, null, 0, null) == pamm.ERR_UNSUPPORTED
    assert i.pamm_compress(fake, 8, 16, 8, pamm.F32, fake, 8, 2, fake, fake, 9, fake, null, 0, null) == pamm.ERR_UNSUPPORTED
    # more generators than the storage type of f can name
    assert i.pamm_compress(fake, 8, 1000, 8, pamm.F32, fake, 8, 257, fake, fake, U8, fake, null, 0, null) == pamm.ERR_INVALID_ARG
    assert i.pamm_contract(fake, U8, fake, fake, 8, 1000, 8, pamm.F32, 257, fake, 8, null, fake, 1 << 30, null) == pamm.ERR_INVALID_ARG
    # a buffer for the sort products that is too small or misaligned
    assert i.pamm_compress(fake, 8, 16, 8, pamm.F32, fake, 8, 2, fake, fake, I32, fake, fake, 8, null) == pamm.ERR_WORKSPACE
    assert i.pamm_compress(fake, 8, 16, 8, pamm.F32, fake, 8, 2, fake, fake, I32, fake, odd, 1 << 20, null) == pamm.ERR_WORKSPACE
    # contract: missing / small / misaligned workspace
    assert i.pamm_contract(fake, I32, fake, fake, 8, 16, 8, pamm.F32, 2, fake, 8, null, null, 0, null) == pamm.ERR_WORKSPACE
    assert i.pamm_contract(fake, I32, fake, fake, 8, 16, 8, pamm.F32, 2, fake, 8, null, fake, 16, null) == pamm.ERR_WORKSPACE
    assert i.pamm_contract(fake, I32, fake, fake, 8, 16, 8, pamm.F32, 2, fake, 8, null, odd, 1 << 20, null) == pamm.ERR_WORKSPACE
    assert i.pamm_contract(fake, I32, fake, fake, 8, 16, 8, pamm.F32, 2, null, 8, null, fake, 1 << 20, null) == pamm.ERR_INVALID_ARG
    # weight grad: NULL output, bad leading dimension of B~, unknown output type / layout, bf16 accumulate is not offered
    NM, MN = pamm.DW_NM, pamm.DW_MN
    assert i.pamm_weight_grad(fake, 8, 2, 8, pamm.F32, fake, 8, 8, null, 8, pamm.F32, NM, null) == pamm.ERR_INVALID_ARG
    assert i.pamm_weight_grad(fake, 8, 2, 8, pamm.F32, fake, 6, 8, fake, 8, pamm.F32, NM, null) == pamm.ERR_INVALID_ARG
    assert i.pamm_weight_grad(fake, 8, 2, 8, pamm.F32, fake, 8, 8, fake, 8, 5, NM, null) == pamm.ERR_UNSUPPORTED
    assert i.pamm_weight_grad(fake, 8, 2, 8, pamm.F32, fake, 8, 8, fake, 8, pamm.F32, 3, null) == pamm.ERR_UNSUPPORTED
    # the leading dimension of dW counts the columns of the chosen layout: n = 8, m = 24
    assert i.pamm_weight_grad(fake, 8, 2, 8, pamm.F32, fake, 24, 24, fake, 8, pamm.F32, NM, null) == pamm.ERR_INVALID_ARG
    assert i.pamm_weight_grad(fake, 8, 2, 8, pamm.F32, fake, 24, 24, fake, 12, pamm.BF16, MN, null) == pamm.ERR_INVALID_ARG
    # host step: arena too small
    assert i.pamm_qkv_step_host(fake, fake, 16, 8, 8, pamm.F32, 2, 0, fake, null, null, fake, 64, null) == pamm.ERR_WORKSPACE
    # limits
    assert i.pamm_select_generators(fake, 8, 1 << 20, 8, pamm.F32, 50000, 0, null, fake, fake, 8, fake, null) == pamm.ERR_UNSUPPORTED


def test_read_probe_argument_errors():
    i = pamm._lib
    fake, null = ctypes.c_void_p(0x1000), None
    assert i.pamm_probe_read(pamm.PROBE_SUM, null, 4, 64, 64, null, fake, null) == pamm.ERR_INVALID_ARG
    assert i.pamm_probe_read(pamm.PROBE_SUM, fake, 4, 60, 64, null, fake, null) == pamm.ERR_INVALID_ARG       # not whole 16-byte words
    assert i.pamm_probe_read(pamm.PROBE_SUM, fake, 4, 64, 48, null, fake, null) == pamm.ERR_INVALID_ARG       # rows overlap
    assert i.pamm_probe_read(pamm.PROBE_SUM, fake, 4, 64, 64, fake, fake, null) == pamm.ERR_INVALID_ARG       # no order with plain loads
    assert i.pamm_probe_read(pamm.PROBE_ROWS, fake, 4, 32768, 32768, null, fake, null) == pamm.ERR_INVALID_ARG  # row too wide for the ring
    assert i.pamm_probe_read(7, fake, 4, 64, 64, null, fake, null) == pamm.ERR_INVALID_ARG


def test_draw_indices_basic_properties():
    for b, k in [(1, 1), (2, 2), (7, 3), (2048, 4), (65536, 128), (65536, 1024), (100003, 517)]:
        idx = pamm.draw_indices_host(b, k, 42).numpy()
        assert idx.shape == (k,) and idx.min() >= 0 and idx.max() < b
        assert np.all(np.diff(idx) > 0)                        # ascending, hence distinct
        assert np.array_equal(idx, pamm.draw_indices_host(b, k, 42).numpy())
    a = pamm.draw_indices_host(65536, 128, 1).numpy()
    c = pamm.draw_indices_host(65536, 128, 2).numpy()
    assert not np.array_equal(a, c)
    # k = b is the whole range
    assert np.array_equal(pamm.draw_indices_host(1000, 1000, 5).numpy(), np.arange(1000))
    # nested: the k-subset is contained in the 2k-subset drawn with the same seed
    big = set(pamm.draw_indices_host(65536, 256, 1).numpy().tolist())
    assert set(a.tolist()) <= big


def test_draw_indices_uniform_chi_square():
    # every row index should be picked with probability k/b: chi-square over many seeds
    b, k, seeds = 96, 8, 6000
    counts = np.zeros(b)
    pair = np.zeros((b, b))
    for s in range(seeds):
        idx = pamm.draw_indices_host(b, k, s).numpy()
        counts[idx] += 1
        pair[np.ix_(idx, idx)] += 1
    expect = seeds * k / b
    chi2 = float(((counts - expect) ** 2 / expect).sum())
    # dof = 95; mean 95, sd ~13.8 -> 5 sigma
    assert chi2 < 95 + 5 * 13.8, chi2
    # pairs: P(i and j both picked) = k(k-1)/(b(b-1))
    iu = np.triu_indices(b, 1)
    pe = seeds * k * (k - 1) / (b * (b - 1))
    chi2p = float(((pair[iu] - pe) ** 2 / pe).sum())
    dof = len(iu[0]) - 1
    assert chi2p < dof + 6 * np.sqrt(2 * dof), (chi2p, dof)


def test_draw_indices_non_power_of_two_uniform():
    b, k, seeds = 37, 5, 8000
    counts = np.zeros(b)
    for s in range(seeds):
        counts[pamm.draw_indices_host(b, k, 1000 + s).numpy()] += 1
    expect = seeds * k / b
    chi2 = float(((counts - expect) ** 2 / expect).sum())
    assert chi2 < 36 + 5 * np.sqrt(72), chi2


def test_prepared_calls_repeat_one_library_call():
    out = torch.zeros(8, dtype=torch.int32)

    def draw(seed):
        pamm._check(pamm._lib.pamm_draw_indices_host(1000, 8, seed, pamm._ptr(out)), "pamm_draw_indices_host")

    run = pamm.prepared(draw, 11)
    assert torch.all(out == 0)                                  # preparing runs nothing
    run()
    assert torch.equal(out, pamm.draw_indices_host(1000, 8, 11))
    out.zero_()
    run()
    assert torch.equal(out, pamm.draw_indices_host(1000, 8, 11))
    # the call's own allocations stay alive with the callable
    keep_alive = pamm.prepared(pamm.draw_indices_host, 1000, 8, 3)
    keep_alive()
    with pytest.raises(ValueError):
        pamm.prepared(lambda: None)
    bad = pamm.prepared(draw, 11)
    assert pamm._lib is not None and callable(bad)
    failing = pamm.prepared(lambda: pamm._check(pamm._lib.pamm_draw_indices_host(4, 8, 0, pamm._ptr(out)), "draw"))
    with pytest.raises(pamm.PammError):
        failing()                                               # k > b is reported when the call is made
