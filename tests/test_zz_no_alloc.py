"""The allocation-free contract entry against the ordinary one.

``pamm_contract_no_alloc`` serves callers that cannot allocate device memory at
the point of the call (no cudaMalloc allowed by their host application, or no
tolerance for its device-wide synchronisation); its scratch is a fixed array in
the library that every call shares and that keeps the previous call's contents.
The check is therefore made on two calls in a row with different inputs: the
second must not be disturbed by what the first left behind.  Collected last on
purpose, so a failure here cannot hide the other tests' results under ``-x``."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2506_02939_b200 import build as pamm_build, synth

pamm_build.build()
from paper_2506_02939_b200 import pamm  # noqa: E402
from tests import parity  # noqa: E402

pytestmark = pytest.mark.gpu

TOL = {"f32": 1e-5, "bf16": 1e-2}     # the relative Frobenius tolerances of the parity tests


def _inputs(b, m, k, dtype, seed):
    rng = np.random.default_rng(seed)
    _, dY = synth.random_case(b, 8, m, dtype, seed=seed, dy_scale=1e-3)
    f = rng.integers(0, k, size=b).astype(np.int32)
    f[f == k // 2] = 0                                   # one empty segment, one crowded one
    a = rng.standard_normal(b).astype(np.float32)
    return torch.from_numpy(f).cuda(), torch.from_numpy(a).cuda(), parity.to_device(dY)


def test_no_alloc_contract_matches_contract_on_two_calls_in_a_row():
    cases = [(3000, 520, 48, "bf16", 31), (1777, 264, 20, "f32", 32)]
    for b, m, k, dtype, seed in cases:
        f, a, dY = _inputs(b, m, k, dtype, seed)
        ref = pamm.contract(f, a, dY, k)                                   # caller-provided workspace
        out = pamm.alloc_matrix(k, m, torch.float32)
        out.fill_(float("nan"))
        pamm.contract_no_alloc(f, a, dY, k, out)
        assert pamm.last_device_status() == pamm.OK
        err = parity.rel_fro(out.cpu().numpy(), ref.cpu().numpy().astype(np.float64))
        assert err <= TOL[dtype], (dtype, err)
        assert torch.equal(out, ref)                                       # same kernels, same order: same bits


def test_no_alloc_contract_rejects_what_does_not_fit():
    b, m, k = 65536, 6144, 128                                            # needs about 36 MiB of scratch
    assert pamm.workspace_bytes(pamm.WS_CONTRACT, b, 1, m, k, pamm.BF16) > pamm.NO_ALLOC_SCRATCH_BYTES
    fake = ctypes.c_void_p(0x1000)
    rc = pamm._lib.pamm_contract_no_alloc(fake, fake, fake, m, b, m, pamm.BF16, k, fake, m, None)
    assert rc == pamm.ERR_WORKSPACE
