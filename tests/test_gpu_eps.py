"""Parity of the neighbourhood-condition path (Eq. 2 and the factor beta, Eq. 4-5) against the oracle.

The keep/drop decision is taken in fp32 by the kernels with a stated rounding
allowance of 2 n 2^-24 relative to ||X_i||^2; rows whose true ratio
||X_i - A~_i||^2 / ||X_i||^2 lies within that allowance above eps^2 may fall on
either side and are counted, every other row must agree with the oracle."""
import numpy as np
import pytest
import torch

from oracle import pamm_oracle as orc
from paper_2506_02939_b200 import build as pamm_build, synth

pamm_build.build()
from paper_2506_02939_b200 import pamm  # noqa: E402
from tests import parity  # noqa: E402

pytestmark = pytest.mark.gpu


def run_eps(X, dY, k, eps, seed=5):
    dtype = "bf16" if X.dtype == np.uint16 else "f32"
    tol = parity.TOL[dtype]
    b, n = X.shape
    m = dY.shape[1]
    Xd, dYd = parity.to_device(X), parity.to_device(dY)
    idx, C, invn = pamm.select_generators(Xd, k, seed)
    f, alpha, dropped = pamm.compress_eps(Xd, C, invn, eps)
    Bt = pamm.contract(f, alpha, dYd, k)
    dW = pamm.weight_grad_beta(C, Bt, b, dropped)
    assert pamm.last_device_status() == pamm.OK
    idx_g, f_g, a_g = idx.cpu().numpy(), f.cpu().numpy(), alpha.cpu().numpy()
    eta_g = int(dropped.item())
    Bt_g, dW_g = Bt.cpu().numpy(), dW.cpu().numpy()

    C64, q = orc.gather(X, idx_g)
    f_o, a_o, t1, t2 = orc.compress(X, C64, q)
    rep = parity.Report(b=b, k=k)
    f_e, a_e = parity.check_assignment(X, C64, q, f_g, f_o, a_o, t1, t2, rep)
    assert rep.unexplained == 0
    # the oracle's neighbourhood step on the assignment the GPU used (tolerated near-tie rows overridden)
    a_m, kept_o, err, rn, eta_o, beta_o = orc.neighbourhood(X, C64, f_e, a_e, eps)
    kept_g = ~((a_g == 0.0) & (a_e != 0.0))
    ratio = np.divide(err ** 2, rn ** 2, out=np.zeros_like(err), where=rn > 0)
    slack = 2.0 * n * 2.0 ** -24
    window = (ratio > eps ** 2 - 2 * slack) & (ratio <= eps ** 2 + 2 * slack)
    disagree = kept_g != kept_o
    assert not np.any(disagree & ~window), f"{int((disagree & ~window).sum())} rows decided differently outside the allowance"
    assert eta_g == int((~kept_g).sum())
    assert abs(eta_g - eta_o) <= int(window.sum())
    # alpha on the rows both keep; then the oracle's remaining steps fed the GPU's decisions
    both = kept_g & kept_o
    assert parity.rel_fro(a_g[both], a_e[both]) <= tol
    a_chain = np.where(kept_g, a_e, 0.0)
    Bt_o = orc.contract(f_g, a_g.astype(np.float64), dY, k)
    assert parity.rel_fro(Bt_g, Bt_o) <= tol
    beta_g = b / (b - eta_g)
    dW_stage = beta_g * orc.weight_grad(C64, Bt_g.astype(np.float64))
    assert parity.rel_fro(dW_g, dW_stage) <= tol
    dW_e2e = beta_g * orc.weight_grad(C64, orc.contract(f_e, a_chain, dY, k))
    assert parity.rel_fro(dW_g, dW_e2e) <= tol
    return dict(kept=int(kept_g.sum()), eta=eta_g, window=int(window.sum()), disagree=int(disagree.sum()), dW=dW_g,
                idx=idx_g, f=f_g, alpha=a_g)


CASES = [
    (1500, 96, 72, 6, "f32"),          # SIMT path
    (3000, 200, 264, 40, "bf16"),      # tcgen05 path, two row tiles per C tile, ragged tiles
    (1111, 520, 136, 200, "bf16"),     # one row tile per C tile (k > 128)
    (700, 64, 40, 300, "bf16"),        # generators in two chunks
    (900, 72, 48, 3, "bf16"),          # k < 16: SIMT path with bf16 inputs
]


@pytest.mark.parametrize("b,n,m,k,dtype", CASES)
@pytest.mark.parametrize("eps", [0.15, 0.35, 0.7])
def test_neighbourhood_parity(b, n, m, k, dtype, eps):
    X, dY = synth.random_case(b, n, m, dtype, seed=b + k, centres=max(3, k // 3), noise=0.25, dy_scale=1e-3)
    r = run_eps(X, dY, k, eps)
    print(dtype, b, n, k, eps, {q: r[q] for q in ("kept", "eta", "window", "disagree")})


def test_largest_generator_count_with_the_row_norm_warps():
    # k = 4096 leaves the least shared memory for the pipeline: the stage count gives way, not the launch
    X, dY = synth.random_case(4500, 128, 72, "bf16", seed=91, centres=300, noise=0.25, dy_scale=1e-3)
    r = run_eps(X, dY, 4096, 0.2)
    assert r["eta"] > 0


def test_both_branches_are_exercised():
    X, dY = synth.random_case(3000, 200, 264, "bf16", seed=77, centres=12, noise=0.25, dy_scale=1e-3)
    r = run_eps(X, dY, 40, 0.3)
    assert 0.05 * 3000 < r["kept"] < 0.95 * 3000


def test_eps_zero_is_uniform_column_row_sampling():
    inp = synth.make_inputs("c2", num_seqs=12)                    # has exact-duplicate and zero padding rows
    X, dY = inp.X, inp.dY
    b, k = X.shape[0], 24
    r = run_eps(X, dY, k, 0.0, seed=9)
    X64, B = synth.to_f64(X), synth.to_f64(dY)
    gens = X64[r["idx"]]
    # kept = rows equal to (a multiple of) a generator, and the zero rows (distance 0 to anything)
    on_line = np.array([np.any(np.all(X64[i] == gens, axis=1)) or not X64[i].any() for i in range(b)])
    kept = r["alpha"] != 0
    assert np.array_equal(kept | ~X64.any(axis=1), on_line)
    crs = (b / on_line.sum()) * X64[kept].T @ B[kept]              # duplicates of a generator count with alpha = 1
    assert parity.rel_fro(r["dW"], crs) <= 1e-2


def test_eps_of_one_or_more_equals_plain_compress():
    X, dY = synth.random_case(2000, 136, 72, "bf16", seed=3, centres=10)
    Xd = parity.to_device(X)
    idx, C, invn = pamm.select_generators(Xd, 32, 4)
    f0, a0 = pamm.compress(Xd, C, invn)
    for eps in (1.0, 3.0, float("inf")):
        f1, a1, dropped = pamm.compress_eps(Xd, C, invn, eps)
        assert torch.equal(f0, f1) and torch.equal(a0, a1) and int(dropped.item()) == 0
    Bt = pamm.contract(f0, a0, parity.to_device(dY), 32)
    assert torch.equal(pamm.weight_grad(C, Bt), pamm.weight_grad_beta(C, Bt, 2000, dropped))
    with pytest.raises(pamm.PammError):
        pamm.compress_eps(Xd, C, invn, -0.5)


def test_full_size_c4_with_neighbourhood():
    inp = synth.make_inputs("c4", num_seqs=16)                    # 16384 rows of the LLaMA-1B-shaped workload
    r = run_eps(inp.X, inp.dY, 128, 0.6, seed=inp.workload.index_seed)
    print("c4/16 seqs eps=0.6", {q: r[q] for q in ("kept", "eta", "window", "disagree")})
