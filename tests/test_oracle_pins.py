"""Pins for the fp64 oracle: each test checks it against something other than
itself -- a definition evaluated by brute force, a closed form, a library
routine on a special case, an invariant, or a value the paper prints."""
from pathlib import Path

import numpy as np
import pytest
from scipy.optimize import minimize_scalar

from oracle import pamm_oracle as orc
from paper_2506_02939_b200 import synth

GOLDEN = Path(__file__).parent / "golden" / "paper_values.txt"


def case(b=96, n=24, m=10, k=7, dtype="f32", seed=0, centres=5):
    X, dY = synth.random_case(b, n, m, dtype, seed, centres=centres)
    rng = np.random.default_rng(seed + 1)
    I = np.sort(rng.choice(b, size=k, replace=False)).astype(np.int32)
    return X, dY, I


def brute_force_assignment(X64, C64):
    """f(i) = argmin_j || A_i - (<A_i,C_j>/||C_j||^2) C_j ||_2, straight from the
    definition under Eq. 1; also returns the distances."""
    b, k = X64.shape[0], C64.shape[0]
    d = np.empty((b, k))
    for i in range(b):
        for j in range(k):
            cj = C64[j]
            a = float(X64[i] @ cj) / float(cj @ cj)
            d[i, j] = np.linalg.norm(X64[i] - a * cj)
    return d


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("seed", [0, 1, 2])
def test_f_is_argmin_point_to_line_distance(dtype, seed):
    X, dY, I = case(dtype=dtype, seed=seed)
    C, q = orc.gather(X, I)
    f, alpha, t1, t2 = orc.compress(X, C, q)
    d = brute_force_assignment(synth.to_f64(X), C)
    dmin = d.min(axis=1)
    # the oracle's choice attains the minimum distance (ties aside, it is the argmin)
    assert np.allclose(d[np.arange(len(f)), f], dmin, rtol=0, atol=1e-9 * (1 + dmin.max()))
    clear = (np.sort(d, axis=1)[:, 1] - dmin) > 1e-9 if d.shape[1] > 1 else np.ones(len(f), bool)
    assert np.array_equal(f[clear], d.argmin(axis=1)[clear])
    assert clear.sum() > 0.8 * len(f)


def test_alpha_is_line_search_minimiser():
    X, dY, I = case(b=40, n=16, k=5, seed=3)
    C, q = orc.gather(X, I)
    f, alpha, _, _ = orc.compress(X, C, q)
    X64 = synth.to_f64(X)
    for i in range(X64.shape[0]):
        cj = C[f[i]]
        res = minimize_scalar(lambda t: float(np.sum((X64[i] - t * cj) ** 2)), method="brent",
                              options=dict(xtol=1e-13))
        assert abs(res.x - alpha[i]) <= 1e-7 * (1 + abs(alpha[i]))


def test_generators_represent_themselves():
    X, dY, I = case(b=200, n=32, k=16, seed=4, centres=0)
    C, q = orc.gather(X, I)
    f, alpha, t1, _ = orc.compress(X, C, q)
    assert np.array_equal(C, synth.to_f64(X)[I])
    assert np.array_equal(f[I], np.arange(len(I)))
    # alpha = <C_j,C_j>/||C_j||^2 = 1 (proof of Lemma 2: a row can always generate itself with alpha = 1)
    assert np.all(alpha[I] == 1.0)
    d = brute_force_assignment(synth.to_f64(X)[I], C)
    assert np.allclose(np.diag(d), 0.0, atol=1e-12)


def test_residual_orthogonal_and_identity():
    X, dY, I = case(b=128, n=48, k=9, dtype="bf16", seed=5)
    C, q = orc.gather(X, I)
    f, alpha, _, _ = orc.compress(X, C, q)
    X64 = synth.to_f64(X)
    At = orc.reconstruct(C, f, alpha)
    assert np.array_equal(At, alpha[:, None] * C[f])
    R = X64 - At
    dots = np.einsum("il,il->i", R, C[f])
    scale = np.linalg.norm(X64, axis=1) * np.linalg.norm(C[f], axis=1)
    assert np.all(np.abs(dots) <= 1e-12 * scale)
    # ||A_i - A~_i||^2 = ||A_i||^2 (1 - csim^2)   (proof of Lemma 1, with the square restored)
    csim = np.einsum("il,il->i", X64, C[f]) / scale
    lhs = np.sum(R * R, axis=1)
    rhs = np.sum(X64 * X64, axis=1) * (1 - csim ** 2)
    assert np.allclose(lhs, rhs, rtol=1e-9, atol=1e-12)
    # Algorithm 1's form: alpha = csim * eta_A / eta_C[f]
    a2 = csim * np.linalg.norm(X64, axis=1) / np.linalg.norm(C[f], axis=1)
    assert np.allclose(alpha, a2, rtol=1e-12, atol=0)


def test_f_maximises_abs_cosine_and_negative_alpha_occurs():
    X, dY, I = case(b=300, n=8, k=3, seed=6, centres=0)
    C, q = orc.gather(X, I)
    f, alpha, t1, t2 = orc.compress(X, C, q)
    X64 = synth.to_f64(X)
    cs = (X64 @ C.T) / (np.linalg.norm(X64, axis=1)[:, None] * np.linalg.norm(C, axis=1)[None, :])
    assert np.array_equal(f, np.abs(cs).argmax(axis=1))
    # abs matters: with only 3 generators in 8 dimensions many winners have negative cosine
    assert (alpha < 0).sum() > 20
    signed = cs.argmax(axis=1)
    assert (signed != f).sum() > 0
    assert np.allclose(t1, np.abs(cs).max(axis=1) * np.linalg.norm(X64, axis=1), rtol=1e-12)
    assert np.allclose(t2, np.sort(np.abs(cs), axis=1)[:, -2] * np.linalg.norm(X64, axis=1), rtol=1e-12)


def test_scaling_invariances():
    X, dY, I = case(b=64, n=20, k=6, seed=7)
    C, q = orc.gather(X, I)
    f, alpha, _, _ = orc.compress(X, C, q)
    # scale generators (exact powers of two, one negative): f unchanged, alpha scales by 1/c, A~ unchanged
    c = np.array([2.0, -4.0, 0.5, 8.0, -0.25, 1.0])
    C2 = C * c[:, None]
    f2, alpha2, _, _ = orc.compress(X, C2, q * c * c)
    assert np.array_equal(f, f2)
    assert np.array_equal(alpha2, alpha / c[f])
    assert np.array_equal(orc.reconstruct(C2, f2, alpha2), orc.reconstruct(C, f, alpha))
    # scale rows of A (incl. negative): f unchanged, alpha scales
    s = np.where(np.arange(64) % 3 == 0, -2.0, 4.0).astype(np.float32)
    Xs = (X * s[:, None]).astype(np.float32)
    f3, alpha3, _, _ = orc.compress(Xs, C, q)
    assert np.array_equal(f, f3)
    assert np.array_equal(alpha3, alpha * s)


def test_duplicate_and_zero_rows_and_zero_generator():
    X, dY, I = case(b=80, n=16, k=5, seed=8)
    X = X.copy()
    X[70:75] = X[3]            # exact duplicates (padding rows)
    X[75:80] = 0.0             # zero rows
    I = np.array([3, 10, 20, 72, 77], np.int32)   # includes a duplicate generator and a zero one
    C, q = orc.gather(X, I)
    assert q[4] == 0.0
    f, alpha, t1, t2 = orc.compress(X, C, q)
    assert np.all(f[70:75] == f[3]) and np.all(alpha[70:75] == alpha[3])
    assert f[3] == 0 and alpha[3] == 1.0          # lowest index among identical generators 0 and 3
    assert f[72] == 0                              # tie between generators 0 and 3 -> lowest
    assert t1[3] == t2[3]                          # exact tie is visible in the top-2 scores
    assert np.all(f[75:80] == 0) and np.all(alpha[75:80] == 0.0)
    assert np.all(np.isfinite(alpha))
    assert not np.any(f == 4)                      # a zero generator never wins against a positive score


def test_k_equals_one():
    X, dY, I = case(b=30, n=12, k=1, seed=9)
    C, q = orc.gather(X, I)
    f, alpha, t1, t2 = orc.compress(X, C, q)
    X64 = synth.to_f64(X)
    assert np.all(f == 0) and np.all(t2 == 0)
    assert np.allclose(alpha, (X64 @ C[0]) / (C[0] @ C[0]), rtol=1e-13)


def test_bf16_widening_matches_torch():
    import torch
    X, _ = synth.random_case(50, 33, 4, "bf16", 11)
    t = torch.from_numpy(X.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    C, q = orc.gather(X, np.arange(50, dtype=np.int32))
    assert np.array_equal(C, t)
    assert np.array_equal(synth.to_f64(X), t)


def test_contract_special_cases():
    X, dY, I = case(b=60, n=8, m=14, k=6, dtype="bf16", seed=12)
    B = synth.to_f64(dY)
    rng = np.random.default_rng(0)
    # alpha = 1, f = 0: row 0 is the column sums, the rest zero
    Bt = orc.contract(np.zeros(60, np.int32), np.ones(60), dY, 6)
    assert np.allclose(Bt[0], B.sum(axis=0), rtol=1e-13, atol=1e-15) and np.all(Bt[1:] == 0)
    # k = b, f = identity: B~ = diag(alpha) B
    a = rng.standard_normal(60)
    Bt = orc.contract(np.arange(60, dtype=np.int32), a, dY, 60)
    assert np.array_equal(Bt, a[:, None] * B)
    # general f: equals numpy's index_add (np.add.at), the routine Algorithm 1 names
    f = rng.integers(0, 6, size=60).astype(np.int32)
    ref = np.zeros((6, 14))
    np.add.at(ref, f, a[:, None] * B)
    Bt = orc.contract(f, a, dY, 6)
    assert np.allclose(Bt, ref, rtol=1e-13, atol=1e-16)
    assert np.allclose(Bt.sum(axis=0), (a[:, None] * B).sum(axis=0), rtol=1e-12, atol=1e-15)
    # linearity in B (fp32 storage so that the sum of inputs is representable)
    _, d1 = synth.random_case(60, 8, 14, "f32", 13)
    _, d2 = synth.random_case(60, 8, 14, "f32", 14)
    d1 = np.round(d1 * 64) / 64
    d2 = np.round(d2 * 64) / 64
    lhs = orc.contract(f, a, (d1 + d2).astype(np.float32), 6)
    rhs = orc.contract(f, a, d1.astype(np.float32), 6) + orc.contract(f, a, d2.astype(np.float32), 6)
    assert np.allclose(lhs, rhs, rtol=1e-12, atol=1e-14)
    with pytest.raises(ValueError):
        orc.contract(np.full(60, 6, np.int32), a, dY, 6)


def test_weight_grad_is_plain_matmul_and_factorisation():
    X, dY, I = case(b=120, n=18, m=11, k=8, seed=15)
    r = orc.pamm(X, I, dY)
    assert np.allclose(r["O"], r["C"].T @ r["Bt"], rtol=1e-12, atol=1e-14)
    # C^T B~ = A~^T B with A~ rebuilt row by row from Eq. 3 (Section 3.2 factorisation)
    At = orc.reconstruct(r["C"], r["f"], r["alpha"])
    assert np.allclose(r["O"], At.T @ synth.to_f64(dY), rtol=1e-10, atol=1e-12)
    # a transposed-operand mistake would change the shape
    assert r["O"].shape == (18, 11)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_k_equals_b_gives_exact_product(dtype):
    X, dY, _ = case(b=48, n=10, m=7, k=1, dtype=dtype, seed=16, centres=0)
    I = np.arange(48, dtype=np.int32)
    r = orc.pamm(X, I, dY)
    assert np.array_equal(r["f"], I) and np.all(r["alpha"] == 1.0)
    exact = synth.to_f64(X).T @ synth.to_f64(dY)
    assert np.allclose(r["O"], exact, rtol=1e-12, atol=1e-14)
    assert np.allclose(orc.exact_product(X, dY), exact, rtol=1e-12, atol=1e-14)


def test_rank_one_input_reproduces_exact_product():
    rng = np.random.default_rng(17)
    u = (rng.integers(1, 9, size=64) * rng.choice([-1, 1], size=64)).astype(np.float32)
    v = rng.integers(-8, 9, size=12).astype(np.float32)
    v[0] = 3
    X = np.outer(u, v).astype(np.float32)      # small integers: exactly representable
    _, dY = synth.random_case(64, 12, 9, "f32", 18)
    I = np.array([5, 17, 40], np.int32)
    r = orc.pamm(X, I, dY)
    exact = X.astype(np.float64).T @ dY.astype(np.float64)
    assert np.allclose(r["O"], exact, rtol=1e-11, atol=1e-13)
    assert np.allclose(r["top1"], r["top2"], rtol=1e-12)     # every generator ties


def test_error_bound_of_section_3_2_1():
    X, dY, I = case(b=150, n=20, m=13, k=10, seed=19)
    r = orc.pamm(X, I, dY)
    X64, B = synth.to_f64(X), synth.to_f64(dY)
    At = orc.reconstruct(r["C"], r["f"], r["alpha"])
    lhs = np.linalg.norm(X64.T @ B - r["O"], "fro")
    rhs = np.linalg.norm(B, 2) * np.linalg.norm(X64 - At, "fro")
    assert lhs <= rhs * (1 + 1e-12)
    # eps = infinity and every row represented: the residual never exceeds the row itself
    assert np.all(np.linalg.norm(X64 - At, axis=1) <= np.linalg.norm(X64, axis=1) * (1 + 1e-12))


def test_row_permutation_equivariance():
    X, dY, I = case(b=90, n=14, m=6, k=7, seed=20)
    r = orc.pamm(X, I, dY)
    p = np.random.default_rng(21).permutation(90)
    inv = np.empty(90, np.int64)
    inv[p] = np.arange(90)
    I2 = inv[I].astype(np.int32)               # same generator rows, same order in C
    r2 = orc.pamm(X[p].copy(), I2, dY[p].copy())
    assert np.array_equal(r2["C"], r["C"])
    assert np.array_equal(r2["f"], r["f"][p]) and np.array_equal(r2["alpha"], r["alpha"][p])
    assert np.allclose(r2["O"], r["O"], rtol=1e-10, atol=1e-13)


def test_row_scores_agree_with_compress():
    X, dY, I = case(b=40, n=30, k=6, dtype="bf16", seed=22)
    C, q = orc.gather(X, I)
    f, alpha, t1, t2 = orc.compress(X, C, q)
    X64 = synth.to_f64(X)
    for i in (0, 7, 39):
        s, sc, ab = orc.row_scores(X, i, C, q)
        assert np.allclose(s, C @ X64[i], rtol=1e-12, atol=1e-14)
        assert np.allclose(ab, np.abs(C * X64[i]).sum(axis=1), rtol=1e-12)
        assert int(np.argmax(sc)) == f[i] and sc[f[i]] == t1[i]


def test_leading_dimension_is_honoured():
    X, dY, I = case(b=32, n=12, m=5, k=4, seed=23)
    Xw = np.full((32, 20), 99.0, np.float32)
    Xw[:, :12] = X
    dYw = np.full((32, 9), 77.0, np.float32)
    dYw[:, :5] = dY
    r = orc.pamm(X, I, dY)
    r2 = orc.pamm(Xw[:, :12], I, dYw[:, :5])
    for key in ("f", "alpha", "Bt", "O"):
        assert np.array_equal(r[key], r2[key])


def test_paper_printed_values():
    vals = {}
    for line in GOLDEN.read_text().splitlines():
        line = line.split("#")[0].strip()
        if line:
            name, v, tol = line.split()
            vals[name] = (v, float(tol))
    g, tol = vals["gamma_llama1b"]
    # LLaMA-1B: b = 16384 tokens, per-projection m = n = 2048, k = b/256 = 64
    assert abs(orc.gamma(16384, 2048, 64) - float(g)) <= tol
    assert abs(orc.gamma(16384, 2048, 64) - 16384 * 2048 / (64 * (16384 + 2048))) < 1e-12
    assert orc.memory_scalars(16384, 2048, 64) == 64 * 2048 + 2 * 16384


def test_clustered_data_error_decreases_with_k():
    """Qualitative claim of the appendix "PAMM Compression EDA": E(r) falls as k grows (here on clustered synthetic rows)."""
    X, dY = synth.random_case(512, 32, 16, "f32", 24, centres=8, noise=0.05)
    exact = X.astype(np.float64).T @ dY.astype(np.float64)
    errs = []
    perm = np.random.default_rng(25).permutation(512)
    for k in (1, 8, 64, 512):
        I = np.sort(perm[:k]).astype(np.int32)
        r = orc.pamm(X, I, dY)
        errs.append(np.linalg.norm(exact - r["O"]) / np.linalg.norm(exact))
    assert errs[0] > errs[1] > errs[2] > errs[3]
    assert errs[3] < 1e-12


# ---- neighbourhood condition (Eq. 2) and the factor beta (Eq. 4-5) -----------------------

def test_neighbourhood_matches_cosine_form():
    """Eq. 2 in its equivalent cosine form: a row is kept iff csim^2 >= 1 - eps^2
    (from ||A_i - A~_i||^2 = ||A_i||^2 (1 - csim^2), proof of Lemma 1)."""
    X, dY, I = case(b=400, n=12, k=6, seed=30, centres=8)
    C, q = orc.gather(X, I)
    f, alpha, _, _ = orc.compress(X, C, q)
    X64 = synth.to_f64(X)
    cs = np.einsum("il,il->i", X64, C[f]) / (np.linalg.norm(X64, axis=1) * np.linalg.norm(C[f], axis=1))
    for eps in (0.05, 0.2, 0.5, 0.9):
        a2, kept, err, rn, eta, beta = orc.neighbourhood(X, C, f, alpha, eps)
        margin = np.abs(cs ** 2 - (1 - eps ** 2))
        clear = margin > 1e-9
        assert np.array_equal(kept[clear], (cs ** 2 >= 1 - eps ** 2)[clear])
        assert 0 < kept.sum() < len(kept)                       # the case exercises both branches
        assert eta == int((~kept).sum()) and beta == 400 / (400 - eta)
        assert np.all(a2[~kept] == 0.0) and np.array_equal(a2[kept], alpha[kept])
        assert np.allclose(rn, np.linalg.norm(X64, axis=1), rtol=1e-13)
        assert np.allclose(err, np.linalg.norm(X64 - alpha[:, None] * C[f], axis=1), rtol=1e-9, atol=1e-13)


def test_epsilon_at_least_one_or_infinite_keeps_everything():
    X, dY, I = case(b=120, n=10, m=6, k=5, seed=31, centres=0)
    base = orc.pamm(X, I, dY)
    for eps in (1.0, 2.5):
        r = orc.pamm(X, I, dY, eps=eps)
        assert r["eta"] == 0 and r["beta"] == 1.0 and r["kept"].all()
        assert np.array_equal(r["alpha"], base["alpha"]) and np.array_equal(r["O"], base["O"])
    assert "eta" not in base                                    # eps = infinity: the steps are skipped


def test_epsilon_zero_is_uniform_column_row_sampling():
    """Section 4.1: eps = 0 makes PAMM the Uniform-CRS estimator (b/k) A_I^T B_I."""
    X, dY, I = case(b=90, n=9, m=7, k=10, seed=32, centres=0)     # generic rows: nothing is parallel
    r = orc.pamm(X, I, dY, eps=0.0)
    assert np.array_equal(np.nonzero(r["kept"])[0], I) and r["eta"] == 80 and r["beta"] == 9.0
    crs = (90 / 10) * synth.to_f64(X)[I].T @ synth.to_f64(dY)[I]
    assert np.allclose(r["O"], crs, rtol=1e-12, atol=1e-14)


def test_epsilon_zero_keeps_exact_duplicates_and_multiples():
    X, dY, I = case(b=60, n=8, m=5, k=3, seed=33, centres=0)
    X = X.copy()
    X[50] = X[I[1]]
    X[51] = -2.0 * X[I[1]]                                        # an exact multiple lies on the generator's line
    r = orc.pamm(X, I, dY, eps=0.0)
    assert r["kept"][50] and r["kept"][51] and r["alpha"][51] == -2.0
    assert r["eta"] == 60 - 5 and abs(r["beta"] - 60 / 5) < 1e-15


def test_single_generator_crs_is_exactly_unbiased():
    """Eq. 5 with k = 1, eps = 0: averaging O~ over every possible choice of the one
    generator gives sum_i A_i^T B_i = O exactly (beta = b)."""
    X, dY, _ = case(b=24, n=6, m=4, k=1, seed=34, centres=0)
    exact = synth.to_f64(X).T @ synth.to_f64(dY)
    mean = np.zeros_like(exact)
    for i in range(24):
        r = orc.pamm(X, np.array([i], np.int32), dY, eps=0.0)
        assert r["beta"] == 24.0 and r["kept"].sum() == 1
        mean += r["O"] / 24
    assert np.allclose(mean, exact, rtol=1e-12, atol=1e-14)


def test_kept_set_grows_with_epsilon_and_error_bound_holds():
    X, dY, I = case(b=300, n=16, m=9, k=8, seed=35, centres=10)
    prev = None
    X64, B = synth.to_f64(X), synth.to_f64(dY)
    for eps in (0.0, 0.1, 0.3, 0.6, 0.95):
        r = orc.pamm(X, I, dY, eps=eps)
        if prev is not None:
            assert np.all(r["kept"] >= prev)
        prev = r["kept"]
        # Section 3.2.1: ||O - O~/beta||_F^2 <= ||B||_2^2 (eps^2 ||A_kept||_F^2 + ||A_dropped||_F^2)
        lhs = np.linalg.norm(X64.T @ B - r["O"] / r["beta"], "fro") ** 2
        rhs = np.linalg.norm(B, 2) ** 2 * (eps ** 2 * np.sum(X64[r["kept"]] ** 2) + np.sum(X64[~r["kept"]] ** 2))
        assert lhs <= rhs * (1 + 1e-12) + 1e-18


# ---- Algorithm 2, first step: the layer's output Z = X W ---------------------------------

def test_linear_forward_hand_computed_two_by_two():
    # [[1, 2], [3, 4]] [[5, 6], [7, 8]] = [[19, 22], [43, 50]], worked by hand
    X = np.array([[1, 2], [3, 4]], np.float32)
    W = np.array([[5, 6], [7, 8]], np.float32)
    assert np.array_equal(orc.linear_forward(X, W), np.array([[19.0, 22.0], [43.0, 50.0]]))
    # not its transpose-side variants: W X, X^T W, X W^T all differ on this example
    assert not np.array_equal(orc.linear_forward(X, W), (W @ X).astype(np.float64))
    assert not np.array_equal(orc.linear_forward(X, W), (X.T @ W).astype(np.float64))
    assert not np.array_equal(orc.linear_forward(X, W), (X @ W.T).astype(np.float64))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_linear_forward_is_the_plain_matrix_product(dtype):
    X, _ = synth.random_case(37, 29, 8, dtype, seed=3)
    W, _ = synth.random_case(29, 23, 8, dtype, seed=4)
    Z = orc.linear_forward(X, W)
    ref = synth.to_f64(X) @ synth.to_f64(W)
    assert Z.shape == (37, 23) and np.allclose(Z, ref, rtol=1e-13, atol=1e-13)
    rows = np.array([5, 0, 36, 5])
    assert np.array_equal(orc.linear_forward(X, W, rows=rows), Z[rows])
    # a padded row stride of either operand changes nothing
    Xp = np.zeros((37, 40), X.dtype); Xp[:, :29] = X
    Wp = np.zeros((29, 32), W.dtype); Wp[:, :23] = W
    assert np.array_equal(orc.linear_forward(Xp[:, :29], Wp[:, :23]), Z)


def test_linear_forward_and_compress_see_the_same_input():
    # Algorithm 2: Z = X W and Compress(X) come from the same X.  The scores are the extra columns of X [W | C^T]:
    # the forward product against C^T reproduces the dot products behind f and alpha (Eq. 1)
    X, _ = synth.random_case(64, 24, 8, "bf16", seed=9, centres=5)
    I = np.array([3, 17, 40], np.int32)
    C64, q = orc.gather(X, I)
    f, alpha, _, _ = orc.compress(X, C64, q)
    S = orc.linear_forward(X, np.ascontiguousarray(X[I].T))          # b x k: X C^T
    assert np.array_equal(np.argmax(np.abs(S) / np.sqrt(q), axis=1), f)
    assert np.allclose(S[np.arange(64), f] / q[f], alpha, rtol=1e-14, atol=0)
