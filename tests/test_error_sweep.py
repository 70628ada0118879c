"""Approximation quality on the synthetic workloads (oracle only, CPU): the relative
error E = ||X^T dY - dW~||_F / ||X^T dY||_F of the appendix "PAMM Compression EDA"
falls as the number of generators grows, and the neighbourhood condition trades
dropped rows against it."""
import numpy as np

from oracle import pamm_oracle as orc
from paper_2506_02939_b200 import synth


def _indices(b, k, seed):
    return np.sort(np.random.default_rng(seed).permutation(b)[:k]).astype(np.int32)


def test_error_falls_with_the_number_of_generators_on_c1():
    inp = synth.make_inputs("c1")                                   # 2048 x 512, 64 clusters, 10% padding rows
    X64, B = synth.to_f64(inp.X), synth.to_f64(inp.dY)
    exact = X64.T @ B
    errs = {}
    for k in (1, 4, 16, 64, 256, 1024, 2048):
        r = orc.pamm(inp.X, _indices(2048, k, 5), inp.dY)            # nested index sets: prefixes of one permutation
        errs[k] = float(np.linalg.norm(exact - r["O"]) / np.linalg.norm(exact))
    ks = sorted(errs)
    assert all(errs[a] > errs[b_] for a, b_ in zip(ks, ks[1:])), errs
    assert errs[2048] < 1e-12                                        # every row its own generator
    assert errs[64] < 0.6 * errs[1]                                  # the clusters are found well before k = b
    # the estimate never does worse than dropping everything (E = 1) by more than the bound allows
    assert all(e < 1.5 for e in errs.values()), errs


def test_neighbourhood_condition_drops_far_rows_on_c1():
    inp = synth.make_inputs("c1")
    I = _indices(2048, 16, 6)
    kept_prev = None
    for eps in (0.0, 0.2, 0.5, 0.9, 1.0):
        r = orc.pamm(inp.X, I, inp.dY, eps=eps)
        kept = int(r["kept"].sum())
        assert kept_prev is None or kept >= kept_prev
        kept_prev = kept
        assert r["beta"] == 2048 / kept
    assert kept_prev == 2048
