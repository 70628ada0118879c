#!/usr/bin/env python
"""Approximation quality of PAMM on the synthetic workloads -- TEST INFRASTRUCTURE, CPU only.

Repeats, on the synthetic stand-ins for the paper's activations, the measurements of the
appendix "PAMM Compression EDA": the relative error of the weight gradient
    E(r, eps) = ||X^T dY - beta C^T B~||_F / ||X^T dY||_F
and the coverage (fraction of rows with alpha != 0) over the compression ratio r = k / b and
the neighbourhood parameter eps; and, for the Conclusion's remark that the generators
could be chosen more strategically than uniformly, two alternative ways of picking C at
eps = infinity.  Everything goes through the fp64 oracle; the exact product X^T dY, the
quantity being approximated, is numpy's matmul.  Writes profiles/error_sweep.md.

    python oracle/error_sweep.py [--rows 8192] [--cols 512]
"""
from __future__ import annotations

import argparse
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

from oracle import pamm_oracle as orc                      # noqa: E402
from paper_2506_02939_b200 import synth                    # noqa: E402  (input generator only)

RATIOS = (64, 128, 256, 512)
EPSILONS = (0.0, 0.2, 0.5, float("inf"))


def pick_uniform(X64, k, rng):
    """The paper's choice: k rows uniformly without replacement (Algorithm 1)."""
    return np.sort(rng.choice(X64.shape[0], size=k, replace=False)).astype(np.int32)


def pick_norm_weighted(X64, k, rng):
    """Rows drawn without replacement with probability proportional to ||X_i||^2 (as norm-based
    column-row sampling does)."""
    w = np.einsum("il,il->i", X64, X64)
    nz = int((w > 0).sum())
    if nz < k:
        return pick_uniform(X64, k, rng)
    return np.sort(rng.choice(X64.shape[0], size=k, replace=False, p=w / w.sum())).astype(np.int32)


def pick_far_from_chosen(X64, k, rng):
    """Seeding in the manner of k-means++ on the method's own distance: the next generator is drawn
    with probability proportional to the squared distance of a row to the closest line chosen so far,
    ||X_i||^2 (1 - max_j csim(X_i, C_j)^2)."""
    b = X64.shape[0]
    norm2 = np.einsum("il,il->i", X64, X64)
    live = norm2 > 0
    first = int(rng.choice(np.nonzero(live)[0])) if live.any() else 0
    chosen = [first]
    best_cos2 = np.zeros(b)
    for _ in range(1, k):
        c = X64[chosen[-1]]
        q = float(c @ c)
        if q > 0:
            s = X64 @ c
            best_cos2 = np.maximum(best_cos2, np.divide(s * s, norm2 * q, out=np.zeros(b), where=live))
        d2 = np.clip(norm2 * (1.0 - best_cos2), 0.0, None)
        d2[chosen] = 0.0
        tot = d2.sum()
        nxt = int(rng.choice(b, p=d2 / tot)) if tot > 0 else int(rng.choice(np.setdiff1d(np.arange(b), chosen)))
        chosen.append(nxt)
    return np.sort(np.array(chosen)).astype(np.int32)


def one_setting(X, dY, I, eps, exact, exact_norm):
    out = orc.pamm(X, I, dY, eps=eps)
    err = float(np.linalg.norm(exact - out["O"]) / exact_norm)
    coverage = float(np.mean(out["alpha"] != 0.0))
    return err, coverage


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--rows", type=int, default=8192, help="tokens per workload (a whole number of sequences)")
    ap.add_argument("--cols", type=int, default=512, help="columns of dY kept (the error does not depend on their number)")
    ap.add_argument("--out", default=str(ROOT / "profiles" / "error_sweep.md"))
    args = ap.parse_args()
    lines = ["# Approximation quality on the synthetic workloads (fp64 oracle, CPU)", "",
             "Written by `python oracle/error_sweep.py`" + ("" if (args.rows, args.cols) == (8192, 512)
                                                            else f" `--rows {args.rows} --cols {args.cols}`") + ".",
             "`E(r, eps) = ||X^T dY - beta C^T B~||_F / ||X^T dY||_F` and coverage (share of rows with alpha != 0), as in the",
             "appendix \"PAMM Compression EDA\", on the first rows of every workload's X and the first columns of its dY",
             f"(at most {args.rows} rows, {args.cols} columns; k = ceil(r b)); generators drawn uniformly with numpy seed 1000 + data seed.",
             "The inputs are synthetic cluster data with a dY that is independent noise, not transformer activations;",
             "what can be compared with the paper are the order of magnitude of E and its trends over r and eps.", ""]
    t_start = time.perf_counter()
    trend_rows = []
    for name, w in synth.WORKLOADS.items():
        seqs = max(1, min(w.num_seqs, args.rows // w.seq_len))
        inp = synth.make_inputs(name, num_seqs=seqs)
        X = inp.X
        dY = np.ascontiguousarray(inp.dY[:, : min(args.cols, w.m)])
        b = X.shape[0]
        X64, B64 = synth.to_f64(X), synth.to_f64(dY)
        exact = X64.T @ B64
        exact_norm = float(np.linalg.norm(exact))
        lines += [f"## {name}: b = {b}, n = {w.n}, {w.dtype}, {w.centres} centres, noise {w.noise}"
                  + (", heavy-tailed" if w.heavy_tail else "") + (f", {w.pad_kind} padding" if w.pad_kind != "none" else ""), "",
                  "| r | k | " + " | ".join(f"E, eps = {e:g}" for e in EPSILONS) + " | " +
                  " | ".join(f"coverage, eps = {e:g}" for e in EPSILONS) + " |",
                  "|---|---|" + "---|" * (2 * len(EPSILONS))]
        e_inf = []
        for ratio in RATIOS:
            k = max(1, -(-b // ratio))
            I = pick_uniform(X64, k, np.random.default_rng(w.index_seed))
            res = [one_setting(X, dY, I, eps, exact, exact_norm) for eps in EPSILONS]
            e_inf.append(res[-1][0])
            lines.append(f"| 1/{ratio} | {k} | " + " | ".join(f"{e:.3f}" for e, _ in res) + " | " +
                         " | ".join(f"{c:.3f}" for _, c in res) + " |")
        # E against log2(1/r): the paper reads its plot as "logarithmic in r"
        slope = np.polyfit(np.log2(np.array(RATIOS, float)), np.array(e_inf), 1)[0]
        trend_rows.append((name, e_inf, slope))
        lines += ["", "Choice of generators at eps = infinity (E; same k as above):", "",
                  "| r | uniform (the paper's) | drawn by squared row norm | drawn by distance to the lines chosen so far |", "|---|---|---|---|"]
        for ratio in RATIOS:
            k = max(1, -(-b // ratio))
            row = []
            for pick in (pick_uniform, pick_norm_weighted, pick_far_from_chosen):
                I = pick(X64, k, np.random.default_rng(w.index_seed))
                row.append(one_setting(X, dY, I, float("inf"), exact, exact_norm)[0])
            lines.append(f"| 1/{ratio} | " + " | ".join(f"{e:.3f}" for e in row) + " |")
        lines.append("")
        print(f"{name} done at {time.perf_counter() - t_start:.0f} s", flush=True)
    lines += ["## Trend of E(r, eps = infinity) over the ratio", "",
              "| workload | " + " | ".join(f"r = 1/{r}" for r in RATIOS) + " | increase of E per halving of r |", "|---|" + "---|" * (len(RATIOS) + 1)]
    for name, e_inf, slope in trend_rows:
        lines.append(f"| {name} | " + " | ".join(f"{e:.3f}" for e in e_inf) + f" | {slope:+.3f} |")
    lines += ["", "At eps = infinity E lies between about 0.7 and 1, the order the appendix reports for real activations",
              "(1/2 to 1), and it rises only slowly as r shrinks -- by a few hundredths per halving, flattening towards 1 --",
              "which is the weak, roughly logarithmic dependence on r the appendix describes.  E falls as eps grows and is",
              "by far the worst at eps = 0 (uniform column-row sampling, beta = b / (b - eta) blowing up the few kept rows);",
              "coverage rises with eps and with r.  Drawing the generators by row norm or by distance to the lines already",
              "chosen moves E by a few hundredths at most on these inputs: uniform sampling loses little here.", ""]
    Path(args.out).write_text("\n".join(lines))
    print(f"wrote {args.out} in {time.perf_counter() - t_start:.0f} s")


if __name__ == "__main__":
    main()
