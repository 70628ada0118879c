"""Seeded synthetic inputs shaped like the paper's LLaMA-style pretraining workloads.

This module only *makes inputs* (activations X, upstream gradients dY) and holds
none of the method's arithmetic; it is the one module that both the CUDA tests /
benchmark and the CPU oracle's tests draw from.  It depends on numpy alone.

Storage types: fp32 arrays are ``np.float32``; bf16 arrays are ``np.uint16`` bit
patterns (round-to-nearest-even from fp32), so the very same bits can be handed
to the GPU library and to the oracle.

The five workloads stand in for the C4 pretraining activations the paper trains
on (Section 4.2), which are not available offline: rows are cluster centres plus
noise (token activations of a batch are highly redundant along the batch/sequence
axis, Section 1), optionally with exact-duplicate / zero "padding" rows at the
tail of each sequence, and dY ~ N(0, 1e-3^2).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (nearest even) and return the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp32."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def to_f64(a: np.ndarray) -> np.ndarray:
    """Exact widening of a stored array (fp32 or bf16 bits) to fp64."""
    if a.dtype == np.uint16:
        return bf16_bits_to_f32(a).astype(np.float64)
    return a.astype(np.float64)


@dataclass(frozen=True)
class Workload:
    name: str
    dtype: str            # "f32" | "bf16"
    num_seqs: int
    seq_len: int
    n: int
    m: int
    ks: tuple             # generator counts to run (one entry except for the ratio sweep)
    centres: int
    noise: float
    pad_frac: float = 0.0
    pad_kind: str = "none"   # "none" | "dup" | "zero+dup"
    heavy_tail: bool = False
    seed: int = 0
    qkv: tuple = ()          # column split of dY = [dQ|dK|dV]
    layers: int = 1

    @property
    def b(self) -> int:
        return self.num_seqs * self.seq_len

    @property
    def index_seed(self) -> int:
        return 1000 + self.seed


WORKLOADS = {
    "c1": Workload("c1", "f32", 8, 256, 512, 1536, (4,), 64, 0.1, 0.10, "dup", seed=0, qkv=(512, 512, 512)),
    "c2": Workload("c2", "bf16", 128, 256, 768, 2304, (64,), 512, 0.2, 0.05, "zero+dup", seed=1, qkv=(768, 768, 768)),
    "c3": Workload("c3", "bf16", 256, 256, 1024, 3072, (1024, 512, 256, 128), 2048, 0.2, 0.0, "none",
                   heavy_tail=True, seed=2, qkv=(1024, 1024, 1024)),
    "c4": Workload("c4", "bf16", 64, 1024, 2048, 6144, (128,), 4096, 0.3, 0.0, "none", seed=3,
                   qkv=(2048, 2048, 2048)),
    "c5": Workload("c5", "bf16", 4, 8192, 4096, 6144, (64,), 8192, 0.3, 0.03, "dup", seed=4,
                   qkv=(4096, 1024, 1024), layers=32),
}


@dataclass
class Inputs:
    workload: Workload
    X: np.ndarray            # b x n, float32 or uint16 (bf16 bits)
    dY: np.ndarray           # b x m, same storage type
    pad_rows: np.ndarray     # indices of padding rows (may be empty)
    meta: dict = field(default_factory=dict)

    @property
    def b(self) -> int:
        return self.X.shape[0]


def _store(x32: np.ndarray, dtype: str) -> np.ndarray:
    return f32_to_bf16_bits(x32) if dtype == "bf16" else np.ascontiguousarray(x32, np.float32)


def _draw(rng: np.random.Generator, shape, heavy: bool) -> np.ndarray:
    if heavy:
        return rng.standard_t(4.0, size=shape).astype(np.float32)
    return rng.standard_normal(size=shape, dtype=np.float32)


def make_inputs(name: str, num_seqs: int | None = None, seed: int | None = None, with_dY: bool = True) -> Inputs:
    """Build X and dY for workload ``name``.

    ``num_seqs`` shrinks the batch (b = num_seqs * seq_len) while keeping the
    per-row recipe; ``seed`` overrides the workload's data seed (the 32-layer
    loop uses one seed per layer).  Independent streams, in this order, are
    spawned from the seed: centres, assignments, noise, padding, dY.
    """
    w = WORKLOADS[name]
    S = w.num_seqs if num_seqs is None else int(num_seqs)
    L, n, m = w.seq_len, w.n, w.m
    b = S * L
    sd = w.seed if seed is None else int(seed)
    r_cent, r_asg, r_noise, r_pad, r_dy = (np.random.default_rng([sd, t]) for t in range(5))

    mu = _draw(r_cent, (w.centres, n), w.heavy_tail)
    g = r_asg.integers(0, w.centres, size=b)
    X = np.empty((b, n), np.float32)
    step = max(1, (1 << 24) // n)
    for r0 in range(0, b, step):
        r1 = min(b, r0 + step)
        X[r0:r1] = mu[g[r0:r1]] + np.float32(w.noise) * _draw(r_noise, (r1 - r0, n), w.heavy_tail)
    if w.heavy_tail:
        rms = float(np.sqrt(np.mean(np.square(X, dtype=np.float64))))
        X *= np.float32(1.0 / rms)

    pad_rows = []
    if w.pad_kind != "none" and w.pad_frac > 0:
        pad_vec = mu[int(r_pad.integers(0, w.centres))] + np.float32(w.noise) * _draw(r_pad, (n,), w.heavy_tail)
        hi = int(2 * w.pad_frac * L)
        lens = r_pad.integers(0, hi + 1, size=S)
        for s in range(S):
            p = int(lens[s])
            if p == 0:
                continue
            rows = np.arange((s + 1) * L - p, (s + 1) * L)
            if w.pad_kind == "zero+dup" and s % 2 == 0:
                X[rows] = 0.0
            else:
                X[rows] = pad_vec
            pad_rows.append(rows)
    pad_rows = np.concatenate(pad_rows) if pad_rows else np.empty(0, np.int64)

    Xs = _store(X, w.dtype)
    del X
    if with_dY:
        if w.dtype == "bf16":
            dY = np.empty((b, m), np.uint16)
        else:
            dY = np.empty((b, m), np.float32)
        step = max(1, (1 << 24) // m)
        for r0 in range(0, b, step):
            r1 = min(b, r0 + step)
            blk = np.float32(1e-3) * r_dy.standard_normal(size=(r1 - r0, m), dtype=np.float32)
            dY[r0:r1] = _store(blk, w.dtype)
    else:
        dY = np.empty((0, m), np.uint16 if w.dtype == "bf16" else np.float32)
    return Inputs(w, Xs, dY, pad_rows, meta=dict(seed=sd, num_seqs=S))


def random_case(b: int, n: int, m: int, dtype: str = "f32", seed: int = 0, centres: int = 0,
                noise: float = 0.2, dy_scale: float = 1.0):
    """Small generic case for unit tests: returns (X, dY) in storage type.

    ``centres == 0`` gives unstructured Gaussian rows, otherwise clustered rows.
    """
    rng = np.random.default_rng([seed, 77])
    if centres > 0:
        mu = rng.standard_normal((centres, n), dtype=np.float32)
        X = mu[rng.integers(0, centres, size=b)] + np.float32(noise) * rng.standard_normal((b, n), dtype=np.float32)
    else:
        X = rng.standard_normal((b, n), dtype=np.float32)
    dY = np.float32(dy_scale) * rng.standard_normal((b, m), dtype=np.float32)
    return _store(X, dtype), _store(dY, dtype)
