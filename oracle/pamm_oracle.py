"""ctypes loader for the PAMM oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Wraps ``pamm_oracle.c`` (plain fp64 C following Algorithm 1 / Section 3.2 of the
paper).  Only tests, the smoke check and the benchmark's CPU-baseline leg import
this module; the CUDA library and its Python binding never do.

Arrays: fp32 inputs are ``np.float32``; bf16 inputs are ``np.uint16`` bit
patterns.  All results are ``np.float64`` (``np.int32`` for f).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "pamm_oracle.c"
_LIB = _HERE / "libpamm_oracle.so"

F32, BF16 = 0, 1


def build(force: bool = False) -> Path:
    """Compile the oracle with gcc (OpenMP across independent outputs only)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".{os.getpid()}.tmp")
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-fno-fast-math", "-ffp-contract=off", "-fPIC", "-shared",
             "-o", str(tmp), str(_SRC), "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(str(_LIB))
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        L.pamm_oracle_gather.argtypes = [vp, ci, i64, i64, i64, vp, i64, vp, vp]
        L.pamm_oracle_gather.restype = ci
        L.pamm_oracle_row_scores.argtypes = [vp, ci, i64, i64, i64, vp, vp, i64, vp, vp, vp]
        L.pamm_oracle_row_scores.restype = None
        L.pamm_oracle_compress.argtypes = [vp, ci, i64, i64, i64, vp, vp, i64, vp, vp, vp, vp]
        L.pamm_oracle_compress.restype = ci
        L.pamm_oracle_contract.argtypes = [vp, vp, vp, ci, i64, i64, i64, i64, vp]
        L.pamm_oracle_contract.restype = ci
        L.pamm_oracle_weight_grad.argtypes = [vp, vp, i64, i64, i64, vp]
        L.pamm_oracle_weight_grad.restype = None
        L.pamm_oracle_reconstruct.argtypes = [vp, vp, vp, i64, i64, vp]
        L.pamm_oracle_reconstruct.restype = None
        L.pamm_oracle_neighbourhood.argtypes = [vp, ci, i64, i64, i64, vp, vp, vp, ctypes.c_double, vp, vp, vp]
        L.pamm_oracle_neighbourhood.restype = i64
        L.pamm_oracle_beta.argtypes = [i64, i64]
        L.pamm_oracle_beta.restype = ctypes.c_double
        L.pamm_oracle_exact_product.argtypes = [vp, ci, i64, vp, ci, i64, i64, i64, i64, vp]
        L.pamm_oracle_exact_product.restype = None
        L.pamm_oracle_linear_forward.argtypes = [vp, ci, i64, vp, ci, i64, i64, i64, i64, vp, i64, vp]
        L.pamm_oracle_linear_forward.restype = None
        L.pamm_oracle_memory_scalars.argtypes = [i64, i64, i64]
        L.pamm_oracle_memory_scalars.restype = i64
        L.pamm_oracle_gamma.argtypes = [i64, i64, i64]
        L.pamm_oracle_gamma.restype = ctypes.c_double
        L.pamm_oracle_num_threads.argtypes = []
        L.pamm_oracle_num_threads.restype = ci
        _lib = L
    return _lib


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError(f"oracle inputs are float32 or uint16 (bf16 bits), got {a.dtype}")


def _mat(a: np.ndarray) -> np.ndarray:
    if a.ndim != 2 or a.strides[1] != a.itemsize or a.strides[0] % a.itemsize:
        raise ValueError("need a 2-D row-major array (a row stride is allowed)")
    return a


def _p(a: np.ndarray):
    return ctypes.c_void_p(a.ctypes.data)


def _ld(a: np.ndarray) -> int:
    return a.strides[0] // a.itemsize


def gather(A: np.ndarray, I: np.ndarray):
    """C = A[I,:] widened to fp64 and q_j = ||C_j||^2 (Algorithm 1)."""
    A = _mat(A)
    I = np.ascontiguousarray(I, dtype=np.int32)
    k, n = I.shape[0], A.shape[1]
    C = np.empty((k, n), np.float64)
    q = np.empty(k, np.float64)
    rc = _load().pamm_oracle_gather(_p(A), _dtype_code(A), A.shape[0], n, _ld(A), _p(I), k, _p(C), _p(q))
    if rc:
        raise ValueError("generator index out of range")
    return C, q


def compress(A: np.ndarray, C: np.ndarray, q: np.ndarray):
    """(f, alpha, top1, top2) per Lemma 1 and Eq. 1, epsilon = infinity."""
    A = _mat(A)
    C = np.ascontiguousarray(C, np.float64)
    q = np.ascontiguousarray(q, np.float64)
    b, n = A.shape
    k = C.shape[0]
    assert C.shape == (k, n) and q.shape == (k,)
    f = np.empty(b, np.int32)
    alpha = np.empty(b, np.float64)
    t1 = np.empty(b, np.float64)
    t2 = np.empty(b, np.float64)
    _load().pamm_oracle_compress(_p(A), _dtype_code(A), b, n, _ld(A), _p(C), _p(q), k,
                                 _p(f), _p(alpha), _p(t1), _p(t2))
    return f, alpha, t1, t2


def row_scores(A: np.ndarray, i: int, C: np.ndarray, q: np.ndarray):
    """(s, score, abssum) of row i against every generator."""
    A = _mat(A)
    C = np.ascontiguousarray(C, np.float64)
    q = np.ascontiguousarray(q, np.float64)
    k = C.shape[0]
    s = np.empty(k, np.float64)
    sc = np.empty(k, np.float64)
    ab = np.empty(k, np.float64)
    _load().pamm_oracle_row_scores(_p(A), _dtype_code(A), A.shape[1], _ld(A), int(i), _p(C), _p(q), k,
                                   _p(s), _p(sc), _p(ab))
    return s, sc, ab


def neighbourhood(A: np.ndarray, C: np.ndarray, f: np.ndarray, alpha: np.ndarray, eps: float):
    """Eq. 2: rows with ||A_i - alpha_i C_f|| > eps ||A_i|| are dropped (alpha_i = 0).

    Returns (alpha_masked, kept, err, rownorm, eta, beta) with beta = b / (b - eta)."""
    A = _mat(A)
    C = np.ascontiguousarray(C, np.float64)
    f = np.ascontiguousarray(f, np.int32)
    a = np.array(alpha, dtype=np.float64, copy=True)
    b, n = A.shape
    kept = np.empty(b, np.uint8)
    err = np.empty(b, np.float64)
    rn = np.empty(b, np.float64)
    L = _load()
    eta = int(L.pamm_oracle_neighbourhood(_p(A), _dtype_code(A), b, n, _ld(A), _p(C), _p(f), _p(a), float(eps),
                                          _p(kept), _p(err), _p(rn)))
    return a, kept.astype(bool), err, rn, eta, float(L.pamm_oracle_beta(b, eta))


def contract(f: np.ndarray, alpha: np.ndarray, B: np.ndarray, k: int) -> np.ndarray:
    """B~[j,:] = sum_{i: f_i=j} alpha_i B_i (ApproxMM, index_add step)."""
    B = _mat(B)
    f = np.ascontiguousarray(f, np.int32)
    alpha = np.ascontiguousarray(alpha, np.float64)
    b, m = B.shape
    assert f.shape == (b,) and alpha.shape == (b,)
    Bt = np.empty((k, m), np.float64)
    rc = _load().pamm_oracle_contract(_p(f), _p(alpha), _p(B), _dtype_code(B), b, m, _ld(B), k, _p(Bt))
    if rc:
        raise ValueError("assignment out of range")
    return Bt


def weight_grad(C: np.ndarray, Bt: np.ndarray) -> np.ndarray:
    """O~ = C^T B~ (ApproxMM, last step)."""
    C = np.ascontiguousarray(C, np.float64)
    Bt = np.ascontiguousarray(Bt, np.float64)
    k, n = C.shape
    m = Bt.shape[1]
    assert Bt.shape[0] == k
    O = np.empty((n, m), np.float64)
    _load().pamm_oracle_weight_grad(_p(C), _p(Bt), k, n, m, _p(O))
    return O


def reconstruct(C: np.ndarray, f: np.ndarray, alpha: np.ndarray) -> np.ndarray:
    """A~_i = alpha_i C_{f(i)} (Eq. 3, all rows kept)."""
    C = np.ascontiguousarray(C, np.float64)
    f = np.ascontiguousarray(f, np.int32)
    alpha = np.ascontiguousarray(alpha, np.float64)
    b, n = f.shape[0], C.shape[1]
    At = np.empty((b, n), np.float64)
    _load().pamm_oracle_reconstruct(_p(C), _p(f), _p(alpha), b, n, _p(At))
    return At


def exact_product(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """O = A^T B by a plain triple loop (reduced sizes only)."""
    A, B = _mat(A), _mat(B)
    b, n = A.shape
    m = B.shape[1]
    assert B.shape[0] == b
    O = np.empty((n, m), np.float64)
    _load().pamm_oracle_exact_product(_p(A), _dtype_code(A), _ld(A), _p(B), _dtype_code(B), _ld(B), b, n, m, _p(O))
    return O


def linear_forward(X: np.ndarray, W: np.ndarray, rows=None) -> np.ndarray:
    """Z = X W (Algorithm 2, the layer's output), optionally for the listed rows of X only."""
    X, W = _mat(X), _mat(W)
    b, n = X.shape
    m = W.shape[1]
    assert W.shape[0] == n
    if rows is None:
        Z = np.empty((b, m), np.float64)
        _load().pamm_oracle_linear_forward(_p(X), _dtype_code(X), _ld(X), _p(W), _dtype_code(W), _ld(W), b, n, m,
                                           None, 0, _p(Z))
        return Z
    rows = np.ascontiguousarray(rows, np.int64)
    assert rows.min() >= 0 and rows.max() < b
    Z = np.empty((rows.size, m), np.float64)
    _load().pamm_oracle_linear_forward(_p(X), _dtype_code(X), _ld(X), _p(W), _dtype_code(W), _ld(W), b, n, m,
                                       _p(rows), rows.size, _p(Z))
    return Z


def memory_scalars(b: int, n: int, k: int) -> int:
    return int(_load().pamm_oracle_memory_scalars(b, n, k))


def gamma(b: int, m: int, k: int) -> float:
    return float(_load().pamm_oracle_gamma(b, m, k))


def num_threads() -> int:
    return int(_load().pamm_oracle_num_threads())


def pamm(A: np.ndarray, I: np.ndarray, B: np.ndarray, eps: float = float("inf")):
    """Whole path given I: returns dict(C, q, f, alpha, top1, top2, Bt, O) and, for a
    finite eps, also kept / err / eta / beta with O = beta * C^T B~."""
    C, q = gather(A, I)
    f, alpha, t1, t2 = compress(A, C, q)
    out = dict(C=C, q=q, f=f, top1=t1, top2=t2)
    beta = 1.0
    if np.isfinite(eps):
        alpha, kept, err, rn, eta, beta = neighbourhood(A, C, f, alpha, eps)
        out.update(kept=kept, err=err, rownorm=rn, eta=eta, beta=beta)
    Bt = contract(f, alpha, B, C.shape[0])
    O = weight_grad(C, Bt)
    if beta != 1.0:
        O = beta * O
    out.update(alpha=alpha, Bt=Bt, O=O)
    return out
