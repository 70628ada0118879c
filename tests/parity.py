"""GPU-vs-oracle comparison used by the parity tests (and by the smoke check).

What is compared, and how tightly:

* f: bit-exact, except rows whose two best scores differ by less than 1e-6 relative in the
  oracle (counted as ``near_tie``).  A mismatch with a larger gap is tolerated only when the
  two competing scores are closer than the rounding of their fp32 n-term sums can resolve,
  ``2 sqrt(n) 2^-24 sum_l |X_il C_jl| / ||C_j||`` for each competitor (counted as
  ``explained_by_rounding``, at most max(2, b/2000) rows); anything else fails.
* alpha, B~, dW~: the relative Frobenius error the method is specified with (1e-5 for fp32
  inputs, 1e-2 for bf16 inputs with fp32 accumulation), a second Frobenius line at what fp32
  accumulation actually delivers (1e-4 for bf16 inputs), and an element-wise bound derived
  from the arithmetic, so that a fault confined to a few elements cannot hide in the norm:
  every sum of L terms accumulated in fp32 may be off by about L 2^-24 times the sum of the
  absolute values of its terms, the bf16 hi + lo split of B~ by 2^-17 of them, and a bf16
  output by half a unit in its last place (2^-9 relative).
"""
from __future__ import annotations

import json
import os
from dataclasses import dataclass, field

import numpy as np
import torch

from oracle import pamm_oracle as orc
from paper_2506_02939_b200 import pamm, synth

NEAR_TIE = 1e-6
TOL = {"f32": 1e-5, "bf16": 1e-2}          # the stated relative Frobenius tolerances
TOL_TIGHT = {"f32": 1e-5, "bf16": 1e-4}    # what fp32 accumulation delivers (measured: <= 1.1e-5)
U32 = 2.0 ** -24                            # unit roundoff of fp32
SAFETY = 2.0                                # accumulation order and rounding mode inside the tensor core are not specified


def to_device(a: np.ndarray, ld: int | None = None) -> torch.Tensor:
    """Storage array (fp32 / bf16 bits) -> CUDA tensor, optionally with a padded row stride."""
    if a.dtype == np.uint16:
        t = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    else:
        t = torch.from_numpy(a)
    t = t.cuda()
    if ld is not None and ld != a.shape[1]:
        buf = torch.zeros((a.shape[0], ld), dtype=t.dtype, device="cuda")
        buf[:, : a.shape[1]] = t
        t = buf[:, : a.shape[1]]
    return t


def from_device_bits(t: torch.Tensor) -> np.ndarray:
    t = t.contiguous().cpu()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def to_f64(t: torch.Tensor) -> np.ndarray:
    """A device result (fp32 or bf16) widened exactly to fp64."""
    return t.detach().to(torch.float64).cpu().numpy()


def abs_bits(a: np.ndarray) -> np.ndarray:
    """|a| in the same storage type (bf16 bit patterns or fp32)."""
    return (a & np.uint16(0x7FFF)) if a.dtype == np.uint16 else np.abs(a)


def rel_fro(a: np.ndarray, ref: np.ndarray) -> float:
    den = float(np.linalg.norm(ref.ravel()))
    num = float(np.linalg.norm((a.astype(np.float64) - ref).ravel()))
    return num / den if den > 0 else num


def worst_ratio(a: np.ndarray, ref: np.ndarray, bound: np.ndarray) -> float:
    """max over the elements of |a - ref| / bound (0 where both vanish)."""
    err = np.abs(a.astype(np.float64) - ref)
    with np.errstate(divide="ignore", invalid="ignore"):
        r = np.where(bound > 0, err / bound, np.where(err > 0, np.inf, 0.0))
    return float(r.max()) if r.size else 0.0


def check_elementwise(name: str, a: np.ndarray, ref: np.ndarray, bound: np.ndarray, rep: "Report") -> None:
    """Every element within its own bound; the worst ratio is recorded."""
    w = worst_ratio(a, ref, bound)
    rep.elem[name] = w
    if not w <= 1.0:
        err = np.abs(a.astype(np.float64) - ref)
        with np.errstate(divide="ignore", invalid="ignore"):
            r = np.where(bound > 0, err / bound, np.where(err > 0, np.inf, 0.0))
        at = np.unravel_index(int(np.argmax(r)), r.shape)
        raise AssertionError(f"{name}: element {at} is off by {err[at]:.3e}, {w:.2f}x its bound {bound[at]:.3e} "
                             f"(got {a[at]!r}, want {ref[at]!r}); {int((r > 1).sum())} elements over")


@dataclass
class Report:
    b: int
    k: int
    mismatches: int = 0
    near_tie: int = 0
    explained_by_rounding: int = 0
    unexplained: int = 0
    near_tie_rows: list = field(default_factory=list)
    rounding_rows: list = field(default_factory=list)     # (row, relative gap) of the rows explained by rounding
    err: dict = field(default_factory=dict)                # relative Frobenius errors
    elem: dict = field(default_factory=dict)               # worst |error| / element-wise bound

    def summary(self) -> dict:
        return dict(b=self.b, k=self.k, f_mismatches=self.mismatches, near_tie=self.near_tie,
                    explained_by_rounding=self.explained_by_rounding, rounding_rows=self.rounding_rows[:8],
                    rel_fro={q: float(f"{v:.3e}") for q, v in self.err.items()},
                    worst_over_bound={q: float(f"{v:.3e}") for q, v in self.elem.items()})


def record(name: str, rep: Report) -> None:
    """Append the report to the file named by PAMM_PARITY_REPORT (one JSON line per case), if set."""
    path = os.environ.get("PAMM_PARITY_REPORT")
    print(name, json.dumps(rep.summary()))
    if path:
        with open(path, "a") as fh:
            fh.write(json.dumps(dict(case=name, **rep.summary())) + "\n")


def check_assignment(X: np.ndarray, C64, q, f_gpu, f_o, alpha_o, t1, t2, rep: Report):
    """Classify rows where the GPU's f differs from the oracle's; returns the
    oracle's (f, alpha) with the tolerated rows overridden by the GPU's choice."""
    n = X.shape[1]
    diff = np.nonzero(f_gpu != f_o)[0]
    rep.mismatches = int(diff.size)
    f_e, a_e = f_o.copy(), alpha_o.copy()
    for i in diff:
        s, sc, ab = orc.row_scores(X, int(i), C64, q)
        g = int(f_gpu[i])
        top = sc[f_o[i]]
        gap = (top - sc[g]) / top if top > 0 else 0.0
        if gap < NEAR_TIE:
            rep.near_tie += 1
            rep.near_tie_rows.append(int(i))
        else:
            # what the rounding of an n-term fp32 sum typically leaves of each competing score
            def bound(j):
                return SAFETY * np.sqrt(n) * U32 * ab[j] / np.sqrt(q[j]) if q[j] > 0 else 0.0
            if top - sc[g] <= bound(int(f_o[i])) + bound(g):
                rep.explained_by_rounding += 1
                rep.rounding_rows.append((int(i), float(f"{gap:.3e}")))
            else:
                rep.unexplained += 1
                continue
        f_e[i] = g
        a_e[i] = s[g] / q[g] if q[g] > 0 else 0.0
    return f_e, a_e


def check_select(X, idx_g, C_g, invn_g, k, idx_in, seed):
    """Step 1: the indices, C as exact row copies, the generator norms."""
    b = X.shape[0]
    if idx_in is None:
        expect = pamm.draw_indices_host(b, k, seed).numpy()
        assert np.array_equal(idx_g, expect), "device-drawn indices differ from the host draw"
        assert np.all(np.diff(idx_g) > 0) and idx_g[0] >= 0 and idx_g[-1] < b
    else:
        assert np.array_equal(idx_g, np.asarray(idx_in, np.int32))
    assert np.array_equal(C_g, X[idx_g]), "C is not an exact copy of the selected rows"
    C64, q = orc.gather(X, idx_g)
    nz = q > 0
    assert np.allclose(invn_g[:k][nz], 1 / np.sqrt(q[nz]), rtol=1e-6, atol=0)
    assert np.allclose(invn_g[k:][nz], 1 / q[nz], rtol=1e-6, atol=0)
    assert np.all(invn_g[:k][~nz] == 0) and np.all(invn_g[k:][~nz] == 0)
    return C64, q


def check_compress(X, C64, q, f_g, a_g, rep: Report, dtype: str):
    """Step 2: f against the oracle row by row, alpha in norm and element by element."""
    b, n = X.shape
    k = C64.shape[0]
    f_o, a_o, t1, t2 = orc.compress(X, C64, q)
    f_e, a_e = check_assignment(X, C64, q, f_g, f_o, a_o, t1, t2, rep)
    assert rep.unexplained == 0, f"{rep.unexplained} rows differ in f beyond the near-tie / rounding allowance"
    assert rep.explained_by_rounding <= max(2, b // 2000), rep
    assert f_g.min() >= 0 and f_g.max() < k
    rep.err["alpha"] = rel_fro(a_g, a_e)
    assert rep.err["alpha"] <= TOL[dtype] and rep.err["alpha"] <= TOL_TIGHT[dtype], rep.err
    # alpha_i = S / q with S an n-term fp32 sum: |X_i| |C_f| / q bounds the sum of its terms' absolute values
    X64 = synth.to_f64(X)
    rown = np.sqrt(np.einsum("il,il->i", X64, X64))
    qf = q[f_e]
    cauchy = np.divide(rown, np.sqrt(qf), out=np.zeros_like(rown), where=qf > 0)
    check_elementwise("alpha", a_g, a_e, SAFETY * (n + 2) * U32 * cauchy, rep)
    return f_e, a_e


def check_contract(f_g, a_g, dY, k, Bt_g, rep: Report, dtype: str, name="Btilde_stage"):
    """Step 3, stage-wise: the oracle's contract fed the GPU's f and alpha."""
    Bt_o = orc.contract(f_g, a_g.astype(np.float64), dY, k)
    rep.err[name] = rel_fro(Bt_g, Bt_o)
    assert np.all(np.isfinite(Bt_g))
    assert rep.err[name] <= TOL[dtype] and rep.err[name] <= TOL_TIGHT[dtype], rep.err
    # segment sums of L_j terms: error <= about L_j 2^-24 times the sum of |alpha_i dY_i|
    Bt_abs = orc.contract(f_g, np.abs(a_g).astype(np.float64), abs_bits(dY), k)
    seg_len = np.bincount(f_g, minlength=k).astype(np.float64)
    check_elementwise(name, Bt_g, Bt_o, SAFETY * (seg_len[:, None] + 2) * U32 * Bt_abs, rep)
    return Bt_o, Bt_abs, seg_len


def product_bound(C64, Bt_abs, k, rel_terms, out_bf16, ref):
    """Element-wise bound of dW = C^T B~: `rel_terms` times sum_j |C_jr| |B~_jc|, plus the rounding of a bf16 output."""
    S = orc.weight_grad(np.abs(C64), Bt_abs)
    bound = SAFETY * rel_terms * S
    if out_bf16:
        bound = bound + 2.0 ** -8 * np.abs(ref)
    return bound


def run_and_compare(X: np.ndarray, dY: np.ndarray, k: int, seed: int = 0, idx_in: np.ndarray | None = None,
                    fused: bool = True, ldx: int | None = None, ldy: int | None = None,
                    dw_dtype=None, layout: int = pamm.DW_NM, f_dtype=None, products: bool = False) -> Report:
    """Run the CUDA path through the C ABI and compare every output with the oracle.

    ``dw_dtype`` / ``layout``: how dW is stored; ``f_dtype``: storage type of f; ``products``: the forward
    pass leaves its per-block counts of f for the backward pass."""
    dtype = "bf16" if X.dtype == np.uint16 else "f32"
    tol = TOL[dtype]
    b, n = X.shape
    m = dY.shape[1]
    rep = Report(b=b, k=k)
    Xd, dYd = to_device(X, ldx), to_device(dY, ldy)
    idx_d = None if idx_in is None else torch.from_numpy(np.asarray(idx_in, np.int32)).cuda()
    out_bf16 = dw_dtype == torch.bfloat16
    sp = pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, k, pamm.BF16 if dtype == "bf16" else pamm.F32) if products else None

    # ---- GPU ------------------------------------------------------------------
    if fused:
        idx, C, invn, f, alpha = pamm.compress_fused(Xd, k, seed, idx_in=idx_d, sort_products=sp, f_dtype=f_dtype)
        Bt = pamm.alloc_matrix(k, m, torch.float32)
        Bt.fill_(float("nan"))
        dW = pamm.contract_weight_grad(C, f, alpha, dYd, Btilde=Bt, dw_dtype=dw_dtype, layout=layout, sort_products=sp)
    else:
        idx, C, invn = pamm.select_generators(Xd, k, seed, idx_in=idx_d)
        f, alpha = pamm.compress(Xd, C, invn, sort_products=sp, f_dtype=f_dtype)
        Bt = pamm.contract(f, alpha, dYd, k, sort_products=sp)
        dW = pamm.weight_grad(C, Bt, dw_dtype=dw_dtype, layout=layout)
    status = pamm.last_device_status()
    assert status == pamm.OK, pamm.status_string(status)
    idx_g = idx.cpu().numpy()
    C_g = from_device_bits(C)
    invn_g = invn.cpu().numpy().astype(np.float64)
    f_g = f.cpu().numpy().astype(np.int64)
    if f.dtype == torch.int16:
        f_g &= 0xFFFF                                                 # unsigned 16-bit entries in int16 storage
    f_g = f_g.astype(np.int32)
    a_g = alpha.cpu().numpy()
    Bt_g = Bt.cpu().numpy()
    dW_g = to_f64(dW)
    if layout == pamm.DW_MN:
        assert dW_g.shape == (m, n)
        dW_g = dW_g.T
    assert dW_g.shape == (n, m)

    C64, q = check_select(X, idx_g, C_g, invn_g, k, idx_in, seed)
    f_e, a_e = check_compress(X, C64, q, f_g, a_g, rep, dtype)
    Bt_o, Bt_abs, seg_len = check_contract(f_g, a_g, dY, k, Bt_g, rep, dtype)

    # ---- step 4 (stage-wise): oracle product fed the GPU's C and B~ --------------
    # 2k accumulated terms in fp32; on the tensor-core path B~ enters as bf16 hi + lo (2^-17)
    split = 2.0 ** -17 if dtype == "bf16" else 0.0
    dW_o = orc.weight_grad(C64, Bt_g.astype(np.float64))
    rep.err["dW_stage"] = rel_fro(dW_g, dW_o)
    # a bf16 dW carries its own rounding (half a unit in the last place, 2^-9 relative) on top of the stated tolerance
    tight = max(TOL_TIGHT[dtype], 2.0 ** -8) if out_bf16 else TOL_TIGHT[dtype]
    tol = max(tol, 2.0 ** -8) if out_bf16 else tol
    assert rep.err["dW_stage"] <= tol and rep.err["dW_stage"] <= tight, rep.err
    Bt_g_abs = np.abs(Bt_g.astype(np.float64))
    check_elementwise("dW_stage", dW_g, dW_o, product_bound(C64, Bt_g_abs, k, (2 * k + 2) * U32 + split, out_bf16, dW_o), rep)

    # ---- end to end: the oracle's own chain, tolerated rows overridden ------------
    # on top of the product's own rounding: alpha carries the n-term sums' error, B~ the segment sums'
    Bt_e = orc.contract(f_e, a_e, dY, k)
    dW_e = orc.weight_grad(C64, Bt_e)
    rep.err["dW_e2e"] = rel_fro(dW_g, dW_e)
    assert rep.err["dW_e2e"] <= tol and rep.err["dW_e2e"] <= tight, rep.err
    Bt_e_abs = orc.contract(f_e, np.abs(a_e), abs_bits(dY), k)
    # alpha's own relative error can exceed n 2^-24 where the row is nearly orthogonal to its generator:
    # bound it through |X_i| |C_f| / q as in check_compress, carried into B~ by |dY|
    X64 = synth.to_f64(X)
    rown = np.sqrt(np.einsum("il,il->i", X64, X64))
    qf = q[f_e]
    cauchy = np.divide(rown, np.sqrt(qf), out=np.zeros_like(rown), where=qf > 0)
    Bt_alpha_err = orc.contract(f_e, (n + 2) * U32 * cauchy, abs_bits(dY), k)
    S_alpha = orc.weight_grad(np.abs(C64), Bt_alpha_err)
    rel_terms = (2 * k + 2) * U32 + split + (float(seg_len.max()) + 2) * U32
    bound = product_bound(C64, Bt_e_abs, k, rel_terms, out_bf16, dW_e) + SAFETY * S_alpha
    check_elementwise("dW_e2e", dW_g, dW_e, bound, rep)
    return rep
