"""A linear layer whose backward pass keeps the compressed input only (Algorithms 2 and 3).

Forward: ``Z = X W`` and ``Compress(flatten(X))``.  For bf16 layers both come out of ONE kernel
of the CUDA library (``pamm_linear_forward``: the scores are extra output columns of the
product, so X is not read a second time); other dtypes take torch's GEMM for Z and the
library's stand-alone compression.  The layer saves (C, f, alpha, W) and lets go of X.
Backward: the weight gradient is ``ApproxMM(C, alpha, f, dZ) = C^T B~`` through the library,
the input gradient ``dX = dZ W^T`` is exact (for bf16 layers the library's tensor-core product
``pamm_linear_backward_input``, else torch).  Meant for the fused Q|K|V projection: ``W`` is n x m
with m = |Q| + |K| + |V|, as in the paper's notation.
"""
from __future__ import annotations

import math

import torch

from . import pamm


def _rows(t: torch.Tensor, cols: int) -> torch.Tensor:
    """(…, cols) -> contiguous (rows, cols) view the library accepts (16-byte aligned rows)."""
    t2 = t.reshape(-1, cols)
    if t2.stride(1) != 1 or (t2.stride(0) * t2.element_size()) % 16 or t2.data_ptr() % 16:
        padded = pamm.alloc_matrix(t2.shape[0], cols, t2.dtype, t2.device)
        padded.copy_(t2)
        t2 = padded
    return t2


class PammLinearFunction(torch.autograd.Function):
    @staticmethod
    def forward(ctx, X, W, k, seed):
        n, m = W.shape
        X2 = _rows(X.detach(), n)
        b = X2.shape[0]
        f_dtype = torch.uint8 if k <= 256 else torch.int16 if k <= 65536 else torch.int32
        # the pass also leaves its per-block counts of f (a few KiB): the backward's counting sort starts from them
        sp = pamm.alloc_workspace(pamm.WS_COMPRESS, b, n, m, int(k), pamm.BF16 if X2.dtype == torch.bfloat16 else pamm.F32,
                                  X2.device)
        Wd = W.detach()
        one_kernel = (X2.dtype == torch.bfloat16 and Wd.dtype == torch.bfloat16 and 16 <= k <= 4096 and n >= 8 and m >= 8
                      and Wd.is_contiguous() and (m * 2) % 16 == 0 and Wd.data_ptr() % 16 == 0)
        if one_kernel:
            Z2, _, C, _, f, alpha = pamm.linear_forward(X2, Wd, int(k), int(seed), sort_products=sp, f_dtype=f_dtype)
            Z = Z2.reshape(*X.shape[:-1], m)
        else:
            Z = X @ W
            _, C, _, f, alpha = pamm.compress_fused(X2, int(k), int(seed), sort_products=sp, f_dtype=f_dtype)
        ctx.save_for_backward(C, f, alpha, sp, W)      # k n + 2 b scalars instead of b n
        return Z

    @staticmethod
    def backward(ctx, dZ):
        C, f, alpha, sp, W = ctx.saved_tensors
        n, m = W.shape
        dX = None
        if ctx.needs_input_grad[0]:
            Wd = W.detach()
            dZr = _rows(dZ, m)
            own = (dZr.dtype == torch.bfloat16 and Wd.dtype == torch.bfloat16 and n >= 8 and m >= 8 and Wd.is_contiguous()
                   and dZr.stride(1) == 1 and (m * 2) % 16 == 0 and (dZr.stride(0) * 2) % 16 == 0
                   and Wd.data_ptr() % 16 == 0 and dZr.data_ptr() % 16 == 0)
            if own:      # Algorithm 3's other product, through the library's tensor-core kernel
                dX = pamm.linear_backward_input(dZr, Wd).reshape(*dZ.shape[:-1], n)
            else:
                dX = dZ @ W.t()
        dW = None
        if ctx.needs_input_grad[1]:
            dZ2 = _rows(dZ.to(C.dtype), m)
            direct = W.dtype in (torch.float32, torch.bfloat16)      # the product kernel writes these itself
            dW = pamm.contract_weight_grad(C, f, alpha, dZ2, dw_dtype=W.dtype if direct else torch.float32, sort_products=sp)
            if not direct:
                dW = dW.to(W.dtype)
        return dX, dW, None, None


class PammLinear(torch.nn.Module):
    """``Z = X W`` with PAMM in the backward pass; ``r`` is the compression ratio k / b (Section 4.1)."""

    def __init__(self, n: int, m: int, r: float = 1.0 / 512, dtype=torch.bfloat16, device="cuda", seed: int = 0):
        super().__init__()
        self.weight = torch.nn.Parameter(torch.empty((n, m), dtype=dtype, device=device))
        torch.nn.init.normal_(self.weight, std=1.0 / math.sqrt(n))
        self.r = float(r)
        self.seed = int(seed)
        self.calls = 0

    def forward(self, X):
        b = X.numel() // X.shape[-1]
        k = max(1, min(b, math.ceil(self.r * b)))
        self.calls += 1                                   # fresh generators every step (Appendix "LLaMA-1B Runtime Breakdown")
        return PammLinearFunction.apply(X, self.weight, k, self.seed + self.calls)
