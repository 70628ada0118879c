"""Thin binding to the PAMM CUDA library (C ABI declared in ``include/pamm.h``).

Argument marshalling only: every step of the path runs in the library's kernels.
torch is used for device memory and streams.  Importing this module fails
loudly when the library has not been built; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libpamm_b200.so"
if not _LIB_PATH.exists():
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2506_02939_b200.build` "
        "(nvcc, sm_100a). The PAMM path has no fallback.")
_lib = ctypes.CDLL(str(_LIB_PATH))

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_BAD_INDEX = range(7)
F32, BF16 = 0, 1
DW_NM, DW_MN = 0, 1                      # layout of the weight gradient: n x m (the paper's), or m x n (out x in)
IDX_I32, IDX_U16, IDX_U8 = 0, 1, 2       # storage type of the assignment f
WS_COMPRESS, WS_CONTRACT, WS_STEP_HOST = 0, 1, 2

_i64, _vp, _ci, _u64, _sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_uint64, ctypes.c_size_t

_SIGNATURES = {
    "pamm_status_string": ([_ci], ctypes.c_char_p),
    "pamm_version": ([], _ci),
    "pamm_last_error_detail": ([], ctypes.c_char_p),
    "pamm_workspace_bytes": ([_ci, _i64, _i64, _i64, _i64, _ci], _sz),
    "pamm_saved_bytes": ([_i64, _i64, _i64, _ci, _ci, _vp], _ci),
    "pamm_draw_indices_host": ([_i64, _i64, _u64, _vp], _ci),
    "pamm_select_generators": ([_vp, _i64, _i64, _i64, _ci, _i64, _u64, _vp, _vp, _vp, _i64, _vp, _vp], _ci),
    "pamm_compress": ([_vp, _i64, _i64, _i64, _ci, _vp, _i64, _i64, _vp, _vp, _ci, _vp, _vp, _sz, _vp], _ci),
    "pamm_compress_fused": ([_vp, _i64, _i64, _i64, _ci, _i64, _u64, _vp, _vp, _vp, _i64, _vp, _vp, _ci, _vp, _vp, _sz, _vp], _ci),
    "pamm_compress_projections": ([_vp, _i64, _i64, _i64, _ci, _vp, _i64, _i64, _i64, _vp, _vp, _ci, _vp, _i64, _vp, _sz, _vp], _ci),
    "pamm_linear_forward": ([_vp, _i64, _i64, _i64, _vp, _i64, _i64, _ci, _i64, _u64, _vp, _vp, _vp, _i64, _vp, _vp, _i64, _vp, _ci,
                             _vp, _vp, _sz, _vp], _ci),
    "pamm_linear_backward_input": ([_vp, _i64, _i64, _i64, _vp, _i64, _i64, _ci, _vp, _i64, _vp], _ci),
    "pamm_contract": ([_vp, _ci, _vp, _vp, _i64, _i64, _i64, _ci, _i64, _vp, _i64, _vp, _vp, _sz, _vp], _ci),
    "pamm_weight_grad": ([_vp, _i64, _i64, _i64, _ci, _vp, _i64, _i64, _vp, _i64, _ci, _ci, _vp], _ci),
    "pamm_compress_eps": ([_vp, _i64, _i64, _i64, _ci, _vp, _i64, _i64, _vp, ctypes.c_float, _vp, _ci, _vp, _vp, _vp, _sz, _vp], _ci),
    "pamm_weight_grad_beta": ([_vp, _i64, _i64, _i64, _ci, _vp, _i64, _i64, _i64, _vp, _vp, _i64, _ci, _ci, _vp], _ci),
    "pamm_weight_grad_accumulate": ([_vp, _i64, _i64, _i64, _ci, _vp, _i64, _i64, _vp, _i64, _ci, _vp], _ci),
    "pamm_contract_weight_grad": ([_vp, _i64, _i64, _vp, _ci, _vp, _vp, _i64, _i64, _i64, _ci, _i64, _vp, _i64, _vp, _i64,
                                   _ci, _ci, _vp, _vp, _sz, _vp], _ci),
    "pamm_qkv_step_host": ([_vp, _vp, _i64, _i64, _i64, _ci, _i64, _u64, _vp, _vp, _vp, _vp, _sz, _vp], _ci),
    "pamm_contract_no_alloc": ([_vp, _vp, _vp, _i64, _i64, _i64, _ci, _i64, _vp, _i64, _vp], _ci),
    "pamm_last_device_status": ([_vp], _ci),
    "pamm_selftest_bounded_wait": ([_vp], _ci),
    "pamm_probe_read": ([_ci, _vp, _i64, _i64, _i64, _vp, _vp, _vp], _ci),
    "pamm_launch_count": ([], ctypes.c_ulonglong),
    "pamm_set_profile_events": ([_ci, _vp, _vp], _ci),
}
for _name, (_args, _res) in _SIGNATURES.items():
    _fn = getattr(_lib, _name)
    _fn.argtypes, _fn.restype = _args, _res

EXPORTED = tuple(_SIGNATURES)


class PammError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = _lib.pamm_last_error_detail().decode() if code == ERR_CUDA else ""
        super().__init__(f"{where}: {status_string(code)} (status {code})" + (f": {detail}" if detail else ""))


def status_string(code: int) -> str:
    return _lib.pamm_status_string(int(code)).decode()


def version() -> int:
    return int(_lib.pamm_version())


def _check(code: int, where: str) -> None:
    if code != OK:
        raise PammError(code, where)


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"PAMM inputs are float32 or bfloat16, got {t.dtype}")


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _ld(t: torch.Tensor) -> int:
    if t.dim() != 2 or t.stride(1) != 1:
        raise ValueError("need a 2-D row-major tensor (a row stride is allowed)")
    return t.stride(0)


def _stream(stream) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


_prep_keep = None      # while a call is being prepared: the tensors it allocates, kept alive with the prepared call


def _empty(*args, **kwargs) -> torch.Tensor:
    t = torch.empty(*args, **kwargs)
    if _prep_keep is not None:
        _prep_keep.append(t)
    return t


def alloc_matrix(rows: int, cols: int, dtype, device="cuda") -> torch.Tensor:
    """rows x cols view whose row stride is padded so that every row starts 16-byte aligned."""
    per = 16 // torch.empty((), dtype=dtype).element_size()
    ld = (cols + per - 1) // per * per
    return _empty((rows, ld), dtype=dtype, device=device)[:, :cols]


def workspace_bytes(kind: int, b: int, n: int, m: int, k: int, dtype: int) -> int:
    r = _lib.pamm_workspace_bytes(kind, b, n, m, k, dtype)
    if r == ctypes.c_size_t(-1).value:
        raise PammError(ERR_INVALID_ARG, "pamm_workspace_bytes")
    return int(r)


def alloc_workspace(kind: int, b: int, n: int, m: int, k: int, dtype: int, device="cuda") -> torch.Tensor:
    return _empty(max(256, workspace_bytes(kind, b, n, m, k, dtype)), dtype=torch.uint8, device=device)


def draw_indices_host(b: int, k: int, seed: int) -> torch.Tensor:
    out = _empty(k, dtype=torch.int32)
    _check(_lib.pamm_draw_indices_host(b, k, seed, _ptr(out)), "pamm_draw_indices_host")
    return out


def select_generators(X, k: int, seed: int = 0, idx_in=None, idx_out=None, C=None, c_invnorm=None, stream=None):
    b, n = X.shape
    idx_out = _empty(k, dtype=torch.int32, device=X.device) if idx_out is None else idx_out
    C = alloc_matrix(k, n, X.dtype, X.device) if C is None else C
    c_invnorm = _empty(2 * k, dtype=torch.float32, device=X.device) if c_invnorm is None else c_invnorm
    _check(_lib.pamm_select_generators(_ptr(X), _ld(X), b, n, _dt(X), k, seed, _ptr(idx_in), _ptr(idx_out),
                                       _ptr(C), _ld(C), _ptr(c_invnorm), _stream(stream)), "pamm_select_generators")
    return idx_out, C, c_invnorm


_F_TYPES = {torch.int32: IDX_I32, torch.uint16: IDX_U16, torch.int16: IDX_U16, torch.uint8: IDX_U8}


def _ft(f: torch.Tensor) -> int:
    """Storage type of an assignment vector (narrow entries are unsigned whatever torch calls them)."""
    try:
        return _F_TYPES[f.dtype]
    except KeyError:
        raise TypeError(f"f is int32, uint16 (or int16 storage) or uint8, got {f.dtype}") from None


def _new_f(shape, f_dtype, device):
    return _empty(shape, dtype=torch.int32 if f_dtype is None else f_dtype, device=device)


def _bytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


def compress(X, C, c_invnorm, f=None, alpha=None, sort_products=None, f_dtype=None, stream=None):
    """``sort_products``: optional uint8 tensor of ``workspace_bytes(WS_COMPRESS, ...)`` bytes that receives the
    per-block counts of f for the backward pass."""
    b, n = X.shape
    k = C.shape[0]
    f = _new_f(b, f_dtype, X.device) if f is None else f
    alpha = _empty(b, dtype=torch.float32, device=X.device) if alpha is None else alpha
    _check(_lib.pamm_compress(_ptr(X), _ld(X), b, n, _dt(X), _ptr(C), _ld(C), k, _ptr(c_invnorm), _ptr(f), _ft(f),
                              _ptr(alpha), _ptr(sort_products), _bytes(sort_products), _stream(stream)), "pamm_compress")
    return f, alpha


def compress_projections(X, C, c_invnorm, sets: int, f=None, alpha=None, sort_products=None, f_dtype=None, stream=None):
    """One compression per projection in one pass over X: ``C`` holds ``sets * k`` generator rows and ``c_invnorm``
    ``sets * 2k`` norms (one ``select_generators`` call per set); returns f and alpha of shape (sets, b)."""
    b, n = X.shape
    k = C.shape[0] // sets
    f = _new_f((sets, b), f_dtype, X.device) if f is None else f
    alpha = _empty((sets, b), dtype=torch.float32, device=X.device) if alpha is None else alpha
    _check(_lib.pamm_compress_projections(_ptr(X), _ld(X), b, n, _dt(X), _ptr(C), _ld(C), k, sets, _ptr(c_invnorm), _ptr(f),
                                          _ft(f), _ptr(alpha), f.stride(0), _ptr(sort_products), _bytes(sort_products),
                                          _stream(stream)), "pamm_compress_projections")
    return f, alpha


def compress_eps(X, C, c_invnorm, eps: float, f=None, alpha=None, dropped=None, sort_products=None, f_dtype=None,
                 stream=None):
    """compress with the neighbourhood condition (Eq. 2): rows farther than eps ||X_i|| from their representative
    get alpha = 0; ``dropped`` (device int32[1]) receives their number."""
    b, n = X.shape
    k = C.shape[0]
    f = _new_f(b, f_dtype, X.device) if f is None else f
    alpha = _empty(b, dtype=torch.float32, device=X.device) if alpha is None else alpha
    dropped = _empty(1, dtype=torch.int32, device=X.device) if dropped is None else dropped
    _check(_lib.pamm_compress_eps(_ptr(X), _ld(X), b, n, _dt(X), _ptr(C), _ld(C), k, _ptr(c_invnorm), float(eps), _ptr(f),
                                  _ft(f), _ptr(alpha), _ptr(dropped), _ptr(sort_products), _bytes(sort_products),
                                  _stream(stream)), "pamm_compress_eps")
    return f, alpha, dropped


def _new_dW(n: int, m: int, dw_dtype, layout: int, device):
    rows, cols = (m, n) if layout == DW_MN else (n, m)
    return alloc_matrix(rows, cols, torch.float32 if dw_dtype is None else dw_dtype, device)


def weight_grad(C, Btilde, dW=None, dw_dtype=None, layout: int = DW_NM, stream=None):
    """dW = C^T B~: n x m (``DW_NM``) or its transpose m x n (``DW_MN``), fp32 or bf16."""
    k, n = C.shape
    m = Btilde.shape[1]
    dW = _new_dW(n, m, dw_dtype, layout, C.device) if dW is None else dW
    _check(_lib.pamm_weight_grad(_ptr(C), _ld(C), k, n, _dt(C), _ptr(Btilde), _ld(Btilde), m, _ptr(dW), _ld(dW), _dt(dW),
                                 layout, _stream(stream)), "pamm_weight_grad")
    return dW


def weight_grad_beta(C, Btilde, b: int, dropped, dW=None, dw_dtype=None, layout: int = DW_NM, stream=None):
    """dW = beta C^T B~ with beta = b / (b - eta), eta read from ``dropped`` on the device (Eq. 4-5)."""
    k, n = C.shape
    m = Btilde.shape[1]
    dW = _new_dW(n, m, dw_dtype, layout, C.device) if dW is None else dW
    _check(_lib.pamm_weight_grad_beta(_ptr(C), _ld(C), k, n, _dt(C), _ptr(Btilde), _ld(Btilde), m, b, _ptr(dropped),
                                      _ptr(dW), _ld(dW), _dt(dW), layout, _stream(stream)), "pamm_weight_grad_beta")
    return dW


def weight_grad_accumulate(C, Btilde, dW, layout: int = DW_NM, stream=None):
    """dW += C^T B~ (gradient accumulation over micro-batches); dW is fp32."""
    k, n = C.shape
    m = Btilde.shape[1]
    if dW.dtype != torch.float32:
        raise TypeError("gradients are accumulated in float32")
    _check(_lib.pamm_weight_grad_accumulate(_ptr(C), _ld(C), k, n, _dt(C), _ptr(Btilde), _ld(Btilde), m, _ptr(dW), _ld(dW),
                                            layout, _stream(stream)), "pamm_weight_grad_accumulate")
    return dW


def compress_fused(X, k: int, seed: int = 0, idx_in=None, idx_out=None, C=None, c_invnorm=None, f=None, alpha=None,
                   sort_products=None, f_dtype=None, stream=None):
    b, n = X.shape
    dev = X.device
    idx_out = _empty(k, dtype=torch.int32, device=dev) if idx_out is None else idx_out
    C = alloc_matrix(k, n, X.dtype, dev) if C is None else C
    c_invnorm = _empty(2 * k, dtype=torch.float32, device=dev) if c_invnorm is None else c_invnorm
    f = _new_f(b, f_dtype, dev) if f is None else f
    alpha = _empty(b, dtype=torch.float32, device=dev) if alpha is None else alpha
    _check(_lib.pamm_compress_fused(_ptr(X), _ld(X), b, n, _dt(X), k, seed, _ptr(idx_in), _ptr(idx_out), _ptr(C),
                                    _ld(C), _ptr(c_invnorm), _ptr(f), _ft(f), _ptr(alpha), _ptr(sort_products),
                                    _bytes(sort_products), _stream(stream)), "pamm_compress_fused")
    return idx_out, C, c_invnorm, f, alpha


def linear_forward(X, W, k: int, seed: int = 0, idx_in=None, Z=None, idx_out=None, C=None, c_invnorm=None, f=None, alpha=None,
                   sort_products=None, f_dtype=None, stream=None):
    """Algorithm 2 in one tensor-core kernel: ``Z = X W`` (W is n x m) and the compression of X.  bf16 only."""
    b, n = X.shape
    m = W.shape[1]
    dev = X.device
    Z = alloc_matrix(b, m, X.dtype, dev) if Z is None else Z
    idx_out = _empty(k, dtype=torch.int32, device=dev) if idx_out is None else idx_out
    C = alloc_matrix(k, n, X.dtype, dev) if C is None else C
    c_invnorm = _empty(2 * k, dtype=torch.float32, device=dev) if c_invnorm is None else c_invnorm
    f = _new_f(b, f_dtype, dev) if f is None else f
    alpha = _empty(b, dtype=torch.float32, device=dev) if alpha is None else alpha
    _check(_lib.pamm_linear_forward(_ptr(X), _ld(X), b, n, _ptr(W), _ld(W), m, _dt(X), k, seed, _ptr(idx_in), _ptr(idx_out),
                                    _ptr(C), _ld(C), _ptr(c_invnorm), _ptr(Z), _ld(Z), _ptr(f), _ft(f), _ptr(alpha),
                                    _ptr(sort_products), _bytes(sort_products), _stream(stream)), "pamm_linear_forward")
    return Z, idx_out, C, c_invnorm, f, alpha


def linear_backward_input(dZ, W, dX=None, stream=None):
    """Algorithm 3's other product through the same tensor-core kernel: ``dX = dZ W^T`` (dZ is b x m, W n x m).  bf16 only."""
    b, m = dZ.shape
    n = W.shape[0]
    dX = alloc_matrix(b, n, dZ.dtype, dZ.device) if dX is None else dX
    _check(_lib.pamm_linear_backward_input(_ptr(dZ), _ld(dZ), b, m, _ptr(W), _ld(W), n, _dt(dZ), _ptr(dX), _ld(dX),
                                           _stream(stream)), "pamm_linear_backward_input")
    return dX


def contract(f, alpha, dY, k: int, Btilde=None, sort_products=None, workspace=None, stream=None):
    b, m = dY.shape
    Btilde = alloc_matrix(k, m, torch.float32, dY.device) if Btilde is None else Btilde
    if workspace is None:
        workspace = alloc_workspace(WS_CONTRACT, b, 1, m, k, _dt(dY), dY.device)
    _check(_lib.pamm_contract(_ptr(f), _ft(f), _ptr(alpha), _ptr(dY), _ld(dY), b, m, _dt(dY), k, _ptr(Btilde), _ld(Btilde),
                              _ptr(sort_products), _ptr(workspace), workspace.numel(), _stream(stream)), "pamm_contract")
    return Btilde


NO_ALLOC_SCRATCH_BYTES = 8 << 20


def contract_no_alloc(f, alpha, dY, k: int, Btilde, stream=None):
    """``contract`` for callers that may not allocate device memory where they need B~ (a plugin inside a host
    application that owns the memory budget, a latency-critical loop that cannot afford cudaMalloc's device
    synchronisation, a callback running while the framework's allocator is locked).  The scratch is a fixed
    8 MiB array inside the library, shared by every call on the device: keep calls on one stream (overlapping
    calls race on it), make the first call on a device outside stream capture, and pass ``Btilde`` yourself --
    this wrapper allocates nothing either.  Problems whose scratch would not fit raise ``ERR_WORKSPACE``."""
    b, m = dY.shape
    _check(_lib.pamm_contract_no_alloc(_ptr(f), _ptr(alpha), _ptr(dY), _ld(dY), b, m, _dt(dY), k, _ptr(Btilde),
                                       _ld(Btilde), _stream(stream)), "pamm_contract_no_alloc")
    return Btilde


def contract_weight_grad(C, f, alpha, dY, Btilde=None, dW=None, dw_dtype=None, layout: int = DW_NM, sort_products=None,
                         workspace=None, stream=None):
    k, n = C.shape
    b, m = dY.shape
    dW = _new_dW(n, m, dw_dtype, layout, C.device) if dW is None else dW
    if workspace is None:
        workspace = alloc_workspace(WS_CONTRACT, b, n, m, k, _dt(dY), dY.device)
    _check(_lib.pamm_contract_weight_grad(_ptr(C), _ld(C), n, _ptr(f), _ft(f), _ptr(alpha), _ptr(dY), _ld(dY), b, m, _dt(dY),
                                          k, _ptr(Btilde), 0 if Btilde is None else _ld(Btilde), _ptr(dW), _ld(dW), _dt(dW),
                                          layout, _ptr(sort_products), _ptr(workspace), workspace.numel(), _stream(stream)),
           "pamm_contract_weight_grad")
    return dW


def qkv_step_host(X_host, dY_host, k: int, seed: int, dW_host, arena, f_host=None, alpha_host=None, stream=None):
    """Whole path from (pinned) host tensors; ``arena`` is device scratch."""
    b, n = X_host.shape
    m = dY_host.shape[1]
    if not (X_host.is_contiguous() and dY_host.is_contiguous() and dW_host.is_contiguous()):
        raise ValueError("host tensors must be contiguous")
    _check(_lib.pamm_qkv_step_host(_ptr(X_host), _ptr(dY_host), b, n, m, _dt(X_host), k, seed, _ptr(dW_host),
                                   _ptr(f_host), _ptr(alpha_host), _ptr(arena), arena.numel(), _stream(stream)),
           "pamm_qkv_step_host")
    return dW_host


class _RecordingLib:
    """Stands in for the library while a call is being prepared: notes the C function and its marshalled arguments."""

    def __init__(self, real):
        self._real, self.calls = real, []

    def __getattr__(self, name):
        fn = getattr(self._real, name)

        def note(*cargs):
            self.calls.append((name, fn, cargs))
            return OK
        return note


def prepared(call, *args, **kwargs):
    """Marshal once, call often.  ``prepared(pamm.compress_fused, X, k, seed, idx_out=..., ...)`` runs nothing; it returns a
    zero-argument callable that repeats exactly that C call (same pointers, sizes, seed and stream), skipping the
    Python-side marshalling -- for loops where a step is only a few microseconds of GPU work.  Outputs the call
    allocates itself stay alive with the callable but are not handed out: pass in the ones you want to read."""
    global _lib, _prep_keep
    real, rec = _lib, _RecordingLib(_lib)
    _lib, _prep_keep = rec, []
    try:
        call(*args, **kwargs)
        keep = (args, kwargs, _prep_keep)          # the tensors behind the pointers, the call's own allocations included
    finally:
        _lib, _prep_keep = real, None
    if len(rec.calls) != 1:
        raise ValueError("prepared() takes a binding function that makes exactly one library call")
    name, fn, cargs = rec.calls[0]

    def run(_fn=fn, _cargs=cargs, _name=name, _keep=keep):
        code = _fn(*_cargs)
        if code != OK:
            raise PammError(code, _name)
    return run


PROBE_SUM, PROBE_ROWS = 0, 1


def probe_read(kind: int, data: torch.Tensor, order=None, sum32=None, stream=None) -> torch.Tensor:
    """A read-only pass over the rows of `data` (2-D, contiguous columns): PROBE_SUM with ordinary loads,
    PROBE_ROWS with bulk copies through a shared-memory ring, optionally in the row order `order` (int32).
    Returns the device word with the 32-bit checksum; time the call with events."""
    if not data.is_cuda or data.dim() != 2 or data.stride(1) != 1:
        raise ValueError("data: a 2-D CUDA tensor with contiguous columns")
    es = data.element_size()
    if sum32 is None:
        sum32 = _empty((1,), dtype=torch.int32, device=data.device)
    if order is not None:
        if not order.is_cuda or order.dtype != torch.int32 or order.numel() != data.shape[0] or not order.is_contiguous():
            raise ValueError("order: contiguous int32, one entry per row")
    _check(_lib.pamm_probe_read(int(kind), _ptr(data), int(data.shape[0]), int(data.shape[1]) * es, int(data.stride(0)) * es,
                                _ptr(order) if order is not None else None, _ptr(sum32), _stream(stream)), "pamm_probe_read")
    return sum32


def selftest_bounded_wait(stream=None) -> None:
    """Launch the kernel whose bounded wait must run out (sets ERR_TIMEOUT in the device status word)."""
    _check(_lib.pamm_selftest_bounded_wait(_stream(stream)), "pamm_selftest_bounded_wait")


def last_device_status(stream=None, synchronize: bool = True) -> int:
    """The device's status word, read and cleared.  The library call itself waits for nothing; by default the
    given (or current) stream is synchronised first, so that the answer covers the work enqueued so far."""
    s = torch.cuda.current_stream() if stream is None else stream
    if synchronize:
        s.synchronize()
    return int(_lib.pamm_last_device_status(ctypes.c_void_p(s.cuda_stream)))


PROF_COMPRESS, PROF_CONTRACT, PROF_WEIGHT_GRAD = 0, 1, 2


def launch_count() -> int:
    return int(_lib.pamm_launch_count())


def set_profile_events(kind: int, start=None, stop=None) -> None:
    """Record torch CUDA events (already recorded once, so their handles exist) around a step's main kernel."""
    a = None if start is None else ctypes.c_void_p(start.cuda_event)
    b = None if stop is None else ctypes.c_void_p(stop.cuda_event)
    _check(_lib.pamm_set_profile_events(kind, a, b), "pamm_set_profile_events")


def saved_bytes(b: int, n: int, k: int, dtype: int, f_type: int = IDX_I32) -> dict:
    """Bytes kept for the backward pass: X itself versus (C, f, alpha); and the paper's scalar counts."""
    out = (ctypes.c_int64 * 4)()
    _check(_lib.pamm_saved_bytes(b, n, k, dtype, f_type, ctypes.cast(out, ctypes.c_void_p)), "pamm_saved_bytes")
    return dict(full=int(out[0]), pamm=int(out[1]), ratio=out[0] / out[1], scalars_full=int(out[2]), scalars_pamm=int(out[3]))
