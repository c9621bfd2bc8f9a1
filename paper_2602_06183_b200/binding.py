"""ctypes binding of libsparseffn.so: argument marshalling only.

Every function has the name of the C entry point it calls (see include/sparseffn.h) and takes
torch tensors (device memory, streams) or raw integers; no step of the method runs in Python.
The shared library must have been built (``python -m paper_2602_06183_b200.build``); loading
fails loudly otherwise and there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsparseffn.so")

SF_OK = 0
SF_ERR_NULL, SF_ERR_SHAPE, SF_ERR_ALIGN, SF_ERR_WORKSPACE = -1, -2, -3, -4
SF_ERR_ARCH, SF_ERR_CUDA, SF_ERR_TIMEOUT, SF_ERR_UNSUPPORTED = -5, -6, -7, -8

SF_CTX_Y2_VALS, SF_CTX_RELU_VALS, SF_CTX_META, SF_CTX_COLIDX, SF_CTX_Y1, SF_CTX_DY1_VALS = range(6)
SF_CTX_Y2_VALS24, SF_CTX_Y2_META24, SF_CTX_DY1_VALS24, SF_CTX_RELU_VALS24 = 6, 7, 8, 9
SF_FFN_SAVE_Y1, SF_FFN_UNFUSED_ACT, SF_FFN_FUSED_ACT, SF_FFN_PACKED_GRAD_OPERANDS, SF_FFN_W2_FD = 1, 2, 4, 8, 16


class sf_ffn_desc(C.Structure):
    _fields_ = [("T", C.c_int64), ("D", C.c_int64), ("F", C.c_int64),
                ("V", C.c_int32), ("N", C.c_int32), ("M", C.c_int32),
                ("prune_mode", C.c_int32), ("flags", C.c_int32)]


class sf_router_desc(C.Structure):
    _fields_ = [("T", C.c_int64), ("D", C.c_int64), ("F", C.c_int64), ("E", C.c_int32), ("prune_mode", C.c_int32),
                ("flags", C.c_int32), ("reserved", C.c_int32)]


(SF_RCTX_EXPERT, SF_RCTX_ROW_OF_TOKEN, SF_RCTX_SRC_OF_ROW, SF_RCTX_SEGMENTS, SF_RCTX_LOGITS, SF_RCTX_Y2_VALS,
 SF_RCTX_RELU_VALS, SF_RCTX_META, SF_RCTX_Y1, SF_RCTX_DY1_VALS) = range(10)


class sf_schedule(C.Structure):
    _fields_ = [("warmup_steps", C.c_int64), ("sparse_steps", C.c_int64), ("total_steps", C.c_int64)]


SF_STEP_DENSE, SF_STEP_SPARSE = 0, 1


class SparseFFNError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (cuda error {last_cuda_error()})")


_lib = None

_vp, _i64, _i32, _sz = C.c_void_p, C.c_int64, C.c_int, C.c_size_t
_SIGNATURES = {
    "sf_status_string": (C.c_char_p, [_i32]),
    "sf_last_cuda_error": (_i32, []),
    "sf_prune24_sizes": (_i32, [_i64, _i64, _i32, C.POINTER(_sz), C.POINTER(_sz)]),
    "sf_prune24_compress": (_i32, [_vp, _i64, _i64, _i64, _i32, _i32, _vp, _vp, _vp, _vp]),
    "sf_vnm_sizes": (_i32, [_i64, _i64, _i32, _i32, _i32, C.POINTER(_sz), C.POINTER(_sz), C.POINTER(_sz)]),
    "sf_vnm_sparsify_act": (_i32, [_vp, _i64, _i64, _i64, _i32, _i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp]),
    "sf_gemm_workspace_size": (_i32, [_i64, _i64, C.POINTER(_sz)]),
    "sf_gemm_dense": (_i32, [_vp, _i32, _vp, _i32, _vp, _i64, _i64, _i64, _vp, _vp]),
    "sf_gemm_sparse24": (_i32, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp, _vp]),
    "sf_gemm_sparse24_rm": (_i32, [_vp, _vp, _vp, _i32, _vp, _i64, _i64, _i64, _vp, _vp]),
    "sf_gemm_sparse24_noalloc": (_i32, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, _vp]),
    "sf_fp8_quantize": (_i32, [_vp, _i64, _i64, _i64, C.c_float, _vp, _vp]),
    "sf_prune24_fp8_sizes": (_i32, [_i64, _i64, _i32, C.POINTER(_sz), C.POINTER(_sz)]),
    "sf_prune24_compress_fp8": (_i32, [_vp, _i64, _i64, _i64, _i32, _i32, C.c_float, _vp, _vp, _vp, _vp]),
    "sf_gemm_fp8_workspace_size": (_i32, [_i64, _i64, C.POINTER(_sz)]),
    "sf_gemm_fp8_dense": (_i32, [_vp, _vp, _vp, _i64, _i64, _i64, C.c_float, _vp, _vp]),
    "sf_gemm_fp8_sparse24": (_i32, [_vp, _vp, _vp, _vp, _i64, _i64, _i64, C.c_float, _vp, _vp]),
    "sf_gemm_venom": (_i32, [_vp, _vp, _vp, _vp, _vp, _i64, _i64, _i64, _i32, _i32, _vp, _vp]),
    "sf_ffn_workspace_size": (_i32, [C.POINTER(sf_ffn_desc), C.POINTER(_sz), C.POINTER(_sz)]),
    "sf_sparse_ffn_fwd": (_i32, [C.POINTER(sf_ffn_desc), _vp, _vp, _vp, _vp, _vp, _sz, _vp, _sz, _vp]),
    "sf_sparse_ffn_bwd": (_i32, [C.POINTER(sf_ffn_desc), _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp, _vp, _vp, _sz, _vp]),
    "sf_dense_ffn_fwd": (_i32, [C.POINTER(sf_ffn_desc), _vp, _vp, _vp, _vp, _vp, _sz, _vp, _sz, _vp]),
    "sf_dense_ffn_bwd": (_i32, [C.POINTER(sf_ffn_desc), _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp, _vp, _vp, _sz, _vp]),
    "sf_ctx_view": (_i32, [C.POINTER(sf_ffn_desc), _vp, _i32, C.POINTER(_vp), C.POINTER(_sz)]),
    "sf_ffn_host_staging_size": (_i32, [C.POINTER(sf_ffn_desc), C.POINTER(_sz)]),
    "sf_ffn_step_host": (_i32, [C.POINTER(sf_ffn_desc), _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp,
                                _sz, _vp]),
    "sf_schedule_step_kind": (_i32, [C.POINTER(sf_schedule), _i64, C.POINTER(_i32)]),
    "sf_schedule_speedup": (_i32, [C.POINTER(sf_schedule), C.c_double, C.POINTER(C.c_double)]),
    "sf_ffn_flop_fraction": (_i32, [_i64, _i64, _i64, _i64, _i64, C.POINTER(C.c_double)]),
    "sf_end_to_end_speedup": (_i32, [C.c_double, C.c_double, C.POINTER(C.c_double)]),
    "sf_ffn_fwd_scheduled": (_i32, [C.POINTER(sf_schedule), _i64, C.POINTER(sf_ffn_desc), _vp, _vp, _vp, _vp, _vp,
                                    _sz, _vp, _sz, _vp]),
    "sf_ffn_bwd_scheduled": (_i32, [C.POINTER(sf_schedule), _i64, C.POINTER(sf_ffn_desc), _vp, _vp, _vp, _vp, _vp,
                                    _sz, _vp, _vp, _vp, _vp, _sz, _vp]),
    "sf_router_fit_host": (_i32, [_vp, _i64, _i64, _i32, _i32, _vp, _vp, _vp]),
    "sf_router_route": (_i32, [_vp, _vp, _i64, _i64, _i32, _vp, _vp, _vp]),
    "sf_routed_ffn_workspace_size": (_i32, [C.POINTER(sf_router_desc), C.POINTER(_sz), C.POINTER(_sz)]),
    "sf_routed_ffn_fwd": (_i32, [C.POINTER(sf_router_desc), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _sz, _vp]),
    "sf_routed_ffn_bwd": (_i32, [C.POINTER(sf_router_desc), _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp, _vp, _vp, _sz, _vp]),
    "sf_routed_ctx_view": (_i32, [C.POINTER(sf_router_desc), _vp, _i32, C.POINTER(_vp), C.POINTER(_sz)]),
    "sf_selftest_wait_expiry": (_i32, [_vp, _i64, _vp]),
    "sf_trace_set": (_i32, [C.POINTER(_vp), _i32]),
    "sf_trace_count": (_i32, []),
    "sf_check_status": (_i32, [_vp, _vp]),
}

EXPORTED_SYMBOLS = tuple(_SIGNATURES)


def lib() -> C.CDLL:
    """Load the shared library (once). Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2602_06183_b200.build` "
                "(there is no fallback implementation)")
        _lib = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(_lib, name)
            fn.restype, fn.argtypes = res, args
    return _lib


def status_string(status: int) -> str:
    return lib().sf_status_string(status).decode()


def last_cuda_error() -> int:
    return lib().sf_last_cuda_error()


def _check(status: int, where: str) -> None:
    if status != SF_OK:
        raise SparseFFNError(status, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream: Optional[torch.cuda.Stream] = None):
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def make_desc(T, D, F, V, M, N=2, prune_mode=0, flags=0) -> sf_ffn_desc:
    return sf_ffn_desc(T, D, F, V, N, M, prune_mode, flags)


# ---- 2:4 pruning -----------------------------------------------------------------------------

def sf_prune24_sizes(rows: int, cols: int, group_dim: int):
    a, b = _sz(), _sz()
    _check(lib().sf_prune24_sizes(rows, cols, group_dim, C.byref(a), C.byref(b)), "sf_prune24_sizes")
    return a.value, b.value


def sf_prune24_compress(W: torch.Tensor, group_dim: int = 1, prune_mode: int = 0, want_dense: bool = False,
                        out=None, stream=None):
    """W: [rows, cols] 16-bit tensor on the device. Returns (vals, meta, dense_or_None)."""
    rows, cols = W.shape
    R, K = (rows, cols) if group_dim == 1 else (cols, rows)
    sf_prune24_sizes(rows, cols, group_dim)
    if out is None:
        vals = torch.empty((R, K // 2), dtype=W.dtype, device=W.device)
        meta = torch.empty((R, K // 16), dtype=torch.int16, device=W.device)
        dense = torch.empty((rows, cols), dtype=W.dtype, device=W.device) if want_dense else None
    else:
        vals, meta, dense = out
    st = lib().sf_prune24_compress(_ptr(W), rows, cols, W.stride(0), group_dim, prune_mode,
                                   _ptr(vals), _ptr(meta), _ptr(dense), _stream(stream))
    _check(st, "sf_prune24_compress")
    return vals, meta, dense


# ---- V:N:M activation sparsification ------------------------------------------------------------

def sf_vnm_sizes(T, F, V, N, M):
    a, b, c = _sz(), _sz(), _sz()
    _check(lib().sf_vnm_sizes(T, F, V, N, M, C.byref(a), C.byref(b), C.byref(c)), "sf_vnm_sizes")
    return a.value, b.value, c.value


def sf_vnm_sparsify_act(P: torch.Tensor, V: int, M: int, N: int = 2, apply_sqrelu: bool = True,
                        want_relu: bool = True, want_dense: bool = False, out=None, stream=None):
    """P: [T, F] 16-bit tensor. Returns (vals, meta, colidx, relu_vals_or_None, dense_or_None)."""
    T, F = P.shape
    sf_vnm_sizes(T, F, V, N, M)
    if out is None:
        G = F // M
        vals = torch.empty((T, 2 * G), dtype=P.dtype, device=P.device)
        meta = torch.empty((T, G // 4), dtype=torch.int16, device=P.device)
        colidx = torch.empty((T // V, G, 4), dtype=torch.uint8, device=P.device)
        relu = torch.empty((T, 2 * G), dtype=P.dtype, device=P.device) if (want_relu and apply_sqrelu) else None
        dense = torch.empty((T, F), dtype=P.dtype, device=P.device) if want_dense else None
    else:
        vals, meta, colidx, relu, dense = out
    st = lib().sf_vnm_sparsify_act(_ptr(P), T, F, P.stride(0), V, N, M, int(apply_sqrelu), _ptr(vals), _ptr(meta),
                                   _ptr(colidx), _ptr(relu), _ptr(dense), _stream(stream))
    _check(st, "sf_vnm_sparsify_act")
    return vals, meta, colidx, relu, dense


# ---- single products -----------------------------------------------------------------------------

def sf_gemm_workspace_size(Mr: int, K: int) -> int:
    a = _sz()
    _check(lib().sf_gemm_workspace_size(Mr, K, C.byref(a)), "sf_gemm_workspace_size")
    return a.value


def _workspace(nbytes: int, device) -> torch.Tensor:
    return torch.zeros((max(nbytes, 256),), dtype=torch.uint8, device=device)


def sf_gemm_dense(A: torch.Tensor, a_kmajor: bool, B: torch.Tensor, b_kmajor: bool, C_out=None,
                  workspace=None, stream=None):
    """C[Mr,Nc] = op(A) op(B)^T. A is [Mr,K] (a_kmajor) or [K,Mr]; B is [Nc,K] (b_kmajor) or [K,Nc]."""
    Mr, K = A.shape if a_kmajor else (A.shape[1], A.shape[0])
    Nc = B.shape[0] if b_kmajor else B.shape[1]
    if C_out is None:
        C_out = torch.empty((Mr, Nc), dtype=A.dtype, device=A.device)
    if workspace is None:
        workspace = _workspace(sf_gemm_workspace_size(Mr, K), A.device)
    st = lib().sf_gemm_dense(_ptr(A), int(a_kmajor), _ptr(B), int(b_kmajor), _ptr(C_out), Mr, Nc, K,
                             _ptr(workspace), _stream(stream))
    _check(st, "sf_gemm_dense")
    return C_out, workspace


def sf_gemm_sparse24(a_vals, a_meta, B, Ct_out=None, workspace=None, stream=None):
    """Ct[Nc,Mr] = (A_s[Mr,K] B[Nc,K]^T)^T with A_s packed (vals [Mr,K/2], meta [Mr,K/16])."""
    Mr, K = a_vals.shape[0], a_vals.shape[1] * 2
    Nc = B.shape[0]
    if Ct_out is None:
        Ct_out = torch.empty((Nc, Mr), dtype=B.dtype, device=B.device)
    if workspace is None:
        workspace = _workspace(sf_gemm_workspace_size(Mr, K), B.device)
    st = lib().sf_gemm_sparse24(_ptr(a_vals), _ptr(a_meta), _ptr(B), _ptr(Ct_out), Mr, Nc, K,
                                _ptr(workspace), _stream(stream))
    _check(st, "sf_gemm_sparse24")
    return Ct_out, workspace


def sf_gemm_sparse24_rm(a_vals, a_meta, B, b_kmajor: bool, C_out=None, workspace=None, stream=None):
    """C[Mr,Nc] = A_s[Mr,K] op(B)^T, row-major output; B is [Nc,K] (b_kmajor) or [K,Nc]."""
    Mr, K = a_vals.shape[0], a_vals.shape[1] * 2
    Nc = B.shape[0] if b_kmajor else B.shape[1]
    if C_out is None:
        C_out = torch.empty((Mr, Nc), dtype=B.dtype, device=B.device)
    if workspace is None:
        workspace = _workspace(sf_gemm_workspace_size(Mr, K), B.device)
    st = lib().sf_gemm_sparse24_rm(_ptr(a_vals), _ptr(a_meta), _ptr(B), int(b_kmajor), _ptr(C_out), Mr, Nc, K,
                                   _ptr(workspace), _stream(stream))
    _check(st, "sf_gemm_sparse24_rm")
    return C_out, workspace


def sf_fp8_quantize(X, scale: float, out=None, stream=None):
    """E4M3 codes (uint8 [rows, cols]) of float(X) * scale; X bf16, may be a strided row view."""
    rows, cols = X.shape
    if out is None:
        out = torch.empty((rows, cols), dtype=torch.uint8, device=X.device)
    _check(lib().sf_fp8_quantize(_ptr(X), rows, cols, X.stride(0) if rows > 1 else cols, float(scale), _ptr(out),
                                 _stream(stream)), "sf_fp8_quantize")
    return out


def sf_prune24_compress_fp8(W, prune_mode: int, scale: float, want_dense: bool = False, out=None, stream=None,
                            group_dim: int = 1):
    """2:4 with the kept values quantised to E4M3 in the same pass. group_dim as for sf_prune24_compress
    (1: groups along a row; 0: along a column, outputs K-major). Returns (vals uint8 [R, K/2], meta int16
    [R, K/16], dense uint8 [rows, cols] or None); ``out`` = a previous result to write into."""
    rows, cols = W.shape
    R, K = (rows, cols) if group_dim == 1 else (cols, rows)
    vb, mb = _sz(), _sz()
    _check(lib().sf_prune24_fp8_sizes(rows, cols, group_dim, C.byref(vb), C.byref(mb)), "sf_prune24_fp8_sizes")
    if out is not None:
        vals, meta, dense = out
    else:
        vals = torch.empty((R, K // 2), dtype=torch.uint8, device=W.device)
        meta = torch.empty((R, K // 16), dtype=torch.int16, device=W.device)
        dense = torch.empty((rows, cols), dtype=torch.uint8, device=W.device) if want_dense else None
    _check(lib().sf_prune24_compress_fp8(_ptr(W), rows, cols, W.stride(0) if rows > 1 else cols, group_dim, prune_mode,
                                         float(scale), _ptr(vals), _ptr(meta), _ptr(dense), _stream(stream)),
           "sf_prune24_compress_fp8")
    return vals, meta, dense


def sf_gemm_fp8_workspace_size(Mr: int, K: int) -> int:
    b = _sz()
    _check(lib().sf_gemm_fp8_workspace_size(Mr, K, C.byref(b)), "sf_gemm_fp8_workspace_size")
    return b.value


def sf_gemm_fp8_dense(A, B, alpha: float, C_out=None, workspace=None, stream=None):
    """C[Mr,Nc] = bf16(alpha * A B^T) on E4M3 codes A [Mr,K], B [Nc,K] (uint8)."""
    Mr, K = A.shape
    Nc = B.shape[0]
    if C_out is None:
        C_out = torch.empty((Mr, Nc), dtype=torch.bfloat16, device=B.device)
    if workspace is None:
        workspace = _workspace(sf_gemm_fp8_workspace_size(Mr, K), B.device)
    _check(lib().sf_gemm_fp8_dense(_ptr(A), _ptr(B), _ptr(C_out), Mr, Nc, K, float(alpha), _ptr(workspace),
                                   _stream(stream)), "sf_gemm_fp8_dense")
    return C_out, workspace


def sf_gemm_fp8_sparse24(a_vals, a_meta, B, alpha: float, C_out=None, workspace=None, stream=None):
    """The same product with A 2:4-packed: a_vals uint8 [Mr,K/2], a_meta canonical [Mr,K/16]."""
    Mr, K = a_vals.shape[0], a_vals.shape[1] * 2
    Nc = B.shape[0]
    if C_out is None:
        C_out = torch.empty((Mr, Nc), dtype=torch.bfloat16, device=B.device)
    if workspace is None:
        workspace = _workspace(sf_gemm_fp8_workspace_size(Mr, K), B.device)
    _check(lib().sf_gemm_fp8_sparse24(_ptr(a_vals), _ptr(a_meta), _ptr(B), _ptr(C_out), Mr, Nc, K, float(alpha),
                                      _ptr(workspace), _stream(stream)), "sf_gemm_fp8_sparse24")
    return C_out, workspace


def sf_gemm_sparse24_noalloc(a_vals, a_meta, B, Ct_out, stream=None):
    """Same product as sf_gemm_sparse24 without a workspace: for callers that cannot allocate device
    memory. ``Ct_out`` [Nc, Mr] must be supplied by the caller; nothing is allocated here either.
    Limit: Mr * K / 8 <= 4 MiB. Calls share one built-in scratch array: keep them on one stream."""
    Mr, K = a_vals.shape[0], a_vals.shape[1] * 2
    Nc = B.shape[0]
    st = lib().sf_gemm_sparse24_noalloc(_ptr(a_vals), _ptr(a_meta), _ptr(B), _ptr(Ct_out), Mr, Nc, K, _stream(stream))
    _check(st, "sf_gemm_sparse24_noalloc")
    return Ct_out


def sf_gemm_venom(a_vals, a_meta, colidx, Bt, V: int, M: int, C_out=None, workspace=None, stream=None):
    """C[T,Nc] = A_vnm[T,F] Bt[F,Nc] with A_vnm in packed V:N:M form."""
    T = a_vals.shape[0]
    F, Nc = Bt.shape
    if C_out is None:
        C_out = torch.empty((T, Nc), dtype=Bt.dtype, device=Bt.device)
    if workspace is None:
        workspace = _workspace(sf_gemm_workspace_size(T, 4 * F // M), Bt.device)
    st = lib().sf_gemm_venom(_ptr(a_vals), _ptr(a_meta), _ptr(colidx), _ptr(Bt), _ptr(C_out), T, F, Nc, V, M,
                             _ptr(workspace), _stream(stream))
    _check(st, "sf_gemm_venom")
    return C_out, workspace


# ---- FFN step --------------------------------------------------------------------------------------

def sf_ffn_workspace_size(desc: sf_ffn_desc):
    a, b = _sz(), _sz()
    _check(lib().sf_ffn_workspace_size(C.byref(desc), C.byref(a), C.byref(b)), "sf_ffn_workspace_size")
    return a.value, b.value


def alloc_ffn_buffers(desc: sf_ffn_desc, device="cuda"):
    """(fwd_ctx, workspace) as zero-initialised uint8 tensors of the sizes the library asks for."""
    c, w = sf_ffn_workspace_size(desc)
    return _workspace(c, device), _workspace(w, device)


def _nbytes(t: torch.Tensor) -> int:
    return t.numel() * t.element_size()


def sf_sparse_ffn_fwd(desc, X, W1, W2, Y, fwd_ctx, workspace, stream=None):
    _check(lib().sf_sparse_ffn_fwd(C.byref(desc), _ptr(X), _ptr(W1), _ptr(W2), _ptr(Y), _ptr(fwd_ctx),
                                   _nbytes(fwd_ctx), _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "sf_sparse_ffn_fwd")


def sf_sparse_ffn_bwd(desc, dY, X, W1, W2, fwd_ctx, dX, dW1, dW2, workspace, stream=None):
    _check(lib().sf_sparse_ffn_bwd(C.byref(desc), _ptr(dY), _ptr(X), _ptr(W1), _ptr(W2), _ptr(fwd_ctx),
                                   _nbytes(fwd_ctx), _ptr(dX), _ptr(dW1), _ptr(dW2), _ptr(workspace),
                                   _nbytes(workspace), _stream(stream)), "sf_sparse_ffn_bwd")


def sf_dense_ffn_fwd(desc, X, W1, W2, Y, fwd_ctx, workspace, stream=None):
    _check(lib().sf_dense_ffn_fwd(C.byref(desc), _ptr(X), _ptr(W1), _ptr(W2), _ptr(Y), _ptr(fwd_ctx),
                                  _nbytes(fwd_ctx), _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "sf_dense_ffn_fwd")


def sf_dense_ffn_bwd(desc, dY, X, W1, W2, fwd_ctx, dX, dW1, dW2, workspace, stream=None):
    _check(lib().sf_dense_ffn_bwd(C.byref(desc), _ptr(dY), _ptr(X), _ptr(W1), _ptr(W2), _ptr(fwd_ctx),
                                  _nbytes(fwd_ctx), _ptr(dX), _ptr(dW1), _ptr(dW2), _ptr(workspace),
                                  _nbytes(workspace), _stream(stream)), "sf_dense_ffn_bwd")


_CTX_DTYPES = {SF_CTX_Y2_VALS: torch.bfloat16, SF_CTX_RELU_VALS: torch.bfloat16, SF_CTX_META: torch.int16,
               SF_CTX_COLIDX: torch.uint8, SF_CTX_Y1: torch.bfloat16, SF_CTX_DY1_VALS: torch.bfloat16,
               SF_CTX_Y2_VALS24: torch.bfloat16, SF_CTX_Y2_META24: torch.int16, SF_CTX_DY1_VALS24: torch.bfloat16,
               SF_CTX_RELU_VALS24: torch.bfloat16}


def sf_ctx_view(desc, buf: torch.Tensor, field: int) -> torch.Tensor:
    """A flat tensor aliasing one field of the forward context (or workspace for DY1_VALS)."""
    p, n = _vp(), _sz()
    _check(lib().sf_ctx_view(C.byref(desc), _ptr(buf), field, C.byref(p), C.byref(n)), "sf_ctx_view")
    off = p.value - buf.data_ptr()
    return buf[off:off + n.value].view(_CTX_DTYPES[field])


def sf_ffn_host_staging_size(desc) -> int:
    a = _sz()
    _check(lib().sf_ffn_host_staging_size(C.byref(desc), C.byref(a)), "sf_ffn_host_staging_size")
    return a.value


def sf_ffn_step_host(desc, dense: bool, hX, hW1, hW2, hdY, hY, hdX, hdW1, hdW2, staging, fwd_ctx, workspace,
                     stream=None):
    """Host tensors in, host tensors out (pinned memory recommended); does not synchronise."""
    _check(lib().sf_ffn_step_host(C.byref(desc), int(dense), _ptr(hX), _ptr(hW1), _ptr(hW2), _ptr(hdY), _ptr(hY),
                                  _ptr(hdX), _ptr(hdW1), _ptr(hdW2), _ptr(staging), _ptr(fwd_ctx), _nbytes(fwd_ctx),
                                  _ptr(workspace), _nbytes(workspace), _stream(stream)), "sf_ffn_step_host")


# ---- routed step (neuron-level experts) ------------------------------------------------------------

def make_router_desc(T, D, F, E, prune_mode=0, flags=0) -> sf_router_desc:
    return sf_router_desc(T, D, F, E, prune_mode, flags, 0)


def sf_router_fit_host(W1_bits, E: int, iters: int = 8):
    """Offline balanced clustering on the host. W1_bits: numpy uint16 [F, D] (bf16 patterns).
    Returns numpy arrays (expert int32 [F], perm int32 [F], means uint16 [E, D])."""
    import numpy as np
    W = np.ascontiguousarray(W1_bits, dtype=np.uint16)
    F, D = W.shape
    expert, perm = np.empty(F, dtype=np.int32), np.empty(F, dtype=np.int32)
    means = np.empty((E, D), dtype=np.uint16)
    _check(lib().sf_router_fit_host(W.ctypes.data_as(_vp), F, D, E, iters, expert.ctypes.data_as(_vp),
                                    perm.ctypes.data_as(_vp), means.ctypes.data_as(_vp)), "sf_router_fit_host")
    return expert, perm, means


def sf_router_route(X: torch.Tensor, means: torch.Tensor, want_logits: bool = True, stream=None):
    """X [T, D], means [E, D] (16-bit tensors). Returns (expert int32 [T], logits float32 [T, E] or None)."""
    T, D = X.shape
    E = means.shape[0]
    expert = torch.empty((T,), dtype=torch.int32, device=X.device)
    logits = torch.empty((T, E), dtype=torch.float32, device=X.device) if want_logits else None
    _check(lib().sf_router_route(_ptr(X), _ptr(means), T, D, E, _ptr(expert), _ptr(logits), _stream(stream)),
           "sf_router_route")
    return expert, logits


def sf_routed_ffn_workspace_size(desc: sf_router_desc):
    a, b = _sz(), _sz()
    _check(lib().sf_routed_ffn_workspace_size(C.byref(desc), C.byref(a), C.byref(b)), "sf_routed_ffn_workspace_size")
    return a.value, b.value


def sf_routed_ffn_fwd(desc, X, W1, W2, means, Y, fwd_ctx, workspace, forced_expert=None, stream=None):
    _check(lib().sf_routed_ffn_fwd(C.byref(desc), _ptr(X), _ptr(W1), _ptr(W2), _ptr(means), _ptr(forced_expert), _ptr(Y),
                                   _ptr(fwd_ctx), _nbytes(fwd_ctx), _ptr(workspace), _nbytes(workspace),
                                   _stream(stream)), "sf_routed_ffn_fwd")


def sf_routed_ffn_bwd(desc, dY, X, W1, W2, fwd_ctx, dX, dW1, dW2, workspace, stream=None):
    _check(lib().sf_routed_ffn_bwd(C.byref(desc), _ptr(dY), _ptr(X), _ptr(W1), _ptr(W2), _ptr(fwd_ctx),
                                   _nbytes(fwd_ctx), _ptr(dX), _ptr(dW1), _ptr(dW2), _ptr(workspace),
                                   _nbytes(workspace), _stream(stream)), "sf_routed_ffn_bwd")


_RCTX_DTYPES = {SF_RCTX_EXPERT: torch.int32, SF_RCTX_ROW_OF_TOKEN: torch.int32, SF_RCTX_SRC_OF_ROW: torch.int32,
                SF_RCTX_SEGMENTS: torch.int32, SF_RCTX_LOGITS: torch.float32, SF_RCTX_Y2_VALS: torch.bfloat16,
                SF_RCTX_RELU_VALS: torch.bfloat16, SF_RCTX_META: torch.int16, SF_RCTX_Y1: torch.bfloat16,
                SF_RCTX_DY1_VALS: torch.bfloat16}


def sf_routed_ctx_view(desc, buf: torch.Tensor, field: int) -> torch.Tensor:
    p, n = _vp(), _sz()
    _check(lib().sf_routed_ctx_view(C.byref(desc), _ptr(buf), field, C.byref(p), C.byref(n)), "sf_routed_ctx_view")
    off = p.value - buf.data_ptr()
    return buf[off:off + n.value].view(_RCTX_DTYPES[field])


def make_schedule(warmup_steps: int, sparse_steps: int, total_steps: int) -> sf_schedule:
    return sf_schedule(warmup_steps, sparse_steps, total_steps)


def sf_schedule_step_kind(schedule, step: int) -> int:
    kind = _i32(0)
    _check(lib().sf_schedule_step_kind(C.byref(schedule), step, C.byref(kind)), "sf_schedule_step_kind")
    return kind.value


def sf_schedule_speedup(schedule, sparse_step_speedup: float) -> float:
    out = C.c_double(0)
    _check(lib().sf_schedule_speedup(C.byref(schedule), sparse_step_speedup, C.byref(out)), "sf_schedule_speedup")
    return out.value


def sf_ffn_flop_fraction(D: int, F: int, n_q_heads: int, n_kv_heads: int, head_dim: int) -> float:
    out = C.c_double(0)
    _check(lib().sf_ffn_flop_fraction(D, F, n_q_heads, n_kv_heads, head_dim, C.byref(out)), "sf_ffn_flop_fraction")
    return out.value


def sf_end_to_end_speedup(ffn_fraction: float, ffn_speedup: float) -> float:
    out = C.c_double(0)
    _check(lib().sf_end_to_end_speedup(ffn_fraction, ffn_speedup, C.byref(out)), "sf_end_to_end_speedup")
    return out.value


def sf_ffn_fwd_scheduled(schedule, step: int, desc, X, W1, W2, Y, fwd_ctx, workspace, stream=None):
    _check(lib().sf_ffn_fwd_scheduled(C.byref(schedule), step, C.byref(desc), _ptr(X), _ptr(W1), _ptr(W2), _ptr(Y),
                                      _ptr(fwd_ctx), _nbytes(fwd_ctx), _ptr(workspace), _nbytes(workspace),
                                      _stream(stream)), "sf_ffn_fwd_scheduled")


def sf_ffn_bwd_scheduled(schedule, step: int, desc, dY, X, W1, W2, fwd_ctx, dX, dW1, dW2, workspace, stream=None):
    _check(lib().sf_ffn_bwd_scheduled(C.byref(schedule), step, C.byref(desc), _ptr(dY), _ptr(X), _ptr(W1), _ptr(W2),
                                      _ptr(fwd_ctx), _nbytes(fwd_ctx), _ptr(dX), _ptr(dW1), _ptr(dW2), _ptr(workspace),
                                      _nbytes(workspace), _stream(stream)), "sf_ffn_bwd_scheduled")


def sf_selftest_wait_expiry(workspace, budget_clocks: int = 1_000_000, stream=None) -> None:
    """One bounded wait on a barrier nothing completes: sets the status word of ``workspace``."""
    _check(lib().sf_selftest_wait_expiry(_ptr(workspace), budget_clocks, _stream(stream)), "sf_selftest_wait_expiry")


def sf_check_status(workspace, stream=None) -> int:
    return lib().sf_check_status(_ptr(workspace), _stream(stream))


class StageTrace:
    """Records CUDA events between the kernels of the FFN step calls made inside the `with` block.

    After the block, ``durations_ms()`` returns the time between consecutive events (the caller
    knows the stage order of the calls it made; see sf_trace_set in the header)."""

    def __init__(self, capacity: int):
        self.events = [torch.cuda.Event(enable_timing=True) for _ in range(capacity)]
        for e in self.events:          # torch creates the CUDA event lazily on first record
            e.record()
        torch.cuda.synchronize()
        self._arr = (C.c_void_p * capacity)(*[C.c_void_p(e.cuda_event) for e in self.events])
        self.count = 0

    def __enter__(self):
        _check(lib().sf_trace_set(self._arr, len(self.events)), "sf_trace_set")
        return self

    def __exit__(self, *exc):
        self.count = lib().sf_trace_count()
        lib().sf_trace_set(None, 0)
        return False

    def durations_ms(self):
        torch.cuda.synchronize()
        return [self.events[i].elapsed_time(self.events[i + 1]) for i in range(self.count - 1)]
