"""Thin ctypes binding of ``libentmax_attn.so``: argument marshalling only.

Same entry-point names as ``include/entmax_attn.h``.  PyTorch supplies device memory and streams;
every step of the computation runs in the library's CUDA kernels.  There is no fallback: if the
library is missing or a call is rejected, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libentmax_attn.so")

DTYPE_BF16, DTYPE_FP32 = 0, 1
STATUS_WORDS = 8
STATUS_FLAGS, STATUS_DENSE_ROWS, STATUS_TILE_SWEEPS, STATUS_TILES = 0, 1, 2, 3
STATUS_SKIPPED_STEPS, STATUS_SCORED_STEPS = 4, 5
FLAG_WAIT_EXPIRED, FLAG_BAD_SCALE, FLAG_BAD_LENGTH = 1, 2, 4


class Params(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads", ctypes.c_int32), ("seq", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("dtype", ctypes.c_int32), ("causal", ctypes.c_int32),
                ("n_mode", ctypes.c_int32), ("alpha", ctypes.c_float), ("sm_scale", ctypes.c_float),
                ("stride_b", ctypes.c_int64), ("stride_h", ctypes.c_int64), ("stride_n", ctypes.c_int64)]


class DecodeParams(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads", ctypes.c_int32), ("q_len", ctypes.c_int32),
                ("kv_capacity", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("alpha", ctypes.c_float),
                ("sm_scale", ctypes.c_float), ("kv_stride_b", ctypes.c_int64), ("kv_stride_h", ctypes.c_int64),
                ("kv_stride_n", ctypes.c_int64)]


class ProjParams(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("heads", ctypes.c_int32), ("seq", ctypes.c_int32), ("d_model", ctypes.c_int32),
                ("x_dtype", ctypes.c_int32), ("causal", ctypes.c_int32), ("n_mode", ctypes.c_int32),
                ("gamma_range", ctypes.c_float)]


class WsLayout(ctypes.Structure):
    _fields_ = [("row_count_offset", ctypes.c_size_t), ("entries_offset", ctypes.c_size_t),
                ("scale_offset", ctypes.c_size_t), ("dense_count_offset", ctypes.c_size_t),
                ("capacity", ctypes.c_int32), ("keep_limit", ctypes.c_int32)]


class Extras(ctypes.Structure):
    _fields_ = [("c_rows", ctypes.c_void_p), ("alibi_slopes", ctypes.c_void_p), ("d_scale_rows", ctypes.c_void_p),
                ("dbeta", ctypes.c_void_p), ("dgamma", ctypes.c_void_p), ("ddelta", ctypes.c_void_p),
                ("fwd_workspace", ctypes.c_void_p), ("saved_supports", ctypes.c_void_p)]


class EntmaxAttnError(RuntimeError):
    pass


_lib = None


def load():
    """Loads the CUDA library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise EntmaxAttnError(
                "libentmax_attn.so is missing: build it with `python -m paper_2506_16640_b200.build` "
                "(there is no CPU or PyTorch fallback)")
        lib = ctypes.CDLL(LIB_PATH)
        vp, fp, ip = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
        pp = ctypes.POINTER(Params)
        lib.entmax_attn_workspace_bytes.restype = ctypes.c_size_t
        lib.entmax_attn_workspace_bytes.argtypes = [pp, ctypes.c_int]
        lib.entmax_attn_workspace_layout.restype = ctypes.c_int
        lib.entmax_attn_workspace_layout.argtypes = [pp, ctypes.POINTER(WsLayout)]
        lib.entmax_attn_fwd.restype = ctypes.c_int
        lib.entmax_attn_fwd.argtypes = [pp, vp, vp, vp, fp, fp, fp, vp, fp, vp, ctypes.c_size_t, ip, vp]
        lib.entmax_attn_bwd.restype = ctypes.c_int
        lib.entmax_attn_bwd.argtypes = [pp, vp, vp, vp, fp, fp, fp, fp, vp, vp, vp, vp, vp, ctypes.c_size_t, ip, vp]
        lib.entmax_attn_bwd_scale.restype = ctypes.c_int
        lib.entmax_attn_bwd_scale.argtypes = [pp, vp, vp, vp, fp, fp, fp, fp, vp, vp, vp, vp, fp, fp, fp, fp, vp,
                                              ctypes.c_size_t, ip, vp]
        ep = ctypes.POINTER(Extras)
        lib.entmax_attn_fwd_ex.restype = ctypes.c_int
        lib.entmax_attn_fwd_ex.argtypes = [pp, vp, vp, vp, fp, fp, fp, ep, vp, fp, vp, ctypes.c_size_t, ip, vp]
        lib.entmax_attn_bwd_ex.restype = ctypes.c_int
        lib.entmax_attn_bwd_ex.argtypes = [pp, vp, vp, vp, fp, fp, fp, ep, fp, vp, vp, vp, vp, vp, ctypes.c_size_t, ip, vp]
        lib.entmax_attn_fwd_rowscale.restype = ctypes.c_int
        lib.entmax_attn_fwd_rowscale.argtypes = [pp, vp, vp, vp, fp, vp, fp, vp, ctypes.c_size_t, ip, vp]
        lib.entmax_attn_bwd_rowscale.restype = ctypes.c_int
        lib.entmax_attn_bwd_rowscale.argtypes = [pp, vp, vp, vp, fp, fp, vp, vp, vp, vp, fp, vp, ctypes.c_size_t, ip, vp]
        lib.entmax_attn_fwd_static.restype = ctypes.c_int
        lib.entmax_attn_fwd_static.argtypes = [pp, vp, vp, vp, fp, fp, fp, vp, fp, ip, vp]
        dp = ctypes.POINTER(DecodeParams)
        lib.entmax_attn_decode_workspace_bytes.restype = ctypes.c_size_t
        lib.entmax_attn_decode_workspace_bytes.argtypes = [dp]
        lib.entmax_attn_decode_fwd.restype = ctypes.c_int
        lib.entmax_attn_decode_fwd.argtypes = [dp, vp, vp, vp, ip, fp, fp, fp, fp, vp, fp, ip, vp, ctypes.c_size_t, ip, vp]
        lib.entmax_attn_saved_bytes.restype = ctypes.c_size_t
        lib.entmax_attn_saved_bytes.argtypes = [pp]
        lib.entmax_attn_save_supports.restype = ctypes.c_int
        lib.entmax_attn_save_supports.argtypes = [pp, vp, vp, ctypes.c_size_t, vp]
        lib.entmax_attn_scores_debug.restype = ctypes.c_int
        lib.entmax_attn_scores_debug.argtypes = [pp, vp, vp, ctypes.c_int32, fp, vp, ctypes.c_size_t, ip, vp]
        lib.entmax_attn_profile_events.restype = ctypes.c_int
        lib.entmax_attn_profile_events.argtypes = [ctypes.c_int, vp, vp]
        jp = ctypes.POINTER(ProjParams)
        lib.entmax_attn_scale_proj_fwd.restype = ctypes.c_int
        lib.entmax_attn_scale_proj_fwd.argtypes = [jp, vp, fp, fp, fp, fp, vp]
        lib.entmax_attn_scale_proj_bwd.restype = ctypes.c_int
        lib.entmax_attn_scale_proj_bwd.argtypes = [jp, vp, fp, fp, fp, fp, fp, fp, vp, vp]
        lib.entmax_attn_selftest_wait_expiry.restype = ctypes.c_int
        lib.entmax_attn_selftest_wait_expiry.argtypes = [ctypes.c_uint64, ip, vp]
        lib.entmax_attn_strerror.restype = ctypes.c_char_p
        lib.entmax_attn_strerror.argtypes = [ctypes.c_int]
        lib.entmax_attn_last_cuda_error.restype = ctypes.c_int
        lib.entmax_attn_version.restype = ctypes.c_int
        _lib = lib
    return _lib


def _check(rc: int, what: str):
    if rc != 0:
        lib = load()
        msg = lib.entmax_attn_strerror(rc).decode()
        extra = ""
        if rc == -7:
            extra = " (cudaError %d)" % lib.entmax_attn_last_cuda_error()
        raise EntmaxAttnError("%s failed: %s%s" % (what, msg, extra))


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def make_params(q: torch.Tensor, alpha: float, causal: bool, sm_scale: float = 0.0, n_mode: int = 0) -> Params:
    if q.dim() != 4:
        raise EntmaxAttnError("expected [batch, heads, seq, head_dim] tensors")
    if q.dtype == torch.bfloat16:
        dt = DTYPE_BF16
    elif q.dtype == torch.float32:
        dt = DTYPE_FP32
    else:
        raise EntmaxAttnError("dtype must be bfloat16 or float32")
    if q.stride(3) != 1:
        raise EntmaxAttnError("head_dim must be the innermost, contiguous dimension")
    B, H, N, D = q.shape
    return Params(B, H, N, D, dt, int(bool(causal)), int(n_mode), float(alpha), float(sm_scale),
                  q.stride(0), q.stride(1), q.stride(2))


def _same_layout(ref: torch.Tensor, *others):
    for t in others:
        if t.shape != ref.shape or t.stride() != ref.stride() or t.dtype != ref.dtype or t.device != ref.device:
            raise EntmaxAttnError("all [B,H,N,D] tensors of a call must share shape, strides, dtype and device")


def entmax_attn_workspace_bytes(params: Params, is_bwd: bool) -> int:
    return int(load().entmax_attn_workspace_bytes(ctypes.byref(params), int(bool(is_bwd))))


def entmax_attn_workspace_layout(params: Params) -> WsLayout:
    out = WsLayout()
    _check(load().entmax_attn_workspace_layout(ctypes.byref(params), ctypes.byref(out)), "entmax_attn_workspace_layout")
    return out


def alloc_workspace(params: Params, is_bwd: bool, device) -> torch.Tensor:
    nbytes = entmax_attn_workspace_bytes(params, is_bwd)
    if nbytes == 0:
        raise EntmaxAttnError("invalid parameters (workspace size query returned 0)")
    return torch.empty(nbytes, dtype=torch.uint8, device=device)   # torch's allocator aligns to >= 512 B


def _stream_ptr(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def entmax_attn_fwd(q, k, v, alpha, causal, beta=None, gamma=None, delta=None, *, sm_scale=0.0, n_mode=0,
                    o=None, tau=None, workspace=None, status=None, stream=None):
    """Forward pass.  Returns (o, tau).  `workspace` (uint8 CUDA tensor) and `status` (int32[4] CUDA
    tensor) are allocated when not given; pass your own to inspect them afterwards."""
    _same_layout(q, k, v)
    params = make_params(q, alpha, causal, sm_scale, n_mode)
    if o is None:
        o = torch.empty_like(q)
    else:
        _same_layout(q, o)
    B, H, N, _ = q.shape
    if tau is None:
        tau = torch.empty((B, H, N), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = alloc_workspace(params, False, q.device)
    rc = load().entmax_attn_fwd(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gamma), _ptr(delta),
                                _ptr(o), _ptr(tau), _ptr(workspace), workspace.numel(), _ptr(status),
                                _stream_ptr(stream))
    _check(rc, "entmax_attn_fwd")
    return o, tau


def entmax_attn_fwd_static(q, k, v, alpha, causal, beta=None, gamma=None, delta=None, *, sm_scale=0.0, n_mode=0,
                           o, tau, status=None, stream=None):
    """Forward pass without a workspace, for callers that cannot allocate device memory: the scratch is
    a fixed array inside the library.  `o` and `tau` must be passed in (this wrapper allocates nothing
    either).  Raises EntmaxAttnError when the problem exceeds the built-in scratch.  Calls that overlap
    on the GPU share that scratch and race; keep them on one stream."""
    _same_layout(q, k, v, o)
    params = make_params(q, alpha, causal, sm_scale, n_mode)
    rc = load().entmax_attn_fwd_static(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gamma),
                                       _ptr(delta), _ptr(o), _ptr(tau), _ptr(status), _stream_ptr(stream))
    _check(rc, "entmax_attn_fwd_static")
    return o, tau


def entmax_attn_decode_fwd(q, k, v, alpha, kv_len=None, beta=None, gamma=None, delta=None, *, alibi_slopes=None,
                           sm_scale=0.0, o=None, tau=None, support_size=None, workspace=None, status=None,
                           stream=None):
    """Decode-shape forward: q [B,H,q_len,d] (contiguous) against the cache k, v [B,H,kv_capacity,d] (any
    strides with d innermost, e.g. a view of a [B,kv_capacity,H,d] cache), kv_len int32 [B] or None.
    Returns (o, tau, support_size)."""
    if q.dtype != torch.bfloat16 or k.dtype != torch.bfloat16 or v.dtype != torch.bfloat16:
        raise EntmaxAttnError("entmax_attn_decode_fwd: bf16 tensors only")
    if not q.is_contiguous() or k.stride() != v.stride() or k.shape != v.shape or k.stride(3) != 1:
        raise EntmaxAttnError("entmax_attn_decode_fwd: q contiguous; k and v the same shape and strides, d innermost")
    B, H, QL, D = q.shape
    if k.shape[0] != B or k.shape[1] != H or k.shape[3] != D:
        raise EntmaxAttnError("entmax_attn_decode_fwd: q and k/v disagree on batch, heads or head_dim")
    params = DecodeParams(B, H, QL, k.shape[2], D, float(alpha), float(sm_scale), k.stride(0), k.stride(1), k.stride(2))
    o = torch.empty_like(q) if o is None else o
    tau = torch.empty((B, H, QL), dtype=torch.float32, device=q.device) if tau is None else tau
    if support_size is None:
        support_size = torch.empty((B, H, QL), dtype=torch.int32, device=q.device)
    if workspace is None:
        nbytes = load().entmax_attn_decode_workspace_bytes(ctypes.byref(params))
        if nbytes == 0:
            raise EntmaxAttnError("entmax_attn_decode_workspace_bytes: invalid parameters")
        workspace = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    rc = load().entmax_attn_decode_fwd(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(kv_len), _ptr(beta),
                                       _ptr(gamma), _ptr(delta), _ptr(alibi_slopes), _ptr(o), _ptr(tau),
                                       _ptr(support_size), _ptr(workspace), workspace.numel(), _ptr(status),
                                       _stream_ptr(stream))
    _check(rc, "entmax_attn_decode_fwd")
    return o, tau, support_size


def entmax_attn_bwd(q, k, v, tau, d_o, alpha, causal, beta=None, gamma=None, delta=None, *, sm_scale=0.0, n_mode=0,
                    dq=None, dk=None, dv=None, workspace=None, status=None, stream=None):
    """Backward pass.  Returns (dq, dk, dv)."""
    _same_layout(q, k, v, d_o)
    params = make_params(q, alpha, causal, sm_scale, n_mode)
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(q) if dk is None else dk
    dv = torch.empty_like(q) if dv is None else dv
    _same_layout(q, dq, dk, dv)
    if workspace is None:
        workspace = alloc_workspace(params, True, q.device)
    rc = load().entmax_attn_bwd(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gamma), _ptr(delta),
                                _ptr(tau), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(workspace),
                                workspace.numel(), _ptr(status), _stream_ptr(stream))
    _check(rc, "entmax_attn_bwd")
    return dq, dk, dv


def entmax_attn_bwd_scale(q, k, v, tau, d_o, alpha, causal, beta, gamma, delta, *, sm_scale=0.0, n_mode=0,
                          dq=None, dk=None, dv=None, d_scale_rows=None, want_param_grads=True, workspace=None,
                          status=None, stream=None):
    """Backward pass with the gradients of the ASEntmax scale.
    Returns (dq, dk, dv, d_scale_rows, (dbeta, dgamma, ddelta) or None)."""
    _same_layout(q, k, v, d_o)
    params = make_params(q, alpha, causal, sm_scale, n_mode)
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(q) if dk is None else dk
    dv = torch.empty_like(q) if dv is None else dv
    _same_layout(q, dq, dk, dv)
    B, H, N, _ = q.shape
    if d_scale_rows is None:
        d_scale_rows = torch.empty((B, H, N), dtype=torch.float32, device=q.device)
    grads = None
    if want_param_grads:
        grads = tuple(torch.empty((H,), dtype=torch.float32, device=q.device) for _ in range(3))
    if workspace is None:
        workspace = alloc_workspace(params, True, q.device)
    g = grads if grads is not None else (None, None, None)
    rc = load().entmax_attn_bwd_scale(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gamma),
                                      _ptr(delta), _ptr(tau), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv),
                                      _ptr(d_scale_rows), _ptr(g[0]), _ptr(g[1]), _ptr(g[2]), _ptr(workspace),
                                      workspace.numel(), _ptr(status), _stream_ptr(stream))
    _check(rc, "entmax_attn_bwd_scale")
    return dq, dk, dv, d_scale_rows, grads


def entmax_attn_fwd_rowscale(q, k, v, c_rows, alpha, causal, *, sm_scale=0.0, o=None, tau=None, workspace=None,
                             status=None, stream=None):
    """Forward pass with a per-query scale table c_rows (float32 [B,H,N]).  Returns (o, tau)."""
    _same_layout(q, k, v)
    params = make_params(q, alpha, causal, sm_scale, 0)
    B, H, N, _ = q.shape
    if c_rows.shape != (B, H, N) or c_rows.dtype != torch.float32 or not c_rows.is_contiguous():
        raise EntmaxAttnError("c_rows must be a contiguous float32 [batch, heads, seq] tensor")
    o = torch.empty_like(q) if o is None else o
    if tau is None:
        tau = torch.empty((B, H, N), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = alloc_workspace(params, False, q.device)
    rc = load().entmax_attn_fwd_rowscale(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(c_rows), _ptr(o),
                                         _ptr(tau), _ptr(workspace), workspace.numel(), _ptr(status), _stream_ptr(stream))
    _check(rc, "entmax_attn_fwd_rowscale")
    return o, tau


def entmax_attn_bwd_rowscale(q, k, v, c_rows, tau, d_o, alpha, causal, *, sm_scale=0.0, dq=None, dk=None, dv=None,
                             d_scale_rows=None, workspace=None, status=None, stream=None):
    """Backward pass with a per-query scale table.  Returns (dq, dk, dv, d_scale_rows)."""
    _same_layout(q, k, v, d_o)
    params = make_params(q, alpha, causal, sm_scale, 0)
    B, H, N, _ = q.shape
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(q) if dk is None else dk
    dv = torch.empty_like(q) if dv is None else dv
    if d_scale_rows is None:
        d_scale_rows = torch.empty((B, H, N), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = alloc_workspace(params, True, q.device)
    rc = load().entmax_attn_bwd_rowscale(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(c_rows), _ptr(tau),
                                         _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(d_scale_rows), _ptr(workspace),
                                         workspace.numel(), _ptr(status), _stream_ptr(stream))
    _check(rc, "entmax_attn_bwd_rowscale")
    return dq, dk, dv, d_scale_rows


def _dp(t):
    return None if t is None else t.data_ptr()


def entmax_attn_fwd_ex(q, k, v, alpha, causal, beta=None, gamma=None, delta=None, *, c_rows=None, alibi_slopes=None,
                       sm_scale=0.0, n_mode=0, o=None, tau=None, workspace=None, status=None, stream=None):
    """Extended forward pass: optional per-query scale table and ALiBi slopes.  Returns (o, tau)."""
    _same_layout(q, k, v)
    params = make_params(q, alpha, causal, sm_scale, n_mode)
    B, H, N, _ = q.shape
    o = torch.empty_like(q) if o is None else o
    if tau is None:
        tau = torch.empty((B, H, N), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = alloc_workspace(params, False, q.device)
    ex = Extras(_dp(c_rows), _dp(alibi_slopes), None, None, None, None, None)
    rc = load().entmax_attn_fwd_ex(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gamma), _ptr(delta),
                                   ctypes.byref(ex), _ptr(o), _ptr(tau), _ptr(workspace), workspace.numel(),
                                   _ptr(status), _stream_ptr(stream))
    _check(rc, "entmax_attn_fwd_ex")
    return o, tau


def entmax_attn_save_supports(q, alpha, causal, fwd_workspace, *, sm_scale=0.0, n_mode=0, saved=None, stream=None):
    """Compact copy of a finished forward call's supports (uint8 CUDA tensor) for entmax_attn_bwd_ex(saved_supports=...)."""
    params = make_params(q, alpha, causal, sm_scale, n_mode)
    nbytes = load().entmax_attn_saved_bytes(ctypes.byref(params))
    if nbytes == 0:
        raise EntmaxAttnError("entmax_attn_saved_bytes: invalid parameters (bf16 problems only)")
    if saved is None:
        saved = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    rc = load().entmax_attn_save_supports(ctypes.byref(params), _ptr(fwd_workspace), _ptr(saved), saved.numel(),
                                          _stream_ptr(stream))
    _check(rc, "entmax_attn_save_supports")
    return saved


def entmax_attn_bwd_ex(q, k, v, tau, d_o, alpha, causal, beta=None, gamma=None, delta=None, *, c_rows=None,
                       alibi_slopes=None, fwd_workspace=None, saved_supports=None, want_scale_rows=False,
                       want_param_grads=False,
                       sm_scale=0.0, n_mode=0, dq=None, dk=None, dv=None, workspace=None, status=None, stream=None):
    """Extended backward pass.  `fwd_workspace`: the forward call's workspace tensor, untouched since
    (the backward pass then reuses the supports it holds instead of sweeping Q K^T again).
    Returns (dq, dk, dv, d_scale_rows or None, (dbeta, dgamma, ddelta) or None)."""
    _same_layout(q, k, v, d_o)
    params = make_params(q, alpha, causal, sm_scale, n_mode)
    B, H, N, _ = q.shape
    dq = torch.empty_like(q) if dq is None else dq
    dk = torch.empty_like(q) if dk is None else dk
    dv = torch.empty_like(q) if dv is None else dv
    dc = torch.empty((B, H, N), dtype=torch.float32, device=q.device) if want_scale_rows else None
    grads = tuple(torch.empty((H,), dtype=torch.float32, device=q.device) for _ in range(3)) if want_param_grads else None
    g = grads if grads is not None else (None, None, None)
    if workspace is None:
        workspace = alloc_workspace(params, True, q.device)
    ex = Extras(_dp(c_rows), _dp(alibi_slopes), _dp(dc), _dp(g[0]), _dp(g[1]), _dp(g[2]), _dp(fwd_workspace),
                _dp(saved_supports))
    rc = load().entmax_attn_bwd_ex(ctypes.byref(params), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(gamma), _ptr(delta),
                                   ctypes.byref(ex), _ptr(tau), _ptr(d_o), _ptr(dq), _ptr(dk), _ptr(dv), _ptr(workspace),
                                   workspace.numel(), _ptr(status), _stream_ptr(stream))
    _check(rc, "entmax_attn_bwd_ex")
    return dq, dk, dv, dc, grads


def entmax_attn_scores_debug(q, k, bh, causal, *, workspace=None, status=None, stream=None):
    """Raw tensor-core accumulators <q_i, k_j> of one (batch, head) pair as a float32 [N, N] tensor
    (NaN where the mask removes the entry)."""
    _same_layout(q, k)
    params = make_params(q, 1.5, causal)
    N = q.shape[2]
    out = torch.full((N, N), float("nan"), dtype=torch.float32, device=q.device)
    if workspace is None:
        workspace = alloc_workspace(params, False, q.device)
    rc = load().entmax_attn_scores_debug(ctypes.byref(params), _ptr(q), _ptr(k), int(bh), _ptr(out), _ptr(workspace),
                                         workspace.numel(), _ptr(status), _stream_ptr(stream))
    _check(rc, "entmax_attn_scores_debug")
    return out


def entmax_attn_profile_events(which: int, start: Optional[torch.cuda.Event], stop: Optional[torch.cuda.Event]):
    """Record `start`/`stop` around the score-sweep kernel of later forward (which=0) or backward (which=1)
    calls of this thread; None, None switches the hook off.  The events must have been created with
    enable_timing=True and recorded once (so that their CUDA handles exist)."""
    a = None if start is None else ctypes.c_void_p(start.cuda_event)
    b = None if stop is None else ctypes.c_void_p(stop.cuda_event)
    _check(load().entmax_attn_profile_events(int(which), a, b), "entmax_attn_profile_events")


def read_support(params: Params, workspace: torch.Tensor, rows):
    """Support lists a forward call left in its workspace, for global row ids `rows`
    (row id = (b*heads + h)*seq + i).  Returns a list of (indices int64 tensor or None, y float32 tensor or None)."""
    lay = entmax_attn_workspace_layout(params)
    total = params.batch * params.heads * params.seq
    cnt = workspace[lay.row_count_offset: lay.row_count_offset + 4 * total].view(torch.int32)
    ent = workspace[lay.entries_offset: lay.entries_offset + 8 * total * lay.capacity].view(torch.int32)
    ent = ent.view(total, lay.capacity, 2)
    rows_t = torch.as_tensor(rows, dtype=torch.long, device=workspace.device)
    cnt_h = cnt[rows_t].cpu()
    ent_h = ent[rows_t].cpu()
    out = []
    for r in range(len(rows)):
        c = int(cnt_h[r])
        if c < 0:
            out.append((None, None))
        else:
            out.append((ent_h[r, :c, 1].to(torch.int64), ent_h[r, :c, 0].contiguous().view(torch.float32)))
    return out


def read_dense_support_sizes(params: Params, workspace: torch.Tensor, rows):
    """Support sizes of rows the dense path computed (row_count == -2), for global row ids `rows`: int64 tensor,
    -1 where the row kept a list instead (use read_support there)."""
    lay = entmax_attn_workspace_layout(params)
    total = params.batch * params.heads * params.seq
    cnt = workspace[lay.row_count_offset: lay.row_count_offset + 4 * total].view(torch.int32)
    dense = workspace[lay.dense_count_offset: lay.dense_count_offset + 8 * total].view(torch.int32).view(total, 2)
    rows_t = torch.as_tensor(rows, dtype=torch.long, device=workspace.device)
    size = dense[rows_t].sum(dim=1).to(torch.int64)
    return torch.where(cnt[rows_t] == -2, size, torch.full_like(size, -1)).cpu()


def entmax_attn_selftest_wait_expiry(limit_ns: int, status: torch.Tensor, stream=None):
    """Runs the bounded-wait self-test: one CTA waits `limit_ns` for a barrier nothing arrives on, then returns with
    FLAG_WAIT_EXPIRED in status[0] and the microseconds it waited in status[1]."""
    _check(load().entmax_attn_selftest_wait_expiry(int(limit_ns), _ptr(status), _stream_ptr(stream)),
           "entmax_attn_selftest_wait_expiry")


def _proj_params(x, heads, causal, n_mode, gamma_range):
    if x.dim() != 3 or not x.is_contiguous():
        raise EntmaxAttnError("x must be a contiguous [batch, seq, d_model] tensor")
    if x.dtype == torch.bfloat16:
        dt = DTYPE_BF16
    elif x.dtype == torch.float32:
        dt = DTYPE_FP32
    else:
        raise EntmaxAttnError("x must be bfloat16 or float32")
    B, N, dm = x.shape
    return ProjParams(B, int(heads), N, dm, dt, int(bool(causal)), int(n_mode), float(gamma_range))


def entmax_attn_scale_proj_fwd(x, w_beta, w_gamma, delta, gamma_range, causal, *, n_mode=0, c_rows=None, stream=None):
    """c_rows [B, H, N] (float32) from the layer input x [B, N, d_model] and per-head weights [H, d_model]."""
    H = w_beta.shape[0]
    params = _proj_params(x, H, causal, n_mode, gamma_range)
    if c_rows is None:
        c_rows = torch.empty((x.shape[0], H, x.shape[1]), dtype=torch.float32, device=x.device)
    _check(load().entmax_attn_scale_proj_fwd(ctypes.byref(params), _ptr(x), _ptr(w_beta), _ptr(w_gamma), _ptr(delta),
                                             _ptr(c_rows), _stream_ptr(stream)), "entmax_attn_scale_proj_fwd")
    return c_rows


def entmax_attn_scale_proj_bwd(x, w_beta, w_gamma, d_scale_rows, gamma_range, causal, *, n_mode=0, want_dx=True,
                               stream=None):
    """Chain rule of the projection.  Returns (dw_beta, dw_gamma, ddelta, dx or None)."""
    H = w_beta.shape[0]
    params = _proj_params(x, H, causal, n_mode, gamma_range)
    dwb, dwg = torch.empty_like(w_beta), torch.empty_like(w_gamma)
    dd = torch.empty((H,), dtype=torch.float32, device=x.device)
    dx = torch.empty_like(x) if want_dx else None
    _check(load().entmax_attn_scale_proj_bwd(ctypes.byref(params), _ptr(x), _ptr(w_beta), _ptr(w_gamma), _ptr(d_scale_rows),
                                             _ptr(dwb), _ptr(dwg), _ptr(dd), _ptr(dx), _stream_ptr(stream)),
           "entmax_attn_scale_proj_bwd")
    return dwb, dwg, dd, dx
