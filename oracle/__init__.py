"""TEST INFRASTRUCTURE -- not part of the product path.

ctypes front end of the plain fp64 CPU oracle (``entmax_oracle.c``).  Only the tests, the smoke
check and the CPU-baseline / reference legs of the benchmark import this package; the CUDA library
and its Python binding never do.

The functions here only marshal arguments: every piece of arithmetic is in the C file, which cites
the passage of the paper each step follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "entmax_oracle.c")
_LIB = os.path.join(_HERE, "libentmax_oracle.so")
_lock = threading.Lock()
_lib = None

METHOD_AUTO, METHOD_BISECT, METHOD_SORT = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (fp64, OpenMP over query rows). Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        cmd = ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True, cwd=_HERE)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            lib = ctypes.CDLL(build())
            dp = ctypes.POINTER(ctypes.c_double)
            fp = ctypes.POINTER(ctypes.c_float)
            ip = ctypes.POINTER(ctypes.c_int64)
            lib.oracle_entmax_row.restype = ctypes.c_int
            lib.oracle_entmax_row.argtypes = [dp, ctypes.c_int, ctypes.c_double, ctypes.c_int, dp, dp]
            lib.oracle_asentmax_scale.restype = ctypes.c_double
            lib.oracle_asentmax_scale.argtypes = [ctypes.c_double] * 3 + [ctypes.c_long]
            common = [ctypes.c_long, ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_int,
                      ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_double]
            lib.oracle_attn_fwd_rows.restype = ctypes.c_int
            lib.oracle_attn_fwd_rows.argtypes = [fp, fp, fp] + common + [ip, ctypes.c_long, dp, dp, dp, ip]
            lib.oracle_attn_bwd_head.restype = ctypes.c_int
            lib.oracle_attn_bwd_head.argtypes = [fp, fp, fp, fp] + common + [dp, dp, dp]
            lib.oracle_attn_bwd_rows.restype = ctypes.c_int
            lib.oracle_attn_bwd_rows.argtypes = [fp, fp, fp, fp] + common + [ip, ctypes.c_long, dp, dp]
            lib.oracle_attn_bwd_scale_head.restype = ctypes.c_int
            lib.oracle_attn_bwd_scale_head.argtypes = [fp, fp, fp, fp] + common + [dp, dp]
            proj = [ctypes.c_long] * 4 + [ctypes.c_double, ctypes.c_int, ctypes.c_int]
            lib.oracle_scale_projection.restype = ctypes.c_int
            lib.oracle_scale_projection.argtypes = [dp, dp, dp, dp] + proj + [dp, dp, dp]
            lib.oracle_scale_projection_bwd.restype = ctypes.c_int
            lib.oracle_scale_projection_bwd.argtypes = [dp, dp, dp, dp] + proj + [dp, dp, dp, dp]
            lib.oracle_num_threads.restype = ctypes.c_int
            lib.oracle_set_num_threads.argtypes = [ctypes.c_int]
            _lib = lib
    return _lib


def _dptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _fptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def _iptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def _f32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(int(n))


def entmax_row(z, alpha: float, method: int = METHOD_AUTO):
    """alpha-entmax of one logit vector. Returns (p, tau, support_size)."""
    z = np.ascontiguousarray(np.asarray(z, dtype=np.float64))
    p = np.empty_like(z)
    tau = ctypes.c_double(0.0)
    supp = _load().oracle_entmax_row(_dptr(z), int(z.shape[0]), float(alpha), int(method), _dptr(p),
                                     ctypes.byref(tau))
    if supp < 0:
        raise ValueError("oracle_entmax_row rejected its arguments (n=%d, alpha=%r)" % (z.shape[0], alpha))
    return p, float(tau.value), int(supp)


def asentmax_scale(beta: float, gamma: float, delta: float, n: int) -> float:
    return float(_load().oracle_asentmax_scale(float(beta), float(gamma), float(delta), int(n)))


def _scale_args(scale):
    if scale is None:
        return 0, 0.0, 0.0, 0.0
    b, g, dl = scale
    return 1, float(b), float(g), float(dl)


def attn_fwd_rows(q, k, v, rows, alpha, sm_scale, causal, scale=None, n_mode=0, want_p=False, alibi=0.0):
    """Forward of one head for the query rows in ``rows``.

    q, k, v: [N, d] arrays (values already rounded to the precision under test).
    scale: None (fixed temperature) or (beta, gamma, delta) of this head.
    alibi: ALiBi slope m of this head (0 = no positional term).
    Returns dict(tau [R], o [R, d], supp [R], p [R, N] or None).
    """
    q, k, v = _f32(q), _f32(k), _f32(v)
    N, d = q.shape
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    R = rows.shape[0]
    tau = np.empty(R, dtype=np.float64)
    o = np.empty((R, d), dtype=np.float64)
    supp = np.empty(R, dtype=np.int64)
    p = np.empty((R, N), dtype=np.float64) if want_p else None
    us, b, g, dl = _scale_args(scale)
    rc = _load().oracle_attn_fwd_rows(_fptr(q), _fptr(k), _fptr(v), N, d, float(alpha), float(sm_scale),
                                      int(bool(causal)), int(n_mode), us, b, g, dl, float(alibi), _iptr(rows), R,
                                      _dptr(tau), _dptr(o), _dptr(p) if want_p else None, _iptr(supp))
    if rc != 0:
        raise RuntimeError("oracle_attn_fwd_rows failed: %d" % rc)
    return {"tau": tau, "o": o, "supp": supp, "p": p}


def attn_bwd_head(q, k, v, d_o, alpha, sm_scale, causal, scale=None, n_mode=0, alibi=0.0):
    """Backward of one head, every row. Returns (dq, dk, dv) as float64 [N, d]."""
    q, k, v, d_o = _f32(q), _f32(k), _f32(v), _f32(d_o)
    N, d = q.shape
    dq = np.empty((N, d), dtype=np.float64)
    dk = np.empty((N, d), dtype=np.float64)
    dv = np.empty((N, d), dtype=np.float64)
    us, b, g, dl = _scale_args(scale)
    rc = _load().oracle_attn_bwd_head(_fptr(q), _fptr(k), _fptr(v), _fptr(d_o), N, d, float(alpha),
                                      float(sm_scale), int(bool(causal)), int(n_mode), us, b, g, dl, float(alibi),
                                      _dptr(dq), _dptr(dk), _dptr(dv))
    if rc != 0:
        raise RuntimeError("oracle_attn_bwd_head failed: %d" % rc)
    return dq, dk, dv


def attn_bwd_rows(q, k, v, d_o, rows, alpha, sm_scale, causal, scale=None, n_mode=0, want_ds=False, alibi=0.0):
    """Row-local backward (dQ rows, optionally dS rows) of one head for ``rows``."""
    q, k, v, d_o = _f32(q), _f32(k), _f32(v), _f32(d_o)
    N, d = q.shape
    rows = np.ascontiguousarray(np.asarray(rows, dtype=np.int64))
    R = rows.shape[0]
    dq = np.empty((R, d), dtype=np.float64)
    ds = np.empty((R, N), dtype=np.float64) if want_ds else None
    us, b, g, dl = _scale_args(scale)
    rc = _load().oracle_attn_bwd_rows(_fptr(q), _fptr(k), _fptr(v), _fptr(d_o), N, d, float(alpha),
                                      float(sm_scale), int(bool(causal)), int(n_mode), us, b, g, dl, float(alibi),
                                      _iptr(rows), R, _dptr(dq), _dptr(ds) if want_ds else None)
    if rc != 0:
        raise RuntimeError("oracle_attn_bwd_rows failed: %d" % rc)
    return dq, ds


def attn_bwd_scale_head(q, k, v, d_o, alpha, sm_scale, causal, scale=None, n_mode=0, alibi=0.0):
    """Gradients with respect to the ASEntmax scale of one head.
    Returns (dc float64 [N], (dbeta, dgamma, ddelta))."""
    q, k, v, d_o = _f32(q), _f32(k), _f32(v), _f32(d_o)
    N, d = q.shape
    dc = np.empty(N, dtype=np.float64)
    grads = np.zeros(3, dtype=np.float64)
    us, b, g, dl = _scale_args(scale)
    rc = _load().oracle_attn_bwd_scale_head(_fptr(q), _fptr(k), _fptr(v), _fptr(d_o), N, d, float(alpha),
                                            float(sm_scale), int(bool(causal)), int(n_mode), us, b, g, dl, float(alibi),
                                            _dptr(dc), _dptr(grads))
    if rc != 0:
        raise RuntimeError("oracle_attn_bwd_scale_head failed: %d" % rc)
    return dc, (float(grads[0]), float(grads[1]), float(grads[2]))


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def scale_projection(x, w_beta, w_gamma, delta, s, causal, n_mode=0):
    """ASEntmax's content-dependent scale (Sec. 4.1) from the layer input x [B, N, dm] and per-head weights [H, dm].
    Returns (c, beta, gamma), each float64 [B, H, N]."""
    x, w_beta, w_gamma, delta = _f64(x), _f64(w_beta), _f64(w_gamma), _f64(delta)
    B, N, dm = x.shape
    H = w_beta.shape[0]
    c, beta, gamma = (np.empty((B, H, N), dtype=np.float64) for _ in range(3))
    rc = _load().oracle_scale_projection(_dptr(x), _dptr(w_beta), _dptr(w_gamma), _dptr(delta), B, H, N, dm, float(s),
                                         int(bool(causal)), int(n_mode), _dptr(c), _dptr(beta), _dptr(gamma))
    if rc != 0:
        raise RuntimeError("oracle_scale_projection failed: %d" % rc)
    return c, beta, gamma


def scale_projection_bwd(x, w_beta, w_gamma, dc, s, causal, n_mode=0):
    """Chain rule of scale_projection. Returns (dw_beta [H, dm], dw_gamma [H, dm], ddelta [H], dx [B, N, dm])."""
    x, w_beta, w_gamma, dc = _f64(x), _f64(w_beta), _f64(w_gamma), _f64(dc)
    B, N, dm = x.shape
    H = w_beta.shape[0]
    dwb, dwg = np.empty((H, dm), dtype=np.float64), np.empty((H, dm), dtype=np.float64)
    dd, dx = np.empty(H, dtype=np.float64), np.empty((B, N, dm), dtype=np.float64)
    rc = _load().oracle_scale_projection_bwd(_dptr(x), _dptr(w_beta), _dptr(w_gamma), _dptr(dc), B, H, N, dm, float(s),
                                             int(bool(causal)), int(n_mode), _dptr(dwb), _dptr(dwg), _dptr(dd), _dptr(dx))
    if rc != 0:
        raise RuntimeError("oracle_scale_projection_bwd failed: %d" % rc)
    return dwb, dwg, dd, dx
