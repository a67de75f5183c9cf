"""ctypes front end of the fp64 CPU oracle (``la_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA package never imports this module and
this module never imports the CUDA package.

Inputs may be torch tensors or numpy arrays of any float dtype; they are widened
exactly to fp32 containers (bf16 -> fp32 is exact) and the C routines do all
arithmetic in fp64.  Outputs are numpy float64 arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "la_oracle.c")
_LIB = os.path.join(_HERE, "libla_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP). Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        fp = ctypes.POINTER(ctypes.c_float)
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int)
        I = ctypes.c_int
        lib.orc_threads.restype = I
        lib.orc_fwd_rec.argtypes = [fp, fp, fp, dp, dp, I, I, I, I, I, dp, dp]
        lib.orc_bwd_rec.argtypes = [fp, fp, fp, fp, dp, dp, dp, I, I, I, I, I, dp, dp, dp, dp]
        lib.orc_fwd_quad.argtypes = [fp, fp, fp, dp, I, I, I, I, I, dp]
        lib.orc_bwd_quad.argtypes = [fp, fp, fp, fp, dp, I, I, I, I, I, dp, dp, dp]
        lib.orc_rows.argtypes = [I, fp, fp, fp, fp, dp, I, I, I, I, I, I, ip, ip, dp]
        lib.orc_decode_step.argtypes = [fp, fp, fp, dp, dp, I, I, I, I, dp]
        lib.orc_fwd_origin.argtypes = [fp, fp, fp, dp, I, I, I, I, I, dp]
        lib.orc_lrpe_fwd_quad.argtypes = [fp, fp, fp, dp, dp, I, I, I, I, I, dp]
        lib.orc_lrpe_bwd_quad.argtypes = [fp, fp, fp, fp, dp, dp, I, I, I, I, I, dp, dp, dp, dp]
        lib.orc_norm_gate_fwd.argtypes = [dp, fp, ctypes.c_long, I, dp, dp]
        lib.orc_norm_gate_bwd.argtypes = [dp, fp, fp, ctypes.c_long, I, dp, dp]
        for name in ("orc_fwd_rec", "orc_bwd_rec", "orc_fwd_quad", "orc_bwd_quad", "orc_rows",
                     "orc_decode_step", "orc_fwd_origin", "orc_norm_gate_fwd", "orc_norm_gate_bwd"):
            getattr(lib, name).restype = I
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().orc_threads())


def _f32(x) -> np.ndarray:
    """Exact widening of the given values into a contiguous fp32 numpy array."""
    if hasattr(x, "detach"):  # torch tensor
        import torch
        x = x.detach().to("cpu").to(torch.float32).contiguous().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float32))


def _f64(x) -> Optional[np.ndarray]:
    if x is None:
        return None
    if hasattr(x, "detach"):
        import torch
        x = x.detach().to("cpu").to(torch.float64).contiguous().numpy()
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _check(rc: int, name: str):
    if rc != 0:
        raise RuntimeError("%s failed (bad sizes or out of memory)" % name)


def _dims(q, v):
    B, H, N, d = q.shape
    e = v.shape[-1]
    assert v.shape[:3] == (B, H, N)
    return B, H, N, d, e


def fwd_rec(q, k, v, lam, kv_in=None, want_state: bool = False):
    """Algorithm 2 over the whole sequence. Returns o [B,H,N,e] (and kv_out [B,H,d,e])."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, H, N, d, e = _dims(q, v)
    lam = _f64(lam)
    assert lam.shape == (H,)
    kv_in = _f64(kv_in)
    o = np.empty((B, H, N, e), np.float64)
    kv_out = np.empty((B, H, d, e), np.float64) if want_state else None
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_fwd_rec(_p(q, F), _p(k, F), _p(v, F), _p(lam, D), _p(kv_in, D),
                               B, H, N, d, e, _p(o, D), _p(kv_out, D)), "orc_fwd_rec")
    return (o, kv_out) if want_state else o


def bwd_rec(q, k, v, do, lam, kv_in=None, grad_kv_out=None, want_state_grad: bool = False):
    """Gradients of <O,dO> (+ <kv_out, grad_kv_out>) by the forward/reverse recurrences."""
    q, k, v, do = _f32(q), _f32(k), _f32(v), _f32(do)
    B, H, N, d, e = _dims(q, v)
    lam = _f64(lam)
    kv_in, grad_kv_out = _f64(kv_in), _f64(grad_kv_out)
    dq = np.empty((B, H, N, d), np.float64)
    dk = np.empty((B, H, N, d), np.float64)
    dv = np.empty((B, H, N, e), np.float64)
    gin = np.empty((B, H, d, e), np.float64) if want_state_grad else None
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_bwd_rec(_p(q, F), _p(k, F), _p(v, F), _p(do, F), _p(lam, D), _p(kv_in, D),
                               _p(grad_kv_out, D), B, H, N, d, e,
                               _p(dq, D), _p(dk, D), _p(dv, D), _p(gin, D)), "orc_bwd_rec")
    return (dq, dk, dv, gin) if want_state_grad else (dq, dk, dv)


def fwd_quad(q, k, v, lam):
    """O = (Q K^T (.) M) V with the N x N matrix materialised."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, H, N, d, e = _dims(q, v)
    lam = _f64(lam)
    o = np.empty((B, H, N, e), np.float64)
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_fwd_quad(_p(q, F), _p(k, F), _p(v, F), _p(lam, D), B, H, N, d, e, _p(o, D)),
           "orc_fwd_quad")
    return o


def bwd_quad(q, k, v, do, lam):
    """dQ = dA K, dK = dA^T Q, dV = A^T dO with A, dA materialised."""
    q, k, v, do = _f32(q), _f32(k), _f32(v), _f32(do)
    B, H, N, d, e = _dims(q, v)
    lam = _f64(lam)
    dq = np.empty((B, H, N, d), np.float64)
    dk = np.empty((B, H, N, d), np.float64)
    dv = np.empty((B, H, N, e), np.float64)
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_bwd_quad(_p(q, F), _p(k, F), _p(v, F), _p(do, F), _p(lam, D), B, H, N, d, e,
                                _p(dq, D), _p(dk, D), _p(dv, D)), "orc_bwd_quad")
    return dq, dk, dv


_KINDS = {"o": 0, "dq": 1, "dk": 2, "dv": 3}


def rows(kind: str, q, k, v, do, lam, bh_idx, t_idx):
    """Single rows of the quadratic form: kind in {'o','dq','dk','dv'}; row r is
    (flattened b*H+h = bh_idx[r], position t_idx[r]).  Returns [nrows, e or d]."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    do = None if do is None else _f32(do)
    B, H, N, d, e = _dims(q, v)
    lam = _f64(lam)
    bh_idx = np.ascontiguousarray(np.asarray(bh_idx, dtype=np.int32))
    t_idx = np.ascontiguousarray(np.asarray(t_idx, dtype=np.int32))
    n = int(bh_idx.shape[0])
    w = e if kind in ("o", "dv") else d
    out = np.empty((n, w), np.float64)
    D, F, I = ctypes.c_double, ctypes.c_float, ctypes.c_int
    _check(_load().orc_rows(_KINDS[kind], _p(q, F), _p(k, F), _p(v, F), _p(do, F), _p(lam, D),
                            B, H, N, d, e, n, _p(bh_idx, I), _p(t_idx, I), _p(out, D)), "orc_rows")
    return out


def decode_step(q, k, v, lam, kv: np.ndarray):
    """One iteration of Algorithm 2 on an fp64 state [B,H,d,e], updated in place. Returns o [B,H,e]."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, H, d = q.shape
    e = v.shape[-1]
    lam = _f64(lam)
    assert kv.dtype == np.float64 and kv.flags["C_CONTIGUOUS"] and kv.shape == (B, H, d, e)
    o = np.empty((B, H, e), np.float64)
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_decode_step(_p(q, F), _p(k, F), _p(v, F), _p(lam, D), _p(kv, D), B, H, d, e,
                                   _p(o, D)), "orc_decode_step")
    return o


def fwd_origin(q, k, v, lam):
    """Algorithm 1 (prescaled recurrence); overflows for long sequences by design."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, H, N, d, e = _dims(q, v)
    lam = _f64(lam)
    o = np.empty((B, H, N, e), np.float64)
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_fwd_origin(_p(q, F), _p(k, F), _p(v, F), _p(lam, D), B, H, N, d, e, _p(o, D)),
           "orc_fwd_origin")
    return o


def norm_gate_fwd(o, u, want_rstd: bool = False):
    """y = SRMSNorm(o) (.) u per row of the last axis (Eq. 3 with Eq. 8). o fp64 array, u any; returns fp64."""
    o = np.ascontiguousarray(np.asarray(o, np.float64))
    u = _f32(u)
    assert o.shape == u.shape
    e = o.shape[-1]
    rows = o.size // e
    y = np.empty_like(o)
    rstd = np.empty(o.shape[:-1], np.float64) if want_rstd else None
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_norm_gate_fwd(_p(o, D), _p(u, F), ctypes.c_long(rows), e, _p(y, D), _p(rstd, D)),
           "orc_norm_gate_fwd")
    return (y, rstd) if want_rstd else y


def norm_gate_bwd(o, u, dy):
    """Gradients of <y, dy> with respect to o and u; returns (do, du) in fp64."""
    o = np.ascontiguousarray(np.asarray(o, np.float64))
    u, dy = _f32(u), _f32(dy)
    assert o.shape == u.shape == dy.shape
    e = o.shape[-1]
    rows = o.size // e
    d_o, d_u = np.empty_like(o), np.empty_like(o)
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_norm_gate_bwd(_p(o, D), _p(u, F), _p(dy, F), ctypes.c_long(rows), e, _p(d_o, D), _p(d_u, D)),
           "orc_norm_gate_bwd")
    return d_o, d_u


def lrpe_fwd_quad(q, k, v, lam, theta):
    """LRPE-d (Eq. 1): o_t = sum_{s<=t} lambda^(t-s) sum_i q_t[i] k_s[i] cos(theta[h,i] (t-s)) v_s.  theta [H, d]."""
    q, k, v = _f32(q), _f32(k), _f32(v)
    B, H, N, d, e = _dims(q, v)
    lam, theta = _f64(lam), _f64(theta)
    assert theta.shape == (H, d)
    o = np.empty((B, H, N, e), np.float64)
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_lrpe_fwd_quad(_p(q, F), _p(k, F), _p(v, F), _p(lam, D), _p(theta, D), B, H, N, d, e, _p(o, D)),
           "orc_lrpe_fwd_quad")
    return o


def lrpe_bwd_quad(q, k, v, do, lam, theta):
    """Gradients of <O, dO> for LRPE-d with respect to q, k, v and theta ([H, d], summed over the batch)."""
    q, k, v, do = _f32(q), _f32(k), _f32(v), _f32(do)
    B, H, N, d, e = _dims(q, v)
    lam, theta = _f64(lam), _f64(theta)
    assert theta.shape == (H, d)
    dq = np.empty((B, H, N, d), np.float64)
    dk = np.empty((B, H, N, d), np.float64)
    dv = np.empty((B, H, N, e), np.float64)
    dth = np.empty((H, d), np.float64)
    D, F = ctypes.c_double, ctypes.c_float
    _check(_load().orc_lrpe_bwd_quad(_p(q, F), _p(k, F), _p(v, F), _p(do, F), _p(lam, D), _p(theta, D), B, H, N, d, e,
                                     _p(dq, D), _p(dk, D), _p(dv, D), _p(dth, D)), "orc_lrpe_bwd_quad")
    return dq, dk, dv, dth
