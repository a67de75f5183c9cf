"""Thin ctypes binding of the C ABI in ``include/la.h``.

Argument marshalling only: every step of the attention path runs in the CUDA
kernels behind ``libla_b200.so``.  PyTorch is used for device memory and streams.
There is no fallback: if the library is missing or the device is not a B200 the
calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libla_b200.so")

LA_BF16, LA_F32 = 0, 1
LA_PATH_AUTO, LA_PATH_SIMT, LA_PATH_TENSOR = 0, 1, 2
LA_SPLIT_SCORES, LA_SPLIT_STATE, LA_SPLIT_DECAYED = 1, 2, 4
LA_PRECISION_DEFAULT = -1
LA_OP_FWD, LA_OP_BWD, LA_OP_DECODE = 0, 1, 2
LA_LAYOUT_BHND, LA_LAYOUT_BNHD = 0, 1

EXPORTS = ("la_workspace_bytes", "la_segment_length", "la_fwd", "la_bwd", "la_decode_step",
           "la_status_string", "la_version", "la_launch_count", "la_profile_enable",
           "la_profile_collect", "la_host_arena_bytes", "la_fwd_bwd_host", "la_device_status", "la_fwd_noalloc", "la_bwd_reuse",
           "la_selftest_bounded_wait", "la_fwd_gated", "la_gate_bwd", "la_gate_fwd", "la_decode_steps", "la_varlen_workspace_bytes", "la_fwd_varlen",
           "la_bwd_varlen", "la_lrpe_workspace_bytes", "la_lrpe_fwd", "la_lrpe_bwd", "la_chunk_state_workspace_bytes", "la_chunk_state", "la_chain_states")
LA_NOALLOC_SCRATCH_BYTES = 32 << 20
KERNEL_KINDS = ("prepass", "scan", "walk", "decode", "walk_pair", "gate", "lrpe")


class LaShape(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int), ("H", ctypes.c_int), ("N", ctypes.c_int), ("d", ctypes.c_int),
                ("e", ctypes.c_int), ("in_dtype", ctypes.c_int), ("out_dtype", ctypes.c_int),
                ("seg_len", ctypes.c_int), ("path", ctypes.c_int), ("precision", ctypes.c_int),
                ("layout", ctypes.c_int)]


class LaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__("%s: %s (status %d)" % (where, status_string(code), code))


_lib = None


def load():
    """Load the shared library (raises if it has not been built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("CUDA library %s is missing; run `python -m paper_2307_14995_b200.build`"
                               % LIB_PATH)
        lib = ctypes.CDLL(LIB_PATH)
        vp, sz, I = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
        sp = ctypes.POINTER(LaShape)
        fp = ctypes.POINTER(ctypes.c_float)
        lib.la_workspace_bytes.argtypes = [I, sp]
        lib.la_workspace_bytes.restype = sz
        lib.la_segment_length.argtypes = [sp]
        lib.la_segment_length.restype = I
        lib.la_fwd.argtypes = [sp, vp, vp, vp, fp, vp, vp, vp, vp, sz, vp]
        lib.la_fwd.restype = I
        lib.la_fwd_gated.argtypes = [sp, vp, vp, vp, vp, fp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.la_fwd_gated.restype = I
        lib.la_gate_fwd.argtypes = [sp, vp, vp, vp, vp, vp]
        lib.la_gate_fwd.restype = I
        lib.la_gate_bwd.argtypes = [sp, vp, vp, vp, vp, vp, vp]
        lib.la_gate_bwd.restype = I
        lib.la_fwd_noalloc.argtypes = [sp, vp, vp, vp, fp, vp, vp, vp, vp]
        lib.la_fwd_noalloc.restype = I
        lib.la_bwd.argtypes = [sp, vp, vp, vp, vp, fp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.la_bwd.restype = I
        lib.la_bwd_reuse.argtypes = [sp, vp, vp, vp, vp, fp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.la_bwd_reuse.restype = I
        lib.la_decode_step.argtypes = [sp, vp, vp, vp, fp, vp, vp, vp]
        lib.la_decode_step.restype = I
        ip = ctypes.POINTER(ctypes.c_int)
        lib.la_varlen_workspace_bytes.argtypes = [I, sp, ip, I]
        lib.la_varlen_workspace_bytes.restype = sz
        lib.la_fwd_varlen.argtypes = [sp, vp, vp, vp, fp, vp, ip, I, vp, vp, vp, sz, vp]
        lib.la_fwd_varlen.restype = I
        lib.la_bwd_varlen.argtypes = [sp, vp, vp, vp, vp, fp, vp, vp, vp, ip, I, vp, vp, vp, vp, sz, vp]
        lib.la_bwd_varlen.restype = I
        LL = ctypes.c_longlong
        lib.la_lrpe_workspace_bytes.argtypes = [I, sp]
        lib.la_lrpe_workspace_bytes.restype = sz
        lib.la_lrpe_fwd.argtypes = [sp, vp, vp, vp, vp, fp, LL, vp, vp, vp, vp, sz, vp]
        lib.la_lrpe_fwd.restype = I
        lib.la_lrpe_bwd.argtypes = [sp, vp, vp, vp, vp, vp, fp, LL, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
        lib.la_lrpe_bwd.restype = I
        lib.la_chunk_state_workspace_bytes.argtypes = [sp]
        lib.la_chunk_state_workspace_bytes.restype = sz
        lib.la_chunk_state.argtypes = [sp, I, vp, vp, fp, vp, vp, sz, vp]
        lib.la_chunk_state.restype = I
        lib.la_chain_states.argtypes = [sp, LL, LL, I, vp, I, I, vp, fp, vp, vp]
        lib.la_chain_states.restype = I
        lib.la_decode_steps.argtypes = [sp, vp, vp, vp, fp, vp, vp, vp]
        lib.la_decode_steps.restype = I
        lib.la_host_arena_bytes.argtypes = [sp]
        lib.la_host_arena_bytes.restype = sz
        lib.la_fwd_bwd_host.argtypes = [sp, vp, vp, vp, vp, fp, vp, vp, vp, vp, vp, sz, vp]
        lib.la_fwd_bwd_host.restype = I
        lib.la_selftest_bounded_wait.argtypes = [ctypes.c_ulonglong, vp]
        lib.la_selftest_bounded_wait.restype = I
        lib.la_device_status.argtypes = [ctypes.POINTER(ctypes.c_uint)]
        lib.la_device_status.restype = I
        lib.la_status_string.argtypes = [I]
        lib.la_status_string.restype = ctypes.c_char_p
        lib.la_version.restype = I
        lib.la_launch_count.restype = ctypes.c_ulonglong
        lib.la_profile_enable.argtypes = [I]
        lib.la_profile_enable.restype = None
        lib.la_profile_collect.argtypes = [ctypes.POINTER(ctypes.c_double),
                                           ctypes.POINTER(ctypes.c_ulonglong)]
        lib.la_profile_collect.restype = I
        _lib = lib
    return _lib


def status_string(code: int) -> str:
    return load().la_status_string(int(code)).decode()


def version() -> int:
    return int(load().la_version())


def launch_count() -> int:
    return int(load().la_launch_count())


def device_status() -> int:
    """Blocks until the device is idle; raises if a tensor-core block gave up on a bounded wait."""
    code = ctypes.c_uint(0)
    rc = load().la_device_status(ctypes.byref(code))
    if rc != 0:
        raise LaError(rc, "la_device_status (device code %d)" % code.value)
    return int(code.value)


def selftest_bounded_wait(budget_clocks: int, stream=None) -> None:
    """Launch the bounded-wait self-test (see la.h); the outcome is read with device_status()."""
    rc = load().la_selftest_bounded_wait(int(budget_clocks), _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_selftest_bounded_wait")


def profile_enable(on: bool) -> None:
    load().la_profile_enable(1 if on else 0)


def profile_collect():
    """{kind: (total_ms, launches)} for the kernels launched while profiling was enabled."""
    ms = (ctypes.c_double * len(KERNEL_KINDS))()
    n = (ctypes.c_ulonglong * len(KERNEL_KINDS))()
    rc = load().la_profile_collect(ms, n)
    if rc != 0:
        raise LaError(rc, "la_profile_collect")
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_KINDS)}


_DT = {torch.bfloat16: LA_BF16, torch.float32: LA_F32}


def make_shape(B, H, N, d, e, in_dtype, out_dtype, seg_len=0, path=LA_PATH_AUTO,
               precision=LA_PRECISION_DEFAULT, layout=LA_LAYOUT_BHND) -> LaShape:
    return LaShape(B, H, N, d, e, _DT[in_dtype], _DT[out_dtype], seg_len, path, precision, layout)


def workspace_bytes(op: int, shape: LaShape) -> int:
    n = load().la_workspace_bytes(op, ctypes.byref(shape))
    if n == ctypes.c_size_t(-1).value:
        raise LaError(2, "la_workspace_bytes")
    return int(n)


def segment_length(shape: LaShape) -> int:
    return int(load().la_segment_length(ctypes.byref(shape)))


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("tensors must be contiguous CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _lam(lam) -> ctypes.Array:
    vals = [float(x) for x in (lam.tolist() if hasattr(lam, "tolist") else lam)]
    return (ctypes.c_float * len(vals))(*vals)


def _stream(stream) -> ctypes.c_void_p:
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def alloc_workspace(op: int, shape: LaShape, device) -> Optional[torch.Tensor]:
    n = workspace_bytes(op, shape)
    if n == 0:
        return None
    return torch.empty(n, dtype=torch.uint8, device=device)  # torch allocations are >= 256-byte aligned


def la_fwd(shape: LaShape, q, k, v, lam, o, kv_in=None, kv_out=None, workspace=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().la_fwd(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _lam(lam), _ptr(o), _ptr(kv_in),
                       _ptr(kv_out), _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_fwd")


def la_fwd_gated(shape: LaShape, q, k, v, u, lam, y, o=None, rstd=None, kv_in=None, kv_out=None, workspace=None,
                 stream=None):
    """la_fwd with y = SRMSNorm(o) (.) u as its output stage; o and rstd are optional outputs."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().la_fwd_gated(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(u), _lam(lam), _ptr(y), _ptr(o),
                             _ptr(rstd), _ptr(kv_in), _ptr(kv_out), _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_fwd_gated")


def la_gate_fwd(shape: LaShape, o, u, y, rstd=None, stream=None):
    rc = load().la_gate_fwd(ctypes.byref(shape), _ptr(o), _ptr(u), _ptr(y), _ptr(rstd), _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_gate_fwd")


def la_gate_bwd(shape: LaShape, o, u, dy, d_o, d_u, stream=None):
    rc = load().la_gate_bwd(ctypes.byref(shape), _ptr(o), _ptr(u), _ptr(dy), _ptr(d_o), _ptr(d_u), _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_gate_bwd")


def la_fwd_noalloc(shape: LaShape, q, k, v, lam, o, kv_in=None, kv_out=None, stream=None):
    """la_fwd with the library's built-in static scratch: for callers that cannot allocate device
    memory when they call (everything was handed to a pool at start-up, no allocator is available,
    or an allocation's device-wide synchronisation is unacceptable).  Calls on different streams
    must not overlap; shapes needing more than LA_NOALLOC_SCRATCH_BYTES raise LaError (status 7)."""
    rc = load().la_fwd_noalloc(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _lam(lam), _ptr(o), _ptr(kv_in),
                               _ptr(kv_out), _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_fwd_noalloc")


def la_bwd(shape: LaShape, q, k, v, do, lam, dq, dk, dv, kv_in=None, grad_kv_out=None, grad_kv_in=None,
           workspace=None, stream=None, fwd_workspace=None):
    """fwd_workspace: the workspace of the matching la_fwd call (same shape, inputs, kv_in), to reuse its
    segment states (la_bwd_reuse); None recomputes them (la_bwd)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    if fwd_workspace is None:
        rc = load().la_bwd(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(do), _lam(lam), _ptr(dq),
                           _ptr(dk), _ptr(dv), _ptr(kv_in), _ptr(grad_kv_out), _ptr(grad_kv_in),
                           _ptr(workspace), ws_bytes, _stream(stream))
    else:
        rc = load().la_bwd_reuse(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(do), _lam(lam), _ptr(dq),
                                 _ptr(dk), _ptr(dv), _ptr(kv_in), _ptr(grad_kv_out), _ptr(grad_kv_in),
                                 _ptr(fwd_workspace), _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_bwd")


def la_decode_step(shape: LaShape, q, k, v, lam, kv, o, stream=None):
    rc = load().la_decode_step(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _lam(lam), _ptr(kv),
                               _ptr(o), _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_decode_step")


def la_decode_steps(shape: LaShape, q, k, v, lam, kv, o, stream=None):
    """shape.N consecutive tokens per call: q, k [B,H,N,d], v, o [B,H,N,e]; kv updated in place once."""
    rc = load().la_decode_steps(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _lam(lam), _ptr(kv),
                                _ptr(o), _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_decode_steps")


def _cu(cu_seqlens):
    vals = [int(x) for x in cu_seqlens]
    return (ctypes.c_int * len(vals))(*vals), len(vals) - 1


def varlen_workspace_bytes(op: int, shape: LaShape, cu_seqlens) -> int:
    cu, S = _cu(cu_seqlens)
    n = load().la_varlen_workspace_bytes(op, ctypes.byref(shape), cu, S)
    if n == ctypes.c_size_t(-1).value:
        raise LaError(2, "la_varlen_workspace_bytes")
    return int(n)


def la_fwd_varlen(shape: LaShape, q, k, v, lam, o, cu_seqlens, kv_in=None, kv_out=None, workspace=None, stream=None):
    """Packed [T,H,d] tensors (shape: B=1, N=T, layout BNHD); cu_seqlens: host ints, first token of each sequence."""
    cu, S = _cu(cu_seqlens)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().la_fwd_varlen(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _lam(lam), _ptr(o), cu, S, _ptr(kv_in),
                              _ptr(kv_out), _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_fwd_varlen")


def la_bwd_varlen(shape: LaShape, q, k, v, do, lam, dq, dk, dv, cu_seqlens, kv_in=None, grad_kv_out=None,
                  grad_kv_in=None, workspace=None, stream=None):
    cu, S = _cu(cu_seqlens)
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().la_bwd_varlen(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(do), _lam(lam), _ptr(dq), _ptr(dk),
                              _ptr(dv), cu, S, _ptr(kv_in), _ptr(grad_kv_out), _ptr(grad_kv_in), _ptr(workspace),
                              ws_bytes, _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_bwd_varlen")


def chunk_state_workspace_bytes(shape: LaShape) -> int:
    n = load().la_chunk_state_workspace_bytes(ctypes.byref(shape))
    if n == ctypes.c_size_t(-1).value:
        raise LaError(2, "la_chunk_state_workspace_bytes")
    return int(n)


def la_chunk_state(shape: LaShape, reverse: int, b, c, lam, state_out, workspace, stream=None):
    """A chunk's own state contribution: reverse=0 (b=k, c=v) or reverse=1 (b=q, c=dO)."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().la_chunk_state(ctypes.byref(shape), int(reverse), _ptr(b), _ptr(c), _lam(lam), _ptr(state_out),
                               _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_chunk_state")


def la_chain_states(shape: LaShape, total_tokens: int, chunk_tokens: int, reverse: int, states, num_chunks: int,
                    chunk: int, boundary, lam, state_out, stream=None):
    """The state at a cut from the gathered per-chunk contributions [num_chunks,B,H,d,e]."""
    rc = load().la_chain_states(ctypes.byref(shape), int(total_tokens), int(chunk_tokens), int(reverse), _ptr(states),
                                int(num_chunks), int(chunk), _ptr(boundary), _lam(lam), _ptr(state_out), _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_chain_states")


def lrpe_workspace_bytes(op: int, shape: LaShape) -> int:
    n = load().la_lrpe_workspace_bytes(op, ctypes.byref(shape))
    if n == ctypes.c_size_t(-1).value:
        raise LaError(2, "la_lrpe_workspace_bytes")
    return int(n)


def la_lrpe_fwd(shape: LaShape, q, k, v, theta, lam, o, pos0=0, kv_in=None, kv_out=None, workspace=None, stream=None):
    """LRPE-d forward (Eq. 1); theta: device fp32 [H,d]; states [2,B,H,d,e]."""
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().la_lrpe_fwd(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(theta), _lam(lam), int(pos0), _ptr(o),
                            _ptr(kv_in), _ptr(kv_out), _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_lrpe_fwd")


def la_lrpe_bwd(shape: LaShape, q, k, v, do, theta, lam, dq, dk, dv, dtheta, pos0=0, kv_in=None, grad_kv_out=None,
                grad_kv_in=None, workspace=None, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    rc = load().la_lrpe_bwd(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(do), _ptr(theta), _lam(lam), int(pos0),
                            _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dtheta), _ptr(kv_in), _ptr(grad_kv_out),
                            _ptr(grad_kv_in), _ptr(workspace), ws_bytes, _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_lrpe_bwd")


def host_arena_bytes(shape: LaShape) -> int:
    n = load().la_host_arena_bytes(ctypes.byref(shape))
    if n == ctypes.c_size_t(-1).value:
        raise LaError(2, "la_host_arena_bytes")
    return int(n)


def la_fwd_bwd_host(shape: LaShape, q, k, v, do, lam, o, dq, dk, dv, arena, stream=None):
    """Host tensors in and out (ideally pinned); `arena` is a CUDA uint8 tensor of host_arena_bytes()."""
    for t in (q, k, v, do, o, dq, dk, dv):
        if t.is_cuda or not t.is_contiguous():
            raise ValueError("host tensors must be contiguous CPU tensors")
    hp = lambda t: ctypes.c_void_p(t.data_ptr())
    rc = load().la_fwd_bwd_host(ctypes.byref(shape), hp(q), hp(k), hp(v), hp(do), _lam(lam), hp(o), hp(dq),
                                hp(dk), hp(dv), _ptr(arena), arena.numel(), _stream(stream))
    if rc != 0:
        raise LaError(rc, "la_fwd_bwd_host")


# ---- convenience wrappers that allocate outputs with torch -------------------------------
def fwd(q, k, v, lam, *, out_dtype=torch.float32, kv_in=None, want_state=False, seg_len=0,
        path=LA_PATH_AUTO, precision=LA_PRECISION_DEFAULT, stream=None):
    B, H, N, d = q.shape
    e = v.shape[-1]
    shape = make_shape(B, H, N, d, e, q.dtype, out_dtype, seg_len, path, precision)
    o = torch.empty((B, H, N, e), dtype=out_dtype, device=q.device)
    kv_out = torch.empty((B, H, d, e), dtype=torch.float32, device=q.device) if want_state else None
    ws = alloc_workspace(LA_OP_FWD, shape, q.device)
    la_fwd(shape, q, k, v, lam, o, kv_in, kv_out, ws, stream)
    return (o, kv_out) if want_state else o


def bwd(q, k, v, do, lam, *, out_dtype=torch.float32, kv_in=None, grad_kv_out=None,
        want_state_grad=False, seg_len=0, path=LA_PATH_AUTO, precision=LA_PRECISION_DEFAULT, stream=None):
    B, H, N, d = q.shape
    e = v.shape[-1]
    shape = make_shape(B, H, N, d, e, q.dtype, out_dtype, seg_len, path, precision)
    dq = torch.empty((B, H, N, d), dtype=out_dtype, device=q.device)
    dk = torch.empty((B, H, N, d), dtype=out_dtype, device=q.device)
    dv = torch.empty((B, H, N, e), dtype=out_dtype, device=q.device)
    gin = torch.empty((B, H, d, e), dtype=torch.float32, device=q.device) if want_state_grad else None
    ws = alloc_workspace(LA_OP_BWD, shape, q.device)
    la_bwd(shape, q, k, v, do, lam, dq, dk, dv, kv_in, grad_kv_out, gin, ws, stream)
    return (dq, dk, dv, gin) if want_state_grad else (dq, dk, dv)


def decode_step(q, k, v, lam, kv, *, out_dtype=torch.float32, stream=None):
    B, H, d = q.shape
    e = v.shape[-1]
    shape = make_shape(B, H, 1, d, e, q.dtype, out_dtype)
    o = torch.empty((B, H, e), dtype=out_dtype, device=q.device)
    la_decode_step(shape, q, k, v, lam, kv, o, stream)
    return o
