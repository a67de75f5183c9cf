"""Host-side checks of the C ABI that need no GPU: the library loads, exports every
symbol the header declares, validates arguments before touching the device, and
sizes its workspace linearly."""
import ctypes
import os
import re

import pytest
import torch

import __graft_entry__ as entry
from paper_2307_14995_b200 import binding as la

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return la.load()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "la.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(la_[a-z_0-9]+)\s*\(", text)))


def test_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert set(la.EXPORTS) <= set(names)
    for n in ("la_fwd", "la_bwd", "la_decode_step", "la_workspace_bytes"):
        assert n in names
    for n in names:
        assert hasattr(lib, n), n


def test_version_and_status_strings(lib):
    assert la.version() >= 100
    seen = {la.status_string(c) for c in range(8)}
    assert len(seen) == 8 and "ok" in seen and "unknown status" not in seen
    assert "scratch" in la.status_string(7)          # LA_ERR_SCRATCH_LIMIT
    assert la.status_string(8) == "unknown status"


def shape(**kw):
    base = dict(B=1, H=2, N=256, d=64, e=64, in_dtype=torch.float32, out_dtype=torch.float32)
    base.update(kw)
    return la.make_shape(**base)


def test_workspace_is_linear_in_segments_not_quadratic(lib):
    s1 = shape(B=1, H=32, N=65536, d=128, e=128, in_dtype=torch.bfloat16, path=la.LA_PATH_SIMT)
    seg = la.segment_length(s1)
    assert seg % 128 == 0 and seg >= 1024
    nseg = -(-65536 // seg)
    assert la.workspace_bytes(la.LA_OP_FWD, s1) == 2 * 32 * nseg * 128 * 128 * 4
    assert la.workspace_bytes(la.LA_OP_BWD, s1) == 3 * 32 * nseg * 128 * 128 * 4
    assert la.workspace_bytes(la.LA_OP_DECODE, s1) == 0
    s2 = shape(N=100)
    assert la.workspace_bytes(la.LA_OP_FWD, s2) == 0  # one segment: no scratch at all
    s3 = shape(N=1000, seg_len=128)
    assert la.workspace_bytes(la.LA_OP_FWD, s3) == 2 * 2 * 8 * 64 * 64 * 4


@pytest.mark.parametrize("bad", [dict(d=48, e=48), dict(d=64, e=128), dict(H=300),
                                 dict(in_dtype=torch.float32, out_dtype=torch.bfloat16)])
def test_unsupported_shapes(lib, bad):
    s = shape(**bad)
    assert lib.la_workspace_bytes(0, ctypes.byref(s)) == ctypes.c_size_t(-1).value


def call_fwd(lib, s, q=256, k=256, v=256, o=256, lam=(1.0, 0.5), ws=None, ws_bytes=0):
    lam_arr = (ctypes.c_float * len(lam))(*lam) if lam is not None else None
    return lib.la_fwd(ctypes.byref(s), q, k, v, lam_arr, o, None, None, ws, ws_bytes, None)


def test_argument_errors_are_found_before_any_launch(lib):
    INVALID, WORKSPACE = 1, 3
    assert call_fwd(lib, shape(N=0)) == INVALID
    assert call_fwd(lib, shape(seg_len=100)) == INVALID
    assert call_fwd(lib, shape(), q=None) == INVALID
    assert call_fwd(lib, shape(), q=264) == INVALID            # not 16-byte aligned
    assert call_fwd(lib, shape(), lam=None) == INVALID
    assert call_fwd(lib, shape(), lam=(1.0, 0.0)) == INVALID    # lambda must be > 0
    assert call_fwd(lib, shape(), lam=(1.0, 1.5)) == INVALID
    assert call_fwd(lib, shape(), lam=(1.0, float("nan"))) == INVALID
    assert call_fwd(lib, shape(N=1000, seg_len=128)) == WORKSPACE
    assert call_fwd(lib, shape(N=1000, seg_len=128), ws=256, ws_bytes=64) == WORKSPACE
    s = shape()
    lam_arr = (ctypes.c_float * 2)(1.0, 0.5)
    assert lib.la_bwd(ctypes.byref(s), 256, 256, 256, 256, lam_arr, 256, 256, 256, None, None, None,
                      None, 0, None) == WORKSPACE
    assert lib.la_decode_step(ctypes.byref(s), 256, 256, 256, lam_arr, None, 256, None) == INVALID


@pytest.mark.skipif(torch.cuda.is_available(), reason="needs a host without a CUDA device")
def test_no_cpu_fallback_without_a_device(lib):
    # With valid arguments but no usable B200 the call must fail, not compute on the host.
    rc = call_fwd(lib, shape())
    assert rc in (4, 5)
