"""la_fwd_noalloc: the forward pass for callers that cannot allocate device memory at call time
(all memory already given to their own pool, no allocator at hand, or no tolerance for the
device-wide synchronisation an allocation brings).  Its scratch is a fixed array inside the
library, so this file checks, through the C ABI, that it gives what la_fwd gives with a
caller-allocated workspace -- and what the CPU oracle's token recurrence gives -- twice in a row,
because the second call finds the first call's leftovers in the shared scratch.  Collected last on purpose (file name), and self-contained so
that it passes alone in a fresh process as well as after the rest of the suite."""
import ctypes

import pytest
import torch

from la_check import TOL_BF16, assert_close
from oracle import la_oracle as orc
from paper_2307_14995_b200 import binding as la, inputs


def test_noalloc_rejects_shapes_beyond_the_static_scratch():
    # 64 heads x 4 segments x 2 sets x 64 KB = 32 MiB fits exactly; one more segment does not.
    la.load()
    fits = la.make_shape(1, 64, 4 * 128, 128, 128, torch.bfloat16, torch.float32, seg_len=128, path=la.LA_PATH_SIMT)
    too_big = la.make_shape(1, 64, 5 * 128, 128, 128, torch.bfloat16, torch.float32, seg_len=128, path=la.LA_PATH_SIMT)
    assert la.workspace_bytes(la.LA_OP_FWD, fits) == la.LA_NOALLOC_SCRATCH_BYTES
    assert la.workspace_bytes(la.LA_OP_FWD, too_big) > la.LA_NOALLOC_SCRATCH_BYTES
    lam = (ctypes.c_float * 64)(*([0.5] * 64))
    rc = la.load().la_fwd_noalloc(ctypes.byref(too_big), 256, 256, 256, lam, 256, None, None, None)
    assert rc == 7 and "scratch" in la.status_string(rc)


@pytest.mark.gpu
@pytest.mark.parametrize("d,path", [(128, la.LA_PATH_AUTO), (64, la.LA_PATH_SIMT)])
def test_noalloc_matches_la_fwd_twice_in_a_row(d, path):
    dev = "cuda:0"
    B, H, N, seg_len = 2, 3, 1000, 256            # four segments per head -> the scratch is really used
    q, k, v, _ = inputs.make_qkvdo(B, H, N, d, d, seed=21)
    lam = torch.tensor([1.0, 0.97, 0.4])
    kv_in = inputs.make_state(B, H, d, d, seed=22).to(dev)
    qg, kg, vg = (x.to(dev) for x in (q, k, v))
    shape = la.make_shape(B, H, N, d, d, torch.bfloat16, torch.float32, seg_len=seg_len, path=path)
    assert 0 < la.workspace_bytes(la.LA_OP_FWD, shape) <= la.LA_NOALLOC_SCRATCH_BYTES

    # existing entry point, caller-allocated workspace
    o_ref = torch.empty((B, H, N, d), dtype=torch.float32, device=dev)
    kv_ref = torch.empty((B, H, d, d), dtype=torch.float32, device=dev)
    la.la_fwd(shape, qg, kg, vg, lam, o_ref, kv_in, kv_ref, la.alloc_workspace(la.LA_OP_FWD, shape, dev))
    torch.cuda.synchronize()
    o_orc, kv_orc = orc.fwd_rec(q, k, v, lam.double().numpy(), kv_in=kv_in.double().cpu().numpy(), want_state=True)
    tol = TOL_BF16 if path != la.LA_PATH_SIMT else 1e-4

    for attempt in range(2):
        o = torch.full((B, H, N, d), float("nan"), dtype=torch.float32, device=dev)
        kv = torch.full((B, H, d, d), float("nan"), dtype=torch.float32, device=dev)
        if attempt == 1:
            # a different problem in between leaves other contents in the shared scratch
            other = la.make_shape(1, 2, 700, d, d, torch.bfloat16, torch.float32, seg_len=128, path=path)
            junk_o = torch.empty((1, 2, 700, d), dtype=torch.float32, device=dev)
            la.la_fwd_noalloc(other, kg[:1, :2, :700].contiguous(), qg[:1, :2, :700].contiguous(),
                              vg[:1, :2, :700].contiguous(), lam[:2], junk_o)
        la.la_fwd_noalloc(shape, qg, kg, vg, lam, o, kv_in, kv)
        torch.cuda.synchronize()
        la.device_status()
        assert_close(o, o_ref.double().cpu().numpy(), TOL_BF16, "o, call %d" % attempt)
        assert_close(kv, kv_ref.double().cpu().numpy(), TOL_BF16, "kv_out, call %d" % attempt)
        assert torch.equal(o, o_ref) and torch.equal(kv, kv_ref)  # same kernels, same order: bitwise equal
        assert_close(o, o_orc, tol, "o vs oracle, call %d" % attempt)
        assert_close(kv, kv_orc, tol, "kv_out vs oracle, call %d" % attempt)
