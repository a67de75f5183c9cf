"""Sequence parallelism (one sequence cut into chunks, one per rank): the chunk-state and chain entry points and
the module that sequences them, against the oracle run on the whole sequence.  One GPU: the ranks are emulated one
after the other in this process (phase by phase; no kernel waits for another rank), with the gather replaced by a
stack of the ranks' contributions; a single-rank NCCL group checks the torch.distributed route."""
import socket

import numpy as np
import pytest
import torch

from la_check import TOL_BF16, assert_close
from oracle import la_oracle as orc
from paper_2307_14995_b200 import binding as la, inputs, seqpar

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_chunk_state_is_the_state_handed_over_by_a_chunk():
    B, H, N, d = 2, 3, 700, 128
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, seed=31)
    lam = torch.tensor([1.0, 0.99, 0.7])
    lam64 = lam.double().numpy()
    for seg_len in (0, 256):
        shape = la.make_shape(B, H, N, d, d, torch.bfloat16, torch.float32, seg_len)
        ws = torch.empty(max(la.chunk_state_workspace_bytes(shape), 256), dtype=torch.uint8, device=DEV)
        s_f = torch.empty((B, H, d, d), dtype=torch.float32, device=DEV)
        s_r = torch.empty_like(s_f)
        la.la_chunk_state(shape, 0, k.to(DEV), v.to(DEV), lam, s_f, ws)
        la.la_chunk_state(shape, 1, q.to(DEV), do.to(DEV), lam, s_r, ws)
        torch.cuda.synchronize()
        la.device_status()
        _, kv = orc.fwd_rec(q, k, v, lam64, want_state=True)
        *_, gin = orc.bwd_rec(q, k, v, do, lam64, want_state_grad=True)
        assert_close(s_f, kv, TOL_BF16, "chunk state, forward")
        assert_close(s_r, gin, TOL_BF16, "chunk state, reverse")


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("world,chunk", [(3, 300), (2, 512), (4, 129)])
def test_emulated_ranks_reproduce_the_whole_sequence(d, world, chunk):
    B, H = 1, 3
    N = (world - 1) * chunk + max(1, chunk // 3)        # the last chunk is shorter
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, seed=32)
    lam = torch.tensor([1.0, 0.98, 0.6])
    lam64 = lam.double().numpy()
    kv_in = inputs.make_state(B, H, d, d, seed=33)
    gko = inputs.make_state(B, H, d, d, seed=34)
    ranks = []

    def stack_gather(dst, src):      # stands in for the all-gather: every emulated rank's contribution, rank-major
        torch.stack([r.local for r in ranks], out=dst)

    ranks.extend(seqpar.SequenceParallel(r, world, N, chunk, B, H, d, d, lam, device=DEV, gather=stack_gather)
                 for r in range(world))
    cut = lambda x, r: x[:, :, r * chunk:min(N, (r + 1) * chunk)].contiguous().to(DEV)
    qs, ks, vs, dos = ([cut(x, r) for r in range(world)] for x in (q, k, v, do))
    new = lambda r: torch.full(qs[r].shape, float("nan"), dtype=torch.float32, device=DEV)
    o, dq, dk, dv = ([new(r) for r in range(world)] for _ in range(4))
    kv_out = torch.empty((B, H, d, d), dtype=torch.float32, device=DEV)
    gin = torch.empty_like(kv_out)
    # forward, phase by phase over the emulated ranks
    for r, sp in enumerate(ranks):
        sp.fwd_local(ks[r], vs[r])
    for sp in ranks:
        sp.fwd_exchange()
    for r, sp in enumerate(ranks):
        sp.fwd_finish(qs[r], ks[r], vs[r], o[r], kv_in.to(DEV), kv_out if r == world - 1 else None)
    # backward
    for r, sp in enumerate(ranks):
        sp.bwd_local(qs[r], dos[r])
    for sp in ranks:
        sp.bwd_exchange()
    for r, sp in enumerate(ranks):
        sp.bwd_finish(qs[r], ks[r], vs[r], dos[r], dq[r], dk[r], dv[r], gko.to(DEV), gin if r == 0 else None)
    torch.cuda.synchronize()
    la.device_status()
    ref_o, ref_kv = orc.fwd_rec(q, k, v, lam64, kv_in=kv_in.double().numpy(), want_state=True)
    rq, rk, rv, rgin = orc.bwd_rec(q, k, v, do, lam64, kv_in=kv_in.double().numpy(),
                                   grad_kv_out=gko.double().numpy(), want_state_grad=True)
    assert_close(torch.cat(o, 2), ref_o, TOL_BF16, "o")
    assert_close(kv_out, ref_kv, TOL_BF16, "kv_out")
    assert_close(torch.cat(dq, 2), rq, TOL_BF16, "dq")
    assert_close(torch.cat(dk, 2), rk, TOL_BF16, "dk")
    assert_close(torch.cat(dv, 2), rv, TOL_BF16, "dv")
    assert_close(gin, rgin, TOL_BF16, "grad_kv_in")
    # the state entering the last chunk is the recurrence's state after the tokens before it
    t_cut = (world - 1) * chunk
    _, kv_cut = orc.fwd_rec(q[:, :, :t_cut], k[:, :, :t_cut], v[:, :, :t_cut], lam64, kv_in=kv_in.double().numpy(),
                            want_state=True)
    assert_close(ranks[-1].kv_in, kv_cut, TOL_BF16, "state at the last cut")


def test_chain_rejects_bad_descriptions():
    shape = la.make_shape(1, 2, 1, 64, 64, torch.bfloat16, torch.float32)
    st = torch.zeros((3, 1, 2, 64, 64), device=DEV)
    out = torch.zeros((1, 2, 64, 64), device=DEV)
    lam = torch.tensor([1.0, 0.5])
    with pytest.raises(la.LaError):
        la.la_chain_states(shape, 1000, 300, 0, st, 3, 0, None, lam, out)     # 1000 tokens in chunks of 300 are 4 chunks
    with pytest.raises(la.LaError):
        la.la_chain_states(shape, 900, 300, 0, st, 3, 4, None, lam, out)      # no such cut
    with pytest.raises(la.LaError):
        la.la_chain_states(shape, 900, 300, 1, st, 3, 3, None, lam, out)


def test_single_rank_nccl_group_equals_the_plain_calls():
    import torch.distributed as dist
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1)
    try:
        B, H, N, d = 1, 2, 600, 128
        q, k, v, do = (x.to(DEV) for x in inputs.make_qkvdo(B, H, N, d, d, seed=35))
        lam = torch.tensor([0.999, 0.8])
        sp = seqpar.SequenceParallel(0, 1, N, N, B, H, d, d, lam, device=DEV)
        o = torch.empty((B, H, N, d), dtype=torch.float32, device=DEV)
        dq, dk, dv = torch.empty_like(o), torch.empty_like(o), torch.empty_like(o)
        sp.fwd(q, k, v, o)
        sp.bwd(q, k, v, do, dq, dk, dv)
        torch.cuda.synchronize()
        assert torch.equal(o, la.fwd(q, k, v, lam))
        for a, b in zip((dq, dk, dv), la.bwd(q, k, v, do, lam)):
            assert torch.equal(a, b)
    finally:
        dist.destroy_process_group()


def test_chunk_state_token_major_layout():
    """la_chunk_state on [B,N,H,d] tensors gives the same states as on [B,H,N,d] ones, bit for bit."""
    B, H, N, d = 2, 3, 600, 128
    q, k, v, do = inputs.make_qkvdo(B, H, N, d, d, seed=36)
    lam = torch.tensor([1.0, 0.95, 0.6])
    out = {}
    for name, layout in (("bhnd", la.LA_LAYOUT_BHND), ("bnhd", la.LA_LAYOUT_BNHD)):
        tm = (lambda x: x.permute(0, 2, 1, 3).contiguous()) if layout == la.LA_LAYOUT_BNHD else (lambda x: x)
        shape = la.make_shape(B, H, N, d, d, torch.bfloat16, torch.float32, 256, layout=layout)
        ws = torch.empty(max(la.chunk_state_workspace_bytes(shape), 256), dtype=torch.uint8, device=DEV)
        s_f = torch.empty((B, H, d, d), dtype=torch.float32, device=DEV)
        s_r = torch.empty_like(s_f)
        la.la_chunk_state(shape, 0, tm(k).to(DEV), tm(v).to(DEV), lam, s_f, ws)
        la.la_chunk_state(shape, 1, tm(q).to(DEV), tm(do).to(DEV), lam, s_r, ws)
        torch.cuda.synchronize()
        out[name] = (s_f.clone(), s_r.clone())
    la.device_status()
    assert torch.equal(out["bhnd"][0], out["bnhd"][0]) and torch.equal(out["bhnd"][1], out["bnhd"][1])
    _, kv = orc.fwd_rec(q, k, v, lam.double().numpy(), want_state=True)
    assert_close(out["bnhd"][0], kv, TOL_BF16, "chunk state, token-major")
