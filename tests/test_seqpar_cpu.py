"""Host logic of the sequence-parallel module with two gloo ranks on the CPU: which contribution goes where in the
gather, which cut each rank chains to, and that the chunks' results put together are the whole sequence's.  The
device calls are replaced by stand-ins built on the CPU oracle (test-only: the module itself has no CPU path), so
what is under test is the choreography, not the kernels."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class OracleDevice:
    """The calls SequenceParallel makes, answered by the fp64 oracle on CPU tensors."""
    LA_OP_FWD, LA_OP_BWD = 0, 1

    def __init__(self):
        from oracle import la_oracle as orc
        from paper_2307_14995_b200 import binding
        self.orc, self.make_shape = orc, binding.make_shape

    def chunk_state_workspace_bytes(self, shape):
        return 0

    def workspace_bytes(self, op, shape):
        return 0

    @staticmethod
    def _lam(lam):
        return np.asarray([float(x) for x in lam], np.float64)

    def la_chunk_state(self, shape, reverse, b, c, lam, out, ws):
        zeros = torch.zeros_like(b)
        if not reverse:
            _, kv = self.orc.fwd_rec(zeros, b, c, self._lam(lam), want_state=True)
            out.copy_(torch.from_numpy(kv))
        else:  # b = q, c = dO; k and v do not enter grad_kv_in
            *_, gin = self.orc.bwd_rec(b, zeros, torch.zeros_like(c), c, self._lam(lam), want_state_grad=True)
            out.copy_(torch.from_numpy(gin))

    def la_chain_states(self, shape, total, chunk_tokens, reverse, states, num, chunk, boundary, lam, out):
        lam = torch.from_numpy(self._lam(lam))[None, :, None, None]
        z = torch.zeros_like(out, dtype=torch.float64) if boundary is None else boundary.double().clone()
        order = range(num - 1, chunk, -1) if reverse else range(0, chunk)
        for j in order:
            n_j = min(total, (j + 1) * chunk_tokens) - j * chunk_tokens
            z = lam ** n_j * z + states[j].double()
        out.copy_(z)

    def la_fwd(self, shape, q, k, v, lam, o, kv_in, kv_out, ws):
        o.copy_(torch.from_numpy(self.orc.fwd_rec(q, k, v, self._lam(lam), kv_in=kv_in.double().numpy())))

    def la_bwd(self, shape, q, k, v, do, lam, dq, dk, dv, kv_in, gko, gin, ws):
        r = self.orc.bwd_rec(q, k, v, do, self._lam(lam), kv_in=kv_in.double().numpy(), grad_kv_out=gko.double().numpy())
        for dst, src in zip((dq, dk, dv), r):
            dst.copy_(torch.from_numpy(src))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


B, H, N, D, CHUNK = 1, 3, 50, 8, 30


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2307_14995_b200 import inputs, seqpar
    q, k, v, do = inputs.make_qkvdo(B, H, N, D, D, dtype=torch.float32, seed=4)
    lam = inputs.decay_rates(H, 0.5)
    kv_in = inputs.make_state(B, H, D, D, seed=5)
    gko = inputs.make_state(B, H, D, D, seed=6)
    sp = seqpar.SequenceParallel(rank, world, N, CHUNK, B, H, D, D, lam, in_dtype=torch.float32, api=OracleDevice())
    lo, hi = rank * CHUNK, min(N, (rank + 1) * CHUNK)
    assert sp.n_local == hi - lo
    ql, kl, vl, dol = (x[:, :, lo:hi].contiguous() for x in (q, k, v, do))
    o = torch.empty((B, H, hi - lo, D), dtype=torch.float64)
    dq, dk, dv = torch.empty_like(o), torch.empty_like(o), torch.empty_like(o)
    kv_out = torch.empty((B, H, D, D), dtype=torch.float32)
    gin = torch.empty_like(kv_out)
    sp.fwd(ql, kl, vl, o, kv_in, kv_out)
    sp.bwd(ql, kl, vl, dol, dq, dk, dv, gko, gin)
    np.savez(os.path.join(out_dir, "r%d.npz" % rank), o=o.numpy(), dq=dq.numpy(), dk=dk.numpy(), dv=dv.numpy(),
             kv_out=kv_out.numpy(), gin=gin.numpy())
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_share_one_sequence(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    from oracle import la_oracle as orc
    from paper_2307_14995_b200 import inputs
    q, k, v, do = inputs.make_qkvdo(B, H, N, D, D, dtype=torch.float32, seed=4)
    lam = inputs.decay_rates(H, 0.5).double().numpy()
    kv_in = inputs.make_state(B, H, D, D, seed=5).double().numpy()
    gko = inputs.make_state(B, H, D, D, seed=6).double().numpy()
    o, kv = orc.fwd_rec(q, k, v, lam, kv_in=kv_in, want_state=True)
    dq, dk, dv, gin = orc.bwd_rec(q, k, v, do, lam, kv_in=kv_in, grad_kv_out=gko, want_state_grad=True)
    parts = [np.load(os.path.join(str(tmp_path), "r%d.npz" % r)) for r in range(world)]
    # states cross the cut as fp32 tensors, so agreement is to fp32 rounding of the states, not bitwise
    tol = dict(rtol=0, atol=2e-5 * max(1.0, float(np.abs(o).max())))
    for name, ref in (("o", o), ("dq", dq), ("dk", dk), ("dv", dv)):
        np.testing.assert_allclose(np.concatenate([p[name] for p in parts], axis=2), ref, err_msg=name, **tol)
    for p in parts:                                   # every rank can compute the whole sequence's end states
        np.testing.assert_allclose(p["kv_out"], kv, **tol)
        np.testing.assert_allclose(p["gin"], gin, **tol)


def test_constructor_rejects_a_cover_that_does_not_match_the_ranks():
    sys.path.insert(0, ROOT)
    import pytest
    from paper_2307_14995_b200 import seqpar
    with pytest.raises(ValueError):
        seqpar.SequenceParallel(0, 2, 100, 30, 1, 1, 8, 8, [1.0], api=OracleDevice())   # 4 chunks for 2 ranks
    with pytest.raises(ValueError):
        seqpar.SequenceParallel(2, 2, 60, 30, 1, 1, 8, 8, [1.0], api=OracleDevice())
