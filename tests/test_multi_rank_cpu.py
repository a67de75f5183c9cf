"""The multi-GPU path is "one process per GPU, (batch, head) slices, no data-path collective".
Its host logic is exercised here with two gloo ranks on the CPU: the head partition is exact,
each rank's slice (computed by the CPU oracle standing in for the device) reproduces the
corresponding part of the full result without any exchange, and the timing reduction is a MAX."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import la_oracle as orc
    from paper_2307_14995_b200 import dist_utils, inputs
    B, H, N, d = 1, 5, 40, 8
    q, k, v, _ = inputs.make_qkvdo(B, H, N, d, d, seed=3)
    lam = inputs.decay_rates(H, 0.5)
    lo, hi = dist_utils.head_range(rank, world, B * H)
    # this rank's heads only; nothing is exchanged to compute them
    o = orc.fwd_rec(q[:, lo:hi], k[:, lo:hi], v[:, lo:hi], lam[lo:hi].double().numpy())
    np.save(os.path.join(out_dir, "o_%d.npy" % rank), o)
    dist_utils.barrier()
    slowest = dist_utils.max_over_ranks(10.0 + rank)
    assert slowest == 10.0 + world - 1
    dist.destroy_process_group()


def test_head_range_partitions_exactly():
    sys.path.insert(0, ROOT)
    from paper_2307_14995_b200.dist_utils import head_range
    for n in (0, 1, 5, 32, 2048):
        for world in (1, 2, 3, 8):
            spans = [head_range(r, world, n) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        head_range(2, 2, 4)


def test_two_gloo_ranks_cover_the_problem_without_exchange(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    sys.path.insert(0, ROOT)
    from oracle import la_oracle as orc
    from paper_2307_14995_b200 import inputs
    q, k, v, _ = inputs.make_qkvdo(1, 5, 40, 8, 8, seed=3)
    lam = inputs.decay_rates(5, 0.5)
    full = orc.fwd_rec(q, k, v, lam.double().numpy())
    parts = [np.load(os.path.join(str(tmp_path), "o_%d.npy" % r)) for r in range(world)]
    assert np.array_equal(np.concatenate(parts, axis=1), full)
