"""The multi-process bookkeeping of bench.py on CPU: world size 2, gloo backend."""
import os
import socket

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp  # noqa: E402

from paper_2609_05709_b200.replicas import job_throughput, max_over_ranks, split_centers  # noqa: E402


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    import torch.distributed as dist
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = [10.0 + rank, 5.0 - rank]               # rank 1 is slower on the first, faster on the second
        dist.barrier()
        out[rank] = max_over_ranks(mine)
    finally:
        dist.destroy_process_group()


def test_max_over_ranks_and_throughput_world2():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        assert out[0] == out[1] == [11.0, 5.0]
        # 3000 centres per replica, slowest rank 11 ms -> whole job
        assert job_throughput(3000, world, out[0][0]) == pytest.approx(2 * 3000 / 11e-3)


def test_single_process_identity_and_split():
    assert max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    ranges = [split_centers(10, 4, r) for r in range(4)]
    assert ranges == [(0, 3), (3, 6), (6, 8), (8, 10)]
    assert split_centers(3, 8, 7) == (3, 3)
