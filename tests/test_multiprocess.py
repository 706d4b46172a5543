"""World-size-2 checks of the multi-process plumbing, on CPU with the gloo backend."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2401_15207_b200 import dist_util


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert dist_util.world() == (rank, world)
        # rank r "measures" r+1 seconds and 10*(r+1) ms: the job is as slow as its slowest rank
        mx = dist_util.max_over_ranks([float(rank + 1), 10.0 * (rank + 1)])
        thr = dist_util.aggregate_throughput(2048.0, float(rank + 1))
        gbuf = torch.full((5,), float(rank + 1))          # rank r holds gradient r+1 everywhere
        dist_util.allreduce_mean_(gbuf)
        assert torch.equal(gbuf, torch.full((5,), 1.5))   # mean of 1 and 2 on both ranks
        seeds = [None] * world
        dist.all_gather_object(seeds, dist_util.rank_seed(77, rank))
        dist.barrier()
        if rank == 0:
            torch.save({"max": mx, "thr": thr, "seeds": seeds}, out)
    finally:
        dist.destroy_process_group()


def test_two_ranks_max_time_and_weak_scaling_throughput(tmp_path):
    out = str(tmp_path / "r0.pt")
    mp.spawn(_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = torch.load(out)
    assert r["max"] == [2.0, 20.0]
    assert r["thr"] == 2048.0 * 2 / 2.0
    assert len(set(r["seeds"])) == 2 and r["seeds"][0] == 77


def test_single_process_is_identity():
    assert dist_util.world() == (0, 1)
    assert dist_util.max_over_ranks([3.5, 1.0]) == [3.5, 1.0]
    assert dist_util.aggregate_throughput(100.0, 4.0) == 25.0
