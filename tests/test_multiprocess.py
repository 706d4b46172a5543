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


def _llama_block_plan(min_elems):
    """Tensors of one LLaMA-shaped block in layout order and the order its backward pass completes them."""
    import synth
    from paper_2401_15207_b200 import binding
    cfg = synth.config_llama_7b()[0].scaled(d_model=256, d_ffn=688, n_heads=2)
    names, sizes = [], []
    for name, shape, _ in synth.unit_tensors(cfg)[1]:
        names.append(name.split(".")[1])
        sizes.append(int(torch.tensor(shape).prod()))
    offsets, o = [], 0
    for n in sizes:
        offsets.append(o)
        o = (o + n + 127) // 128 * 128
    order = [names.index(x) for x in ("w_down", "w_gu", "rms2_g", "w_o", "w_qkv", "rms1_g")]
    return offsets, sizes, o, binding.plan_grad_chunks(offsets, sizes, o, order, min_elems)


def test_chunk_plan_tiles_the_span_in_completion_order():
    offsets, sizes, span, plan = _llama_block_plan(100_000)
    assert sum(n for _, n, _ in plan) == span
    assert plan[0][0] + plan[0][1] == span and plan[-1][0] == 0
    for (o1, n1, a1), (o2, n2, a2) in zip(plan, plan[1:]):
        assert o2 + n2 == o1 and a2 > a1                        # descending, gap-free, released in completion order
    assert all(n >= 100_000 for _, n, _ in plan[:-1])
    # the first chunk is exactly the down projection, released after the first completion
    assert plan[0] == (offsets[-1], span - offsets[-1], 0)
    # a huge minimum gives one chunk, released after the last completion
    _, _, _, one = _llama_block_plan(1 << 40)
    assert one == [(0, span, 5)]
    # an out-of-order completion (a low tensor early) releases nothing by itself
    from paper_2401_15207_b200 import binding
    early = binding.plan_grad_chunks(offsets, sizes, span, [0, 5, 4, 3, 2, 1], 1)
    assert [a for _, _, a in early] == [1, 2, 3, 4, 5] and early[-1][0] == 0


def _chunk_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        offsets, sizes, span, plan = _llama_block_plan(100_000)
        g = torch.Generator().manual_seed(100 + rank)
        grad = torch.randn(span, generator=g)
        whole = grad.clone()
        dist_util.allreduce_mean_(whole)
        waited = []
        flag = torch.tensor([101 if rank == 1 else 0], dtype=torch.int32)
        dist_util.allreduce_chunks_mean_(grad, plan, wait_for_chunk=waited.append, flag=flag)
        assert waited == list(range(len(plan)))                 # every chunk was waited for, in order, before its exchange
        assert torch.equal(grad, whole)                         # chunk by chunk = all at once
        assert int(flag.item()) == 101                          # one rank's failure is every rank's
        dist.barrier()
        if rank == 0:
            torch.save({"ok": True, "chunks": len(plan)}, out)
    finally:
        dist.destroy_process_group()


def test_two_ranks_chunked_exchange_equals_one_all_reduce(tmp_path):
    out = str(tmp_path / "c0.pt")
    mp.spawn(_chunk_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    r = torch.load(out)
    assert r["ok"] and r["chunks"] >= 3


def _pieces_worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        n = 1000
        pieces = [(0, 640), (640, 360)]                          # whole 128-element lines first, the rest last
        g = torch.Generator().manual_seed(7 + rank)
        grad = torch.randn(n, generator=g)
        mean = grad.clone()
        dist_util.allreduce_mean_(mean)
        dist_util.reduce_pieces_mean_(grad, pieces, rank)
        lo, cnt = pieces[rank]
        assert torch.allclose(grad[lo:lo + cnt], mean[lo:lo + cnt], rtol=0, atol=1e-7)   # the owner holds the mean of its piece
        # each rank "updates" its own piece of the parameters, then the pieces travel
        params = torch.zeros(n)
        params[lo:lo + cnt] = float(rank + 1)
        dist_util.broadcast_pieces_(params, pieces)
        assert torch.equal(params[:640], torch.full((640,), 1.0)) and torch.equal(params[640:], torch.full((360,), 2.0))
        dist.barrier()
        if rank == 0:
            torch.save({"ok": True}, out)
    finally:
        dist.destroy_process_group()


def test_two_ranks_piecewise_reduce_and_broadcast(tmp_path):
    out = str(tmp_path / "p0.pt")
    mp.spawn(_pieces_worker, args=(2, _free_port(), out), nprocs=2, join=True)
    assert torch.load(out)["ok"]
