"""Host-side plumbing for running one HiFT context per GPU (one process per GPU).

The step has no exchange inside it on one GPU, so ranks are independent replicas with their own
batches; the only cross-rank operations are a barrier around the timed region and the maximum
over ranks of the measured times.  Works with any torch.distributed backend (nccl on GPUs, gloo
on CPU for the tests)."""
from __future__ import annotations

from typing import List, Sequence


def world() -> tuple:
    """(rank, world_size); (0, 1) when torch.distributed is not initialised."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        return dist.get_rank(), dist.get_world_size()
    return 0, 1


def rank_seed(base: int, rank: int) -> int:
    """Distinct, reproducible data/weight seed per replica."""
    return int(base) + 1000003 * int(rank)


def max_over_ranks(values: Sequence[float], device: str = "cpu") -> List[float]:
    """Element-wise maximum of a few floats over all ranks (identity for a single process)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def aggregate_throughput(units_per_rank: float, seconds_per_rank: float, device: str = "cpu") -> float:
    """Whole-job throughput under weak scaling: every rank processed `units_per_rank`; the job took
    as long as its slowest rank."""
    _, n = world()
    (slowest,) = max_over_ranks([seconds_per_rank], device)
    return units_per_rank * n / slowest


def allreduce_mean_(tensor):
    """In-place mean over ranks of a gradient buffer (sum all-reduce, then 1/world): the one exchange
    of data-parallel HiFT, over the active group's flat gradient only."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(tensor, op=dist.ReduceOp.SUM)
        tensor.mul_(1.0 / dist.get_world_size())
    return tensor


def allreduce_chunks_mean_(tensor, chunks, wait_for_chunk=None, flag=None):
    """Mean over ranks of `tensor`, exchanged chunk by chunk in the given order (each (offset, length, ...)),
    every chunk as its own asynchronous all-reduce so that later chunks can still be produced while earlier
    ones travel.  wait_for_chunk(i) is called before chunk i is handed to the collective (on GPUs: makes
    the communication stream wait for the event that says the chunk is final).  `flag` (one integer
    element, optional) is reduced with MAX after the last chunk: non-zero on any rank means non-zero on
    all.  Returns when every collective has been waited for (on GPUs: enqueued on the current stream)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        if wait_for_chunk is not None:
            for i in range(len(chunks)):
                wait_for_chunk(i)
        return tensor
    n = dist.get_world_size()
    works = []
    for i, ch in enumerate(chunks):
        if wait_for_chunk is not None:
            wait_for_chunk(i)
        works.append(dist.all_reduce(tensor[ch[0]:ch[0] + ch[1]], op=dist.ReduceOp.SUM, async_op=True))
    if flag is not None:
        works.append(dist.all_reduce(flag, op=dist.ReduceOp.MAX, async_op=True))
    for w in works:
        w.wait()
    tensor.mul_(1.0 / n)
    return tensor


def reduce_pieces_mean_(grad, pieces, rank):
    """Sharded optimizer state: piece r of the gradient (pieces[r] = (offset, length)) is summed over the ranks
    onto rank r, which alone will use it; this rank's piece is then scaled to the mean.  The volume of a
    reduce-scatter, with pieces that need not have equal lengths."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return grad
    works = [dist.reduce(grad[lo:lo + n], dst=r, op=dist.ReduceOp.SUM, async_op=True) for r, (lo, n) in enumerate(pieces) if n]
    for w in works:
        w.wait()
    lo, n = pieces[rank]
    grad[lo:lo + n].mul_(1.0 / dist.get_world_size())
    return grad


def broadcast_pieces_(params, pieces):
    """After the sharded update: every rank's piece of the group's parameters goes to all the others
    (an all-gather with pieces of unequal length)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return params
    works = [dist.broadcast(params[lo:lo + n], src=r, async_op=True) for r, (lo, n) in enumerate(pieces) if n]
    for w in works:
        w.wait()
    return params


def data_parallel_step_sharded(h, tokens, labels) -> float:
    """The data-parallel step with the optimizer state split over the ranks (contexts created with
    shard_rank / shard_world): forward + truncated backward, each piece of the group's gradient reduced to the
    rank that holds its master and state, the update of that piece, and the updated pieces of the parameters
    sent to everyone.  State memory and state paging per rank shrink by the number of ranks; the parameters
    every rank ends up with are bit for bit those of the unsharded step, because the update is element-wise."""
    import torch
    import torch.distributed as dist
    rank, world_size = world()
    g = h.active_group()
    pieces = [h.shard_range(g, r) for r in range(world_size)]
    h.step_begin_async(tokens, labels)
    grad, gate = h.grad_view(), h.gate_view()
    for i in range(len(h.grad_chunks())):
        h.grad_chunk_wait(i, torch.cuda.current_stream().cuda_stream)
    reduce_pieces_mean_(grad, pieces, rank)
    if world_size > 1:
        dist.all_reduce(gate, op=dist.ReduceOp.MAX)
    loss = h.step_finish()
    broadcast_pieces_(h.param_view(), pieces)
    return loss


_comm_streams = {}


def data_parallel_step(h, tokens, labels, overlap: bool = True) -> float:
    """One data-parallel step of context `h` on this rank's shard: forward + truncated backward,
    mean of the group's gradient over ranks, update.  Every rank follows the same group schedule,
    so no communication is needed to agree on the group.

    overlap=True: the backward pass is enqueued without waiting, and the gradient is reduced chunk by
    chunk on a communication stream in the order the backward pass completes the chunks (top of the
    group's span first), so that all but the last exchange run under the remaining GEMMs; the ranks
    also share the step's gate word, and all of them skip the update when one of them failed.
    overlap=False: one all-reduce between the two synchronous halves of the step."""
    import torch
    if not overlap:
        loss = h.step_begin(tokens, labels)
        allreduce_mean_(h.grad_view())
        h.step_end()
        return loss
    dev = torch.cuda.current_device()
    comm = _comm_streams.get(dev)
    if comm is None:
        comm = _comm_streams[dev] = torch.cuda.Stream()
    h.step_begin_async(tokens, labels)
    grad, gate = h.grad_view(), h.gate_view()
    chunks = h.grad_chunks()
    with torch.cuda.stream(comm):
        allreduce_chunks_mean_(grad, chunks, wait_for_chunk=lambda i: h.grad_chunk_wait(i, comm.cuda_stream), flag=gate)
    torch.cuda.current_stream().wait_stream(comm)       # hift_step_finish orders itself after the current stream
    return h.step_finish()
