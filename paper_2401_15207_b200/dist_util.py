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


def data_parallel_step(h, tokens, labels) -> float:
    """One data-parallel step of context `h` on this rank's shard: forward + truncated backward,
    mean of the group's gradient over ranks, update.  Every rank follows the same group schedule,
    so no communication is needed to agree on the group."""
    loss = h.step_begin(tokens, labels)
    allreduce_mean_(h.grad_view())
    h.step_end()
    return loss
