"""Host-side logic for running the layer on several GPUs.

Tokens are independent (every step of the layer is per token; the histogram, scan and token
lists are per-batch bookkeeping), so the layer shards by tokens with no data-path collective:
every rank holds the whole layer and runs the single-GPU path on its own slice.  The only
cross-rank traffic is the benchmark's barrier and the max-over-ranks reduction of its timing.
"""
from __future__ import annotations


def token_shard(T: int, rank: int, world: int) -> tuple[int, int]:
    """[begin, end) of the tokens rank `rank` of `world` owns: contiguous, sizes differ by at most one."""
    if world <= 0 or not (0 <= rank < world) or T < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(T, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def max_over_ranks(value: float, group=None) -> float:
    """Maximum of a host float over the ranks of a torch.distributed group (identity when not initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    device = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    return float(t.item())


def whole_job_throughput(units_per_rank: int, seconds_local: float, group=None) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    import torch
    import torch.distributed as dist
    slowest = max_over_ranks(seconds_local, group)
    total = units_per_rank
    if dist.is_available() and dist.is_initialized():
        device = "cuda" if dist.get_backend(group) == "nccl" else "cpu"
        t = torch.tensor([float(units_per_rank)], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
        total = float(t.item())
    return total / slowest
