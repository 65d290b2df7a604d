"""Work assignment and timing reduction for runs with one process per GPU.

The path shards only along the inputs (they are independent of one another): every rank holds a full
replica of the net and works on its own inputs; nothing is exchanged on the data path.  The only
collective is the reduction of the measured time (max over ranks) that turns per-rank work into a
whole-job throughput.  These helpers hold no arithmetic of the method and run on CPU process groups
(gloo) as well as on NCCL.
"""
from __future__ import annotations


def rank_inputs(rank: int, world: int, per_rank: int) -> tuple[int, int]:
    """Weak scaling: rank r works on inputs [r * per_rank, (r + 1) * per_rank) of the job's input stream."""
    if not (0 <= rank < world) or per_rank < 0:
        raise ValueError("need 0 <= rank < world and per_rank >= 0")
    return rank * per_rank, per_rank


def split_inputs(n_inputs: int, rank: int, world: int) -> tuple[int, int]:
    """Strong scaling: a fixed batch of n_inputs cut into `world` contiguous, balanced ranges (sizes differ by
    at most one, earlier ranks get the larger ones).  Returns (start, count) of this rank's range."""
    if not (0 <= rank < world) or n_inputs < 0:
        raise ValueError("need 0 <= rank < world and n_inputs >= 0")
    base, extra = divmod(n_inputs, world)
    start = rank * base + min(rank, extra)
    return start, base + (1 if rank < extra else 0)


def max_over_ranks(value: float, device=None) -> float:
    """Max of `value` over all ranks of the default process group (the value itself without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, local_ms: float, world: int, device=None) -> tuple[float, float]:
    """(whole-job units per second, ms per step) for `world` ranks that each processed `units_per_rank` units
    in `local_ms` milliseconds: total units divided by the slowest rank's time."""
    ms = max_over_ranks(local_ms, device)
    return world * units_per_rank / (ms * 1e-3), ms
