"""Multi-GPU plumbing: the path shards by sequence with no data-path collective.

Every rank owns its own sequences (its own cache, its own seeded inputs) and runs
the same per-GPU workload; the only communication is the timing contract of the
benchmark: a barrier around the timed region and the maximum of the ranks' device
times.  The functions work on any torch.distributed backend (nccl on GPUs, gloo
in the CPU tests).
"""
from __future__ import annotations


def rank_workload(w: dict, rank: int) -> dict:
    """The workload of one rank: same shapes, a seed of its own, so that the
    ranks hold different sequences (weak scaling)."""
    out = dict(w)
    out["seed"] = w["seed"] + 101 * rank
    return out


def max_over_ranks(ms: float, device="cpu") -> float:
    """Maximum over all ranks of a local time (the local value if no process
    group is initialised)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_rate(units_per_rank: float, ms_max: float, world: int) -> float:
    """Whole-job rate: every rank processed `units_per_rank` in at most ms_max."""
    return world * units_per_rank / (ms_max * 1e-3)
