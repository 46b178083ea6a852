"""Host logic of the multi-GPU run: lanes are independent, so N GPUs are N replicas that each decode their own
batch.  No data-path collective exists; ranks only agree on the slowest device time."""
from __future__ import annotations

import torch


def rank_seed(base_seed: int, rank: int) -> int:
    """Every rank draws its own stream so the replicas do not decode identical batches."""
    return int(base_seed) + 3 + 1000 * int(rank)


def max_over_ranks(value: float, dist=None, device="cpu") -> float:
    """Maximum of a per-rank scalar (device-measured milliseconds) over all ranks; identity without a process group."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_steps_per_s(world: int, steps: int, elapsed_ms: float) -> float:
    """Whole-job rate: every rank completed `steps` decode steps of its own batch within the slowest rank's time."""
    return world * steps / (elapsed_ms * 1e-3)
