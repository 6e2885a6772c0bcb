"""Multi-GPU plumbing of the benchmark: one process per GPU, every rank runs
its own independent FFN problems (other layers / other batches), so the path
shards with no data-path collective.  The only communication is the timing
reduction: the slowest rank's device time decides, and throughput is the work
of all ranks over that time.

Works on any torch.distributed backend (nccl on GPUs, gloo in the CPU tests).
"""
from __future__ import annotations

import os
from typing import Sequence


def rank_world_local():
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) without a launcher."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of the problems rank `rank` runs: disjoint streams per rank, rank 0 keeps the base seed."""
    return base_seed + rank


def max_over_ranks(values_ms: Sequence[float], device=None):
    """Element-wise maximum over all ranks of a few per-rank times (all-reduce MAX); identity for one process."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values_ms]
    t = torch.tensor(list(values_ms), dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_throughput(units_per_rank_per_step: float, world: int, steps: int, total_ms_max: float) -> float:
    """Units all ranks processed per second: world * units * steps / (slowest rank's total time)."""
    return world * units_per_rank_per_step * steps / (total_ms_max * 1e-3)
