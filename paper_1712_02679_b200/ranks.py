"""Host-side rank logic of the multi-GPU runs: one process per GPU, no data-path collective.

Learners are independent (in the paper a learner is one GPU and only exchange() couples
them), so N GPUs run N copies of the per-GPU workload on their own seeded learners (weak
scaling) or split a fixed list of units (learners, tensors) between them.  The only
collectives are a barrier and a max-reduction of the device-measured times; both work on
the gloo backend with CPU tensors, which is how this module is tested without GPUs.
"""
from __future__ import annotations

import os
from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def rank_env() -> Tuple[int, int, int]:
    """(rank, world_size, local_rank) from the torchrun environment; (0, 1, 0) outside it."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def learner_seed(rank: int, learner: int, step: int) -> int:
    """Seed of one learner's gradient at one step; distinct for every (rank, learner, step)
    with learner < 1000 and step < 1009, so no two GPUs ever compress the same gradient."""
    return 171202679 + 1000003 * rank + 1009 * learner + step


def shard_units(n_units: int, world: int, rank: int) -> range:
    """Contiguous, balanced split of units 0..n_units-1; the first n_units % world ranks take one more."""
    base, extra = divmod(n_units, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def max_over_ranks(values: Sequence[float], device=None) -> List[float]:
    """Element-wise maximum of `values` over all ranks (identity when not distributed)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_throughput(bytes_per_rank: float, world: int, ms_max: float) -> float:
    """GB/s over all ranks: every rank moved bytes_per_rank, the job took the slowest rank's time."""
    return bytes_per_rank * world / (ms_max * 1e-3) / 1e9
