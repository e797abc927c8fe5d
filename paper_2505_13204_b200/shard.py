"""Host-side logic of running the path on several GPUs of one node.

Rows, hence sequences, are independent on this path: nothing is exchanged between GPUs while
it runs.  Each rank (one process per GPU) owns a contiguous block of sequences, draws its
inputs from its own seed, and the only cross-rank operation is the reduction of the timing
(max over ranks) that turns per-rank work into a whole-job rate.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def rank_sequences(sequences_per_rank: int, world: int, rank: int) -> range:
    """Global ids of the sequences rank ``rank`` owns (weak scaling: every rank owns
    ``sequences_per_rank`` of them)."""
    if not (0 <= rank < world) or sequences_per_rank < 0:
        raise ValueError("rank %d of %d, %d sequences" % (rank, world, sequences_per_rank))
    return range(rank * sequences_per_rank, (rank + 1) * sequences_per_rank)


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's synthetic inputs: distinct per rank, equal to the base on rank 0."""
    return int(base_seed) + 1000 * int(rank)


def max_over_ranks(value: float, device=None) -> float:
    """Largest ``value`` of any rank (the job is as slow as its slowest rank)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_per_step: float, steps: int, world: int, ms_max: float) -> float:
    """Units per second of all ranks together, given the slowest rank's time for ``steps``."""
    return world * units_per_rank_per_step * steps / (ms_max * 1e-3)
