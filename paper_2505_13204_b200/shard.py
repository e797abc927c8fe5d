"""Host-side logic of running the path on several GPUs of one node.

Rows, hence sequences, are independent on this path: nothing is exchanged between GPUs while
it runs.  Each rank (one process per GPU) owns a contiguous block of sequences, draws its
inputs from its own seed, and the only cross-rank operation is the reduction of the timing
(max over ranks) that turns per-rank work into a whole-job rate.
"""
from __future__ import annotations

import os
import socket
import subprocess
import sys

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


def launch_plan(gpus: int, env=None) -> str:
    """What a program asked to use ``gpus`` GPUs has to do, given its environment:
    "run" (it is the only rank, or one rank of a launcher's group of that size), or "spawn"
    (it was started plainly and has to start the ranks itself).  A launcher's group of
    another size than asked for is an error: the two would silently disagree."""
    env = os.environ if env is None else env
    if gpus < 1:
        raise ValueError("--gpus must be at least 1")
    world = env.get("WORLD_SIZE")
    if world is None:
        return "run" if gpus == 1 else "spawn"
    if int(world) != gpus:
        raise ValueError("--gpus %d but the launcher started %s ranks" % (gpus, world))
    return "run"


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(script: str, argv, gpus: int, port: int | None = None, extra_env=None) -> int:
    """Starts ``gpus`` ranks of ``script argv`` on this node, one process per GPU, through
    torch's launcher (rendezvous on 127.0.0.1) and returns its exit code.  The ranks find
    RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* in their environment; their output goes to
    this process's stdout and stderr (NCCL's communicator lines with NCCL_DEBUG=INFO too)."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(int(gpus)),
           "--master-addr", "127.0.0.1", "--master-port", str(port or free_port()), script] + list(argv)
    env = dict(os.environ)
    env.update(extra_env or {})
    return subprocess.call(cmd, env=env)
