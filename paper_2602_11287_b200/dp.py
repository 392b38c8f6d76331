"""Host-side helpers for running the HiF4 path on several GPUs of one node.

The path has no exchange step: units, rows and experts are independent, so ranks are data-parallel
replicas over disjoint row ranges (or independent token batches) and the only collectives are the
barrier around the timed region and the maximum of the per-rank times.  Nothing here touches a GPU;
the functions work with any initialised ``torch.distributed`` backend (``nccl`` on GPUs, ``gloo`` in
the CPU tests) and degrade to the single-process answer when no process group exists.
"""
from __future__ import annotations

import os
from typing import Tuple

import torch


def rank_info() -> Tuple[int, int, int]:
    """(rank, local_rank, world_size) as torchrun exports them; (0, 0, 1) outside torchrun."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def shard_rows(total_rows: int, world: int, rank: int) -> Tuple[int, int]:
    """Contiguous, balanced [lo, hi) row range of `rank`; the ranges of all ranks tile [0, total_rows)."""
    if world < 1 or not 0 <= rank < world or total_rows < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(total_rows, world)
    lo = rank * base + min(rank, extra)
    return lo, lo + base + (1 if rank < extra else 0)


def rank_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's private synthetic batch (weak scaling: every rank draws its own tokens)."""
    return int(base_seed) + 7919 * int(rank)


def _dist():
    import torch.distributed as dist
    return dist if dist.is_available() and dist.is_initialized() else None


def barrier() -> None:
    d = _dist()
    if d is not None:
        d.barrier()


def max_over_ranks(value: float, device=None) -> float:
    """Largest `value` over all ranks (the job's time is its slowest rank's)."""
    d = _dist()
    if d is None:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    d.all_reduce(t, op=d.ReduceOp.MAX)
    return float(t.item())


def job_throughput(units_per_rank: float, world: int, max_seconds: float) -> float:
    """Whole-job rate under weak scaling: every rank processed `units_per_rank` in at most `max_seconds`."""
    return world * units_per_rank / max_seconds
