"""Host-side logic of a multi-rank (one process per GPU) run.

The iteration itself runs on one GPU; N ranks are N independent replicas (one problem each, seeded by
rank, no data-path collective).  What the ranks share is the timing protocol: a barrier on both sides
of the timed region and the maximum of the per-rank device times."""
from __future__ import annotations

import dataclasses
import os


def rank_world_local() -> tuple[int, int, int]:
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_spec(spec, rank: int):
    """The rank's own problem: the same recipe with the seed offset by the rank."""
    return dataclasses.replace(spec, seed=spec.seed + rank)


def max_over_ranks(ms: float, device=None) -> float:
    """Largest per-rank time; the identity when no process group is initialised."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def whole_job_rate(world: int, steps: int, iters_per_step: int, ms: float) -> float:
    """Iterations per second over all replicas: every rank did steps x iters_per_step iterations in ms."""
    return world * steps * iters_per_step / (ms * 1e-3)
