"""Host-side plumbing for running one process per GPU.

The path shards by independent problems: every rank convolves its own signals (or its own batch
of images) with no exchange on the data path, so the only collective is the reduction of the timing
(maximum over ranks) after the timed region.  Nothing here touches the arithmetic; it works with
the ``nccl`` backend on GPUs and with ``gloo`` on CPU, which is how it is tested.
"""
from __future__ import annotations

import os
from typing import Optional, Tuple

RANK_SEED_STRIDE = 100000      # added to a case's seed per rank, so that ranks hold different data


def rank_info() -> Tuple[int, int, int]:
    """(world size, rank, local rank) from the launcher's environment; (1, 0, 0) when run alone."""
    return (int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")),
            int(os.environ.get("LOCAL_RANK", "0")))


def rank_seed(seed: int, rank: int) -> int:
    return seed + RANK_SEED_STRIDE * rank


def init(backend: str, device=None) -> bool:
    """Joins the process group when the launcher started more than one rank.  Returns True if it did."""
    world, _, _ = rank_info()
    if world <= 1:
        return False
    import torch.distributed as dist
    if backend == "nccl":
        dist.init_process_group("nccl", device_id=device)
    else:
        dist.init_process_group(backend)
    return True


def barrier() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(value: float, device=None) -> float:
    """The slowest rank's time: what a job that waits for all ranks observes."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank_step: float, steps: int, total_ms: float, world: Optional[int] = None) -> float:
    """Units per second over all ranks: every rank processed `units_per_rank_step` per step (weak scaling)
    and the job took `total_ms` (already the maximum over ranks) for `steps` steps."""
    if world is None:
        world = rank_info()[0]
    return world * units_per_rank_step * steps / (total_ms * 1e-3)


def shutdown() -> None:
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
