"""Host-side logic of a multi-process run: one process per GPU, each with an independent replica.

The iteration has no cross-GPU exchange, so the only collective work is bookkeeping: a barrier around
the timed region, the maximum over ranks of the measured device time, and the whole-job throughput.
The functions take any initialised ``torch.distributed`` process group (NCCL on GPUs, gloo on CPU).
"""

from __future__ import annotations

import os
from typing import Optional


def env_rank_world():
    """(rank, world size, local rank) from the launcher's environment; a single process is (0, 1, 0)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def device_for(local_rank: int, world: int) -> int:
    """CUDA ordinal a rank runs its replica on: its local rank under a launcher, device 0 alone."""
    return local_rank if world > 1 else 0


def max_over_ranks(value: float, dist=None, device: Optional[str] = None) -> float:
    """Maximum of a per-rank scalar (the slowest rank defines the step time)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_throughput(world: int, steps: int, max_ms: float) -> float:
    """Iterations per second of the whole job: every rank did ``steps`` iterations of its own replica
    within ``max_ms`` (weak scaling: work per GPU is fixed)."""
    return world * steps / (max_ms * 1e-3)
