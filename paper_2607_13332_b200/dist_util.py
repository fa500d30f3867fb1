"""The little multi-process plumbing the benchmark needs: ranks never exchange codec data (every
step is independent per token), they only meet at a barrier and agree on the slowest rank's time."""

from __future__ import annotations

import os
from typing import Tuple

import torch
import torch.distributed as dist


def rank_world() -> Tuple[int, int, int]:
    """(rank, world size, local rank) from the launcher's environment; (0, 1, 0) when alone."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def barrier() -> None:
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def max_over_ranks(value: float, device: str = "cpu") -> float:
    """The largest `value` any rank holds (device-timed durations are reported this way)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())
