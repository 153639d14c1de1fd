"""Host-side plumbing of the multi-GPU run: prompts are independent units (Eq. 4 of the paper), so every
rank decodes its own shard with no collective on the data path; only the timing scalars are reduced."""
from __future__ import annotations

from typing import Sequence, Tuple

import torch
import torch.distributed as dist


def reduce_timing(times_ms: Sequence[float], units: float, device="cpu") -> Tuple[list, float]:
    """MAX over ranks of each time, SUM over ranks of the processed units (no-op without a process group)."""
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    u = torch.tensor([float(units)], dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return [float(x) for x in t.tolist()], float(u.item())


def aggregate_throughput(times_ms: Sequence[float], units: float, steps: int, device="cpu") -> Tuple[float, list, float]:
    """Whole-job units per second: all ranks' units over the slowest rank's time (first entry of times_ms)."""
    tmax, total = reduce_timing(times_ms, units, device)
    return total * steps / (tmax[0] * 1e-3), tmax, total
