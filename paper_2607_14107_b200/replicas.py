"""Multi-GPU = independent replicas.

The decoding path has no exchange step (sequences are independent; the paper is single-GPU,
batch 1), so N GPUs run N replicas of the decoder, each on its own prompts, with no data-path
collective.  The only communication is bookkeeping for the benchmark: a barrier, the maximum over
ranks of the device-measured times and the sum over ranks of the token counts.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def replica_prompt_seed(base_seed: int, rank: int) -> int:
    """Every replica decodes a different batch of synthetic prompts."""
    return base_seed + rank


def aggregate(times_ms: Sequence[float], counts: Sequence[float], device="cpu") -> Tuple[List[float], List[float]]:
    """(max over ranks of each time, sum over ranks of each count).  Identity when not distributed."""
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    c = torch.tensor(list(counts), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(c, op=dist.ReduceOp.SUM)
    return t.tolist(), c.tolist()


def whole_job_rate(total_units: float, max_time_ms: float) -> float:
    """Units all ranks processed divided by the slowest rank's time."""
    return total_units / (max_time_ms / 1e3)
