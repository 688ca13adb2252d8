"""Host-side bookkeeping for running independent replicas of the scoring step, one per rank.

SAPO nodes never synchronise weights or gradients (each node owns its policy), so ranks only
agree on timing: the slowest rank's device time and the total number of tokens scored.
"""
from __future__ import annotations

from typing import Tuple

import torch
import torch.distributed as dist


def rank_seed(workload: int, rank: int) -> int:
    """Every rank draws its own batch of the same workload."""
    return 1000 * workload + rank


def aggregate(ms_local: float, tokens_local: float, device="cpu") -> Tuple[float, float]:
    """(max over ranks of the elapsed milliseconds, sum over ranks of the tokens)."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms_local), float(tokens_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    n = torch.tensor([tokens_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), float(n.item())


def throughput(ms_max: float, tokens_total: float, steps: int) -> float:
    """Whole-job tokens per second."""
    return tokens_total * steps / (ms_max / 1e3)
