"""Multi-GPU layout of the reduction pass: independent prompts, one per rank, no data-path exchange.

The units of the pass (layer, sequence, KV head, K or V) never interact, so more GPUs means more
prompts.  The only communication is bookkeeping for the benchmark: a sum of token counts and a
maximum of step times.  Works with any ``torch.distributed`` backend (NCCL on GPUs, gloo in tests).
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch


def rank_workload(wl, rank: int):
    """The prompt rank ``rank`` compresses: same shape, its own seed."""
    return wl.replace(seed=wl.seed + rank)


def aggregate(tokens_local: int, ms_local: float, dist=None, device: Optional[torch.device] = None) -> Tuple[int, float]:
    """Whole-job token count (sum over ranks) and step time (max over ranks)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return int(tokens_local), float(ms_local)
    dev = device if device is not None else torch.device("cpu")
    tok = torch.tensor([float(tokens_local)], dtype=torch.float64, device=dev)
    ms = torch.tensor([float(ms_local)], dtype=torch.float64, device=dev)
    dist.all_reduce(tok, op=dist.ReduceOp.SUM)
    dist.all_reduce(ms, op=dist.ReduceOp.MAX)
    return int(round(tok.item())), float(ms.item())


def throughput(tokens_total: int, steps: int, ms_total: float) -> float:
    """Tokens per second of the whole job."""
    return tokens_total * steps / (ms_total * 1e-3)
