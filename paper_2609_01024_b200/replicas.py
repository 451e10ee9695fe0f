"""Token data parallelism over replicas: the only multi-GPU form the layer needs.

Tokens are independent units of the layer, so N ranks hold the same weights and each processes its own
batch of T tokens; there is no exchange step on the data path.  The helpers here give every rank its own
seeded batch, and reduce the timing the way the benchmark reports it (max over ranks).
"""
from __future__ import annotations

import numpy as np

from . import workloads as wl


def rank_token_config(cfg: wl.LayerConfig, rank: int) -> wl.LayerConfig:
    """Config whose token tensors (hidden states, logits) are rank `rank`'s batch.  Rank 0 uses the layer's own
    seed; mask, bias and weights are always drawn with the layer's seed, whatever the rank."""
    return cfg if rank == 0 else cfg.scaled(seed=cfg.seed + 100 * rank)


def rank_inputs(cfg: wl.LayerConfig, rank: int):
    """(hidden states, logits) of one rank."""
    c = rank_token_config(cfg, rank)
    h = wl.make_hidden(c)
    logits = wl.make_logits(c, wl.hidden_as_f32(c, h) if cfg.logits == "router" else None)
    return h, logits


def max_over_ranks(value: float, device="cpu") -> float:
    """Max of a scalar over the ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(tokens_per_rank: int, world: int, ms_per_step: float) -> float:
    return world * tokens_per_rank / (ms_per_step * 1e-3)
