"""One decision shared by several ranks: each draws a contiguous range of the Monte-Carlo samples.

The decision shards over samples (rows are independent until the mean): rank r draws the samples
[r*S, (r+1)*S) of a decision with world*S samples -- the noise is addressed by the global sample
index, so the union is exactly what one context with world*S samples would draw -- sorts them and
keeps the per-position sums.  The only exchange is one all-reduce(sum) of N doubles; every rank
then finishes the same decision from the total.  No other collective is needed.
"""
from __future__ import annotations

import numpy as np


def shard_config(rank: int, world: int, samples_per_rank: int) -> dict:
    """Keyword arguments for binding.Cutoff that place `rank` in a decision of world*S samples."""
    if not 0 <= rank < world:
        raise ValueError("rank out of range")
    return {"n_samples": samples_per_rank, "sample_offset": rank * samples_per_rank,
            "total_samples": world * samples_per_rank}


class ShardedDecision:
    """Wraps a context (anything with predict / get_partial_sums / decide_from_sums) and a process group."""

    def __init__(self, ctx, group=None, device=None):
        self.ctx = ctx
        self.group = group
        self.device = device           # where the all-reduce buffer lives ("cuda" for NCCL, None/cpu for gloo)

    def predict(self):
        """(code, c): the decision over all ranks' samples; identical on every rank."""
        import torch
        import torch.distributed as dist

        code, c = self.ctx.predict()
        if code == 1:                  # warm-up: nothing was drawn, nothing to exchange
            return code, c
        sums = torch.from_numpy(np.ascontiguousarray(self.ctx.get_partial_sums()))
        if self.device is not None:
            sums = sums.to(self.device)
        dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=self.group)
        return self.ctx.decide_from_sums(sums.cpu().numpy())
