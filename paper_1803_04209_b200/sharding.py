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
    """Wraps a context and a process group.

    With ``device="cuda"`` the context must be a library context whose stream is torch's current stream:
    its part of the decision is enqueued up to the per-position sums, those N doubles are all-reduced in
    place in the library's own device array (NCCL orders itself after the work already on the current
    stream), and the decision is finished from them -- nothing passes through the host.  With
    ``device=None`` (gloo on CPU) the sums travel through host arrays via get_partial_sums /
    decide_from_sums.
    """

    def __init__(self, ctx, group=None, device=None):
        self.ctx = ctx
        self.group = group
        self.device = device           # "cuda" for NCCL, None for gloo on CPU
        self._sums = None

    def predict(self):
        """(code, c): the decision over all ranks' samples; identical on every rank."""
        import torch
        import torch.distributed as dist

        if self.device is not None and hasattr(self.ctx, "predict_partial_async"):
            code = self.ctx.predict_partial_async()
            if code == 1:              # warm-up: nothing was drawn, nothing to exchange
                return code, self.ctx.N
            if self._sums is None:
                self._sums = self.ctx.partial_sums_tensor()
            dist.all_reduce(self._sums, op=dist.ReduceOp.SUM, group=self.group)
            return self.ctx.decide_from_device_sums(self._sums)
        code, c = self.ctx.predict()
        if code == 1:
            return code, c
        sums = torch.from_numpy(np.ascontiguousarray(self.ctx.get_partial_sums()))
        dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=self.group)
        return self.ctx.decide_from_sums(sums.numpy())
