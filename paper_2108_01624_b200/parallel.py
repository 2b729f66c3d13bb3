"""Data-parallel macro-step: one process per GPU, examples sharded across ranks.

Per-example clipping needs no exchange (clip factors are per example), so ranks accumulate their own
microbatches independently.  Once per macro-batch the fp32 accumulators are summed across ranks -- the
gradient reduction that large batches amortise (Section 5.3) -- as a reduce-scatter; each rank then runs
the fused noise + AdamW pass on its own shard of the flat parameter vector and theta is all-gathered.
The noise is keyed by the GLOBAL element index, so it is added exactly once and the result does not depend
on the number of ranks.
"""
from __future__ import annotations

from typing import Callable, Optional

import torch


def shard_bounds(n_flat: int, world: int, rank: int):
    """Equal shards whose length is a multiple of 4 elements (one Philox block, one 16-byte vector);
    the last shard may be shorter.  Returns (start, stop)."""
    per = (n_flat + world - 1) // world
    per = (per + 3) // 4 * 4
    lo = min(rank * per, n_flat)
    return lo, min(lo + per, n_flat)


class ShardedUpdate:
    """Finishes a macro-batch across `world` ranks for a DPStep-like state object.

    `update_fn(theta, m, v, acc, elem_offset, batch_size, t)` applies noise + scaling + AdamW in place to
    one shard; by default it is the library's fused kernel.  The state object supplies theta, m, v, acc,
    t, examples_seen (already the global count) and the hyper-parameters.
    """

    def __init__(self, state, dist, world: int, rank: int, update_fn: Optional[Callable] = None):
        self.state, self.dist, self.world, self.rank = state, dist, world, rank
        self.lo, self.hi = shard_bounds(state.acc.numel(), world, rank)
        self.per = shard_bounds(state.acc.numel(), world, 0)[1]
        self.padded = torch.zeros(self.per * world, dtype=state.acc.dtype, device=state.acc.device)
        self.update_fn = update_fn or self._fused_kernel
        self.use_reduce_scatter = dist.get_backend() == "nccl"

    def _fused_kernel(self, theta, m, v, acc, elem_offset, batch_size, t):
        from . import binding as b
        s = self.state
        b.dp_noise_scale_adamw_step(theta, m, v, acc, True, s.sigma, s.C, batch_size, s.seed, t, s.lr, s.beta1,
                                    s.beta2, s.xi, s.weight_decay, t, elem_offset)

    def finish_macro_batch(self):
        s, dist = self.state, self.dist
        n = s.acc.numel()
        s.t += 1
        self.padded[:n].copy_(s.acc)
        mine = self.padded[self.rank * self.per:(self.rank + 1) * self.per]
        if self.use_reduce_scatter:
            dist.reduce_scatter_tensor(mine, self.padded)
        else:
            dist.all_reduce(self.padded)
        lo, hi = self.lo, self.hi
        if hi > lo:
            self.update_fn(s.theta[lo:hi], s.m[lo:hi], s.v[lo:hi], mine[:hi - lo], lo, s.examples_seen, s.t)
        # gather the updated shards of theta
        th = torch.zeros_like(self.padded)
        th[lo:hi].copy_(s.theta[lo:hi])
        if self.use_reduce_scatter:
            dist.all_gather_into_tensor(th, th[self.rank * self.per:(self.rank + 1) * self.per].clone())
        else:
            parts = [torch.zeros(self.per, dtype=th.dtype, device=th.device) for _ in range(self.world)]
            dist.all_gather(parts, th[self.rank * self.per:(self.rank + 1) * self.per].clone())
            th = torch.cat(parts)
        s.theta.copy_(th[:n])
        s.acc.zero_()
        s.examples_seen = 0
