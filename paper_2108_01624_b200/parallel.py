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

    def __init__(self, state, dist, world: int, rank: int, update_fn: Optional[Callable] = None,
                 peer_acc=None, peer_theta=None, fused_fn: Optional[Callable] = None):
        """peer_acc / peer_theta (optional, one entry per rank): every rank's full accumulator and full replica of
        theta as this GPU can address them (tensors, or raw device addresses of peer-mapped memory, e.g. the
        buffer pointers of a symmetric-memory rendezvous).  With both given, the macro-batch ends with ONE kernel
        per rank that sums the shard over all ranks, applies noise + AdamW and writes theta into every replica
        (`fused_fn`, by default the library's dp_reduce_noise_adamw_step), between two barriers."""
        self.state, self.dist, self.world, self.rank = state, dist, world, rank
        self.peer_acc, self.peer_theta = peer_acc, peer_theta
        self.fused_fn = fused_fn or self._fused_reduce_kernel
        if (peer_acc is None) != (peer_theta is None):
            raise ValueError("peer_acc and peer_theta go together")
        if peer_acc is not None and (len(peer_acc) != world or len(peer_theta) != world):
            raise ValueError("one accumulator and one replica per rank")
        self.lo, self.hi = shard_bounds(state.acc.numel(), world, rank)
        self.per = shard_bounds(state.acc.numel(), world, 0)[1]
        self.update_fn = update_fn or self._fused_kernel
        self.use_reduce_scatter = dist.get_backend() == "nccl"
        # staging for the collectives of the two-step path (the fused path reads the peers' buffers in place)
        self.padded = None if peer_acc is not None else torch.zeros(self.per * world, dtype=state.acc.dtype,
                                                                     device=state.acc.device)

    def _fused_kernel(self, theta, m, v, acc, elem_offset, batch_size, t):
        from . import binding as b
        s = self.state
        b.dp_noise_scale_adamw_step(theta, m, v, acc, True, s.sigma, s.C, batch_size, s.seed, t, s.lr, s.beta1,
                                    s.beta2, s.xi, s.weight_decay, t, elem_offset)

    def _fused_reduce_kernel(self, theta, m, v, acc_shards, theta_shards, elem_offset, batch_size, t):
        from . import binding as b
        s = self.state
        b.dp_reduce_noise_adamw_step(theta, m, v, acc_shards, theta_shards, True, s.sigma, s.C, batch_size, s.seed, t,
                                     s.lr, s.beta1, s.beta2, s.xi, s.weight_decay, t, elem_offset)

    @staticmethod
    def _shard_of(buf, lo, hi):
        return buf + 4 * lo if isinstance(buf, int) else buf[lo:hi]      # fp32: 4 bytes per element

    def _finish_fused(self):
        s, dist = self.state, self.dist
        s.t += 1
        lo, hi = self.lo, self.hi
        dist.barrier()          # stream-ordered: every rank's accumulate kernels precede the reads below
        if hi > lo:
            self.fused_fn(s.theta[lo:hi], s.m[lo:hi], s.v[lo:hi], [self._shard_of(a, lo, hi) for a in self.peer_acc],
                          [self._shard_of(t, lo, hi) for t in self.peer_theta], lo, s.examples_seen, s.t)
        dist.barrier()          # every shard of every replica is written, every accumulator is zero
        s.examples_seen = 0

    def finish_macro_batch(self):
        if self.peer_acc is not None:
            return self._finish_fused()
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
