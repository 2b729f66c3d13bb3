"""Data-parallel macro-step: one process per GPU, examples sharded across ranks.

Per-example clipping needs no exchange (clip factors are per example), so ranks accumulate their own
microbatches independently.  Once per macro-batch the fp32 accumulators are summed across ranks -- the
gradient reduction that large batches amortise (Section 5.3) -- and each rank runs the fused noise + AdamW
pass on its own shard of the flat parameter vector.  The noise is keyed by the GLOBAL element index, so it
is added exactly once and the result does not depend on the number of ranks.

Two ways to end a macro-batch:
  * collectives, in place: reduce-scatter of the accumulator into this rank's shard of it, the fused update on
    the shard, all-gather of theta from this rank's shard of it (no staging copies: the flat buffers are
    allocated with room for `world` equal shards);
  * one kernel over peer-addressable memory (dp_reduce_noise_adamw_step): the shard owner loads the shard from
    every rank's accumulator, updates, and stores the new theta into every replica.  `exchange_peer_buffers`
    makes the ranks' buffers addressable (CUDA IPC between processes; plain loads and stores only).
"""
from __future__ import annotations

from typing import Callable, List, Optional

import torch


def shard_length(n_flat: int, world: int) -> int:
    """Elements per shard: equal shards whose length is a multiple of 4 (one Philox block, one 16-byte vector)."""
    per = (n_flat + world - 1) // world
    return (per + 3) // 4 * 4


def padded_length(n_flat: int, world: int) -> int:
    """Length of a flat buffer that holds `world` whole shards (>= n_flat; the tail is padding)."""
    return n_flat if world <= 1 else shard_length(n_flat, world) * world


def shard_bounds(n_flat: int, world: int, rank: int):
    """(start, stop) of rank's shard within the n_flat real elements; the last shards may be short or empty."""
    per = shard_length(n_flat, world)
    lo = min(rank * per, n_flat)
    return lo, min(lo + per, n_flat)


def exchange_peer_buffers(tensor: torch.Tensor, dist, world: int, rank: int) -> List[torch.Tensor]:
    """Every rank passes its own buffer; returns one tensor per rank that aliases THAT rank's buffer and that this
    process can address: entry `rank` is `tensor` itself, the others are mapped from handles exchanged over the
    process group (CUDA IPC for device memory -- the peer's allocation is mapped into this process and peer
    access is enabled by the mapping; a shared-memory file for host memory, which is what the CPU tests use).
    The mapping is plain memory: kernels reach it with ordinary loads and stores.  Keep the returned tensors
    alive as long as kernels use their addresses, and the owner must keep `tensor` alive as long as any peer
    maps it."""
    from torch.multiprocessing import reductions
    if tensor.is_cuda:
        handle = reductions.reduce_tensor(tensor)        # (rebuild function, plain-data arguments incl. the IPC handle)
    else:
        import torch.multiprocessing as mp
        if mp.get_sharing_strategy() != "file_system":   # the handle must be plain data (a name), not an open descriptor
            mp.set_sharing_strategy("file_system")
        # moves the storage to a shared-memory file in place; `tensor` keeps pointing at it
        rebuild_storage, storage_args = reductions.reduce_storage(tensor.untyped_storage())
        meta = (tensor.storage_offset(), tuple(tensor.size()), tuple(tensor.stride()), tensor.dtype)
        handle = (_rebuild_host_tensor, (rebuild_storage, storage_args, meta))
    gathered = [None] * world
    dist.all_gather_object(gathered, handle)
    out = []
    for r in range(world):
        out.append(tensor if r == rank else gathered[r][0](*gathered[r][1]))
    return out


def _rebuild_host_tensor(rebuild_storage, storage_args, meta):
    offset, size, stride, dtype = meta
    storage = rebuild_storage(*storage_args)
    return torch.empty(0, dtype=dtype).set_(storage, offset, size, stride)


class ShardedUpdate:
    """Finishes a macro-batch across `world` ranks for a DPStep-like state object.

    `update_fn(theta, m, v, acc, elem_offset, batch_size, t)` applies noise + scaling + AdamW in place to
    one shard and zeroes that shard of the accumulator; by default it is the library's fused kernel.  The state
    object supplies theta, m, v, acc, t, examples_seen (already the global count) and the hyper-parameters.

    The flat accumulator and theta must have room for `world` whole shards.  DPStep(shard_world=world) allocates
    them that way (acc_store / theta_store).  For any other state object the constructor re-allocates the two
    buffers once and re-points state.acc / state.theta at them: build descriptor lists after that.
    """

    def __init__(self, state, dist, world: int, rank: int, update_fn: Optional[Callable] = None,
                 peer_acc=None, peer_theta=None, fused_fn: Optional[Callable] = None,
                 poll_fn: Optional[Callable] = None):
        """peer_acc / peer_theta (optional, one entry per rank): every rank's full accumulator and full replica of
        theta as this GPU can address them (tensors from exchange_peer_buffers, or raw device addresses of
        peer-mapped memory).  With both given, the macro-batch ends with ONE kernel per rank that sums the shard
        over all ranks, applies noise + AdamW and writes theta into every replica (`fused_fn`, by default the
        library's dp_reduce_noise_adamw_step), between two barriers.
        poll_fn() returns this rank's device status code (0 = clean); by default the library's dp_poll_status."""
        self.state, self.dist, self.world, self.rank = state, dist, world, rank
        self.peer_acc, self.peer_theta = peer_acc, peer_theta
        self.fused_fn = fused_fn or self._fused_reduce_kernel
        if (peer_acc is None) != (peer_theta is None):
            raise ValueError("peer_acc and peer_theta go together")
        if peer_acc is not None and (len(peer_acc) != world or len(peer_theta) != world):
            raise ValueError("one accumulator and one replica per rank")
        self.n = state.acc.numel()
        self.lo, self.hi = shard_bounds(self.n, world, rank)
        self.per = shard_length(self.n, world)
        self.update_fn = update_fn or self._fused_kernel
        self.poll_fn = poll_fn or self._poll_library
        self.nccl = dist.get_backend() == "nccl"
        self._events = None
        self._in_place = True          # collectives on aliased buffers; cleared if the process group refuses them
        if peer_acc is None:
            self.acc_full = self._padded(state, "acc")
            self.theta_full = self._padded(state, "theta")

    # ---- plumbing ---------------------------------------------------------------------------------------------
    def _padded(self, state, name: str) -> torch.Tensor:
        total = self.per * self.world
        store = getattr(state, name + "_store", None)
        if store is not None and store.numel() == total and getattr(state, name).data_ptr() == store.data_ptr():
            return store
        old = getattr(state, name)
        store = torch.zeros(total, dtype=old.dtype, device=old.device)
        store[:self.n].copy_(old)
        setattr(state, name + "_store", store)
        setattr(state, name, store[:self.n])
        return store

    def _poll_library(self) -> int:
        from . import binding as b
        return b.dp_poll_status()

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

    def _barrier(self):
        """All ranks' work enqueued so far is complete when this returns on any rank.  NCCL's barrier is ordered
        after the current stream's work; other backends only meet on the host, so the device is drained first."""
        if not self.nccl and self.state.acc.is_cuda:
            torch.cuda.synchronize(self.state.acc.device)
        self.dist.barrier()
        if self.nccl:
            torch.cuda.synchronize(self.state.acc.device)

    def _agreed_status(self) -> int:
        """This rank's device status, then the worst over all ranks, so that every rank takes the same branch
        (a rank that stopped alone would leave the others waiting in the collectives)."""
        code = int(self.poll_fn())
        t = torch.tensor([code], dtype=torch.int32, device=self.state.acc.device if self.nccl else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MIN)       # status codes are <= 0
        return int(t.item())

    def _check_or_discard(self):
        from .step import DeviceStatusError
        code = self._agreed_status()
        if code != 0:
            s = self.state
            s.acc.zero_()
            s.examples_seen = 0
            raise DeviceStatusError(code)

    def _mark(self, k: int):
        if self._events is not None:
            if k == 0:
                self._events.append([torch.cuda.Event(enable_timing=True) for _ in range(4)])
            self._events[-1][k].record()

    def time_phases(self, on: bool = True):
        """From now on every finished macro-batch records four device events around its three phases."""
        self._events = [] if on and self.state.acc.is_cuda else None

    def timings(self):
        """Mean device milliseconds of the phases of the macro-batches finished since time_phases() (or since the
        last call): {"reduce": reduce-scatter (or the opening barrier of the one-kernel way), "update": the shard
        update, "gather": all-gather + zeroing (or the closing barrier), "macro_batches": how many}.
        Synchronises the device; None when nothing was recorded."""
        if not self._events:
            return None
        torch.cuda.synchronize()
        ev, self._events = self._events, []
        names = ("reduce", "update", "gather")
        out = {n: sum(e[i].elapsed_time(e[i + 1]) for e in ev) / len(ev) for i, n in enumerate(names)}
        out["macro_batches"] = len(ev)
        return out

    # ---- the two ways to end a macro-batch ----------------------------------------------------------------------
    def _finish_fused(self):
        s = self.state
        lo, hi = self.lo, self.hi
        self._mark(0)
        self._barrier()         # every rank's accumulate kernels precede the reads below
        self._mark(1)
        if hi > lo:
            self.fused_fn(s.theta[lo:hi], s.m[lo:hi], s.v[lo:hi], [self._shard_of(a, lo, hi) for a in self.peer_acc],
                          [self._shard_of(t, lo, hi) for t in self.peer_theta], lo, s.examples_seen, s.t)
        self._mark(2)
        self._barrier()         # every shard of every replica is written, every accumulator is zero
        self._mark(3)

    def _finish_collectives(self):
        s, dist, per, r = self.state, self.dist, self.per, self.rank
        acc, theta = self.acc_full, self.theta_full
        mine_acc = acc[r * per:(r + 1) * per]
        mine_theta = theta[r * per:(r + 1) * per]
        lo, hi = self.lo, self.hi
        self._mark(0)
        if self.nccl and self._in_place:
            try:
                dist.reduce_scatter_tensor(mine_acc, acc)       # in place: the output is this rank's slice of the input
            except (RuntimeError, ValueError):                  # a front end that refuses aliased buffers: stage once
                self._in_place = False
        if self.nccl and not self._in_place:
            out = torch.empty_like(mine_acc)
            dist.reduce_scatter_tensor(out, acc)
            mine_acc.copy_(out)
        elif not self.nccl:
            dist.all_reduce(acc)
        self._mark(1)
        if hi > lo:
            self.update_fn(s.theta[lo:hi], s.m[lo:hi], s.v[lo:hi], acc[lo:hi], lo, s.examples_seen, s.t)
        self._mark(2)
        if self.nccl and self._in_place:
            try:
                dist.all_gather_into_tensor(theta, mine_theta)  # in place: the input is this rank's slice of the output
            except (RuntimeError, ValueError):
                self._in_place = False
        if self.nccl and not self._in_place:
            dist.all_gather_into_tensor(theta, mine_theta.clone())
        elif not self.nccl:
            dist.all_gather([theta[k * per:(k + 1) * per] for k in range(self.world)], mine_theta.clone())
        # the other ranks' shards of the accumulator still hold this rank's sums
        acc[:r * per].zero_()
        acc[(r + 1) * per:].zero_()
        self._mark(3)

    def finish_macro_batch(self, check_status: bool = True):
        """Ends the macro-batch on every rank (collective call).  With check_status, a device-side error on ANY
        rank since the last poll makes every rank discard its accumulator and raise before anything is applied."""
        if check_status:
            self._check_or_discard()
        s = self.state
        s.t += 1
        if self.peer_acc is not None:
            self._finish_fused()
        else:
            self._finish_collectives()
        s.examples_seen = 0

