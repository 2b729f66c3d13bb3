"""world_size-2 (and 3) gloo runs on CPU of the data-parallel macro-step's host logic: sharding, the
accumulator reduction, shard-local noise + AdamW keyed by the global element index, and the gather."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


class _State:
    def __init__(self, n, acc):
        self.acc = acc.clone()
        self.theta = torch.linspace(-1, 1, n, dtype=torch.float64)
        self.m = torch.zeros(n, dtype=torch.float64)
        self.v = torch.zeros(n, dtype=torch.float64)
        self.t, self.examples_seen = 0, 0
        self.sigma, self.C, self.seed = 1.3, 0.5, 11
        self.lr, self.beta1, self.beta2, self.xi, self.weight_decay = 1e-2, 0.9, 0.999, 1e-11, 0.5


def _oracle_update(state):
    from oracle import dp_oracle as O

    def fn(theta, m, v, acc, elem_offset, batch_size, t):
        g = O.add_noise_and_scale(acc.numpy(), state.sigma, state.C, batch_size, state.seed, t, elem_offset)
        th, mm, vv = O.adamw_step(theta.numpy(), m.numpy(), v.numpy(), g, state.lr, state.beta1, state.beta2,
                                  state.xi, state.weight_decay, t)
        theta.copy_(torch.from_numpy(th)); m.copy_(torch.from_numpy(mm)); v.copy_(torch.from_numpy(vv))
        acc.zero_()
    return fn


def _worker(rank, world, port, n, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2108_01624_b200.parallel import ShardedUpdate
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.Generator().manual_seed(100 + rank)
    local_acc = torch.randn(n, generator=g, dtype=torch.float64)
    st = _State(n, local_acc)
    sh = ShardedUpdate(st, dist, world, rank, update_fn=_oracle_update(st), poll_fn=lambda: 0)
    for step in range(2):
        st.acc.copy_(local_acc * (step + 1))
        st.examples_seen = 64 * world
        sh.finish_macro_batch()
    torch.save({"theta": st.theta, "acc": st.acc, "lo": sh.lo, "hi": sh.hi, "m": st.m}, f"{out_dir}/r{rank}.pt")
    dist.destroy_process_group()


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


@pytest.mark.parametrize("world,n", [(2, 1003), (3, 64)])
def test_sharded_update_equals_single_process(world, n, tmp_path):
    from oracle import dp_oracle as O
    mp.spawn(_worker, args=(world, _free_port(), n, str(tmp_path)), nprocs=world, join=True)
    outs = [torch.load(f"{tmp_path}/r{r}.pt") for r in range(world)]
    # single-process reference: summed accumulators, one update over the whole vector
    accs = [torch.randn(n, generator=torch.Generator().manual_seed(100 + r), dtype=torch.float64) for r in range(world)]
    st = _State(n, sum(accs))
    fn = _oracle_update(st)
    for step in range(2):
        st.t += 1
        acc = (sum(accs) * (step + 1)).clone()
        fn(st.theta, st.m, st.v, acc, 0, 64 * world, st.t)
    for r, o in enumerate(outs):
        np.testing.assert_allclose(o["theta"].numpy(), st.theta.numpy(), rtol=1e-12, atol=1e-14)
        assert float(o["acc"].abs().max()) == 0.0
        np.testing.assert_allclose(o["m"][o["lo"]:o["hi"]].numpy(), st.m[o["lo"]:o["hi"]].numpy(), rtol=1e-12)
    covered = sorted((o["lo"], o["hi"]) for o in outs)
    assert covered[0][0] == 0 and covered[-1][1] == n
    assert all(a[1] == b[0] for a, b in zip(covered[:-1], covered[1:]))
    assert all(lo % 4 == 0 for lo, _ in covered)


def test_shard_bounds_cover_and_align():
    from paper_2108_01624_b200.parallel import shard_bounds
    for n in (1, 5, 64, 1003, 333_563_904):
        for world in (1, 2, 3, 8):
            spans = [shard_bounds(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            for (a, b_), (c, d) in zip(spans[:-1], spans[1:]):
                assert b_ == c and a <= b_
            assert all(lo % 4 == 0 or lo == n for lo, _ in spans)


def _oracle_fused(state):
    """CPU stand-in for dp_reduce_noise_adamw_step: rank-ordered sum of the accumulator shards, noise + AdamW,
    theta into every replica, accumulator shards zeroed."""
    from oracle import dp_oracle as O

    def fn(theta, m, v, acc_shards, theta_shards, elem_offset, batch_size, t):
        total = np.zeros(theta.numel())
        for a in acc_shards:
            total += a.numpy()
        g = O.add_noise_and_scale(total, state.sigma, state.C, batch_size, state.seed, t, elem_offset)
        th, mm, vv = O.adamw_step(theta.numpy(), m.numpy(), v.numpy(), g, state.lr, state.beta1, state.beta2,
                                  state.xi, state.weight_decay, t)
        m.copy_(torch.from_numpy(mm)); v.copy_(torch.from_numpy(vv))
        for ts in theta_shards:
            ts.copy_(torch.from_numpy(th))
        for a in acc_shards:
            a.zero_()
    return fn


def _fused_worker(rank, world, port, n, accs, thetas, out_dir):
    """accs / thetas live in shared memory: every process addresses every rank's buffers, as peer-mapped GPU
    memory would be."""
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2108_01624_b200.parallel import ShardedUpdate
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.Generator().manual_seed(100 + rank)
    local_acc = torch.randn(n, generator=g, dtype=torch.float64)
    st = _State(n, local_acc)
    st.acc, st.theta = accs[rank], thetas[rank]          # this rank's buffers are the shared ones
    st.theta.copy_(torch.linspace(-1, 1, n, dtype=torch.float64))
    sh = ShardedUpdate(st, dist, world, rank, peer_acc=accs, peer_theta=thetas, fused_fn=_oracle_fused(st),
                       poll_fn=lambda: 0)
    for step in range(2):
        st.acc.copy_(local_acc * (step + 1))
        st.examples_seen = 64 * world
        sh.finish_macro_batch()
        assert st.examples_seen == 0 and st.t == step + 1
    torch.save({"theta": st.theta.clone(), "acc": st.acc.clone(), "lo": sh.lo, "hi": sh.hi, "m": st.m},
               f"{out_dir}/f{rank}.pt")
    dist.destroy_process_group()


@pytest.mark.parametrize("world,n", [(2, 1003), (3, 64)])
def test_fused_peer_memory_update_equals_single_process(world, n, tmp_path):
    accs = [torch.zeros(n, dtype=torch.float64).share_memory_() for _ in range(world)]
    thetas = [torch.zeros(n, dtype=torch.float64).share_memory_() for _ in range(world)]
    mp.spawn(_fused_worker, args=(world, _free_port(), n, accs, thetas, str(tmp_path)), nprocs=world, join=True)
    outs = [torch.load(f"{tmp_path}/f{r}.pt") for r in range(world)]
    src = [torch.randn(n, generator=torch.Generator().manual_seed(100 + r), dtype=torch.float64) for r in range(world)]
    st = _State(n, sum(src))
    fn = _oracle_update(st)
    for step in range(2):
        st.t += 1
        fn(st.theta, st.m, st.v, (sum(src) * (step + 1)).clone(), 0, 64 * world, st.t)
    for o in outs:
        np.testing.assert_allclose(o["theta"].numpy(), st.theta.numpy(), rtol=1e-12, atol=1e-14)
        assert float(o["acc"].abs().max()) == 0.0
        np.testing.assert_allclose(o["m"][o["lo"]:o["hi"]].numpy(), st.m[o["lo"]:o["hi"]].numpy(), rtol=1e-12)


def test_peer_buffers_given_as_addresses():
    from paper_2108_01624_b200.parallel import ShardedUpdate
    assert ShardedUpdate._shard_of(4096, 8, 16) == 4096 + 32
    t = torch.arange(20.0)
    assert torch.equal(ShardedUpdate._shard_of(t, 8, 16), t[8:16])


def _rendezvous_worker(rank, world, port, n, out_dir):
    """Every rank allocates its own accumulator and replica, the ranks exchange handles over the process group
    (exchange_peer_buffers) and finish two macro-batches with the one-kernel way over the mapped buffers."""
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2108_01624_b200.parallel import ShardedUpdate, exchange_peer_buffers
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    g = torch.Generator().manual_seed(100 + rank)
    local_acc = torch.randn(n, generator=g, dtype=torch.float64)
    st = _State(n, local_acc)
    accs = exchange_peer_buffers(st.acc, dist, world, rank)
    thetas = exchange_peer_buffers(st.theta, dist, world, rank)
    assert accs[rank] is st.acc and thetas[rank] is st.theta
    # a write through the mapping is seen by the owner
    dist.barrier()
    if rank == 0:
        accs[world - 1][n - 1] = 12345.0
    dist.barrier()
    if rank == world - 1:
        assert float(st.acc[n - 1]) == 12345.0
    dist.barrier()
    sh = ShardedUpdate(st, dist, world, rank, peer_acc=accs, peer_theta=thetas, fused_fn=_oracle_fused(st),
                       poll_fn=lambda: 0)
    for step in range(2):
        st.acc.copy_(local_acc * (step + 1))
        st.examples_seen = 64 * world
        sh.finish_macro_batch()
    torch.save({"theta": st.theta.clone(), "acc": st.acc.clone(), "lo": sh.lo, "hi": sh.hi, "m": st.m},
               f"{out_dir}/x{rank}.pt")
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,n", [(2, 1003), (3, 257)])
def test_handle_exchange_then_fused_update(world, n, tmp_path):
    mp.spawn(_rendezvous_worker, args=(world, _free_port(), n, str(tmp_path)), nprocs=world, join=True)
    outs = [torch.load(f"{tmp_path}/x{r}.pt") for r in range(world)]
    src = [torch.randn(n, generator=torch.Generator().manual_seed(100 + r), dtype=torch.float64) for r in range(world)]
    st = _State(n, sum(src))
    fn = _oracle_update(st)
    for step in range(2):
        st.t += 1
        fn(st.theta, st.m, st.v, (sum(src) * (step + 1)).clone(), 0, 64 * world, st.t)
    for o in outs:
        np.testing.assert_allclose(o["theta"].numpy(), st.theta.numpy(), rtol=1e-12, atol=1e-14)
        assert float(o["acc"].abs().max()) == 0.0


def _status_worker(rank, world, port, n, bad_rank, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2108_01624_b200.parallel import ShardedUpdate
    from paper_2108_01624_b200.step import DeviceStatusError
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    st = _State(n, torch.ones(n, dtype=torch.float64))
    calls = []
    codes = iter([-5 if rank == bad_rank else 0, 0])      # first macro-batch: one rank reports a timeout

    def update(theta, m, v, acc, elem_offset, batch_size, t):
        calls.append(t)
        acc.zero_()
    sh = ShardedUpdate(st, dist, world, rank, update_fn=update, poll_fn=lambda: next(codes))
    theta0 = st.theta.clone()
    st.examples_seen = 8
    raised = None
    try:
        sh.finish_macro_batch()
    except DeviceStatusError as e:
        raised = e.code
    ok_first = (raised == -5 and not calls and st.t == 0 and st.examples_seen == 0
                and float(st.acc.abs().max()) == 0.0 and torch.equal(st.theta, theta0))
    st.acc.fill_(1.0)
    st.examples_seen = 8
    sh.finish_macro_batch()                               # the next macro-batch goes through on every rank
    ok_second = calls == [1] and st.t == 1
    torch.save({"ok_first": ok_first, "ok_second": ok_second}, f"{out_dir}/s{rank}.pt")
    dist.destroy_process_group()


def test_device_error_on_one_rank_discards_the_macro_batch_on_all(tmp_path):
    world = 2
    mp.spawn(_status_worker, args=(world, _free_port(), 40, 1, str(tmp_path)), nprocs=world, join=True)
    for r in range(world):
        o = torch.load(f"{tmp_path}/s{r}.pt")
        assert o["ok_first"] and o["ok_second"], (r, o)


def test_padded_storage_is_reused_or_made():
    from paper_2108_01624_b200.parallel import padded_length, shard_length
    assert padded_length(1003, 1) == 1003
    assert padded_length(1003, 2) == 2 * shard_length(1003, 2) == 1008
    assert padded_length(333_563_904, 8) == 333_563_904
