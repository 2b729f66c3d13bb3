"""Two ranks as two processes that share cuda:0: the ranks map each other's accumulator and replica of theta through
CUDA IPC handles exchanged over the process group and end two macro-batches with the one-kernel way
(dp_reduce_noise_adamw_step over the mapped buffers), then with the in-place collectives.  The kernels wait for
nobody on the device; the ranks meet on the host (gloo barriers after a device synchronisation)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.multiprocessing as mp

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HP = dict(C=0.5, sigma=1.3, lr=1e-2, beta1=0.9, beta2=0.999, xi=1e-11, weight_decay=0.5, seed=11)


class _State:
    """The fields ShardedUpdate needs, on the GPU."""

    def __init__(self, n, dev):
        self.acc = torch.zeros(n, dtype=torch.float32, device=dev)
        self.theta = torch.linspace(-1, 1, n, dtype=torch.float32, device=dev)
        self.m = torch.zeros(n, dtype=torch.float32, device=dev)
        self.v = torch.zeros(n, dtype=torch.float32, device=dev)
        self.t, self.examples_seen = 0, 0
        for k, val in HP.items():
            setattr(self, k, val)


def _local_acc(rank, n):
    return torch.randn(n, generator=torch.Generator().manual_seed(100 + rank), dtype=torch.float32)


def _worker(rank, world, port, n, fused, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    from paper_2108_01624_b200.parallel import ShardedUpdate, exchange_peer_buffers
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    st = _State(n, dev)
    if fused:
        accs = exchange_peer_buffers(st.acc, dist, world, rank)
        thetas = exchange_peer_buffers(st.theta, dist, world, rank)
        sh = ShardedUpdate(st, dist, world, rank, peer_acc=accs, peer_theta=thetas)
    else:
        sh = ShardedUpdate(st, dist, world, rank)
    src = _local_acc(rank, n).to(dev)
    for step in range(2):
        st.acc.copy_(src * (step + 1))
        st.examples_seen = 64 * world
        sh.finish_macro_batch()
    torch.cuda.synchronize()
    torch.save({"theta": st.theta.cpu(), "acc": st.acc.cpu(), "m": st.m.cpu(), "lo": sh.lo, "hi": sh.hi},
               f"{out_dir}/g{rank}.pt")
    dist.barrier()                       # nobody unmaps or frees while a peer may still touch the buffers
    if fused:
        del sh, accs, thetas
        torch.cuda.ipc_collect()
    dist.barrier()
    dist.destroy_process_group()


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


@pytest.mark.parametrize("fused", [True, False])
def test_two_processes_finish_a_macro_batch_together(fused, tmp_path):
    from oracle import dp_oracle as O
    world, n = 2, 100_003
    mp.spawn(_worker, args=(world, _free_port(), n, fused, str(tmp_path)), nprocs=world, join=True)
    outs = [torch.load(f"{tmp_path}/g{r}.pt") for r in range(world)]
    total = sum(_local_acc(r, n).double().numpy() for r in range(world))
    theta = np.linspace(-1, 1, n).astype(np.float32).astype(np.float64)
    m, v = np.zeros(n), np.zeros(n)
    for step in range(2):
        g = O.add_noise_and_scale(total * (step + 1), HP["sigma"], HP["C"], 64 * world, HP["seed"], step + 1, 0)
        theta, m, v = O.adamw_step(theta, m, v, g, HP["lr"], HP["beta1"], HP["beta2"], HP["xi"], HP["weight_decay"],
                                   step + 1)
    assert torch.equal(outs[0]["theta"], outs[1]["theta"])               # both replicas hold the same bits
    for o in outs:
        assert float(o["acc"].abs().max()) == 0.0
        np.testing.assert_allclose(o["theta"].double().numpy(), theta, rtol=2e-4, atol=2e-6)
        lo, hi = o["lo"], o["hi"]
        np.testing.assert_allclose(o["m"][lo:hi].double().numpy(), m[lo:hi], rtol=1e-4, atol=1e-7)
