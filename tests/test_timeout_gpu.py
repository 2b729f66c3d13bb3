"""A bounded device-side wait that runs out: the kernel returns, the status word says so, and the library goes on
working.  The wait limit is shortened for the test; nothing hangs, traps or faults."""
import numpy as np
import pytest
import torch

from .helpers import LINEAR, LayerSpec, O, b, gpu_norms_clip, make_layer_list, random_layers, to_np, to_oracle_layers

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = "cuda:0"


def test_wait_that_nobody_satisfies_gives_up_and_is_reported():
    torch.cuda.synchronize()
    assert b.dp_poll_status() == 0
    try:
        b.dp_set_wait_limit_cycles(2_000_000)            # about a millisecond
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        b.dp_selftest_wait_timeout()
        t1.record()
        torch.cuda.synchronize()
        assert t0.elapsed_time(t1) < 100.0                # it returned at the limit, not at the default of seconds
        assert b.dp_poll_status() == -5                   # DP_ERR_TIMEOUT
        info = b.dp_last_timeout_info()
        assert info[0] in (98, 99) and info[1] == 0       # the self-test's wait sites, block 0
        assert info[2] == (7 if info[0] == 99 else 8) and info[4] == (0 if info[0] == 99 else 32)
        assert b.dp_poll_status() == 0                    # the poll cleared the word
    finally:
        b.dp_set_wait_limit_cycles(0)                     # back to the default
    # an ordinary call afterwards runs clean and right
    data = random_layers([LayerSpec(LINEAR, 256, 128, True, "fc")], 4, 64, torch.bfloat16, DEV, seed=3, g_scale=0.02)
    ll, accs = make_layer_list(data, DEV)
    n, c, ws = gpu_norms_clip(ll, 1.0)
    b.dp_clipped_accumulate(ll, c, ws)
    assert b.dp_poll_status() == 0
    n_ref = O.per_example_sqnorms(to_oracle_layers(data))
    np.testing.assert_allclose(to_np(n), n_ref, rtol=2e-3)


def test_macro_batch_is_not_applied_after_a_timeout():
    """DPStep reads the status before the update: after a timeout theta, m and v stay put and the accumulator is dropped."""
    from paper_2108_01624_b200 import DeviceStatusError, DPStep
    specs = [LayerSpec(LINEAR, 128, 64, True, "fc")]
    step = DPStep(specs, DEV, C=1.0, sigma=1.0, lr=1e-2, beta1=0.9, beta2=0.999, xi=1e-11, weight_decay=0.1)
    step.theta.fill_(0.5)
    data = random_layers(specs, 4, 32, torch.bfloat16, DEV, seed=5, g_scale=0.02)
    step.accumulate_microbatch(step.layer_list(data))
    try:
        b.dp_set_wait_limit_cycles(2_000_000)
        b.dp_selftest_wait_timeout()
        with pytest.raises(DeviceStatusError) as e:
            step.finish_macro_batch()
    finally:
        b.dp_set_wait_limit_cycles(0)
    assert e.value.code == -5
    assert step.t == 0 and step.examples_seen == 0
    assert float(step.acc.abs().max()) == 0.0 and float(step.m.abs().max()) == 0.0
    assert bool(torch.all(step.theta == 0.5))
    step.accumulate_microbatch(step.layer_list(data))
    step.finish_macro_batch()
    assert step.t == 1 and not bool(torch.all(step.theta == 0.5))
