"""Host logic of DPStep that needs no GPU: the device status is read before a macro-batch is applied."""
import pytest
import torch

from paper_2108_01624_b200 import step as step_mod
from paper_2108_01624_b200.synth import LAYERNORM, LINEAR, LayerSpec


class _FakeBinding:
    """Stands in for the ctypes binding: records the update calls, reports a chosen status code."""
    DP_OK = 0

    def __init__(self, code):
        self.code, self.calls = code, []

    def dp_poll_status(self, stream=None):
        c, self.code = self.code, 0          # the real word is cleared by the poll
        return c

    def status_string(self, code):
        return {-5: "device-side wait timed out", -7: "token id out of range"}.get(code, "?")

    def dp_noise_scale_adamw_step(self, theta, m, v, acc, zero_acc, *rest):
        self.calls.append("fused")
        theta.add_(1.0)
        acc.zero_()

    def dp_add_noise_and_scale(self, *a):
        self.calls.append("noise")

    def dp_adamw_step(self, *a):
        self.calls.append("adamw")


@pytest.mark.parametrize("code", [-5, -7])
def test_bad_device_status_leaves_the_parameters_alone(monkeypatch, code):
    fake = _FakeBinding(code)
    monkeypatch.setattr(step_mod, "b", fake)
    specs = [LayerSpec(LINEAR, 8, 4, True, "fc"), LayerSpec(LAYERNORM, 4, 4, False, "ln")]
    st = step_mod.DPStep(specs, "cpu", C=1.0, sigma=1.0, lr=1e-3, beta1=0.9, beta2=0.999, xi=1e-11, weight_decay=0.1)
    st.theta.fill_(0.25)
    st.acc.fill_(3.0)
    st.examples_seen = 16
    with pytest.raises(step_mod.DeviceStatusError) as e:
        st.finish_macro_batch()
    assert e.value.code == code
    assert fake.calls == []                                   # nothing was applied
    assert st.t == 0 and st.examples_seen == 0
    assert float(st.acc.abs().max()) == 0.0                   # the macro-batch is discarded
    assert torch.all(st.theta == 0.25) and float(st.m.abs().max()) == 0.0 and float(st.v.abs().max()) == 0.0
    # the next macro-batch is applied as usual
    st.acc.fill_(1.0)
    st.examples_seen = 16
    st.finish_macro_batch()
    assert fake.calls == ["fused"] and st.t == 1 and torch.all(st.theta == 1.25)


def test_flat_buffers_have_room_for_whole_shards():
    specs = [LayerSpec(LINEAR, 5, 3, True, "fc")]              # 15 -> 16, 3 -> 4: 20 elements
    st = step_mod.DPStep(specs, "cpu", 1.0, 1.0, 1e-3, 0.9, 0.999, 1e-11, 0.0, shard_world=3)
    assert st.n_flat == 20 and st.acc.numel() == 20 and st.theta.numel() == 20
    assert st.acc_store.numel() == 24 and st.theta_store.numel() == 24          # 3 shards of 8
    assert st.acc.data_ptr() == st.acc_store.data_ptr() and st.theta.data_ptr() == st.theta_store.data_ptr()
