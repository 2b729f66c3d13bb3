"""GPU check of dp_layernorm_sqnorms_static, the entry point for callers that cannot allocate device memory
(their framework or server owns the device's memory, or cudaMalloc's synchronisation is not acceptable where
they run).  Its scratch is a fixed array inside the library, so the test calls it through the C ABI twice in a
row -- the second call meets the first call's leftovers in that array -- and compares each result with the
workspace-based dp_per_example_sqnorms on the same layer and with the CPU checker.  Collected last on purpose."""
import numpy as np
import pytest
import torch

from .helpers import LAYERNORM, LayerSpec, O, b, make_layer_list, random_layers, to_np, to_oracle_layers

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = "cuda:0"


def _reference(ll):
    n = torch.empty(ll.B, dtype=torch.float32, device=DEV)
    b.dp_per_example_sqnorms(ll, n, False, b.alloc_workspace(ll))
    return to_np(n)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_static_scratch_matches_workspace_path_twice_in_a_row(dtype):
    cases = [(64, 128, 1024, 11), (7, 33, 200, 12)]       # second call is smaller: stale tail stays in the array
    for B, T, d, seed in cases:
        data = random_layers([LayerSpec(LAYERNORM, d, d, False, "ln")], B, T, dtype, DEV, seed=seed, g_scale=0.3)
        ll, _ = make_layer_list(data, DEV)
        ref = _reference(ll)
        got = torch.full((B,), float("nan"), dtype=torch.float32, device=DEV)
        b.dp_layernorm_sqnorms_static(ll, got, False)
        np.testing.assert_allclose(to_np(got), ref, rtol=2e-3)
        # and against the CPU checker directly, not only against the library's other path
        np.testing.assert_allclose(to_np(got), O.per_example_sqnorms(to_oracle_layers(data)), rtol=2e-3)
        # accumulate_into adds to what is there
        b.dp_layernorm_sqnorms_static(ll, got, True)
        np.testing.assert_allclose(to_np(got), 2 * ref, rtol=2e-3)
    assert b.dp_poll_status() == 0


def test_static_scratch_rejects_sizes_beyond_the_limit():
    B, T, d = 1024, 2, 1024                                 # B * 2d = 2^21 floats > 2^20
    assert B * 2 * d > b.STATIC_SCRATCH_FLOATS
    data = random_layers([LayerSpec(LAYERNORM, d, d, False, "ln")], B, T, torch.bfloat16, DEV, seed=1)
    ll, _ = make_layer_list(data, DEV)
    n = torch.zeros(B, dtype=torch.float32, device=DEV)
    with pytest.raises(b.DpError) as e:
        b.dp_layernorm_sqnorms_static(ll, n, False)
    assert e.value.code == -6
    assert float(n.abs().max()) == 0.0                      # nothing was launched
    # a linear layer is not accepted
    lin = random_layers([LayerSpec("linear", 64, 64, False, "fc")], 2, 4, torch.bfloat16, DEV, seed=2)
    ll2, _ = make_layer_list(lin, DEV)
    with pytest.raises(b.DpError) as e2:
        b.dp_layernorm_sqnorms_static(ll2, n[:2], False)
    assert e2.value.code == -1
