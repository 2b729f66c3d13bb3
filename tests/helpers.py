"""Shared plumbing for the GPU parity tests: build descriptor lists, run the library, run the checker."""
from __future__ import annotations

import numpy as np
import torch

from oracle import dp_oracle as O
from paper_2108_01624_b200 import binding as b
from paper_2108_01624_b200.synth import EMBEDDING, LAYERNORM, LINEAR, LayerData, LayerSpec

from .conftest import to_oracle_layers


def acc_shapes(spec: LayerSpec):
    if spec.kind == LINEAR:
        return [(spec.d_in, spec.d_out)] + ([(spec.d_out,)] if spec.has_bias else [])
    if spec.kind == LAYERNORM:
        return [(spec.d_out,), (spec.d_out,)]
    return [(spec.d_in, spec.d_out)]


def make_layer_list(data, device, paths=None, accs=None):
    """Returns (LayerList, accs) with fresh zero fp32 accumulators unless given."""
    if accs is None:
        accs = [[torch.zeros(s, dtype=torch.float32, device=device) for s in acc_shapes(ld.spec)] for ld in data]
    layers = []
    for k, (ld, acc) in enumerate(zip(data, accs)):
        sp = ld.spec
        layers.append(b.Layer(kind=sp.kind, G=ld.G, A=ld.A, ids=ld.ids, acc_w=acc[0],
                              acc_b=acc[1] if len(acc) > 1 else None, has_bias=sp.has_bias,
                              vocab=sp.d_in if sp.kind == EMBEDDING else 0,
                              path=b.DP_PATH_AUTO if paths is None else paths[k]))
    return b.LayerList(layers), accs


def gpu_norms_clip(ll, C):
    dev = ll.layers[0].G.device
    ws = b.alloc_workspace(ll)
    n = torch.full((ll.B,), float("nan"), dtype=torch.float32, device=dev)
    c = torch.empty(ll.B, dtype=torch.float32, device=dev)
    b.dp_per_example_sqnorms(ll, n, False, ws)
    b.dp_clip_factors(n, C, c)
    return n, c, ws


def rel_l2(x, ref):
    x = np.asarray(x, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(x - ref) / den) if den > 0 else float(np.linalg.norm(x))


def rel_max(x, ref):
    x = np.asarray(x, dtype=np.float64).ravel()
    ref = np.asarray(ref, dtype=np.float64).ravel()
    den = np.max(np.abs(ref))
    return float(np.max(np.abs(x - ref)) / den) if den > 0 else float(np.max(np.abs(x)))


def assert_update_close(theta_new, theta_old, ref_new, v_ref, tol=1e-4, ill_rel=1e-5):
    """The parameter update itself (theta_new - theta_old), element by element against the checker's, relative to
    the largest update with a floor from the fp32 rounding of theta.

    Algorithm 1 divides by sqrt(v_hat) + xi with xi = 1e-11.  Where the reference sqrt(v_hat) is itself within
    the fp32 resolution of the gradient (the noise sigma C z / N is O(sigma C / N) and is added to the sum in fp32,
    so g carries an absolute error near 1e-7 of that scale), the quotient m_hat / (sqrt(v_hat) + xi) of a
    first step is g / (|g| + xi): it swings from -1 to 1 over a range that fp32 cannot resolve.  Such elements
    (sqrt(v_ref) below `ill_rel` of its root mean square: about one in 10^5 draws) are only required to stay within
    twice the largest update; there must be few of them, and every other element meets the tight bound."""
    theta_new, theta_old, ref_new = (np.asarray(x, dtype=np.float64) for x in (theta_new, theta_old, ref_new))
    d, rd = theta_new - theta_old, ref_new - theta_old
    err = np.abs(d - rd)
    big = float(np.max(np.abs(rd)))
    bound = tol * big + 1e-7 * float(np.max(np.abs(theta_old)))
    root = np.sqrt(np.asarray(v_ref, dtype=np.float64))
    ill = root < ill_rel * np.sqrt(np.mean(root ** 2))
    assert ill.mean() <= 1e-3, f"{int(ill.sum())} of {ill.size} elements are ill-conditioned"
    assert np.all(err[~ill] <= bound), f"max update error {err[~ill].max():.3e} over bound {bound:.3e}"
    assert np.all(err[ill] <= 2.0 * big + bound)


def to_np(t):
    return t.detach().to("cpu").double().numpy()


def random_layers(specs, B, T, dtype, device, seed, g_scale=1.0, vocab_dup=None):
    """Small ad-hoc layer data on `device` (CPU generator, then moved): A ~ N(0,1), G ~ g_scale*N(0,1)*s_i."""
    g = torch.Generator().manual_seed(seed)
    s = torch.pow(10.0, torch.rand(B, generator=g) * 2 - 1).view(B, 1, 1)
    out = []
    for sp in specs:
        G = (torch.randn(B, T, sp.d_out, generator=g) * s * g_scale).to(dtype).to(device)
        if sp.kind == EMBEDDING:
            hi = sp.d_in if vocab_dup is None else min(sp.d_in, vocab_dup)
            ids = torch.randint(0, hi, (B, T), generator=g, dtype=torch.int32).to(device)
            out.append(LayerData(sp, G=G, ids=ids))
        else:
            A = torch.randn(B, T, sp.d_in, generator=g).to(dtype).to(device)
            out.append(LayerData(sp, G=G, A=A))
    return out


__all__ = ["O", "b", "np", "torch", "to_oracle_layers", "make_layer_list", "gpu_norms_clip", "rel_l2", "rel_max",
           "to_np", "assert_update_close", "random_layers", "acc_shapes", "LayerSpec", "LayerData", "LINEAR", "LAYERNORM", "EMBEDDING"]
