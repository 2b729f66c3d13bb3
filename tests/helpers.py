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
           "to_np", "random_layers", "acc_shapes", "LayerSpec", "LayerData", "LINEAR", "LAYERNORM", "EMBEDDING"]
