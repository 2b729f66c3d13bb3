"""Seeded synthetic inputs with the shapes of BERT pretraining under DP-SGD.

This module only draws inputs (layer inputs A, output-gradients G, token ids,
initial weights).  It contains none of the step's arithmetic, so both the CUDA
library's callers and the CPU checker may be fed from it.

The shapes follow the paper's workload (Section 4: BERT-Large, 24 blocks,
hidden 1024, 128 tokens per example, ~32K word-pieces; Section 5.3: 2M-example
mega-batches built from microbatches).  The corpus itself is not used: values
are Gaussian, token ids follow a truncated Zipf law.

Scaling of G.  With A, G ~ N(0, 1) every per-example gradient norm is in the
tens of thousands, so every example would clip at C = 1.  To exercise both
branches of the clip, G of example i is N(0, 1) * s_i / kappa, with s_i
log-uniform in [0.1, 10] and kappa the root of the expected squared norm of a
unit-scale example, so that the per-example norm is close to s_i.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch

LINEAR, LAYERNORM, EMBEDDING = "linear", "layernorm", "embedding"


@dataclass
class LayerSpec:
    kind: str
    d_in: int           # LINEAR: input width; LAYERNORM: d; EMBEDDING: vocab V
    d_out: int
    has_bias: bool = False
    name: str = ""
    ids: str = "zipf"   # EMBEDDING: "zipf" word-pieces, "position" 0..T-1, "segment" two sentence segments

    def n_params(self) -> int:
        if self.kind == LINEAR:
            return self.d_in * self.d_out + (self.d_out if self.has_bias else 0)
        if self.kind == LAYERNORM:
            return 2 * self.d_out
        return self.d_in * self.d_out


@dataclass
class LayerData:
    spec: LayerSpec
    G: torch.Tensor                       # [B, T, d_out]
    A: Optional[torch.Tensor] = None      # [B, T, d_in]  (None for EMBEDDING)
    ids: Optional[torch.Tensor] = None    # [B, T] int32  (EMBEDDING only)


@dataclass
class Workload:
    name: str
    B: int
    T: int
    dtype: torch.dtype
    specs: List[LayerSpec]
    C: float = 1.0
    sigma: float = 1.0
    lr: float = 6.0902e-4
    beta1: float = 0.9
    beta2: float = 0.999
    xi: float = 1e-11
    weight_decay: float = 0.5
    scaled_G: bool = True
    microbatches: int = 1
    extra: dict = field(default_factory=dict)

    def n_params(self) -> int:
        return sum(s.n_params() for s in self.specs)


def encoder_layer_specs(hidden: int, ffn: int, tag: str = "") -> List[LayerSpec]:
    """Trainables of one transformer encoder block: QKV, attention output,
    the two FFN linears (all with biases) and two LayerNorms."""
    return [
        LayerSpec(LINEAR, hidden, 3 * hidden, True, f"{tag}qkv"),
        LayerSpec(LINEAR, hidden, hidden, True, f"{tag}attn_out"),
        LayerSpec(LAYERNORM, hidden, hidden, False, f"{tag}ln1"),
        LayerSpec(LINEAR, hidden, ffn, True, f"{tag}ffn1"),
        LayerSpec(LINEAR, ffn, hidden, True, f"{tag}ffn2"),
        LayerSpec(LAYERNORM, hidden, hidden, False, f"{tag}ln2"),
    ]


def workload(name: str) -> Workload:
    """The five named workloads (small linear layer; BERT-Base block;
    BERT-Large stack with token embedding; mega-batch accumulation; T=512)."""
    if name == "tiny_linear":
        return Workload(name, 32, 16, torch.float32, [LayerSpec(LINEAR, 64, 64, True, "fc")],
                        C=1.0, sigma=1.1, lr=1e-3, beta1=0.9, beta2=0.999, weight_decay=0.01,
                        scaled_G=False)
    if name == "bert_base_layer":
        return Workload(name, 256, 128, torch.bfloat16, encoder_layer_specs(768, 3072))
    if name in ("bert_large", "bert_large_megabatch"):
        specs = []
        for l in range(24):
            specs += encoder_layer_specs(1024, 4096, f"l{l}.")
        specs.append(LayerSpec(EMBEDDING, 30522, 1024, False, "tok_emb"))
        mb = 8192 if name == "bert_large_megabatch" else 1
        return Workload(name, 256, 128, torch.bfloat16, specs, microbatches=mb)
    if name == "bert_large_embeddings":
        # the input layer of BERT: word-piece, positional and token-type embeddings summed, then LayerNorm
        specs = [LayerSpec(EMBEDDING, 30522, 1024, False, "tok_emb", "zipf"),
                 LayerSpec(EMBEDDING, 512, 1024, False, "pos_emb", "position"),
                 LayerSpec(EMBEDDING, 2, 1024, False, "type_emb", "segment"),
                 LayerSpec(LAYERNORM, 1024, 1024, False, "emb_ln")]
        return Workload(name, 256, 128, torch.bfloat16, specs)
    if name == "bert_large_layer_t512":
        return Workload(name, 64, 512, torch.bfloat16, encoder_layer_specs(1024, 4096))
    raise KeyError(name)


def kappa(specs: List[LayerSpec], T: int) -> float:
    """Root of the expected squared gradient norm of one example whose A and G
    are unit Gaussians (embedding rows counted as if ids were distinct)."""
    s = 0.0
    for sp in specs:
        if sp.kind == LINEAR:
            s += T * sp.d_out * (sp.d_in + (1 if sp.has_bias else 0))
        elif sp.kind == LAYERNORM:
            s += 2 * T * sp.d_out
        else:
            s += T * sp.d_out
    return math.sqrt(s)


def _gen(device, *key) -> torch.Generator:
    g = torch.Generator(device=device)
    h = 0x9E3779B97F4A7C15
    for k in key:
        h = (h * 6364136223846793005 + int(k) + 1442695040888963407) & 0x7FFFFFFFFFFFFFFF
    g.manual_seed(h)
    return g


def zipf_ids(B: int, T: int, vocab: int, exponent: float, gen: torch.Generator, device) -> torch.Tensor:
    """Token ids with P(id = k) proportional to (k + 1)^-exponent, 0 <= k < vocab,
    drawn by inverse CDF on an fp64 cumulative table."""
    w = torch.arange(1, vocab + 1, dtype=torch.float64, device=device).pow(-exponent)
    cdf = torch.cumsum(w, 0)
    cdf = cdf / cdf[-1]
    u = torch.rand(B * T, generator=gen, device=device, dtype=torch.float64)
    ids = torch.searchsorted(cdf, u).clamp_(max=vocab - 1)
    return ids.to(torch.int32).reshape(B, T)


def example_scales(B: int, seed: int, microbatch: int, device) -> torch.Tensor:
    """s_i = 10^U(-1, 1), one per example."""
    g = _gen(device, seed, microbatch, 999_983)
    return torch.pow(10.0, torch.rand(B, generator=g, device=device, dtype=torch.float32) * 2.0 - 1.0)


def generate(wl: Workload, seed: int = 0, device="cpu", microbatch: int = 0,
             B: Optional[int] = None, specs: Optional[List[LayerSpec]] = None) -> List[LayerData]:
    """Draw one microbatch of inputs for every layer of the workload.

    Each tensor has its own stream keyed by (seed, microbatch, layer index,
    tensor id), so a subset of layers reproduces the same bytes.  `specs`
    selects layers by identity from wl.specs (default: all)."""
    B = wl.B if B is None else B
    T = wl.T
    if wl.name == "tiny_linear":
        rng = np.random.default_rng(seed)
        A = torch.from_numpy(rng.standard_normal((B, T, 64), dtype=np.float32)).to(device)
        G = torch.from_numpy(rng.standard_normal((B, T, 64), dtype=np.float32)).to(device)
        return [LayerData(wl.specs[0], G=G, A=A)]
    kap = kappa(wl.specs, T)
    s = example_scales(B, seed, microbatch, device) / kap if wl.scaled_G else None
    out = []
    for li, sp in enumerate(wl.specs):
        if specs is not None and not any(sp is q for q in specs):
            continue
        gG = _gen(device, seed, microbatch, li, 1)
        G = torch.randn(B, T, sp.d_out, generator=gG, device=device, dtype=torch.float32)
        if s is not None:
            G = G * s.view(B, 1, 1)
        G = G.to(wl.dtype)
        if sp.kind == EMBEDDING:
            gi = _gen(device, seed, microbatch, li, 2)
            if sp.ids == "position":
                ids = torch.arange(T, dtype=torch.int32, device=device).repeat(B, 1)
            elif sp.ids == "segment":      # sentence A then sentence B, split point drawn per example
                cut = torch.randint(1, max(T, 2), (B, 1), generator=gi, device=device)
                ids = (torch.arange(T, device=device).view(1, T) >= cut).to(torch.int32)
            else:
                ids = zipf_ids(B, T, sp.d_in, 1.1, gi, device)
            out.append(LayerData(sp, G=G, ids=ids.contiguous()))
        else:
            gA = _gen(device, seed, microbatch, li, 0)
            A = torch.randn(B, T, sp.d_in, generator=gA, device=device, dtype=torch.float32).to(wl.dtype)
            out.append(LayerData(sp, G=G, A=A))
    return out


def initial_weights(n: int, seed: int, device, std: float = 0.02) -> torch.Tensor:
    """theta_0 ~ N(0, std^2), fp32."""
    g = _gen(device, seed, 424_243)
    return torch.randn(n, generator=g, device=device, dtype=torch.float32) * std
