"""CPU oracle for the DP-SGD privatised-gradient step (test infrastructure only).

This module is the slow, plain, fp64 statement of what the step computes.  It
exists so that tests, the smoke check and the benchmark's CPU-baseline leg have
something obviously correct to compare the CUDA library against.  It is NOT
part of the product: the library never imports it, and it imports nothing from
the library.  Every per-example gradient is materialised explicitly; there is
no blocking, fusion or reordering beyond what the definitions state.

What follows the paper (Algorithm 1 and Sections 3, 4.3, 5.3):

* per-example gradient of a fully connected layer, grad_W = sum over tokens of
  x * (dL/ds)^T, i.e. A_i^T G_i for token inputs A_i and output-gradients G_i
  (Section 4.3; stored [d_in, d_out]);
* LayerNorm gain/bias gradients (Section 4.3) and the token-embedding gradient
  (Section 4.3, last paragraph), both as plain sums over tokens;
* clip(g, C) = g * min(1, C / ||g||_2) over the WHOLE per-example gradient
  (Algorithm 1, the g_t line; the operator is the standard DP-SGD one the
  paper cites, since the paper does not spell it out);
* g_t = (N(0, sigma^2 C^2 I) + sum_j clip(grad_j, C)) / |B_t| (Algorithm 1),
  with the sum taken over every microbatch of the macro-batch (Section 5.3);
* the Adam recurrences with bias correction and the decoupled weight-decay
  update theta <- theta - eta * (m_hat / (sqrt(v_hat) + xi) + lambda * theta),
  xi = 1e-11 (Algorithm 1).

The Gaussian draw is a construction the paper leaves open; it is fixed here as
Philox4x32-10 (Salmon et al., SC'11) keyed by (seed, step, element) followed by
the Box-Muller transform, with the uniforms formed in IEEE binary32 so that a
GPU can reproduce the same uniforms bit for bit and the transcendental part
evaluated in fp64.

A table shared by the embedding and the output projection (BERT's masked-LM
head) is clipped by the norm of its summed gradient (shared_table_*).

Pins (tests/test_oracle_pins.py): C -> infinity equals the batch GEMM; every
clipped contribution has norm <= C; Gram-identity norm equals brute force on
tiny inputs; rank-one closed form; Philox known-answer vectors and an
independent library generator; normal moments; AdamW closed forms.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

LINEAR = "linear"
LAYERNORM = "layernorm"
EMBEDDING = "embedding"


@dataclass
class OracleLayer:
    """One trainable layer's per-token tensors for a microbatch of B examples.

    kind       LINEAR, LAYERNORM or EMBEDDING.
    G          [B, T, d_out] float64: gradient of the per-example (un-averaged)
               loss with respect to the layer output, per token.
    A          LINEAR: [B, T, d_in] layer input.  LAYERNORM: [B, T, d] the
               normalised input x_hat.  EMBEDDING: None.
    ids        EMBEDDING only: [B, T] integer token ids in [0, vocab).
    has_bias   LINEAR only: whether a bias vector [d_out] is trained.
    vocab      EMBEDDING only: number of rows V of the table.
    """

    kind: str
    G: np.ndarray
    A: Optional[np.ndarray] = None
    ids: Optional[np.ndarray] = None
    has_bias: bool = False
    vocab: int = 0

    @property
    def B(self) -> int:
        return int(self.G.shape[0])


# ---------------------------------------------------------------------------
# Per-example gradients (Section 4.3) -- explicit materialisation
# ---------------------------------------------------------------------------

def per_example_gradient(layer: OracleLayer, i: int) -> List[np.ndarray]:
    """Gradient tensors of example i for one layer, each fully materialised.

    LINEAR    [A_i^T G_i  (d_in x d_out)] and, with a bias, [sum_t G_i[t, :]].
    LAYERNORM [sum_t x_hat_i[t, :] * G_i[t, :]] (gain) and [sum_t G_i[t, :]] (bias).
    EMBEDDING a dense [V, d] table of zeros with G_i[t, :] added to row ids_i[t].
    """
    G = np.asarray(layer.G[i], dtype=np.float64)
    if layer.kind == LINEAR:
        A = np.asarray(layer.A[i], dtype=np.float64)
        out = [A.T @ G]
        if layer.has_bias:
            out.append(G.sum(axis=0))
        return out
    if layer.kind == LAYERNORM:
        X = np.asarray(layer.A[i], dtype=np.float64)
        return [(X * G).sum(axis=0), G.sum(axis=0)]
    if layer.kind == EMBEDDING:
        table = np.zeros((layer.vocab, G.shape[1]), dtype=np.float64)
        for t in range(G.shape[0]):
            table[int(layer.ids[i, t]), :] += G[t, :]
        return [table]
    raise ValueError(f"unknown layer kind {layer.kind!r}")


def per_example_sqnorms(layers: Sequence[OracleLayer]) -> np.ndarray:
    """n_i = squared L2 norm of example i's whole flat gradient (all layers)."""
    B = layers[0].B
    n = np.zeros(B, dtype=np.float64)
    for i in range(B):
        total = 0.0
        for layer in layers:
            for g in per_example_gradient(layer, i):
                total += float(np.sum(g * g))
        n[i] = total
    return n


# ---------------------------------------------------------------------------
# A table shared by the token embedding and the output projection
# ---------------------------------------------------------------------------
# The paper trains BERT-Large (Section 4) and does not restate its architecture;
# in that model the masked-LM output projection reuses the word-piece table E
# of Section 4.3's embeddings: logits[s, v] = <h[s, :], E[v, :]>.  Example i's
# gradient for E is then ONE tensor, the sum of the embedding's scatter and of
# the projection's dlogits_i^T h_i, and Algorithm 1 clips by the norm of that
# sum, not by the two parts' norms added up.

def shared_table_gradient(emb: OracleLayer, proj: OracleLayer, i: int) -> np.ndarray:
    """[V, d] gradient of example i for a table used by both layers.

    emb   EMBEDDING layer (ids [B, T], G [B, T, d]).
    proj  LINEAR layer without bias whose A is dlogits [B, T_out, V] and whose
          G is the projection's input h [B, T_out, d], so that its A_i^T G_i is
          the [V, d] gradient of the table.
    """
    scatter = per_example_gradient(emb, i)[0]
    dense = per_example_gradient(proj, i)[0]
    assert scatter.shape == dense.shape
    return scatter + dense


def shared_table_cross_terms(emb: OracleLayer, proj: OracleLayer) -> np.ndarray:
    """x_i = <scatter_i, dense_i> (sum of elementwise products of the two
    materialised [V, d] parts): ||scatter_i + dense_i||^2 exceeds the two
    parts' squared norms by 2 x_i."""
    B = emb.B
    x = np.zeros(B, dtype=np.float64)
    for i in range(B):
        scatter = per_example_gradient(emb, i)[0]
        dense = per_example_gradient(proj, i)[0]
        x[i] = float(np.sum(scatter * dense))
    return x


def per_example_sqnorms_shared_table(layers: Sequence[OracleLayer], emb_index: int, proj_index: int) -> np.ndarray:
    """n_i over all layers when layers[emb_index] and layers[proj_index] train
    the same table: every other layer as in per_example_sqnorms, the shared
    table once, by the norm of its summed gradient."""
    B = layers[0].B
    n = np.zeros(B, dtype=np.float64)
    for i in range(B):
        total = 0.0
        for k, layer in enumerate(layers):
            if k in (emb_index, proj_index):
                continue
            for g in per_example_gradient(layer, i):
                total += float(np.sum(g * g))
        g = shared_table_gradient(layers[emb_index], layers[proj_index], i)
        total += float(np.sum(g * g))
        n[i] = total
    return n


def clip_factors(sqnorm: np.ndarray, C: float) -> np.ndarray:
    """c_i = min(1, C / sqrt(n_i)); an all-zero gradient is left unscaled."""
    n = np.asarray(sqnorm, dtype=np.float64)
    c = np.ones_like(n)
    nz = n > 0.0
    c[nz] = np.minimum(1.0, float(C) / np.sqrt(n[nz]))
    return c


def zero_accumulators(layers: Sequence[OracleLayer]) -> List[List[np.ndarray]]:
    """Accumulators shaped like each layer's gradient tensors, all zero."""
    accs = []
    for layer in layers:
        d_out = layer.G.shape[2]
        if layer.kind == LINEAR:
            a = [np.zeros((layer.A.shape[2], d_out))]
            if layer.has_bias:
                a.append(np.zeros(d_out))
        elif layer.kind == LAYERNORM:
            a = [np.zeros(d_out), np.zeros(d_out)]
        else:
            a = [np.zeros((layer.vocab, d_out))]
        accs.append(a)
    return accs


def clipped_accumulate(layers: Sequence[OracleLayer], clip: np.ndarray,
                       accs: List[List[np.ndarray]]) -> List[List[np.ndarray]]:
    """accs += sum_i c_i * g_i, example by example in index order (in place)."""
    B = layers[0].B
    for i in range(B):
        for layer, acc in zip(layers, accs):
            for dst, g in zip(acc, per_example_gradient(layer, i)):
                dst += float(clip[i]) * g
    return accs


# ---------------------------------------------------------------------------
# Philox4x32-10 and the normal draw (the noise term of Algorithm 1)
# ---------------------------------------------------------------------------

_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = np.uint64(0x9E3779B9)
_PHILOX_W1 = np.uint64(0xBB67AE85)
_MASK32 = np.uint64(0xFFFFFFFF)
_SH32 = np.uint64(32)


def philox4x32_10(counter: np.ndarray, key: Sequence[int]) -> np.ndarray:
    """Ten rounds of the Philox-4x32 bijection.

    counter  [..., 4] array of 32-bit words (c0, c1, c2, c3).
    key      two 32-bit words (k0, k1).
    Each round: (hi0, lo0) = M0 * c0, (hi1, lo1) = M1 * c2, then
    c <- (hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0); the key is bumped by the
    Weyl constants (W0, W1) between rounds.  Returns uint32 words [..., 4].
    """
    c = np.asarray(counter).astype(np.uint64) & _MASK32
    c0, c1, c2, c3 = c[..., 0], c[..., 1], c[..., 2], c[..., 3]
    k0 = np.uint64(int(key[0]) & 0xFFFFFFFF)
    k1 = np.uint64(int(key[1]) & 0xFFFFFFFF)
    for _ in range(10):
        p0 = _PHILOX_M0 * c0
        p1 = _PHILOX_M1 * c2
        hi0, lo0 = p0 >> _SH32, p0 & _MASK32
        hi1, lo1 = p1 >> _SH32, p1 & _MASK32
        c0, c1, c2, c3 = hi1 ^ c1 ^ k0, lo1, hi0 ^ c3 ^ k1, lo0
        k0 = (k0 + _PHILOX_W0) & _MASK32
        k1 = (k1 + _PHILOX_W1) & _MASK32
    return np.stack([c0, c1, c2, c3], axis=-1).astype(np.uint32)


def _blocks_for_elements(first_elem: int, n: int, seed: int, step: int) -> np.ndarray:
    """Philox output words for the blocks covering elements [first, first+n).

    Element e lives in block j = e >> 2 at lane e & 3.  The counter of block j
    is (lo32(j), hi32(j), lo32(step), hi32(step)); the key is
    (lo32(seed), hi32(seed)).  Returns (first_block, words[n_blocks, 4]).
    """
    j0 = first_elem >> 2
    j1 = (first_elem + n + 3) >> 2
    j = np.arange(j0, j1, dtype=np.uint64)
    ctr = np.empty((j.size, 4), dtype=np.uint64)
    ctr[:, 0] = j & _MASK32
    ctr[:, 1] = j >> _SH32
    ctr[:, 2] = np.uint64(step & 0xFFFFFFFF)
    ctr[:, 3] = np.uint64((step >> 32) & 0xFFFFFFFF)
    words = philox4x32_10(ctr, (seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF))
    return j0, words


def philox_u32(n: int, elem_offset: int, seed: int, step: int) -> np.ndarray:
    """The raw 32-bit word attached to each of n elements from elem_offset on."""
    if n == 0:
        return np.zeros(0, dtype=np.uint32)
    j0, words = _blocks_for_elements(elem_offset, n, seed, step)
    flat = words.reshape(-1)
    lo = elem_offset - 4 * j0
    return flat[lo:lo + n].copy()


def standard_normals(n: int, elem_offset: int, seed: int, step: int) -> np.ndarray:
    """z_e ~ N(0, 1) for elements e = elem_offset .. elem_offset + n - 1.

    Box-Muller on the word pairs (x0, x1) and (x2, x3) of each block:
      u1 = fl32(fl32(x_a) * 2^-32 + 2^-33)  in (0, 1],
      u2 = fl32(fl32(x_b) * 2^-32)          in [0, 1],
      r = sqrt(-2 ln u1), z_even = r cos(2 pi u2), z_odd = r sin(2 pi u2).
    The uniforms are rounded exactly as binary32 arithmetic rounds them; the
    logarithm, root and trigonometry are fp64.
    """
    if n == 0:
        return np.zeros(0, dtype=np.float64)
    j0, words = _blocks_for_elements(elem_offset, n, seed, step)
    xa = words[:, 0::2].astype(np.float32)          # x0, x2 (uint32 -> binary32, RN)
    xb = words[:, 1::2].astype(np.float32)          # x1, x3
    u1 = (xa * np.float32(2.0 ** -32) + np.float32(2.0 ** -33)).astype(np.float32)
    u2 = (xb * np.float32(2.0 ** -32)).astype(np.float32)
    r = np.sqrt(-2.0 * np.log(u1.astype(np.float64)))
    ang = 2.0 * np.pi * u2.astype(np.float64)
    z = np.empty(words.shape, dtype=np.float64)
    z[:, 0::2] = r * np.cos(ang)
    z[:, 1::2] = r * np.sin(ang)
    flat = z.reshape(-1)
    lo = elem_offset - 4 * j0
    return flat[lo:lo + n].copy()


def add_noise_and_scale(acc: np.ndarray, sigma: float, C: float, batch_size: int,
                        seed: int, step: int, elem_offset: int = 0) -> np.ndarray:
    """g = (acc + sigma * C * z) / batch_size over the flattened tensor."""
    S = np.asarray(acc, dtype=np.float64)
    z = standard_normals(S.size, elem_offset, seed, step).reshape(S.shape)
    return (S + float(sigma) * float(C) * z) / float(batch_size)


# ---------------------------------------------------------------------------
# Adam with decoupled weight decay (Algorithm 1)
# ---------------------------------------------------------------------------

def adamw_step(theta: np.ndarray, m: np.ndarray, v: np.ndarray, g: np.ndarray,
               lr: float, beta1: float, beta2: float, xi: float,
               weight_decay: float, t: int):
    """One update of (theta, m, v) at step t >= 1; returns new arrays."""
    theta = np.asarray(theta, dtype=np.float64)
    g = np.asarray(g, dtype=np.float64)
    m_new = beta1 * np.asarray(m, dtype=np.float64) + (1.0 - beta1) * g
    v_new = beta2 * np.asarray(v, dtype=np.float64) + (1.0 - beta2) * g * g
    m_hat = m_new / (1.0 - beta1 ** t)
    v_hat = v_new / (1.0 - beta2 ** t)
    theta_new = theta - lr * (m_hat / (np.sqrt(v_hat) + xi) + weight_decay * theta)
    return theta_new, m_new, v_new


# ---------------------------------------------------------------------------
# The whole step (Algorithm 1 with Section 5.3's accumulation)
# ---------------------------------------------------------------------------

def privatised_gradient(microbatches: Sequence[Sequence[OracleLayer]], C: float,
                        sigma: float, seed: int, step: int,
                        elem_offsets: Optional[Sequence[Sequence[int]]] = None):
    """Noisy mean gradient of one macro-batch.

    microbatches  a list of microbatches, each a list of layers with identical
                  structure; N = sum of their B is the divisor |B_t|.
    elem_offsets  per layer, per gradient tensor, the index of that tensor's
                  first element in the caller's flat parameter ordering (it
                  selects the Philox block); default: tensors laid end to end.
    Returns (g, clip) with g shaped like zero_accumulators() and clip the list
    of per-microbatch clip-factor vectors.
    """
    accs = zero_accumulators(microbatches[0])
    clips = []
    N = 0
    for layers in microbatches:
        c = clip_factors(per_example_sqnorms(layers), C)
        clipped_accumulate(layers, c, accs)
        clips.append(c)
        N += layers[0].B
    if elem_offsets is None:
        elem_offsets, pos = [], 0
        for acc in accs:
            offs = []
            for a in acc:
                offs.append(pos)
                pos += a.size
            elem_offsets.append(offs)
    g = [[add_noise_and_scale(a, sigma, C, N, seed, step, off)
          for a, off in zip(acc, offs)] for acc, offs in zip(accs, elem_offsets)]
    return g, clips


# ---------------------------------------------------------------------------
# Diagnostics of Section 5.2.1: gradient-SNR and clipping statistics
# ---------------------------------------------------------------------------

def gradient_snr_sums(acc: np.ndarray, sigma: float, C: float, seed: int, step: int, elem_offset: int = 0):
    """(sum acc^2, sum (sigma C z)^2) over one tensor; gradient-SNR of a macro-batch is the root of the ratio
    of the two sums taken over ALL tensors: ||aggregated clipped gradient|| / ||noise vector||."""
    S = np.asarray(acc, dtype=np.float64).ravel()
    z = standard_normals(S.size, elem_offset, seed, step)
    return float(np.sum(S * S)), float(np.sum((float(sigma) * float(C) * z) ** 2))


def clip_stats(clip: np.ndarray):
    """(fraction of examples that were clipped, mean clip factor)."""
    c = np.asarray(clip, dtype=np.float64)
    return float(np.mean(c < 1.0)), float(np.mean(c))
