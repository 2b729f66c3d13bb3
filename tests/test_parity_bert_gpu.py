"""GPU parity at BERT shapes: a BERT-Base block in full, the 24-layer BERT-Large stack with its Zipf token
embedding (checker on an 8-example subset plus sampled accumulator entries at the full launch size), the
T=512 crossover layer under all three path settings, and the mega-batch accumulation invariants."""
import numpy as np
import pytest
import torch

from paper_2108_01624_b200 import DPStep, synth

from .helpers import (LAYERNORM, LINEAR, O, assert_update_close, b, gpu_norms_clip, make_layer_list, rel_l2, to_np,
                      to_oracle_layers)

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = "cuda:0"
CLIP_TOL = 1e-3
BF16_TOL = 2e-2


def _subset(data, rows):
    return [synth.LayerData(ld.spec, G=ld.G[rows].contiguous(), A=None if ld.A is None else ld.A[rows].contiguous(),
                            ids=None if ld.ids is None else ld.ids[rows].contiguous()) for ld in data]


ENTRY_TOL = 0.01      # of the root-sum-square of an entry's terms; see _tile_sampled_check


def _tile_sampled_check(data, accs, clips, seed, counts=None, bias_layers=3):
    """The clipped sum at the full launch size, one sampled entry for EVERY 128 x 128 block of every linear layer's
    accumulator (eight per 256 x 512 tile of the accumulate GEMM: each CTA of a pair, each half of its accumulator,
    each 128-column group), recomputed in fp64 on the host from columns gathered on the device:
        acc_w[p, q] = sum over the microbatches of  sum_r clip[r / T] A[r, p] G[r, q].
    `data`, `clips`: one entry per distinct microbatch, `counts[k]` = how often microbatch k was accumulated.
    Bound per entry: 1 % of the root-sum-square of its terms.  The bf16 rounding of clip * G (relative 2^-9 per term,
    independent) puts the error near 0.1 % of that scale; a dropped or unscaled 64-token stage is 1 / 512 of the
    terms, about 4 % of it, and a dropped tile or a misplaced block is of order 100 %.
    Every bias element of `bias_layers` layers is checked the same way."""
    rng = np.random.default_rng(seed)
    counts = [1] * len(data) if counts is None else counts
    lin = [k for k, ld in enumerate(data[0]) if ld.spec.kind == LINEAR]
    n_entries = 0
    for k in lin:
        sp = data[0][k].spec
        nb_in, nb_out = (sp.d_in + 127) // 128, (sp.d_out + 127) // 128
        ps = np.array([min(sp.d_in - 1, bi * 128 + int(rng.integers(128))) for bi in range(nb_in) for _ in range(nb_out)])
        qs = np.array([min(sp.d_out - 1, bo * 128 + int(rng.integers(128))) for _ in range(nb_in) for bo in range(nb_out)])
        ref = np.zeros(len(ps))
        sq = np.zeros(len(ps))
        for mb, clip, cnt in zip(data, clips, counts):
            ld = mb[k]
            B, T, _ = ld.G.shape
            w = np.repeat(to_np(clip), T)
            a = to_np(ld.A.reshape(B * T, -1)[:, torch.from_numpy(ps).to(ld.A.device)])       # [B T, n]
            g = to_np(ld.G.reshape(B * T, -1)[:, torch.from_numpy(qs).to(ld.G.device)])
            terms = a * g * w[:, None]
            ref += cnt * terms.sum(0)
            sq += cnt * cnt * (terms ** 2).sum(0)
        got = to_np(accs[k][0][torch.from_numpy(ps).to(DEV), torch.from_numpy(qs).to(DEV)])
        err = np.abs(got - ref)
        bound = ENTRY_TOL * np.sqrt(sq) + 1e-30
        worst = int(np.argmax(err / bound))
        assert np.all(err <= bound), (f"{sp.name}: entry ({ps[worst]}, {qs[worst]}) off by {err[worst]:.3e}, "
                                      f"bound {bound[worst]:.3e}")
        n_entries += len(ps)
    with_bias = [k for k in lin if data[0][k].spec.has_bias]
    for k in rng.choice(with_bias, size=min(bias_layers, len(with_bias)), replace=False):
        k = int(k)
        ref = np.zeros(data[0][k].spec.d_out)
        sq = np.zeros_like(ref)
        for mb, clip, cnt in zip(data, clips, counts):
            G = to_np(mb[k].G) * to_np(clip)[:, None, None]
            ref += cnt * G.sum((0, 1))
            sq += cnt * cnt * (G ** 2).sum((0, 1))
        err = np.abs(to_np(accs[k][1]) - ref)
        assert np.all(err <= 1e-3 * np.sqrt(sq) + 1e-30), data[0][k].spec.name      # fp32 sums of exact products
    return n_entries


def _sampled_entries_check(data, accs, clip, seed):
    return _tile_sampled_check([data], accs, [clip], seed)


def _full_size_ln_and_embedding_check(data, accs, clip, n_ln, seed):
    """At the full launch size: a few LayerNorm layers (every element of gain and bias sums) and the embedding
    (every row) recomputed in fp64 on the host with the GPU's clip factors."""
    rng = np.random.default_rng(seed)
    c = to_np(clip)
    ln_idx = [k for k, ld in enumerate(data) if ld.spec.kind == LAYERNORM]
    for k in rng.choice(ln_idx, size=min(n_ln, len(ln_idx)), replace=False):
        ld, acc = data[int(k)], accs[int(k)]
        G, X = to_np(ld.G), to_np(ld.A)
        gain = np.einsum("i,itd->d", c, X * G)
        bias = np.einsum("i,itd->d", c, G)
        assert rel_l2(to_np(acc[0]), gain) <= 1e-3 and rel_l2(to_np(acc[1]), bias) <= 1e-3, ld.spec.name
    for ld, acc in zip(data, accs):
        if ld.spec.kind != synth.EMBEDDING:
            continue
        G = to_np(ld.G) * c[:, None, None]
        ref = np.zeros((ld.spec.d_in, ld.spec.d_out))
        np.add.at(ref, ld.ids.cpu().numpy().reshape(-1), G.reshape(-1, ld.spec.d_out))
        assert rel_l2(to_np(acc[0]), ref) <= 1e-3, ld.spec.name
        untouched = np.setdiff1d(np.arange(ld.spec.d_in), ld.ids.cpu().numpy().reshape(-1))
        assert float(acc[0][torch.from_numpy(untouched).to(acc[0].device)].abs().max()) == 0.0


def test_bert_base_block_full_batch():
    wl = synth.workload("bert_base_layer")
    data = synth.generate(wl, seed=0, device=DEV)
    ll, accs = make_layer_list(data, DEV)
    n, c, ws = gpu_norms_clip(ll, wl.C)
    b.dp_clipped_accumulate(ll, c, ws)
    assert b.dp_poll_status() == 0
    ol = to_oracle_layers(data)
    n_ref = O.per_example_sqnorms(ol)
    c_ref = O.clip_factors(n_ref, wl.C)
    frac = float(np.mean(c_ref < 1.0))
    assert 0.2 < frac < 0.8                      # the input recipe makes some examples clip and some not
    np.testing.assert_allclose(to_np(c), c_ref, rtol=CLIP_TOL)
    np.testing.assert_allclose(to_np(n), n_ref, rtol=2 * CLIP_TOL)
    ref = O.clipped_accumulate(ol, c_ref, O.zero_accumulators(ol))
    for ld, acc, racc in zip(data, accs, ref):
        for x, y in zip(acc, racc):
            assert rel_l2(to_np(x), y) <= BF16_TOL, ld.spec.name
    # every clipped contribution is bounded by C: ||sum|| <= (number of examples) * C
    tot = np.sqrt(sum(float((x.double() ** 2).sum()) for acc in accs for x in acc))
    assert tot <= wl.B * wl.C * (1 + 1e-3)


@pytest.mark.parametrize("n_layers", [24])
def test_bert_large_stack_subset_and_samples(n_layers):
    wl = synth.workload("bert_large")
    specs = wl.specs[:6 * n_layers] + [wl.specs[-1]]
    data = synth.generate(wl, seed=0, device=DEV, specs=specs)
    assert len(data) == 6 * n_layers + 1
    ll, accs = make_layer_list(data, DEV)
    # the call sequence bench.py times: the model in two lists (linear layers; LayerNorm + embedding), each with
    # its own workspace, the second accumulate reusing the column sums of its norm call
    lin = b.LayerList([l for l in ll.layers if l.kind == "linear"])
    rest = b.LayerList([l for l in ll.layers if l.kind != "linear"])
    ws, ws_rest = b.alloc_workspace(lin), b.alloc_workspace(rest)
    n = torch.empty(wl.B, dtype=torch.float32, device=DEV)
    c = torch.empty(wl.B, dtype=torch.float32, device=DEV)
    b.dp_per_example_sqnorms(lin, n, False, ws)
    b.dp_per_example_sqnorms(rest, n, True, ws_rest)
    b.dp_clip_factors(n, wl.C, c)
    b.dp_clipped_accumulate(lin, c, ws)
    b.dp_clipped_accumulate_after_sqnorms(rest, c, ws_rest)
    torch.cuda.synchronize()
    assert b.dp_poll_status() == 0
    # (a) checker on eight examples spread over the batch (first, last, and both sides of the half-way and
    # quarter marks, where an indexing slip would show), all layers and the embedding
    rows = [0, 1, 63, 64, 127, 128, 254, 255]
    sub = _subset(data, rows)
    ol = to_oracle_layers(sub)
    n_ref = O.per_example_sqnorms(ol)
    c_ref = O.clip_factors(n_ref, wl.C)
    np.testing.assert_allclose(to_np(n[rows]), n_ref, rtol=2 * CLIP_TOL)
    np.testing.assert_allclose(to_np(c[rows]), c_ref, rtol=CLIP_TOL)
    # (b) full launch size: sampled accumulator entries in fp64
    n_entries = _sampled_entries_check(data, accs, c, seed=1)
    assert n_entries == 24 * (8 * 24 + 8 * 8 + 8 * 32 + 32 * 8)       # every 128 x 128 block of all 96 linear layers
    _full_size_ln_and_embedding_check(data, accs, c, n_ln=3, seed=2)
    # (b') all 256 norms of the linear layers: the Gram kernel against the materialised-tile kernel, two different
    # algorithms for the same quantity (the identity of Section 4.3 holds at any size)
    n_gram = torch.empty(wl.B, dtype=torch.float32, device=DEV)
    b.dp_per_example_sqnorms(lin, n_gram, False, ws)
    lin_mat = b.LayerList([b.Layer(kind=l.kind, G=l.G, A=l.A, ids=None, acc_w=l.acc_w, acc_b=l.acc_b, has_bias=l.has_bias,
                                   vocab=0, path=b.DP_PATH_MATERIALIZED) for l in lin.layers])
    n_mat = torch.empty(wl.B, dtype=torch.float32, device=DEV)
    b.dp_per_example_sqnorms(lin_mat, n_mat, False, b.alloc_workspace(lin_mat))
    assert b.dp_poll_status() == 0
    np.testing.assert_allclose(to_np(n_gram), to_np(n_mat), rtol=2 * CLIP_TOL)
    # (c) the same eight examples as a microbatch of their own through the GPU path, element by element
    ll8, acc8 = make_layer_list(sub, DEV)
    n8, c8, ws8 = gpu_norms_clip(ll8, wl.C)
    b.dp_clipped_accumulate(ll8, c8, ws8)
    np.testing.assert_allclose(to_np(c8), c_ref, rtol=CLIP_TOL)
    ref = O.clipped_accumulate(ol, c_ref, O.zero_accumulators(ol))
    for ld, acc, racc in zip(sub, acc8, ref):
        for x, y in zip(acc, racc):
            assert rel_l2(to_np(x), y) <= BF16_TOL, ld.spec.name
    # embedding ids follow the Zipf recipe: id 0 is the most frequent by far
    ids = data[-1].ids
    assert float((ids == 0).float().mean()) > 0.10


def test_long_sequence_crossover_all_paths():
    wl = synth.workload("bert_large_layer_t512")
    data = synth.generate(wl, seed=0, device=DEV)
    sub = _subset(data, slice(0, 4))
    ol = to_oracle_layers(sub)
    n_ref = O.per_example_sqnorms(ol)
    c_ref = O.clip_factors(n_ref, wl.C)
    norms = {}
    for path in (b.DP_PATH_AUTO, b.DP_PATH_GRAM, b.DP_PATH_MATERIALIZED):
        ll, accs = make_layer_list(data, DEV, [path] * len(data))
        n, c, ws = gpu_norms_clip(ll, wl.C)
        norms[path] = to_np(n)
        np.testing.assert_allclose(norms[path][:4], n_ref, rtol=2 * CLIP_TOL)
        np.testing.assert_allclose(to_np(c[:4]), c_ref, rtol=CLIP_TOL)
    np.testing.assert_allclose(norms[b.DP_PATH_GRAM], norms[b.DP_PATH_MATERIALIZED], rtol=2 * CLIP_TOL)
    np.testing.assert_allclose(norms[b.DP_PATH_AUTO], norms[b.DP_PATH_GRAM], rtol=2 * CLIP_TOL)
    # clipped sum of the 4-example subset, element by element
    ll4, acc4 = make_layer_list(sub, DEV)
    n4, c4, ws4 = gpu_norms_clip(ll4, wl.C)
    b.dp_clipped_accumulate(ll4, c4, ws4)
    ref = O.clipped_accumulate(ol, c_ref, O.zero_accumulators(ol))
    for ld, acc, racc in zip(sub, acc4, ref):
        for x, y in zip(acc, racc):
            assert rel_l2(to_np(x), y) <= BF16_TOL, ld.spec.name
    # and sampled entries at the full B = 64 launch
    ll, accs = make_layer_list(data, DEV)
    n, c, ws = gpu_norms_clip(ll, wl.C)
    b.dp_clipped_accumulate(ll, c, ws)
    _sampled_entries_check(data, accs, c, seed=2)


def test_mega_batch_accumulation_invariants():
    """K distinct microbatches against the checker, then the loop invariants: the same microbatch M times
    gives M times the single result, and ||acc|| <= N * C."""
    wl = synth.workload("bert_base_layer")
    B = 16
    step = DPStep(wl.specs, DEV, wl.C, wl.sigma, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay, seed=3)
    ref = None
    for mb in range(4):
        data = synth.generate(wl, seed=1, device=DEV, microbatch=mb, B=B)
        step.accumulate_microbatch(step.layer_list(data))
        ol = to_oracle_layers(data)
        ref = O.zero_accumulators(ol) if ref is None else ref
        O.clipped_accumulate(ol, O.clip_factors(O.per_example_sqnorms(ol), wl.C), ref)
    assert step.examples_seen == 4 * B
    for li in range(len(wl.specs)):
        for k in range(len(ref[li])):
            assert rel_l2(to_np(step.view(step.acc, li, k)), ref[li][k]) <= BF16_TOL
    assert float(step.acc.double().norm()) <= 4 * B * wl.C * (1 + 1e-3)
    # same microbatch M times
    single = DPStep(wl.specs, DEV, wl.C, wl.sigma, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay)
    many = DPStep(wl.specs, DEV, wl.C, wl.sigma, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay)
    data = synth.generate(wl, seed=2, device=DEV, B=B)
    single.accumulate_microbatch(single.layer_list(data))
    M = 8
    ll = many.layer_list(data)
    for _ in range(M):
        many.accumulate_microbatch(ll)
    assert rel_l2(to_np(many.acc), M * to_np(single.acc)) <= 1e-5
    # finish: fused noise + AdamW against the checker on the whole flat vector
    acc_before = to_np(many.acc)
    th0 = synth.initial_weights(many.n_flat, 0, DEV)
    many.theta.copy_(th0)
    many.finish_macro_batch()
    assert float(many.acc.abs().max()) == 0.0 and many.examples_seen == 0 and many.t == 1
    g = O.add_noise_and_scale(acc_before, wl.sigma, wl.C, M * B, seed=0, step=1, elem_offset=0)
    rt, rm, rv = O.adamw_step(to_np(th0), 0 * acc_before, 0 * acc_before, g, wl.lr, wl.beta1, wl.beta2, wl.xi,
                              wl.weight_decay, 1)
    assert rel_l2(to_np(many.m), rm) <= 1e-5 and rel_l2(to_np(many.v), rv) <= 1e-5
    assert_update_close(to_np(many.theta), to_np(th0), rt, rv)


def test_mega_batch_at_bert_large_shapes():
    """The mega-batch accumulation of Section 5.3 at the full 24-block shapes: two DISTINCT microbatches of 256
    examples clipped and summed in place (norms and clip factors of a spread subset against the checker, one sampled
    entry per 128 x 128 accumulator block against fp64), then one microbatch accumulated M = 16 times against 16 times
    the single pass, the bound ||acc|| <= N C, and the macro-batch's noise + AdamW update on sampled windows."""
    wl = synth.workload("bert_large")
    step = DPStep(wl.specs, DEV, wl.C, wl.sigma, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay, seed=5)
    pool = [synth.generate(wl, seed=11, device=DEV, microbatch=k) for k in range(2)]
    lists = [step.layer_list(d) for d in pool]
    clips = []
    rows = [0, 77, 128, 255]
    for d, ll in zip(pool, lists):
        sq, clip = step.accumulate_microbatch(ll)
        clips.append(clip.clone())
        ol = to_oracle_layers(_subset(d, rows))
        n_ref = O.per_example_sqnorms(ol)
        np.testing.assert_allclose(to_np(sq[rows]), n_ref, rtol=2 * CLIP_TOL)
        np.testing.assert_allclose(to_np(clip[rows]), O.clip_factors(n_ref, wl.C), rtol=CLIP_TOL)
    torch.cuda.synchronize()
    assert b.dp_poll_status() == 0 and step.examples_seen == 2 * wl.B
    assert not torch.equal(clips[0], clips[1])                       # the microbatches are distinct
    accs = [[step.view(step.acc, li, k) for k in range(len(step.shapes[li]))] for li in range(len(wl.specs))]
    _tile_sampled_check(pool, accs, clips, seed=3)
    two = step.acc.clone()
    assert float(two.double().norm()) <= 2 * wl.B * wl.C * (1 + 1e-3)
    # the same microbatch M times: M x the single pass (equal addends round the same way every time)
    step.discard_macro_batch()
    step.accumulate_microbatch(lists[0])
    single = step.acc.clone()
    M = 16
    for _ in range(M - 1):
        step.accumulate_microbatch(lists[0])
    torch.cuda.synchronize()
    assert b.dp_poll_status() == 0 and step.examples_seen == M * wl.B
    diff = float((step.acc.double() - M * single.double()).norm() / (M * single.double().norm()))
    assert diff <= 1e-5, diff
    assert float(step.acc.double().norm()) <= M * wl.B * wl.C * (1 + 1e-3)
    # once per macro-batch: noise + AdamW over all 333.6M parameters, the checker on windows of the flat vector
    del two, single
    th0 = synth.initial_weights(step.n_flat, 0, DEV)
    step.theta.copy_(th0)
    acc_before = step.acc.clone()
    step.finish_macro_batch()
    assert step.t == 1 and float(step.acc.abs().max()) == 0.0
    n = step.n_flat
    for lo in (0, 4 * 1_000_003, n // 2 - 12, n - 50_000):
        hi = min(n, lo + 50_000)
        g = O.add_noise_and_scale(to_np(acc_before[lo:hi]), wl.sigma, wl.C, M * wl.B, seed=5, step=1, elem_offset=lo)
        z = np.zeros(hi - lo)
        rt, rm, rv = O.adamw_step(to_np(th0[lo:hi]), z, z, g, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay, 1)
        assert rel_l2(to_np(step.m[lo:hi]), rm) <= 1e-5 and rel_l2(to_np(step.v[lo:hi]), rv) <= 1e-5
        assert_update_close(to_np(step.theta[lo:hi]), to_np(th0[lo:hi]), rt, rv)
