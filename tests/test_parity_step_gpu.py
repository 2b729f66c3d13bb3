"""GPU parity of whole macro-steps through DPStep: varying batch size per step (the increasing schedule of
Section 5.2.2 in miniature), gradient-SNR tracking, and the BERT input layer with its three embeddings."""
import numpy as np
import pytest
import torch

from paper_2108_01624_b200 import DPStep, synth

from .helpers import (EMBEDDING, LAYERNORM, LINEAR, LayerSpec, O, assert_update_close, b, gpu_norms_clip, make_layer_list, random_layers,
                      rel_l2, to_np, to_oracle_layers)

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = "cuda:0"
SPECS = [LayerSpec(LINEAR, 128, 256, True, "fc1"), LayerSpec(LAYERNORM, 128, 128, False, "ln"),
         LayerSpec(EMBEDDING, 30, 64, False, "emb")]


def test_macro_steps_with_a_growing_batch_and_snr():
    B, T = 8, 64
    hp = dict(C=0.05, sigma=0.8, lr=1e-2, beta1=0.9, beta2=0.999, xi=1e-11, weight_decay=0.5)
    step = DPStep(SPECS, DEV, seed=9, track_snr=True, **hp)
    th = synth.initial_weights(step.n_flat, 1, DEV)
    step.theta.copy_(th)
    r_th, r_m, r_v = to_np(th), np.zeros(step.n_flat), np.zeros(step.n_flat)
    seed_ctr = 0
    for t, n_mb in enumerate((2, 3), start=1):              # the batch grows from 16 to 24 examples
        mbs = []
        for _ in range(n_mb):
            data = random_layers(SPECS, B, T, torch.bfloat16, DEV, seed=100 + seed_ctr, g_scale=0.02, vocab_dup=6)
            seed_ctr += 1
            step.accumulate_microbatch(step.layer_list(data))
            mbs.append(to_oracle_layers(data))
        assert step.examples_seen == n_mb * B
        acc = to_np(step.acc)
        step.finish_macro_batch()
        # checker: clipped sums -> flat layout -> noise / N -> AdamW
        accs = O.zero_accumulators(mbs[0])
        for ol in mbs:
            O.clipped_accumulate(ol, O.clip_factors(O.per_example_sqnorms(ol), hp["C"]), accs)
        flat = np.zeros(step.n_flat)
        for li in range(len(SPECS)):
            for k, a in enumerate(accs[li]):
                off = step.offsets[li][k]
                flat[off:off + a.size] = a.ravel()
        assert rel_l2(acc, flat) <= 2e-2
        g = O.add_noise_and_scale(acc, hp["sigma"], hp["C"], n_mb * B, seed=9, step=t, elem_offset=0)
        new = O.adamw_step(r_th, r_m, r_v, g, hp["lr"], hp["beta1"], hp["beta2"], hp["xi"], hp["weight_decay"], t)
        assert_update_close(to_np(step.theta), r_th, new[0], new[2])
        r_th, r_m, r_v = to_np(step.theta), to_np(step.m), to_np(step.v)
        s2, n2 = O.gradient_snr_sums(acc, hp["sigma"], hp["C"], 9, t, 0)
        assert step.gradient_snr() == pytest.approx(np.sqrt(s2 / n2), rel=1e-4)
    assert step.t == 2 and step.examples_seen == 0


def test_bert_input_layer_three_embeddings():
    """Word-piece (Zipf), positional (all ids distinct) and token-type (two ids) embeddings plus their LayerNorm."""
    wl = synth.workload("bert_large_embeddings")
    data = synth.generate(wl, seed=3, device=DEV, B=8)
    ol = to_oracle_layers(data)
    n_ref = O.per_example_sqnorms(ol)
    c_ref = O.clip_factors(n_ref, 1e-3)
    for path in (b.DP_PATH_AUTO, b.DP_PATH_MATERIALIZED):
        ll, accs = make_layer_list(data, DEV, [path] * len(data))
        n, c, ws = gpu_norms_clip(ll, 1e-3)
        np.testing.assert_allclose(to_np(n), n_ref, rtol=2e-3)
        np.testing.assert_allclose(to_np(c), c_ref, rtol=1e-3)
        b.dp_clipped_accumulate(ll, c, ws)
        ref = O.clipped_accumulate(ol, c_ref, O.zero_accumulators(ol))
        for ld, acc, racc in zip(data, accs, ref):
            for x, y in zip(acc, racc):
                assert rel_l2(to_np(x), y) <= 2e-2, ld.spec.name
    # closed forms: positions are all distinct -> |G|_F^2; a single segment id per half -> two row sums
    G = to_np(data[1].G)
    ll1, _ = make_layer_list([data[1]], DEV)
    n1, _, _ = gpu_norms_clip(ll1, 1.0)
    np.testing.assert_allclose(to_np(n1), (G ** 2).sum((1, 2)), rtol=2e-3)
    assert b.dp_poll_status() == 0


def test_checkpoint_resume_in_the_middle_of_a_macro_batch(tmp_path):
    """Save after two of three microbatches, reload into a fresh object, finish: the linear and LayerNorm tensors
    are bit-identical to the uninterrupted run (one owner per element and launch), the embedding rows agree within
    fp32 atomics order, and the noise is the same draw (counter-based generator keyed by seed, step, element)."""
    wl = synth.workload("bert_base_layer")
    specs = list(wl.specs) + [synth.LayerSpec(synth.EMBEDDING, 300, 768, False, "emb")]
    mk = lambda: DPStep(specs, DEV, wl.C, wl.sigma, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay, seed=9)
    wl2 = synth.Workload("ckpt", 8, 64, torch.bfloat16, specs)
    mbs = [synth.generate(wl2, seed=4, device=DEV, microbatch=k) for k in range(3)]
    th0 = synth.initial_weights(mk().n_flat, 1, DEV)

    full = mk()
    full.theta.copy_(th0)
    for d in mbs:
        full.accumulate_microbatch(full.layer_list(d))
    full.finish_macro_batch()

    first = mk()
    first.theta.copy_(th0)
    for d in mbs[:2]:
        first.accumulate_microbatch(first.layer_list(d))
    torch.save(first.state_dict(), tmp_path / "ckpt.pt")
    resumed = mk()
    resumed.load_state_dict(torch.load(tmp_path / "ckpt.pt"))
    assert resumed.examples_seen == 16 and resumed.t == 0
    resumed.accumulate_microbatch(resumed.layer_list(mbs[2]))
    resumed.finish_macro_batch()
    torch.cuda.synchronize()
    assert b.dp_poll_status() == 0
    emb_lo = full.offsets[-1][0]
    assert torch.equal(resumed.theta[:emb_lo], full.theta[:emb_lo])
    assert torch.equal(resumed.m[:emb_lo], full.m[:emb_lo]) and torch.equal(resumed.v[:emb_lo], full.v[:emb_lo])
    assert rel_l2(to_np(resumed.m[emb_lo:]), to_np(full.m[emb_lo:])) <= 1e-6
    assert resumed.t == full.t == 1 and resumed.examples_seen == 0


def test_outputs_stay_inside_their_buffers_and_repeat_bit_for_bit():
    """Canary words around the accumulators, the norms and the clip factors survive a full microbatch, and a
    second run of the same calls gives the same bits (the only order-dependent adds, the embedding atomics,
    are left out of this list)."""
    wl = synth.workload("bert_base_layer")
    wl2 = synth.Workload("canary", 5, 100, torch.bfloat16, wl.specs)
    data = synth.generate(wl2, seed=6, device=DEV)
    results = []
    for rep in range(2):
        pad = 64
        accs, raws = [], []
        for ld in data:
            acc = []
            for shp in ([(ld.spec.d_in, ld.spec.d_out)] + ([(ld.spec.d_out,)] if ld.spec.has_bias else [])
                        if ld.spec.kind == synth.LINEAR else [(ld.spec.d_out,), (ld.spec.d_out,)]):
                n = int(np.prod(shp))
                raw = torch.full((n + 2 * pad,), 12345.0, dtype=torch.float32, device=DEV)
                raw[pad:pad + n].zero_()
                raws.append((raw, n))
                acc.append(raw[pad:pad + n].view(shp))
            accs.append(acc)
        ll = b.LayerList([b.Layer(kind=ld.spec.kind, G=ld.G, A=ld.A, ids=None, acc_w=a[0], acc_b=a[1] if len(a) > 1 else None,
                                  has_bias=ld.spec.has_bias, vocab=0, path=b.DP_PATH_AUTO) for ld, a in zip(data, accs)])
        nraw = torch.full((5 + 2 * pad,), 777.0, dtype=torch.float32, device=DEV)
        craw = torch.full((5 + 2 * pad,), 777.0, dtype=torch.float32, device=DEV)
        n, c = nraw[pad:pad + 5], craw[pad:pad + 5]
        ws = b.alloc_workspace(ll)
        b.dp_per_example_sqnorms(ll, n, False, ws)
        b.dp_clip_factors(n, wl.C, c)
        b.dp_clipped_accumulate_after_sqnorms(ll, c, ws)
        torch.cuda.synchronize()
        assert b.dp_poll_status() == 0
        for raw, k in raws:
            assert bool((raw[:pad] == 12345.0).all()) and bool((raw[pad + k:] == 12345.0).all())
        for raw in (nraw, craw):
            assert bool((raw[:pad] == 777.0).all()) and bool((raw[pad + 5:] == 777.0).all())
        results.append([x.clone() for acc in accs for x in acc] + [n.clone(), c.clone()])
    for x, y in zip(*results):
        assert torch.equal(x, y)


def test_microbatch_and_update_replay_from_a_cuda_graph():
    """The calls of a microbatch (norms, clip factors, clipped accumulate) and of the fused update only enqueue
    work on the caller's stream, so a stream capture records them; replaying the graph with new input values in
    the same buffers gives what the eager calls give, up to the order of the fp32 adds where small layers split
    their example range over several CTA pairs."""
    specs = [LayerSpec(LINEAR, 256, 512, True, "fc1"), LayerSpec(LAYERNORM, 256, 256, False, "ln"),
             LayerSpec(LINEAR, 512, 128, False, "fc2")]
    hp = dict(C=0.05, sigma=0.8, lr=1e-2, beta1=0.9, beta2=0.999, xi=1e-11, weight_decay=0.5)
    B, T = 12, 128
    batches = [random_layers(specs, B, T, torch.bfloat16, DEV, seed=300 + k, g_scale=0.02) for k in range(3)]

    def fresh():
        s = DPStep(specs, DEV, seed=4, **hp)
        s.theta.copy_(synth.initial_weights(s.n_flat, 2, DEV))
        return s

    eager = fresh()
    for data in batches:
        eager.accumulate_microbatch(eager.layer_list(data))
    acc_eager = eager.acc.clone()
    eager.finish_macro_batch()

    graphed = fresh()
    resident = random_layers(specs, B, T, torch.bfloat16, DEV, seed=1, g_scale=0.02)   # the buffers the graph reads
    ll = graphed.layer_list(resident)
    graphed.accumulate_microbatch(ll)            # warm-up outside the capture: scratch buffers, library state
    graphed.acc.zero_()
    graphed.examples_seen = 0
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(g, stream=side):
            graphed.accumulate_microbatch(ll)
    graphed.examples_seen = 0                    # the capture counted a microbatch that did not run
    for data in batches:
        for dst, src in zip(resident, data):
            dst.G.copy_(src.G)
            dst.A.copy_(src.A)
        g.replay()
        graphed.examples_seen += B
    torch.cuda.synchronize()
    assert b.dp_poll_status() == 0
    assert rel_l2(to_np(graphed.acc), to_np(acc_eager)) <= 1e-6
    graphed.finish_macro_batch()
    assert rel_l2(to_np(graphed.m), to_np(eager.m)) <= 1e-6
    assert rel_l2(to_np(graphed.theta), to_np(eager.theta)) <= 1e-6
