"""GPU parity for a table trained through two layers (token embedding + output projection onto the same table, the
masked-LM head of BERT): the cross term of the squared norm, the whole norm -> clip -> accumulate flow into one
accumulator, the BERT-Large-sized case on sampled examples, and the report of an out-of-range token id."""
import numpy as np
import pytest
import torch

from .helpers import (EMBEDDING, LINEAR, LayerData, LayerSpec, O, assert_update_close, b, rel_l2, to_np,
                      to_oracle_layers)

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = "cuda:0"
CLIP_TOL = 1e-3
BF16_TOL = 2e-2


def _case(B, T, T_out, V, d, dtype, seed, scale=1.0, correlated=False):
    """Embedding (ids repeat when V < T) and projection (A = dlogits, G = h) on the device, as LayerData.
    correlated: position s of the projection sees a hidden state aligned with token s's embedding gradient and
    pushes on that token's own vocabulary entry, so that the two parts of the table's gradient overlap."""
    g = torch.Generator().manual_seed(seed)
    ids = torch.randint(0, V, (B, T), generator=g, dtype=torch.int32)
    G_emb = torch.randn(B, T, d, generator=g) * scale
    dlogits = torch.randn(B, T_out, V, generator=g) * scale
    h = torch.randn(B, T_out, d, generator=g)
    if correlated:
        h = h + 2.0 * G_emb[:, :T_out, :] / scale
        dlogits.scatter_add_(2, ids[:, :T_out, None].long(), torch.full((B, T_out, 1), 3.0 * scale))
    ids, G_emb, dlogits, h = ids.to(DEV), G_emb.to(dtype).to(DEV), dlogits.to(dtype).to(DEV), h.to(dtype).to(DEV)
    emb = LayerData(LayerSpec(EMBEDDING, V, d, False, "tok_emb"), G=G_emb, ids=ids)
    proj = LayerData(LayerSpec(LINEAR, V, d, False, "mlm_decoder"), G=h, A=dlogits)
    return emb, proj


def _layers(emb, proj, acc):
    le = b.Layer(kind=EMBEDDING, G=emb.G, ids=emb.ids, acc_w=acc, vocab=emb.spec.d_in)
    lp = b.Layer(kind=LINEAR, G=proj.G, A=proj.A, acc_w=acc, has_bias=False)
    return le, lp


@pytest.mark.parametrize("dtype,tol", [(torch.float32, 1e-4), (torch.bfloat16, 1e-3)])
@pytest.mark.parametrize("B,T,T_out,V,d", [(3, 37, 20, 50, 96), (2, 150, 130, 40, 72), (1, 1, 1, 3, 5), (4, 64, 65, 700, 33)])
def test_cross_term_matches_checker(dtype, tol, B, T, T_out, V, d):
    emb, proj = _case(B, T, T_out, V, d, dtype, seed=T + T_out)
    oe, op = to_oracle_layers([emb, proj])
    x_ref = O.shared_table_cross_terms(oe, op)
    scale = np.sqrt(O.per_example_sqnorms([oe]) * O.per_example_sqnorms([op]))     # |<s, d>| <= ||s|| ||d||
    le, lp = _layers(emb, proj, torch.zeros(V, d, device=DEV))
    sq = torch.full((B,), 3.0, dtype=torch.float32, device=DEV)                     # adds into what is there
    b.dp_shared_table_cross_sqnorms(le, lp, sq)
    assert b.dp_poll_status() == 0
    assert np.max(np.abs(to_np(sq) - 3.0 - 2.0 * x_ref) / (scale + 3.0)) <= tol


@pytest.mark.parametrize("dtype,V,d", [(torch.float32, 50, 40), (torch.bfloat16, 128, 64), (torch.bfloat16, 100, 64)])
def test_shared_table_norm_clip_accumulate(dtype, V, d):
    """Two calls with different token counts, the cross term, one clip, both layers summed into ONE accumulator."""
    B, T, T_out = 6, 48, 20
    emb, proj = _case(B, T, T_out, V, d, dtype, seed=11, scale=0.05, correlated=True)
    oe, op = to_oracle_layers([emb, proj])
    n_ref = O.per_example_sqnorms_shared_table([oe, op], 0, 1)
    C = float(np.sqrt(np.median(n_ref)))
    c_ref = O.clip_factors(n_ref, C)
    acc = torch.zeros(V, d, device=DEV)
    le, lp = _layers(emb, proj, acc)
    ll_e, ll_p = b.LayerList([le]), b.LayerList([lp])
    ws_e, ws_p = b.alloc_workspace(ll_e), b.alloc_workspace(ll_p)
    sq = torch.empty(B, dtype=torch.float32, device=DEV)
    clip = torch.empty_like(sq)
    b.dp_per_example_sqnorms(ll_e, sq, False, ws_e)
    b.dp_per_example_sqnorms(ll_p, sq, True, ws_p)
    b.dp_shared_table_cross_sqnorms(le, lp, sq)
    b.dp_clip_factors(sq, C, clip)
    b.dp_clipped_accumulate(ll_e, clip, ws_e)
    b.dp_clipped_accumulate(ll_p, clip, ws_p)
    assert b.dp_poll_status() == 0
    np.testing.assert_allclose(to_np(sq), n_ref, rtol=2 * CLIP_TOL)
    np.testing.assert_allclose(to_np(clip), c_ref, rtol=CLIP_TOL)
    assert 0 < int((c_ref < 1).sum()) < B                      # both branches of the clip
    accs = O.zero_accumulators([oe, op])
    accs[1][0] = accs[0][0]
    O.clipped_accumulate([oe, op], c_ref, accs)
    assert rel_l2(to_np(acc), accs[0][0]) <= (1e-4 if dtype == torch.float32 else BF16_TOL)
    # without the cross term the norms would be visibly off on these inputs
    assert np.max(np.abs(O.per_example_sqnorms([oe, op]) / n_ref - 1.0)) > 10 * CLIP_TOL


def test_bert_large_sized_table_on_sampled_examples():
    """30528 x 1024 table (the vocabulary padded to a multiple of 64), 128 tokens, 20 masked positions, B = 256 in
    one launch; the checker materialises the [V, d] gradient of three examples spread over the batch."""
    B, T, T_out, V, d = 256, 128, 20, 30528, 1024
    emb, proj = _case(B, T, T_out, V, d, torch.bfloat16, seed=5, scale=0.01)
    ids = emb.ids.clone()
    ids[:, ::3] = ids[:, ::3] % 50                              # frequent ids, as under a Zipf law: rows repeat
    emb = LayerData(emb.spec, G=emb.G, ids=ids.contiguous())
    le, lp = _layers(emb, proj, None)
    sq = torch.zeros(B, dtype=torch.float32, device=DEV)
    b.dp_shared_table_cross_sqnorms(le, lp, sq)
    assert b.dp_poll_status() == 0
    got = to_np(sq)
    for i in (0, 131, 255):
        sub = [LayerData(emb.spec, G=emb.G[i:i + 1].contiguous(), ids=emb.ids[i:i + 1].contiguous()),
               LayerData(proj.spec, G=proj.G[i:i + 1].contiguous(), A=proj.A[i:i + 1].contiguous())]
        oe, op = to_oracle_layers(sub)
        x = O.shared_table_cross_terms(oe, op)[0]
        scale = float(np.sqrt(O.per_example_sqnorms([oe])[0] * O.per_example_sqnorms([op])[0]))
        assert abs(got[i] - 2.0 * x) <= 1e-3 * scale, (i, got[i], 2.0 * x, scale)


def test_out_of_range_id_is_skipped_and_reported():
    emb, proj = _case(2, 9, 4, 10, 8, torch.float32, seed=3)
    ids = emb.ids.clone()
    ids[1, 4] = 10                                              # == V
    oe, op = to_oracle_layers([emb, proj])
    # the checker with that token's row zeroed = the token skipped
    G0 = emb.G.clone()
    G0[1, 4] = 0
    oe0 = to_oracle_layers([LayerData(emb.spec, G=G0, ids=emb.ids)])[0]
    x_ref = O.shared_table_cross_terms(oe0, op)
    bad = LayerData(emb.spec, G=emb.G, ids=ids.contiguous())
    le, lp = _layers(bad, proj, None)
    sq = torch.zeros(2, dtype=torch.float32, device=DEV)
    b.dp_shared_table_cross_sqnorms(le, lp, sq)
    assert b.dp_poll_status() == -7                             # DP_ERR_BAD_ID
    assert b.dp_poll_status() == 0                              # the report is read once
    np.testing.assert_allclose(to_np(sq), 2.0 * x_ref, rtol=1e-4, atol=1e-5)


def test_bert_heads_in_three_token_groups_with_tied_decoder():
    """The tensors of BERT outside the encoder stack, through the C ABI in three calls with their own token counts:
    per token (word-piece table, a stand-in encoder layer), per masked position (MLM transform, its LayerNorm, the
    decoder tied to the word-piece table, the output bias as a 1 x V linear layer over a column of ones), per
    example (pooler and next-sentence classifier on the first token).  One norm over everything, one clip, every
    tensor's clipped sum against the checker; the table receives both of its contributions."""
    B, T, T_out, V, d = 5, 24, 20, 128, 64
    g = torch.Generator().manual_seed(21)
    dt = torch.bfloat16

    def rnd(*shape, scale=1.0):
        return (torch.randn(*shape, generator=g) * scale).to(dt).to(DEV)

    ids = torch.randint(0, V, (B, T), generator=g, dtype=torch.int32).to(DEV)
    dlogits = rnd(B, T_out, V, scale=0.05)
    ones = torch.ones(B, T_out, 1, dtype=dt, device=DEV)
    specs = {
        "tok_emb": LayerData(LayerSpec(EMBEDDING, V, d, False, "tok_emb"), G=rnd(B, T, d, scale=0.05), ids=ids),
        "enc": LayerData(LayerSpec(LINEAR, d, d, True, "enc"), G=rnd(B, T, d, scale=0.02), A=rnd(B, T, d)),
        "mlm_dense": LayerData(LayerSpec(LINEAR, d, d, True, "mlm_dense"), G=rnd(B, T_out, d, scale=0.05), A=rnd(B, T_out, d)),
        "mlm_ln": LayerData(LayerSpec("layernorm", d, d, False, "mlm_ln"), G=rnd(B, T_out, d, scale=0.05), A=rnd(B, T_out, d)),
        "decoder": LayerData(LayerSpec(LINEAR, V, d, False, "decoder"), G=rnd(B, T_out, d), A=dlogits),
        "out_bias": LayerData(LayerSpec(LINEAR, 1, V, False, "out_bias"), G=dlogits, A=ones),
        "pooler": LayerData(LayerSpec(LINEAR, d, d, True, "pooler"), G=rnd(B, 1, d, scale=0.3), A=rnd(B, 1, d)),
        "nsp": LayerData(LayerSpec(LINEAR, d, 2, True, "nsp"), G=rnd(B, 1, 2, scale=0.3), A=rnd(B, 1, d)),
    }
    groups = [["tok_emb", "enc"], ["mlm_dense", "mlm_ln", "decoder", "out_bias"], ["pooler", "nsp"]]
    names = [n for grp in groups for n in grp]
    table = torch.zeros(V, d, device=DEV)

    def acc_for(name):
        sp = specs[name].spec
        if name in ("tok_emb", "decoder"):
            return [table]
        if sp.kind == LINEAR:
            return [torch.zeros(sp.d_in, sp.d_out, device=DEV)] + ([torch.zeros(sp.d_out, device=DEV)] if sp.has_bias else [])
        return [torch.zeros(d, device=DEV), torch.zeros(d, device=DEV)]

    accs = {n: acc_for(n) for n in names}
    layer = {}
    for n in names:
        ld, a = specs[n], accs[n]
        layer[n] = b.Layer(kind=ld.spec.kind, G=ld.G, A=ld.A, ids=ld.ids, acc_w=a[0], acc_b=a[1] if len(a) > 1 else None,
                           has_bias=ld.spec.has_bias, vocab=V if ld.spec.kind == EMBEDDING else 0)
    lists = [b.LayerList([layer[n] for n in grp]) for grp in groups]
    wss = [b.alloc_workspace(ll) for ll in lists]
    sq = torch.empty(B, dtype=torch.float32, device=DEV)
    clip = torch.empty_like(sq)
    for k, (ll, ws) in enumerate(zip(lists, wss)):
        b.dp_per_example_sqnorms(ll, sq, k > 0, ws)
    b.dp_shared_table_cross_sqnorms(layer["tok_emb"], layer["decoder"], sq)

    ol = to_oracle_layers([specs[n] for n in names])
    n_ref = O.per_example_sqnorms_shared_table(ol, names.index("tok_emb"), names.index("decoder"))
    C = float(np.sqrt(np.median(n_ref)))
    c_ref = O.clip_factors(n_ref, C)
    b.dp_clip_factors(sq, C, clip)
    for ll, ws in zip(lists, wss):
        b.dp_clipped_accumulate(ll, clip, ws)
    assert b.dp_poll_status() == 0
    np.testing.assert_allclose(to_np(sq), n_ref, rtol=2 * CLIP_TOL)
    np.testing.assert_allclose(to_np(clip), c_ref, rtol=CLIP_TOL)
    ref = O.zero_accumulators(ol)
    ref[names.index("decoder")][0] = ref[names.index("tok_emb")][0]
    O.clipped_accumulate(ol, c_ref, ref)
    for k, n in enumerate(names):
        for x, y in zip(accs[n], ref[k]):
            assert x.shape == y.shape and rel_l2(to_np(x), y) <= BF16_TOL, n


def test_dpstep_with_token_groups_and_a_shared_table():
    """The same model through DPStep: layers grouped by token count, the decoder aliased onto the word-piece table
    (no storage of its own in the flat parameter vector), two microbatches, then noise + AdamW over the flat vector
    against the checker."""
    from paper_2108_01624_b200 import DPStep, synth
    B, T, T_out, V, d = 4, 24, 20, 128, 64
    dt = torch.bfloat16
    spec_list = [LayerSpec(EMBEDDING, V, d, False, "tok_emb"), LayerSpec(LINEAR, d, d, True, "enc"),
                 LayerSpec(LINEAR, d, d, True, "mlm_dense"), LayerSpec("layernorm", d, d, False, "mlm_ln"),
                 LayerSpec(LINEAR, V, d, False, "decoder"), LayerSpec(LINEAR, 1, V, False, "out_bias"),
                 LayerSpec(LINEAR, d, d, True, "pooler"), LayerSpec(LINEAR, d, 2, True, "nsp")]
    tokens = [T, T, T_out, T_out, T_out, T_out, 1, 1]
    hp = dict(C=0.3, sigma=0.7, lr=1e-2, beta1=0.9, beta2=0.999, xi=1e-11, weight_decay=0.5)
    step = DPStep(spec_list, DEV, seed=5, shared_tables={4: 0}, **hp)
    assert step.offsets[4] == step.offsets[0]
    assert step.n_flat == sum((sp.n_params() + 3) // 4 * 4 if sp.kind != LINEAR or not sp.has_bias else
                              (sp.d_in * sp.d_out + 3) // 4 * 4 + (sp.d_out + 3) // 4 * 4
                              for k, sp in enumerate(spec_list) if k != 4)
    th0 = synth.initial_weights(step.n_flat, 3, DEV)
    step.theta.copy_(th0)
    g = torch.Generator().manual_seed(33)
    mbs = []
    for mb in range(2):
        data = []
        dlogits = (torch.randn(B, T_out, V, generator=g) * 0.05).to(dt).to(DEV)
        for sp, tk in zip(spec_list, tokens):
            G = (torch.randn(B, tk, sp.d_out, generator=g) * 0.05).to(dt).to(DEV)
            if sp.kind == EMBEDDING:
                data.append(LayerData(sp, G=G, ids=torch.randint(0, V, (B, tk), generator=g, dtype=torch.int32).to(DEV)))
            elif sp.name == "decoder":
                data.append(LayerData(sp, G=torch.randn(B, tk, d, generator=g).to(dt).to(DEV), A=dlogits))
            elif sp.name == "out_bias":
                data.append(LayerData(sp, G=dlogits, A=torch.ones(B, tk, 1, dtype=dt, device=DEV)))
            else:
                data.append(LayerData(sp, G=G, A=torch.randn(B, tk, sp.d_in, generator=g).to(dt).to(DEV)))
        mbs.append(to_oracle_layers(data))
        if mb == 0:                                # a clip norm that some examples exceed and some do not
            step.C = hp["C"] = float(np.sqrt(np.median(O.per_example_sqnorms_shared_table(mbs[0], 0, 4))))
        lists = step.layer_lists(data)
        assert [ll.layers[0].G.shape[1] for ll in lists] == [T, T_out, 1]
        step.accumulate_microbatch(lists)
    assert b.dp_poll_status() == 0 and step.examples_seen == 2 * B
    ref = O.zero_accumulators(mbs[0])
    ref[4][0] = ref[0][0]
    clipped = 0
    for ol in mbs:
        c = O.clip_factors(O.per_example_sqnorms_shared_table(ol, 0, 4), hp["C"])
        clipped += int((c < 1).sum())
        O.clipped_accumulate(ol, c, ref)
    assert 0 < clipped < 2 * B
    flat = np.zeros(step.n_flat)
    for li in range(len(spec_list)):
        for k, a in enumerate(ref[li]):
            off = step.offsets[li][k]
            flat[off:off + a.size] = a.ravel()
    acc = to_np(step.acc)
    assert rel_l2(acc, flat) <= BF16_TOL
    step.finish_macro_batch()
    gref = O.add_noise_and_scale(acc, hp["sigma"], hp["C"], 2 * B, seed=5, step=1, elem_offset=0)
    rt, rm, rv = O.adamw_step(to_np(th0), np.zeros(step.n_flat), np.zeros(step.n_flat), gref, hp["lr"], hp["beta1"],
                              hp["beta2"], hp["xi"], hp["weight_decay"], 1)
    assert_update_close(to_np(step.theta), to_np(th0), rt, rv)
