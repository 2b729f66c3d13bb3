"""GPU parity for the layer passes (per-example norms, clip factors, clipped accumulate) against the CPU
checker, from the tiny fp32 layer up to BERT-shaped bf16 blocks, including ragged and degenerate cases."""
import numpy as np
import pytest
import torch

from paper_2108_01624_b200 import synth

from .helpers import (EMBEDDING, LAYERNORM, LINEAR, LayerSpec, O, b, gpu_norms_clip, make_layer_list, random_layers,
                      rel_l2, rel_max, to_np, to_oracle_layers)

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = "cuda:0"
CLIP_TOL = 1e-3       # clip factors: relative error bound
F32_TOL = 1e-4        # fp32-input paths
BF16_TOL = 2e-2       # bf16-input / fp32-accumulate clipped sums, relative L2


def check_against_checker(data, C, paths=None, sum_tol=BF16_TOL, rows=None):
    """Runs norms -> clip -> accumulate on the GPU and compares all three with the checker."""
    ll, accs = make_layer_list(data, DEV, paths)
    n, c, ws = gpu_norms_clip(ll, C)
    b.dp_clipped_accumulate(ll, c, ws)
    assert b.dp_poll_status() == 0
    ol = to_oracle_layers(data)
    n_ref = O.per_example_sqnorms(ol)
    c_ref = O.clip_factors(n_ref, C)
    np.testing.assert_allclose(to_np(n), n_ref, rtol=2 * CLIP_TOL)
    np.testing.assert_allclose(to_np(c), c_ref, rtol=CLIP_TOL)
    ref = O.clipped_accumulate(ol, c_ref, O.zero_accumulators(ol))
    for ld, acc, racc in zip(data, accs, ref):
        for k, (x, y) in enumerate(zip(acc, racc)):
            assert x.shape == y.shape
            err = rel_l2(to_np(x), y)
            assert err <= sum_tol, f"{ld.spec.name or ld.spec.kind}[{k}] rel L2 {err:.3e}"
            if ld.G.dtype == torch.float32:      # fp32 paths: every element within 1e-4 of the tensor's largest
                emax = rel_max(to_np(x), y)
                assert emax <= F32_TOL, f"{ld.spec.name or ld.spec.kind}[{k}] max error {emax:.3e} of the largest entry"
    return n_ref, c_ref, accs


# ------------------------------------------------------------------ the tiny fp32 layer, end to end

@pytest.mark.parametrize("path", [b.DP_PATH_AUTO, b.DP_PATH_GRAM, b.DP_PATH_MATERIALIZED])
def test_tiny_linear_fp32_full_step(path):
    wl = synth.workload("tiny_linear")
    data = synth.generate(wl, seed=0, device=DEV)
    n_ref, c_ref, accs = check_against_checker(data, wl.C, [path], sum_tol=F32_TOL)
    assert np.all(c_ref < 1.0)                    # unit-variance inputs: every example clips at C = 1
    # noise + AdamW on the 64x64 weight and the bias, laid end to end
    rng = np.random.default_rng(0)
    W0 = (rng.standard_normal((64, 64)) * 0.02).astype(np.float32)
    ol = to_oracle_layers(data)
    g_ref, _ = O.privatised_gradient([ol], wl.C, wl.sigma, seed=0, step=1)
    flat = torch.cat([accs[0][0].reshape(-1), accs[0][1].reshape(-1)])
    b.dp_add_noise_and_scale(flat, wl.sigma, wl.C, wl.B, 0, 1, 0)
    g_ref_flat = np.concatenate([g_ref[0][0].ravel(), g_ref[0][1].ravel()])
    assert rel_max(to_np(flat), g_ref_flat) <= F32_TOL
    theta = torch.cat([torch.from_numpy(W0).reshape(-1), torch.zeros(64)]).to(DEV)
    th0 = to_np(theta)
    m, v = torch.zeros_like(theta), torch.zeros_like(theta)
    b.dp_adamw_step(theta, m, v, flat, wl.lr, wl.beta1, wl.beta2, wl.xi, wl.weight_decay, 1)
    rt, rm, rv = O.adamw_step(th0, np.zeros_like(th0), np.zeros_like(th0), g_ref_flat, wl.lr, wl.beta1, wl.beta2,
                              wl.xi, wl.weight_decay, 1)
    assert rel_max(to_np(m), rm) <= F32_TOL and rel_max(to_np(v), rv) <= F32_TOL
    d, rd = to_np(theta) - th0, rt - th0
    assert np.max(np.abs(d - rd)) <= F32_TOL * np.max(np.abs(rd)) + 1e-7 * np.max(np.abs(th0))


# ------------------------------------------------------------------ small mixed models, ragged shapes

SMALL = [LayerSpec(LINEAR, 128, 192, True, "fc1"), LayerSpec(LINEAR, 192, 64, False, "fc2"),
         LayerSpec(LAYERNORM, 128, 128, False, "ln"), LayerSpec(EMBEDDING, 50, 64, False, "emb")]
ODD = [LayerSpec(LINEAR, 72, 40, True, "fc_odd"), LayerSpec(LINEAR, 33, 17, True, "fc_unaligned"),
       LayerSpec(LAYERNORM, 100, 100, False, "ln_odd"), LayerSpec(EMBEDDING, 11, 24, False, "emb_dup")]


@pytest.mark.parametrize("dtype,tol", [(torch.float32, F32_TOL), (torch.bfloat16, BF16_TOL)])
@pytest.mark.parametrize("specs,B,T", [(SMALL, 6, 40), (SMALL, 3, 128), (SMALL, 2, 200), (ODD, 5, 19), (ODD, 1, 1)])
@pytest.mark.parametrize("path", [b.DP_PATH_AUTO, b.DP_PATH_GRAM, b.DP_PATH_MATERIALIZED])
def test_small_models_all_paths(dtype, tol, specs, B, T, path):
    data = random_layers(specs, B, T, dtype, DEV, seed=B * 1000 + T, g_scale=0.02, vocab_dup=7)
    ol = to_oracle_layers(data)
    C = float(np.sqrt(np.median(O.per_example_sqnorms(ol))))       # about half the examples clip
    check_against_checker(data, C, [path] * len(specs), sum_tol=tol)


def test_accumulates_in_place_over_microbatches():
    """Two microbatches into the same accumulators equal the checker's sum; linear in the microbatch."""
    accs = None
    ref = None
    for mb in range(2):
        data = random_layers(SMALL, 4, 64, torch.bfloat16, DEV, seed=50 + mb, g_scale=0.02)
        ll, accs = make_layer_list(data, DEV, accs=accs)
        n, c, ws = gpu_norms_clip(ll, 0.5)
        b.dp_clipped_accumulate(ll, c, ws)
        ol = to_oracle_layers(data)
        ref = O.zero_accumulators(ol) if ref is None else ref
        O.clipped_accumulate(ol, O.clip_factors(O.per_example_sqnorms(ol), 0.5), ref)
    for acc, racc in zip(accs, ref):
        for x, y in zip(acc, racc):
            assert rel_l2(to_np(x), y) <= BF16_TOL


def test_sqnorm_accumulate_into_splits_the_model():
    data = random_layers(SMALL, 4, 64, torch.bfloat16, DEV, seed=8, g_scale=0.02)
    ll_all, _ = make_layer_list(data, DEV)
    n_all, _, _ = gpu_norms_clip(ll_all, 1.0)
    n_split = torch.empty(4, dtype=torch.float32, device=DEV)
    for k, part in enumerate((data[:2], data[2:])):
        ll, _ = make_layer_list(part, DEV)
        b.dp_per_example_sqnorms(ll, n_split, accumulate_into=(k > 0), workspace=b.alloc_workspace(ll))
    np.testing.assert_allclose(to_np(n_split), to_np(n_all), rtol=1e-5)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_accumulate_after_sqnorms_reuses_the_layernorm_sums(dtype):
    """The entry point that takes the LayerNorm column sums from the workspace gives bit-identical accumulators
    for every layer kind (the GEMM's L2 reductions have one owner per element here: no example split)."""
    data = random_layers(SMALL, 6, 80, dtype, DEV, seed=13, g_scale=0.02, vocab_dup=7)
    ol = to_oracle_layers(data)
    C = float(np.sqrt(np.median(O.per_example_sqnorms(ol))))
    ll_a, acc_a = make_layer_list(data, DEV)
    n, c, ws = gpu_norms_clip(ll_a, C)
    b.dp_clipped_accumulate(ll_a, c, ws)
    ll_b, acc_b = make_layer_list(data, DEV)
    n2, c2, ws2 = gpu_norms_clip(ll_b, C)
    b.dp_clipped_accumulate_after_sqnorms(ll_b, c2, ws2)
    assert b.dp_poll_status() == 0
    ref = O.clipped_accumulate(ol, O.clip_factors(O.per_example_sqnorms(ol), C), O.zero_accumulators(ol))
    for ld, xa, xb, r in zip(data, acc_a, acc_b, ref):
        for x, y, z in zip(xa, xb, r):
            if ld.spec.kind == LAYERNORM:
                assert torch.equal(x, y), ld.spec.name
            assert rel_l2(to_np(y), z) <= (BF16_TOL if dtype == torch.bfloat16 else 1e-4), ld.spec.name


# ------------------------------------------------------------------ tensor-core tile edges (bf16, widths % 64 == 0)

WIDE = [LayerSpec(LINEAR, 576, 320, True, "w576x320"),      # d_in spans two 512-wide tiles, d_out two 256-wide ones
        LayerSpec(LINEAR, 64, 64, True, "w64x64"),          # one CTA of the pair has no rows at all
        LayerSpec(LINEAR, 1088, 192, False, "w1088x192"),   # three tiles along d_in, the last one 64 wide
        LayerSpec(LINEAR, 256, 512, True, "w256x512")]


@pytest.mark.parametrize("B,T", [(1, 1), (5, 16), (3, 63), (4, 64), (2, 65), (3, 130), (9, 128)])
def test_tensor_core_tile_edges(B, T):
    """Tiles that overhang d_in / d_out, token counts around the 64-token stage, one example, bias on and off."""
    data = random_layers(WIDE, B, T, torch.bfloat16, DEV, seed=100 * B + T, g_scale=0.02)
    ol = to_oracle_layers(data)
    C = float(np.sqrt(np.median(O.per_example_sqnorms(ol))))
    check_against_checker(data, C)
    check_against_checker(data, C, [b.DP_PATH_MATERIALIZED] * len(WIDE))


RAGGED = [LayerSpec(LINEAR, 200, 72, True, "r200x72"),        # widths that are multiples of 8 but not of 64:
          LayerSpec(LINEAR, 136, 264, False, "r136x264"),     # the last 64-feature group overhangs the row and must
          LayerSpec(LINEAR, 584, 328, True, "r584x328"),      # arrive as zeros; tiles overhang as well
          LayerSpec(LINEAR, 1096, 200, True, "r1096x200"),
          LayerSpec(LINEAR, 64, 40, True, "r64x40"),          # one operand ragged, the other not
          LayerSpec(LINEAR, 8, 8, True, "r8x8"),
          LayerSpec(EMBEDDING, 30, 200, False, "emb200")]


@pytest.mark.parametrize("B,T", [(1, 1), (5, 16), (4, 64), (3, 130), (2, 300)])
def test_tensor_core_ragged_widths(B, T):
    """bf16 widths with d % 8 == 0 and d % 64 != 0 on the tensor-core kernels: every norm path and the accumulate."""
    data = random_layers(RAGGED, B, T, torch.bfloat16, DEV, seed=300 * B + T, g_scale=0.02, vocab_dup=9)
    ol = to_oracle_layers(data)
    C = float(np.sqrt(np.median(O.per_example_sqnorms(ol))))
    ll, _ = make_layer_list(data, DEV)
    units = torch.cuda.get_device_properties(0).multi_processor_count // 2
    assert all(x >= 0 for x in b.dp_accumulate_schedule(ll, units)["launch"][:6])     # they are on the tensor-core GEMM
    check_against_checker(data, C)
    check_against_checker(data, C, [b.DP_PATH_GRAM] * len(RAGGED))
    check_against_checker(data, C, [b.DP_PATH_MATERIALIZED] * len(RAGGED))


@pytest.mark.parametrize("B,T", [(3, 129), (2, 256), (3, 300), (2, 384), (2, 640), (1, 700), (2, 2050)])
def test_long_examples_gram_and_tiles(B, T):
    """More than one 128-token block per example: the Gram kernel pairs the column blocks of every row block
    (two blocks = one item; three and five blocks leave a lone last column, with and without the row block in it;
    token counts that end inside a block), and the tile kernel runs several token stages per tile.  Both forced
    paths against the checker, with embedding and LayerNorm layers beside the linear ones."""
    specs = [LayerSpec(LINEAR, 192, 320, True, "w192x320"), LayerSpec(LINEAR, 64, 128, False, "w64x128"),
             LayerSpec(LAYERNORM, 128, 128, False, "ln"), LayerSpec(EMBEDDING, 50, 64, False, "emb")]
    data = random_layers(specs, B, T, torch.bfloat16, DEV, seed=7 * T + B, g_scale=0.02, vocab_dup=12)
    ol = to_oracle_layers(data)
    C = float(np.sqrt(np.median(O.per_example_sqnorms(ol))))
    check_against_checker(data, C, [b.DP_PATH_GRAM] * len(specs))
    check_against_checker(data, C, [b.DP_PATH_MATERIALIZED] * len(specs))


def test_more_long_gram_layers_than_one_launch_holds():
    """60 linear layers at T = 160: the Gram launch for examples of several token blocks takes 48 layers, so this
    needs two, widest layers first; the partial sums still land in the caller's layer order."""
    specs = [LayerSpec(LINEAR, 64 * (1 + k % 3), 64 * (1 + (k // 3) % 2), k % 2 == 0, f"l{k}") for k in range(60)]
    data = random_layers(specs, 2, 160, torch.bfloat16, DEV, seed=9, g_scale=0.02)
    ol = to_oracle_layers(data)
    C = float(np.sqrt(np.median(O.per_example_sqnorms(ol))))
    check_against_checker(data, C, [b.DP_PATH_GRAM] * len(specs))


def test_more_linear_layers_than_one_launch_holds():
    """130 small linear layers: the tensor-core launches take at most 96 layers each, and the accumulate GEMM packs
    every launch's layers into waves of its own."""
    specs = [LayerSpec(LINEAR, 64 * (1 + k % 3), 64 * (1 + (k // 3) % 2), k % 2 == 0, f"l{k}") for k in range(130)]
    data = random_layers(specs, 3, 32, torch.bfloat16, DEV, seed=5, g_scale=0.02)
    ol = to_oracle_layers(data)
    C = float(np.sqrt(np.median(O.per_example_sqnorms(ol))))
    check_against_checker(data, C)


def test_uniform_tiny_clip_factor_reaches_every_stage():
    """c_i = 1e-3 for every example: a stage of G that reached the tensor cores unscaled would weigh 1000 times
    its share, so every accumulator ELEMENT (not only the L2 norm) must stay within rounding of the checker."""
    specs = [LayerSpec(LINEAR, 512, 512, True, "sq"), LayerSpec(LINEAR, 1024, 256, True, "wide")]
    data = random_layers(specs, 16, 128, torch.bfloat16, DEV, seed=77, g_scale=0.02)
    ll, accs = make_layer_list(data, DEV)
    clip = torch.full((16,), 1e-3, dtype=torch.float32, device=DEV)
    for _ in range(3):
        for acc in accs:
            for x in acc:
                x.zero_()
        b.dp_clipped_accumulate(ll, clip, b.alloc_workspace(ll))
        assert b.dp_poll_status() == 0
        ol = to_oracle_layers(data)
        ref = O.clipped_accumulate(ol, np.full(16, 1e-3), O.zero_accumulators(ol))
        for acc, racc in zip(accs, ref):
            for x, y in zip(acc, racc):
                assert np.max(np.abs(to_np(x) - y)) <= 0.05 * np.sqrt(np.mean(y ** 2))


def test_layer_with_more_tiles_than_one_wave():
    """A 4096 x 4096 layer has 128 accumulate tiles, more than the CTA pairs of one wave: it takes whole waves of
    its own and the small layer beside it shares its last one."""
    specs = [LayerSpec(LINEAR, 4096, 4096, True, "big"), LayerSpec(LINEAR, 512, 256, False, "small")]
    data = random_layers(specs, 2, 64, torch.bfloat16, DEV, seed=41, g_scale=0.02)
    ol = to_oracle_layers(data)
    C = float(np.sqrt(np.median(O.per_example_sqnorms(ol))))
    check_against_checker(data, C)


def test_vocabulary_sized_output_layer():
    """An output projection onto a vocabulary padded to a multiple of 64 (30528): 120 x 1 accumulate tiles, 477
    feature tiles per example in the Gram kernel."""
    specs = [LayerSpec(LINEAR, 256, 30528, True, "mlm_head")]
    data = random_layers(specs, 3, 48, torch.bfloat16, DEV, seed=17, g_scale=0.01)
    ol = to_oracle_layers(data)
    C = float(np.sqrt(np.median(O.per_example_sqnorms(ol))))
    check_against_checker(data, C)


def test_accumulate_twice_adds_twice():
    """acc += ...: a second call over the same microbatch doubles every accumulator (the GEMM adds through L2
    reductions, the other kernels read-modify-write)."""
    data = random_layers(SMALL + WIDE[:1], 4, 96, torch.bfloat16, DEV, seed=31, g_scale=0.02, vocab_dup=9)
    ll, accs = make_layer_list(data, DEV)
    n, c, ws = gpu_norms_clip(ll, 0.5)
    b.dp_clipped_accumulate(ll, c, ws)
    once = [[x.clone() for x in acc] for acc in accs]
    b.dp_clipped_accumulate(ll, c, ws)
    for a1, a2 in zip(once, accs):
        for x, y in zip(a1, a2):
            assert rel_l2(to_np(y), 2 * to_np(x)) <= 1e-6


def test_zero_gradient_example_is_left_unscaled():
    data = random_layers(SMALL[:3], 3, 32, torch.bfloat16, DEV, seed=4, g_scale=0.02)
    for ld in data:
        ld.G[1].zero_()
    ll, accs = make_layer_list(data, DEV)
    n, c, ws = gpu_norms_clip(ll, 1e-3)
    assert float(n[1]) == 0.0 and float(c[1]) == 1.0
    b.dp_clipped_accumulate(ll, c, ws)
    assert all(torch.isfinite(x).all() for acc in accs for x in acc)


def test_no_clipping_equals_batch_gradient():
    """C -> infinity: every c_i = 1 and the clipped sum is the plain batch gradient A^T G."""
    data = random_layers(SMALL, 5, 96, torch.bfloat16, DEV, seed=21, g_scale=0.02)
    ll, accs = make_layer_list(data, DEV)
    n, c, ws = gpu_norms_clip(ll, 1e30)
    assert torch.all(c == 1.0)
    b.dp_clipped_accumulate(ll, c, ws)
    A = to_np(data[0].A).reshape(-1, 128)
    G = to_np(data[0].G).reshape(-1, 192)
    assert rel_l2(to_np(accs[0][0]), A.T @ G) <= 1e-5
    assert rel_l2(to_np(accs[0][1]), G.sum(0)) <= 1e-5


def test_out_of_range_token_id_is_skipped_and_reported():
    data = random_layers([SMALL[3]], 2, 16, torch.float32, DEV, seed=2)
    data[0].ids[0, 3] = 50          # == V
    data[0].ids[1, 0] = -1
    ll, accs = make_layer_list(data, DEV)
    n, c, ws = gpu_norms_clip(ll, 1e30)
    b.dp_clipped_accumulate(ll, c, ws)
    assert b.dp_poll_status() == -7
    assert b.dp_poll_status() == 0                     # sticky word is cleared by the poll
    ids = data[0].ids.cpu().numpy()
    G = to_np(data[0].G)
    E = np.zeros((50, 64))
    for i in range(2):
        for t in range(16):
            if 0 <= ids[i, t] < 50:
                E[ids[i, t]] += G[i, t]
    assert rel_l2(to_np(accs[0][0]), E) <= 1e-6


def test_embedding_mask_gram_equals_grouped_rows():
    """Token-id equality Gram (tensor cores) against the grouped-row kernel and the checker, heavy duplicates."""
    spec = [LayerSpec(EMBEDDING, 40, 128, False, "emb")]
    for B, T in ((5, 128), (3, 200), (4, 33)):
        data = random_layers(spec, B, T, torch.bfloat16, DEV, seed=T, g_scale=0.05, vocab_dup=9)
        n_ref = O.per_example_sqnorms(to_oracle_layers(data))
        got = {}
        for path in (b.DP_PATH_GRAM, b.DP_PATH_MATERIALIZED):
            ll, _ = make_layer_list(data, DEV, [path])
            n, _, _ = gpu_norms_clip(ll, 1.0)
            got[path] = to_np(n)
            np.testing.assert_allclose(got[path], n_ref, rtol=2 * CLIP_TOL)
        np.testing.assert_allclose(got[b.DP_PATH_GRAM], got[b.DP_PATH_MATERIALIZED], rtol=1e-4)
    assert b.dp_poll_status() == 0
    assert len(b.dp_last_timeout_info()) == 5


def test_embedding_mask_counts_equal_pairs_exactly():
    """G of all ones makes every entry of G G^T equal d, so the embedding norm is d times the NUMBER of token pairs
    with equal ids: an integer that fp32 holds exactly.  The id compares inside the norm kernels (the mask applied
    to the Gram in the tensor-core kernel's epilogue, and the grouping of equal ids in the CUDA-core kernel) must
    reproduce it bit for bit."""
    for B, T, d, V, dup in ((6, 128, 128, 40, 9), (3, 200, 64, 500, 30), (4, 33, 192, 11, 11), (2, 300, 128, 7, 3)):
        spec = [LayerSpec(EMBEDDING, V, d, False, "emb")]
        data = random_layers(spec, B, T, torch.bfloat16, DEV, seed=T + d, g_scale=1.0, vocab_dup=dup)
        data[0].G.fill_(1.0)
        ids = data[0].ids.cpu().numpy()
        pairs = np.array([int((row[:, None] == row[None, :]).sum()) for row in ids], dtype=np.int64)
        assert pairs.max() * d < 2 ** 24
        for path in (b.DP_PATH_GRAM, b.DP_PATH_MATERIALIZED):
            ll, _ = make_layer_list(data, DEV, [path])
            n, _, _ = gpu_norms_clip(ll, 1.0)
            got = n.cpu().numpy().astype(np.float64)
            assert np.array_equal(got, (pairs * d).astype(np.float64)), (path, T, got, pairs * d)
        # the checker agrees with the count as well
        np.testing.assert_array_equal(O.per_example_sqnorms(to_oracle_layers(data)), (pairs * d).astype(np.float64))
    assert b.dp_poll_status() == 0


def test_unsplit_accumulate_is_bitwise_repeatable():
    """With no example split every accumulator element has one owner and a fixed summation order, so repeated runs
    with clip factors other than 1 (every stage of G rescaled in shared memory before the tensor cores read it)
    must agree bit for bit; a stage consumed before its scaling was visible would show up as a difference."""
    specs = []
    for blk in range(2):
        specs += [LayerSpec(LINEAR, 1024, 3072, True, f"qkv{blk}"), LayerSpec(LINEAR, 1024, 1024, True, f"o{blk}"),
                  LayerSpec(LINEAR, 1024, 4096, True, f"f1{blk}"), LayerSpec(LINEAR, 4096, 1024, True, f"f2{blk}")]
    B, T = 24, 128
    data = random_layers(specs, B, T, torch.bfloat16, DEV, seed=91, g_scale=0.02)
    ll, accs = make_layer_list(data, DEV)
    units = torch.cuda.get_device_properties(0).multi_processor_count // 2
    sched = b.dp_accumulate_schedule(ll, units)
    assert sched["splits"] == [1], sched                 # the case this test is about
    g = torch.Generator().manual_seed(4)
    clip = (0.05 + 0.9 * torch.rand(B, generator=g)).to(DEV)
    ws = b.alloc_workspace(ll)
    first = None
    for rep in range(6):
        for acc in accs:
            for x in acc:
                x.zero_()
        b.dp_clipped_accumulate(ll, clip, ws)
        torch.cuda.synchronize()
        snap = [[x.clone() for x in acc] for acc in accs]
        if first is None:
            first = snap
        else:
            for sp, a0, a1 in zip(specs, first, snap):
                for x, y in zip(a0, a1):
                    assert torch.equal(x, y), f"{sp.name}: run {rep} differs from run 0"
    assert b.dp_poll_status() == 0
    # and the result is the checker's on a few sampled entries per layer (fp64 on the host)
    c = to_np(clip)
    w = np.repeat(c, T)
    rng = np.random.default_rng(0)
    for ld, acc in zip(data, first):
        for _ in range(4):
            p, q = int(rng.integers(ld.spec.d_in)), int(rng.integers(ld.spec.d_out))
            ref = float(np.sum(w * to_np(ld.A[:, :, p]).reshape(-1) * to_np(ld.G[:, :, q]).reshape(-1)))
            scale = float(np.sqrt(np.sum((w * to_np(ld.A[:, :, p]).reshape(-1) * to_np(ld.G[:, :, q]).reshape(-1)) ** 2)))
            assert abs(float(acc[0][p, q]) - ref) <= 0.01 * scale + 1e-12


@pytest.mark.parametrize("dtype,slack", [(torch.bfloat16, 2.0 ** -8), (torch.float32, 1e-5)])
def test_each_clipped_contribution_is_bounded_by_C(dtype, slack):
    """The sensitivity that the noise is calibrated to: one example's clipped contribution to the whole accumulator
    (every layer kind) has norm at most C -- up to the rounding of c * G to bf16 on the tensor-core path (2^-9 per
    element, hence per norm) plus the 1e-3 tolerance of the clip factor's own norm.  One example per call, so the
    accumulator IS that contribution."""
    specs = SMALL + WIDE[:2]
    C = 0.37
    for seed in range(4):
        data = random_layers(specs, 1, 96, dtype, DEV, seed=400 + seed, g_scale=3.0, vocab_dup=5)
        ll, accs = make_layer_list(data, DEV)
        n, c, ws = gpu_norms_clip(ll, C)
        assert float(c[0]) < 1.0                              # the example clips
        b.dp_clipped_accumulate(ll, c, ws)
        total = np.sqrt(sum(float((x.double() ** 2).sum()) for acc in accs for x in acc))
        n_ref = float(O.per_example_sqnorms(to_oracle_layers(data))[0])
        true_c = min(1.0, C / np.sqrt(n_ref))
        assert total <= C * (1 + slack) * (float(c[0]) / true_c), (total, C)
        assert total <= C * (1 + slack + CLIP_TOL)
        assert total >= C * (1 - slack - CLIP_TOL)            # and it is not over-clipped either
    assert b.dp_poll_status() == 0


def test_workspace_too_small_is_refused():
    data = random_layers(SMALL, 2, 16, torch.bfloat16, DEV, seed=2)
    ll, _ = make_layer_list(data, DEV)
    need = b.dp_workspace_bytes(ll)
    assert need > 0
    n = torch.empty(2, dtype=torch.float32, device=DEV)
    with pytest.raises(b.DpError) as e:
        b.dp_per_example_sqnorms(ll, n, False, torch.empty(need - 1, dtype=torch.uint8, device=DEV))
    assert e.value.code == -6
