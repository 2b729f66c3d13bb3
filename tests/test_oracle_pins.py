"""Pins for the CPU checker: every function is tied to something other than itself
(a textbook routine, a closed form, brute force, published vectors, an independent
library generator, distribution moments).  No GPU is needed."""
import ctypes
import math
import os

import numpy as np
import pytest

from oracle import dp_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _layers(rng, B=3, T=5, d_in=4, d_out=6, V=7, dup=False):
    lin = O.OracleLayer(O.LINEAR, G=rng.standard_normal((B, T, d_out)),
                        A=rng.standard_normal((B, T, d_in)), has_bias=True)
    lin2 = O.OracleLayer(O.LINEAR, G=rng.standard_normal((B, T, d_in)),
                         A=rng.standard_normal((B, T, d_out)), has_bias=False)
    ln = O.OracleLayer(O.LAYERNORM, G=rng.standard_normal((B, T, d_out)),
                       A=rng.standard_normal((B, T, d_out)))
    ids = rng.integers(0, 3 if dup else V, size=(B, T))
    emb = O.OracleLayer(O.EMBEDDING, G=rng.standard_normal((B, T, d_out)), ids=ids, vocab=V)
    return [lin, lin2, ln, emb]


# ---------------------------------------------------------------- per-example gradients

def test_per_example_gradient_matches_scalar_loops(rng):
    """Brute force with Python loops: catches a transposed operand or a wrong index."""
    layers = _layers(rng, B=2, T=3, d_in=2, d_out=3, V=4, dup=True)
    for layer in layers:
        for i in range(2):
            got = O.per_example_gradient(layer, i)
            T, d_out = layer.G.shape[1:]
            if layer.kind == O.LINEAR:
                d_in = layer.A.shape[2]
                W = [[sum(layer.A[i, t, p] * layer.G[i, t, q] for t in range(T)) for q in range(d_out)]
                     for p in range(d_in)]
                assert got[0].shape == (d_in, d_out)
                np.testing.assert_allclose(got[0], np.array(W), rtol=1e-13, atol=1e-13)
                if layer.has_bias:
                    b = [sum(layer.G[i, t, q] for t in range(T)) for q in range(d_out)]
                    np.testing.assert_allclose(got[1], np.array(b), rtol=1e-13, atol=1e-13)
                else:
                    assert len(got) == 1
            elif layer.kind == O.LAYERNORM:
                gam = [sum(layer.A[i, t, q] * layer.G[i, t, q] for t in range(T)) for q in range(d_out)]
                bet = [sum(layer.G[i, t, q] for t in range(T)) for q in range(d_out)]
                np.testing.assert_allclose(got[0], np.array(gam), rtol=1e-13, atol=1e-13)
                np.testing.assert_allclose(got[1], np.array(bet), rtol=1e-13, atol=1e-13)
            else:
                E = np.zeros((layer.vocab, d_out))
                for t in range(T):
                    for q in range(d_out):
                        E[layer.ids[i, t], q] += layer.G[i, t, q]
                np.testing.assert_allclose(got[0], E, rtol=1e-13, atol=1e-13)


def test_sqnorm_equals_gram_identity_and_brute_force(rng):
    """||A^T G||_F^2 + ||1^T G||^2 = <A A^T + 1 1^T, G G^T>; LayerNorm and embedding analogues."""
    layers = _layers(rng, B=4, T=8, d_in=16, d_out=12, V=9, dup=True)
    for layer in layers:
        n = O.per_example_sqnorms([layer])
        for i in range(4):
            G = layer.G[i]
            Q = G @ G.T
            if layer.kind == O.LINEAR:
                P = layer.A[i] @ layer.A[i].T
                if layer.has_bias:
                    P = P + 1.0
                ref = float(np.sum(P * Q))
            elif layer.kind == O.LAYERNORM:
                X = layer.A[i]
                ref = sum(float(np.sum(X[:, q] * G[:, q]) ** 2 + np.sum(G[:, q]) ** 2) for q in range(G.shape[1]))
            else:
                mask = (layer.ids[i][:, None] == layer.ids[i][None, :]).astype(np.float64)
                ref = float(np.sum(mask * Q))
            assert n[i] == pytest.approx(ref, rel=1e-12)


def test_embedding_sqnorm_degenerate_ids(rng):
    G = rng.standard_normal((2, 6, 5))
    same = O.OracleLayer(O.EMBEDDING, G=G, ids=np.full((2, 6), 3), vocab=8)
    distinct = O.OracleLayer(O.EMBEDDING, G=G, ids=np.tile(np.arange(6), (2, 1)), vocab=8)
    np.testing.assert_allclose(O.per_example_sqnorms([same]), (G.sum(1) ** 2).sum(1), rtol=1e-12)
    np.testing.assert_allclose(O.per_example_sqnorms([distinct]), (G ** 2).sum((1, 2)), rtol=1e-12)


def test_rank_one_closed_form(rng):
    """A_i = 1 a^T, G_i = 1 b^T  =>  A_i^T G_i = T a b^T: weight part T^2|a|^2|b|^2, bias part T^2|b|^2."""
    T, a, b = 7, rng.standard_normal(5), rng.standard_normal(3)
    layer = O.OracleLayer(O.LINEAR, A=np.tile(a, (1, T, 1)), G=np.tile(b, (1, T, 1)), has_bias=True)
    n = O.per_example_sqnorms([layer])[0]
    assert n == pytest.approx(T * T * (a @ a) * (b @ b) + T * T * (b @ b), rel=1e-12)


def test_sqnorm_sums_over_layers(rng):
    layers = _layers(rng)
    total = O.per_example_sqnorms(layers)
    parts = sum(O.per_example_sqnorms([l]) for l in layers)
    np.testing.assert_allclose(total, parts, rtol=1e-12)


# ---------------------------------------------------------------- clip factors and the clipped sum

def test_clip_factor_special_values():
    C = 3.2429e-3   # the paper's tuned clipping norm (Table 1)
    n = np.array([0.0, C * C, 4 * C * C, 0.25 * C * C, 1e30])
    c = O.clip_factors(n, C)
    np.testing.assert_allclose(c, [1.0, 1.0, 0.5, 1.0, C / 1e15], rtol=1e-12)


def test_no_clipping_equals_batch_gemm(rng):
    """C -> infinity: the clipped sum is the ordinary batch gradient, a textbook GEMM."""
    layers = _layers(rng, B=5, T=4, d_in=6, d_out=3, V=8, dup=True)
    c = O.clip_factors(O.per_example_sqnorms(layers), 1e30)
    assert np.all(c == 1.0)
    accs = O.clipped_accumulate(layers, c, O.zero_accumulators(layers))
    for layer, acc in zip(layers, accs):
        Gf = layer.G.reshape(-1, layer.G.shape[2])
        if layer.kind == O.LINEAR:
            Af = layer.A.reshape(-1, layer.A.shape[2])
            np.testing.assert_allclose(acc[0], Af.T @ Gf, rtol=1e-12, atol=1e-12)
            if layer.has_bias:
                np.testing.assert_allclose(acc[1], Gf.sum(0), rtol=1e-12, atol=1e-12)
        elif layer.kind == O.LAYERNORM:
            Xf = layer.A.reshape(Gf.shape)
            np.testing.assert_allclose(acc[0], (Xf * Gf).sum(0), rtol=1e-12, atol=1e-12)
            np.testing.assert_allclose(acc[1], Gf.sum(0), rtol=1e-12, atol=1e-12)
        else:
            E = np.zeros((layer.vocab, Gf.shape[1]))
            np.add.at(E, layer.ids.reshape(-1), Gf)
            np.testing.assert_allclose(acc[0], E, rtol=1e-12, atol=1e-12)


def test_each_clipped_contribution_is_bounded(rng):
    layers = _layers(rng, B=6)
    n = O.per_example_sqnorms(layers)
    C = float(np.sqrt(np.median(n)))          # about half the examples clip
    c = O.clip_factors(n, C)
    assert 0 < np.sum(c < 1.0) < len(c)
    for i in range(6):
        sq = sum(float(np.sum((c[i] * g) ** 2)) for l in layers for g in O.per_example_gradient(l, i))
        assert math.sqrt(sq) <= C * (1 + 1e-12)
        if n[i] < C * C:
            assert c[i] == 1.0              # short gradients pass unscaled
        else:
            assert math.sqrt(sq) == pytest.approx(C, rel=1e-12)


def test_accumulation_is_linear_and_permutation_invariant(rng):
    layers = _layers(rng, B=6)
    c = O.clip_factors(O.per_example_sqnorms(layers), 2.0)
    full = O.clipped_accumulate(layers, c, O.zero_accumulators(layers))

    def sub(rows):
        return [O.OracleLayer(l.kind, G=l.G[rows], A=None if l.A is None else l.A[rows],
                              ids=None if l.ids is None else l.ids[rows], has_bias=l.has_bias, vocab=l.vocab)
                for l in layers]
    two = O.zero_accumulators(layers)
    for rows in (slice(0, 2), slice(2, 6)):           # two microbatches into the same accumulators
        part = sub(rows)
        O.clipped_accumulate(part, O.clip_factors(O.per_example_sqnorms(part), 2.0), two)
    perm = rng.permutation(6)
    shuffled = sub(perm)
    shuf = O.clipped_accumulate(shuffled, O.clip_factors(O.per_example_sqnorms(shuffled), 2.0),
                                O.zero_accumulators(layers))
    for a, b, s in zip(full, two, shuf):
        for x, y, z in zip(a, b, s):
            np.testing.assert_allclose(x, y, rtol=1e-12, atol=1e-13)
            np.testing.assert_allclose(x, z, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- Philox and the normal draw

def _kat():
    rows = []
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([int(x, 16) for x in line.split()])
    return rows


def test_philox_known_answers():
    rows = _kat()
    assert len(rows) >= 3
    for r in rows:
        out = O.philox4x32_10(np.array(r[0:4]), r[4:6])
        assert [int(x) for x in out] == r[6:10]


def _curand_host():
    for name in ("libcurand.so", "libcurand.so.10", "/usr/local/cuda/lib64/libcurand.so"):
        try:
            return ctypes.CDLL(name)
        except OSError:
            continue
    try:
        import nvidia.curand
        return ctypes.CDLL(os.path.join(os.path.dirname(nvidia.curand.__file__), "lib", "libcurand.so.10"))
    except Exception:
        return None


def test_philox_matches_independent_library_generator():
    """cuRAND's HOST Philox4_32_10 stream (no GPU involved): block b of the stream is the
    bijection at counter (b >> 16, 0, b & 0xffff, 0) under key (lo32(seed), hi32(seed))."""
    lib = _curand_host()
    if lib is None:
        pytest.skip("libcurand not loadable")
    gen = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) != 0:
        pytest.skip("host generator unavailable")
    seed = 0x0123456789ABCDEF
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    nb = 70000
    buf = (ctypes.c_uint32 * (4 * nb))()
    assert lib.curandGenerate(gen, buf, ctypes.c_size_t(4 * nb)) == 0
    lib.curandDestroyGenerator(gen)
    got = np.frombuffer(buf, dtype=np.uint32).reshape(nb, 4)
    b = np.arange(nb)
    ctr = np.stack([b >> 16, np.zeros_like(b), b & 0xFFFF, np.zeros_like(b)], axis=1)
    ref = O.philox4x32_10(ctr, (seed & 0xFFFFFFFF, seed >> 32))
    assert np.array_equal(got, ref)


def test_philox_element_indexing():
    """Element e uses lane e & 3 of block e >> 2, counter (lo(j), hi(j), lo(step), hi(step))."""
    seed, step = 0xDEADBEEF12345678, (5 << 32) | 9
    e0 = (1 << 34) + 6                       # crosses into the high counter word, odd lane start
    w = O.philox_u32(11, e0, seed, step)
    for k in range(11):
        e = e0 + k
        j = e >> 2
        blk = O.philox4x32_10(np.array([j & 0xFFFFFFFF, j >> 32, 9, 5]), (0x12345678, 0xDEADBEEF))
        assert int(w[k]) == int(blk[e & 3])
    # any split of a range gives the same words
    whole = O.philox_u32(1000, 3, 7, 1)
    parts = np.concatenate([O.philox_u32(333, 3, 7, 1), O.philox_u32(667, 336, 7, 1)])
    assert np.array_equal(whole, parts)


def test_uniform_extremes_are_finite():
    """u1 lies in (0, 1]: word 0 gives 2^-33, word 2^32-1 gives exactly 1; |z| <= sqrt(66 ln 2)."""
    z = O.standard_normals(4096, 0, 1, 1)
    assert np.all(np.isfinite(z))
    assert np.max(np.abs(z)) <= math.sqrt(66 * math.log(2)) + 1e-9
    u1_min = np.float32(np.float32(0) * np.float32(2.0 ** -32) + np.float32(2.0 ** -33))
    u1_max = np.float32(np.float32(0xFFFFFFFF) * np.float32(2.0 ** -32) + np.float32(2.0 ** -33))
    assert u1_min == np.float32(2.0 ** -33) and u1_max == np.float32(1.0)


def test_normal_moments_and_ks():
    from scipy import stats
    n = 10_000_000
    z = O.standard_normals(n, 0, 2024, 3)
    assert abs(z.mean()) < 5 / math.sqrt(n)
    assert abs(z.var() - 1.0) < 5 * math.sqrt(2.0 / n)
    assert abs(stats.skew(z)) < 5 * math.sqrt(6.0 / n)
    assert abs(stats.kurtosis(z)) < 5 * math.sqrt(24.0 / n)
    # even (cos) and odd (sin) lanes separately, and their independence
    assert abs(np.mean(z[0::2] * z[1::2])) < 5 / math.sqrt(n / 2)
    assert stats.kstest(z[:1_000_000], "norm").pvalue > 1e-4
    # different steps / seeds give different, uncorrelated streams
    z2 = O.standard_normals(1_000_000, 0, 2024, 4)
    assert abs(np.mean(z[:1_000_000] * z2)) < 5 / math.sqrt(1_000_000)


def test_noise_term_has_variance_sigma2_C2_over_N2(rng):
    S = rng.standard_normal(2_000_000)
    sigma, C, N = 1.1, 0.7, 4096
    g = O.add_noise_and_scale(S, sigma, C, N, seed=5, step=2)
    resid = g - S / N
    assert abs(resid.mean()) < 5 * sigma * C / N / math.sqrt(S.size)
    assert resid.var() == pytest.approx((sigma * C / N) ** 2, rel=5 * math.sqrt(2.0 / S.size))
    # sigma = 0 is the plain mean
    np.testing.assert_allclose(O.add_noise_and_scale(S, 0.0, C, N, 5, 2), S / N, rtol=1e-15)
    # the draw depends on the global element index only
    a = O.add_noise_and_scale(S[:1000], sigma, C, N, 5, 2, elem_offset=0)
    b = O.add_noise_and_scale(S[501:1000], sigma, C, N, 5, 2, elem_offset=501)
    np.testing.assert_array_equal(a[501:], b)


# ---------------------------------------------------------------- AdamW closed forms (Algorithm 1)

def test_adamw_first_step_closed_form(rng):
    th, g = rng.standard_normal(50), rng.standard_normal(50)
    lr, b1, b2, xi, wd = 6.0902e-4, 0.75, 0.9, 1e-11, 1.0        # the paper's tuned values
    t1, m1, v1 = O.adamw_step(th, np.zeros(50), np.zeros(50), g, lr, b1, b2, xi, wd, 1)
    np.testing.assert_allclose(m1, (1 - b1) * g, rtol=1e-14)
    np.testing.assert_allclose(v1, (1 - b2) * g * g, rtol=1e-14)
    np.testing.assert_allclose(t1, th - lr * (g / (np.abs(g) + xi) + wd * th), rtol=1e-12)


def test_adamw_zero_gradient_is_pure_decay():
    th = np.array([1.0, -2.0, 0.5])
    t1, m1, v1 = O.adamw_step(th, np.zeros(3), np.zeros(3), np.zeros(3), 1e-2, 0.9, 0.999, 1e-11, 0.5, 1)
    np.testing.assert_allclose(t1, th * (1 - 1e-2 * 0.5), rtol=1e-15)
    assert np.all(m1 == 0) and np.all(v1 == 0)


def test_adamw_constant_gradient_keeps_unit_ratio():
    """lambda = 0 and a constant g: m_hat = g and v_hat = g^2 at every t, so each step moves by
    -eta * sign(g) (up to xi); a wrong exponent in the bias correction breaks this at t >= 2."""
    g = np.array([0.3, -1.7, 2.5e-3])
    th, m, v = np.zeros(3), np.zeros(3), np.zeros(3)
    lr = 1e-3
    for t in range(1, 8):
        th, m, v = O.adamw_step(th, m, v, g, lr, 0.9, 0.999, 1e-11, 0.0, t)
        np.testing.assert_allclose(m / (1 - 0.9 ** t), g, rtol=1e-12)
        np.testing.assert_allclose(v / (1 - 0.999 ** t), g * g, rtol=1e-12)
        np.testing.assert_allclose(th, -lr * t * np.sign(g), rtol=1e-7)


def test_adamw_decay_is_scaled_by_learning_rate():
    """The decay term sits inside the parenthesis multiplied by eta: doubling eta doubles it."""
    th = np.array([2.0])
    z = np.zeros(1)
    a = O.adamw_step(th, z, z, z, 1e-2, 0.9, 0.999, 1e-11, 0.5, 1)[0]
    b = O.adamw_step(th, z, z, z, 2e-2, 0.9, 0.999, 1e-11, 0.5, 1)[0]
    assert (th - b)[0] == pytest.approx(2 * (th - a)[0], rel=1e-14)


# ---------------------------------------------------------------- whole step

def test_privatised_gradient_composes(rng):
    mb = [_layers(rng, B=3), _layers(rng, B=3)]
    g, clips = O.privatised_gradient(mb, C=1.5, sigma=0.0, seed=1, step=1)
    acc = O.zero_accumulators(mb[0])
    for layers, c in zip(mb, clips):
        O.clipped_accumulate(layers, c, acc)
    for ga, aa in zip(g, acc):
        for x, y in zip(ga, aa):
            np.testing.assert_allclose(x, y / 6.0, rtol=1e-14)
    # with noise: residual equals sigma*C*z/N at the flat offsets
    g2, _ = O.privatised_gradient(mb, C=1.5, sigma=2.0, seed=1, step=1)
    pos = 0
    for ga, gb in zip(g, g2):
        for x, y in zip(ga, gb):
            z = O.standard_normals(x.size, pos, 1, 1).reshape(x.shape)
            np.testing.assert_allclose(y - x, 2.0 * 1.5 * z / 6.0, rtol=1e-9, atol=1e-12)
            pos += x.size


# ---------------------------------------------------------------- gradient-SNR and clip statistics (Section 5.2.1)

def test_gradient_snr_sums_closed_forms(rng):
    n = 1_000_000
    S = rng.standard_normal(n) * 3.0
    sig2, noi2 = O.gradient_snr_sums(S, 1.3, 0.5, seed=8, step=2)
    assert sig2 == pytest.approx(float(S @ S), rel=1e-13)
    # ||sigma C z||^2 / (sigma^2 C^2 n) -> 1 (chi-square with n degrees of freedom)
    assert noi2 / ((1.3 * 0.5) ** 2 * n) == pytest.approx(1.0, abs=5 * math.sqrt(2.0 / n))
    # scaling the gradient by k scales the SNR by k; sigma scales it by 1/sigma
    s2, n2 = O.gradient_snr_sums(2 * S, 2.6, 0.5, seed=8, step=2)
    assert math.sqrt(s2 / n2) == pytest.approx(math.sqrt(sig2 / noi2), rel=1e-12)
    # additive over a partition when the offsets follow the flat layout
    a = O.gradient_snr_sums(S[:1234], 1.3, 0.5, 8, 2, 0)
    b = O.gradient_snr_sums(S[1234:], 1.3, 0.5, 8, 2, 1234)
    assert a[0] + b[0] == pytest.approx(sig2, rel=1e-12) and a[1] + b[1] == pytest.approx(noi2, rel=1e-12)
    # the noise term is the residual of add_noise_and_scale
    g = O.add_noise_and_scale(S[:5000], 1.3, 0.5, 7, 8, 2, 0)
    resid = g * 7 - S[:5000]
    assert float(resid @ resid) == pytest.approx(O.gradient_snr_sums(S[:5000], 1.3, 0.5, 8, 2, 0)[1], rel=1e-9)


def test_clip_stats_values():
    assert O.clip_stats(np.array([1.0, 1.0, 0.5, 0.25])) == (0.5, 0.6875)
    assert O.clip_stats(np.ones(7)) == (0.0, 1.0)


# ------------------------------------------------------------------ a table shared by embedding and output projection

def _shared_table_case(rng, B=3, T=5, T_out=4, V=7, d=6):
    emb = O.OracleLayer(kind=O.EMBEDDING, G=rng.standard_normal((B, T, d)), ids=rng.integers(0, V, (B, T)), vocab=V)
    proj = O.OracleLayer(kind=O.LINEAR, A=rng.standard_normal((B, T_out, V)), G=rng.standard_normal((B, T_out, d)))
    return emb, proj


def test_shared_table_gradient_matches_scalar_loops(rng):
    """dE[v, :] = sum_{t: id_t = v} G_emb[t, :] + sum_s dlogits[s, v] h[s, :], written out with scalar loops."""
    emb, proj = _shared_table_case(rng)
    B, T, d = emb.G.shape
    T_out, V = proj.A.shape[1], proj.A.shape[2]
    for i in range(B):
        ref = np.zeros((V, d))
        for t in range(T):
            for q in range(d):
                ref[emb.ids[i, t], q] += emb.G[i, t, q]
        for s in range(T_out):
            for v in range(V):
                for q in range(d):
                    ref[v, q] += proj.A[i, s, v] * proj.G[i, s, q]
        np.testing.assert_allclose(O.shared_table_gradient(emb, proj, i), ref, rtol=1e-12, atol=1e-12)


def test_shared_table_norm_is_the_parts_plus_twice_the_cross_term(rng):
    """Polarisation: ||s + d||^2 = ||s||^2 + ||d||^2 + 2 <s, d>, with the parts' norms taken from the functions
    pinned above, and <s, d> also by the token-pair form sum_{t,s} dlogits[s, id_t] <h[s], G_emb[t]>."""
    emb, proj = _shared_table_case(rng, B=4, T=6, T_out=3, V=5, d=8)     # V < T: ids repeat
    other = O.OracleLayer(kind=O.LAYERNORM, A=rng.standard_normal((4, 6, 8)), G=rng.standard_normal((4, 6, 8)))
    x = O.shared_table_cross_terms(emb, proj)
    n_sep = O.per_example_sqnorms([emb, other, proj])
    n_tied = O.per_example_sqnorms_shared_table([emb, other, proj], 0, 2)
    np.testing.assert_allclose(n_tied, n_sep + 2.0 * x, rtol=1e-12)
    for i in range(4):
        pair = 0.0
        for t in range(6):
            for s in range(3):
                pair += proj.A[i, s, emb.ids[i, t]] * float(np.dot(proj.G[i, s], emb.G[i, t]))
        assert abs(pair - x[i]) <= 1e-12 * max(1.0, abs(x[i]))
    assert np.max(np.abs(x)) > 1e-3            # the term is not negligible on random inputs


def test_shared_table_cross_term_closed_forms(rng):
    """One token with id k and one output position whose dlogits is alpha on vocabulary entry k': the scatter is
    g at row k, the dense part alpha h at row k', so <s, d> = alpha <h, g> if k' = k and 0 otherwise."""
    d, V = 5, 4
    g, h = rng.standard_normal(d), rng.standard_normal(d)
    for k, kp in ((2, 2), (2, 3)):
        emb = O.OracleLayer(kind=O.EMBEDDING, G=g.reshape(1, 1, d), ids=np.array([[k]]), vocab=V)
        A = np.zeros((1, 1, V))
        A[0, 0, kp] = 0.7
        proj = O.OracleLayer(kind=O.LINEAR, A=A, G=h.reshape(1, 1, d))
        x = O.shared_table_cross_terms(emb, proj)[0]
        assert abs(x - (0.7 * float(h @ g) if k == kp else 0.0)) <= 1e-14
    # zero output gradients: the shared table's norm is the embedding's alone
    emb, proj = _shared_table_case(rng)
    proj.A[:] = 0.0
    np.testing.assert_allclose(O.per_example_sqnorms_shared_table([emb, proj], 0, 1), O.per_example_sqnorms([emb]),
                               rtol=1e-12)


def test_shared_table_accumulates_into_one_tensor(rng):
    """Both layers add into the same [V, d] accumulator; with C -> infinity the result is the batch gradient of
    the table, scatter of all rows plus dlogits^T h over all examples and positions."""
    emb, proj = _shared_table_case(rng, B=5)
    accs = O.zero_accumulators([emb, proj])
    accs[1][0] = accs[0][0]                     # one tensor, two contributors
    O.clipped_accumulate([emb, proj], np.ones(5), accs)
    V, d = accs[0][0].shape
    ref = np.zeros((V, d))
    np.add.at(ref, emb.ids.reshape(-1), emb.G.reshape(-1, d))
    ref += proj.A.reshape(-1, V).T @ proj.G.reshape(-1, d)
    np.testing.assert_allclose(accs[0][0], ref, rtol=1e-12, atol=1e-12)
    # every clipped contribution of the shared table stays within C
    n = O.per_example_sqnorms_shared_table([emb, proj], 0, 1)
    c = O.clip_factors(n, 0.5)
    for i in range(5):
        assert c[i] * np.linalg.norm(O.shared_table_gradient(emb, proj, i)) <= 0.5 * (1 + 1e-12)
