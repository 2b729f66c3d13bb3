"""GPU parity: Philox words, equality masks, noise + scaling, AdamW, fused pass -- all through the C ABI,
element by element against the CPU checker on the same seeded inputs."""
import numpy as np
import pytest
import torch

from .helpers import O, b, rel_l2, rel_max, to_np

pytestmark = pytest.mark.gpu

if not torch.cuda.is_available():
    pytest.skip("needs a CUDA device", allow_module_level=True)

DEV = "cuda:0"
F32_TOL = 1e-4        # fp32 paths: relative error bound stated for this step


@pytest.mark.parametrize("n,off,seed,step", [
    (10007, 0, 0, 0),
    (4099, 5, 0xDEADBEEF12345678, (7 << 32) | 11),
    (2051, (1 << 34) + 3, 1, 2),        # block index crosses into the second counter word
    (1, 2, 3, 4),
])
def test_philox_words_bit_exact(n, off, seed, step):
    out = torch.empty(n, dtype=torch.int32, device=DEV)
    b.dp_philox_u32(out, off, seed, step)
    got = out.cpu().numpy().view(np.uint32)
    assert np.array_equal(got, O.philox_u32(n, off, seed, step))


def test_philox_independent_of_launch_split():
    whole = torch.empty(100_000, dtype=torch.int32, device=DEV)
    b.dp_philox_u32(whole, 13, 99, 5)
    parts = [torch.empty(k, dtype=torch.int32, device=DEV) for k in (1, 33_333, 66_666)]
    off = 13
    for p in parts:
        b.dp_philox_u32(p, off, 99, 5)
        off += p.numel()
    assert torch.equal(whole, torch.cat(parts))


def test_token_equality_mask_bit_exact():
    g = torch.Generator().manual_seed(3)
    ids = torch.randint(0, 9, (5, 37), generator=g, dtype=torch.int32)
    mask = torch.empty(5, 37, 37, dtype=torch.uint8, device=DEV)
    b.dp_token_equality_mask(ids.to(DEV), mask)
    ref = (ids[:, :, None] == ids[:, None, :]).to(torch.uint8)
    assert torch.equal(mask.cpu(), ref)


@pytest.mark.parametrize("n,off", [(1 << 20, 0), ((1 << 20) + 3, 0), (50_001, 7), (5, 2), (3, 1)])
def test_noise_and_scale_matches_checker(n, off):
    rng = np.random.default_rng(n + off)
    S = rng.standard_normal(n).astype(np.float32) * 3
    sigma, C, N, seed, step = 1.1, 0.7, 4096, 0xABCDEF0123, 3
    base = torch.zeros(n + 8, dtype=torch.float32, device=DEV)
    # a deliberately misaligned view when off is odd-ish: exercises the element-wise tail path
    acc = base[(off % 4):(off % 4) + n]
    acc.copy_(torch.from_numpy(S))
    b.dp_add_noise_and_scale(acc, sigma, C, N, seed, step, elem_offset=off)
    ref = O.add_noise_and_scale(S.astype(np.float64), sigma, C, N, seed, step, elem_offset=off)
    got = to_np(acc)
    assert rel_max(got, ref) <= F32_TOL
    assert rel_l2(got, ref) <= 1e-5
    # the noise itself: recover z and compare with the fp64 normals
    z = (got * N - S.astype(np.float64)) / (sigma * C)
    zr = O.standard_normals(n, off, seed, step)
    assert np.max(np.abs(z - zr)) <= 2e-5 * max(1.0, np.max(np.abs(zr))) + 6e-6 * np.max(np.abs(S)) / (sigma * C)
    # untouched guard elements
    assert float(base[(off % 4) + n:].abs().max()) == 0.0


def test_noise_same_draw_for_any_partition():
    n = 70_001
    a = torch.zeros(n, dtype=torch.float32, device=DEV)
    b.dp_add_noise_and_scale(a, 1.0, 1.0, 1, 42, 9, elem_offset=0)
    parts = torch.zeros(n, dtype=torch.float32, device=DEV)
    cuts = [0, 1, 4, 4099, 30_000, n]
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        b.dp_add_noise_and_scale(parts[lo:hi], 1.0, 1.0, 1, 42, 9, elem_offset=lo)
    assert torch.equal(a, parts)
    # another step gives another draw
    c = torch.zeros(n, dtype=torch.float32, device=DEV)
    b.dp_add_noise_and_scale(c, 1.0, 1.0, 1, 42, 10, elem_offset=0)
    assert not torch.equal(a, c)
    z = to_np(a)
    assert abs(z.mean()) < 5 / np.sqrt(n) and abs(z.var() - 1) < 5 * np.sqrt(2 / n)


def _adam_case(n, seed):
    rng = np.random.default_rng(seed)
    th = rng.standard_normal(n).astype(np.float32) * 0.02
    m = rng.standard_normal(n).astype(np.float32) * 1e-3
    v = (rng.standard_normal(n).astype(np.float32) * 1e-3) ** 2
    g = rng.standard_normal(n).astype(np.float32) * 1e-3
    g[::97] = 0.0
    return th, m, v, g


def _check_adam(got, ref, old_theta):
    th, m, v = got
    rt, rm, rv = ref
    assert rel_max(m, rm) <= F32_TOL and rel_max(v, rv) <= F32_TOL
    assert rel_max(th, rt) <= F32_TOL
    d, rd = th - old_theta, rt - old_theta
    # the update itself, not hidden behind theta: relative with a floor from fp32 rounding of theta
    floor = 1e-7 * np.max(np.abs(old_theta)) + 1e-7 * np.max(np.abs(rd))
    assert np.max(np.abs(d - rd)) <= F32_TOL * np.max(np.abs(rd)) + floor


@pytest.mark.parametrize("hp", [
    dict(lr=1e-3, b1=0.9, b2=0.999, xi=1e-11, wd=0.01, t=1),
    dict(lr=6.0902e-4, b1=0.75, b2=0.9, xi=1e-11, wd=1.0, t=7),      # the paper's tuned values (Table 1)
    dict(lr=6.0902e-4, b1=0.9, b2=0.999, xi=1e-11, wd=0.5, t=20000),
])
@pytest.mark.parametrize("n", [1 << 18, 1001])
def test_adamw_matches_checker(hp, n):
    th, m, v, g = _adam_case(n, n)
    if hp["t"] == 1:
        m[:] = 0
        v[:] = 0
    dth, dm, dv, dg = (torch.from_numpy(x.copy()).to(DEV) for x in (th, m, v, g))
    b.dp_adamw_step(dth, dm, dv, dg, hp["lr"], hp["b1"], hp["b2"], hp["xi"], hp["wd"], hp["t"])
    ref = O.adamw_step(th.astype(np.float64), m, v, g, hp["lr"], hp["b1"], hp["b2"], hp["xi"], hp["wd"], hp["t"])
    _check_adam((to_np(dth), to_np(dm), to_np(dv)), ref, th.astype(np.float64))
    assert torch.equal(dg.cpu(), torch.from_numpy(g))       # g is read-only


def test_adamw_zero_state_zero_gradient_stays_finite():
    n = 64
    th = torch.ones(n, device=DEV)
    z = torch.zeros(n, device=DEV)
    m, v = z.clone(), z.clone()
    b.dp_adamw_step(th, m, v, z, 1e-2, 0.9, 0.999, 1e-11, 0.5, 1)
    assert torch.isfinite(th).all()
    np.testing.assert_allclose(to_np(th), 1 - 1e-2 * 0.5, rtol=1e-6)


@pytest.mark.parametrize("n,off", [(1 << 19, 0), (77_777, 0), (4097, 6)])
def test_fused_pass_matches_split_calls_and_checker(n, off):
    th, m, v, _ = _adam_case(n, 5)
    rng = np.random.default_rng(9)
    S = rng.standard_normal(n).astype(np.float32) * 50
    hp = dict(lr=6.0902e-4, b1=0.9, b2=0.999, xi=1e-11, wd=0.5, t=3)
    sigma, C, N, seed, step = 1.0, 1.0, 2048, 77, 3
    # fused
    f = [torch.from_numpy(x.copy()).to(DEV) for x in (th, m, v, S)]
    b.dp_noise_scale_adamw_step(f[0], f[1], f[2], f[3], True, sigma, C, N, seed, step, hp["lr"], hp["b1"], hp["b2"],
                                hp["xi"], hp["wd"], hp["t"], elem_offset=off)
    assert float(f[3].abs().max()) == 0.0                   # accumulator cleared
    # split
    s = [torch.from_numpy(x.copy()).to(DEV) for x in (th, m, v, S)]
    b.dp_add_noise_and_scale(s[3], sigma, C, N, seed, step, elem_offset=off)
    b.dp_adamw_step(s[0], s[1], s[2], s[3], hp["lr"], hp["b1"], hp["b2"], hp["xi"], hp["wd"], hp["t"])
    for x, y in zip(f[:3], s[:3]):
        assert rel_max(to_np(x), to_np(y)) <= 1e-6
    g = O.add_noise_and_scale(S.astype(np.float64), sigma, C, N, seed, step, elem_offset=off)
    ref = O.adamw_step(th.astype(np.float64), m, v, g, hp["lr"], hp["b1"], hp["b2"], hp["xi"], hp["wd"], hp["t"])
    _check_adam(tuple(to_np(x) for x in f[:3]), ref, th.astype(np.float64))
    # zero_acc = 0 leaves the accumulator as it was
    k = [torch.from_numpy(x.copy()).to(DEV) for x in (th, m, v, S)]
    b.dp_noise_scale_adamw_step(k[0], k[1], k[2], k[3], False, sigma, C, N, seed, step, hp["lr"], hp["b1"],
                                hp["b2"], hp["xi"], hp["wd"], hp["t"], elem_offset=off)
    assert torch.equal(k[3].cpu(), torch.from_numpy(S))
    assert torch.equal(k[0], f[0])


def test_clip_factors_special_values():
    C = 3.2429e-3
    n = torch.tensor([0.0, C * C, 4 * C * C, 0.25 * C * C, 1e30, 1e-30], dtype=torch.float32, device=DEV)
    c = torch.empty_like(n)
    b.dp_clip_factors(n, C, c)
    ref = O.clip_factors(to_np(n), C)
    np.testing.assert_allclose(to_np(c), ref, rtol=1e-6)


@pytest.mark.parametrize("n,off", [(1 << 20, 0), (50_003, 5)])
def test_gradient_snr_sums_in_the_fused_pass(n, off):
    """Same update as the plain fused call, plus sum acc^2 and sum (sigma C z)^2 against the checker."""
    th, m, v, _ = _adam_case(n, 3)
    S = (np.random.default_rng(4).standard_normal(n) * 20).astype(np.float32)
    hp = dict(lr=6.0902e-4, b1=0.9, b2=0.999, xi=1e-11, wd=0.5, t=2)
    sigma, C, N, seed, step = 1.1, 0.9, 1024, 5, 2
    a = [torch.from_numpy(x.copy()).to(DEV) for x in (th, m, v, S)]
    b_ = [torch.from_numpy(x.copy()).to(DEV) for x in (th, m, v, S)]
    sums = torch.zeros(2, dtype=torch.float64, device=DEV)
    b.dp_noise_scale_adamw_step_snr(a[0], a[1], a[2], a[3], True, sigma, C, N, seed, step, hp["lr"], hp["b1"],
                                    hp["b2"], hp["xi"], hp["wd"], hp["t"], sums, elem_offset=off)
    b.dp_noise_scale_adamw_step(b_[0], b_[1], b_[2], b_[3], True, sigma, C, N, seed, step, hp["lr"], hp["b1"],
                                hp["b2"], hp["xi"], hp["wd"], hp["t"], elem_offset=off)
    for x, y in zip(a, b_):
        assert torch.equal(x, y)
    ref = O.gradient_snr_sums(S.astype(np.float64), sigma, C, seed, step, off)
    got = sums.cpu().numpy()
    assert got[0] == pytest.approx(ref[0], rel=1e-5) and got[1] == pytest.approx(ref[1], rel=1e-4)
    # accumulates across calls (tensors of one macro-batch)
    c = [torch.from_numpy(x.copy()).to(DEV) for x in (th, m, v, S)]
    b.dp_noise_scale_adamw_step_snr(c[0], c[1], c[2], c[3], False, sigma, C, N, seed, step, hp["lr"], hp["b1"],
                                    hp["b2"], hp["xi"], hp["wd"], hp["t"], sums, elem_offset=off)
    np.testing.assert_allclose(sums.cpu().numpy(), 2 * got, rtol=1e-9)


def test_clip_stats_matches_checker():
    g = torch.Generator().manual_seed(1)
    for B in (1, 33, 256, 1000):
        clip = torch.where(torch.rand(B, generator=g) < 0.4, torch.ones(B), torch.rand(B, generator=g)).to(DEV)
        out = torch.empty(2, dtype=torch.float32, device=DEV)
        b.dp_clip_stats(clip, out)
        np.testing.assert_allclose(to_np(out), O.clip_stats(to_np(clip)), rtol=1e-5)


@pytest.mark.parametrize("n_flat,world", [(40_003, 3), (1 << 18, 8), (7, 2)])
def test_fused_cross_rank_update_matches_checker(n_flat, world):
    """Virtual ranks on one GPU: every rank has a full accumulator and a full replica of theta; the shard owners
    run dp_reduce_noise_adamw_step one after the other (no launch waits for another).  Afterwards every replica
    holds the checker's update of the SUMMED accumulator and every accumulator is zero."""
    from paper_2108_01624_b200.parallel import shard_bounds
    rng = np.random.default_rng(n_flat + world)
    hp = dict(sigma=0.9, C=0.5, N=4096, seed=0x1234567, step=5, lr=1e-3, b1=0.9, b2=0.999, xi=1e-11, wd=0.1, t=3)
    accs = [rng.standard_normal(n_flat).astype(np.float32) for _ in range(world)]
    th0 = rng.standard_normal(n_flat).astype(np.float32)
    m0 = (rng.standard_normal(n_flat) * 0.1).astype(np.float32)
    v0 = (rng.random(n_flat) * 0.01).astype(np.float32)
    acc_d = [torch.from_numpy(a).to(DEV) for a in accs]
    th_d = [torch.from_numpy(th0).to(DEV) for _ in range(world)]
    m_d = [torch.from_numpy(m0).to(DEV) for _ in range(world)]
    v_d = [torch.from_numpy(v0).to(DEV) for _ in range(world)]
    for r in range(world):
        lo, hi = shard_bounds(n_flat, world, r)
        if hi <= lo:
            continue
        b.dp_reduce_noise_adamw_step(th_d[r][lo:hi], m_d[r][lo:hi], v_d[r][lo:hi], [a[lo:hi] for a in acc_d],
                                     [t[lo:hi] for t in th_d], True, hp["sigma"], hp["C"], hp["N"], hp["seed"],
                                     hp["step"], hp["lr"], hp["b1"], hp["b2"], hp["xi"], hp["wd"], hp["t"],
                                     elem_offset=lo)
    torch.cuda.synchronize()
    total = np.sum(np.stack([a.astype(np.float64) for a in accs]), axis=0)
    g = O.add_noise_and_scale(total, hp["sigma"], hp["C"], hp["N"], seed=hp["seed"], step=hp["step"], elem_offset=0)
    rt, rm, rv = O.adamw_step(th0.astype(np.float64), m0.astype(np.float64), v0.astype(np.float64), g, hp["lr"],
                              hp["b1"], hp["b2"], hp["xi"], hp["wd"], hp["t"])
    for r in range(world):
        assert torch.equal(th_d[r], th_d[0])                      # every replica got the same bits
        assert float(acc_d[r].abs().max()) == 0.0
        lo, hi = shard_bounds(n_flat, world, r)
        if hi > lo:
            assert rel_max(to_np(m_d[r][lo:hi]), rm[lo:hi]) <= F32_TOL
            assert rel_max(to_np(v_d[r][lo:hi]), rv[lo:hi]) <= F32_TOL
    d, rd = to_np(th_d[0]) - th0, rt - th0
    assert np.max(np.abs(d - rd)) <= F32_TOL * np.max(np.abs(rd)) + 1e-7 * np.max(np.abs(th0))
    # and it is the single-GPU fused call on the summed accumulator, bit for bit, when the sum is exact
    if world == 2:
        th1, m1, v1 = (torch.from_numpy(x).to(DEV) for x in (th0, m0, v0))
        s = torch.from_numpy(accs[0]).to(DEV) + torch.from_numpy(accs[1]).to(DEV)
        b.dp_noise_scale_adamw_step(th1, m1, v1, s, True, hp["sigma"], hp["C"], hp["N"], hp["seed"], hp["step"],
                                    hp["lr"], hp["b1"], hp["b2"], hp["xi"], hp["wd"], hp["t"], 0)
        assert torch.equal(th1, th_d[0])


def test_fused_update_at_full_parameter_count_on_sampled_windows():
    """One fused launch over 333,563,904 parameters (the BERT-Large vector of the benchmark); the checker
    recomputes windows at the start, around 2^28 and 2^32 bytes into the vector, and at the ragged end."""
    n = 333_563_904
    hp = dict(sigma=0.9, C=0.5, N=2_097_152, seed=0xC0FFEE, step=7, lr=1e-3, b1=0.9, b2=0.999, xi=1e-11, wd=0.5, t=2)
    g = torch.Generator(device=DEV).manual_seed(5)
    acc = torch.randn(n, generator=g, device=DEV) * 100.0
    theta = torch.randn(n, generator=g, device=DEV) * 0.02
    m = torch.randn(n, generator=g, device=DEV) * 1e-5
    v = torch.rand(n, generator=g, device=DEV) * 1e-9
    windows = [(0, 4096), ((1 << 26) - 100, 300), ((1 << 28) + 1, 2047), (n - 4099, 4099)]
    before = {lo: tuple(to_np(x[lo:lo + k]) for x in (acc, theta, m, v)) for lo, k in windows}
    b.dp_noise_scale_adamw_step(theta, m, v, acc, True, hp["sigma"], hp["C"], hp["N"], hp["seed"], hp["step"],
                                hp["lr"], hp["b1"], hp["b2"], hp["xi"], hp["wd"], hp["t"], 0)
    torch.cuda.synchronize()
    assert float(acc.abs().max()) == 0.0
    for lo, k in windows:
        a0, t0, m0, v0 = before[lo]
        gref = O.add_noise_and_scale(a0, hp["sigma"], hp["C"], hp["N"], seed=hp["seed"], step=hp["step"], elem_offset=lo)
        rt, rm, rv = O.adamw_step(t0, m0, v0, gref, hp["lr"], hp["b1"], hp["b2"], hp["xi"], hp["wd"], hp["t"])
        assert rel_max(to_np(m[lo:lo + k]), rm) <= F32_TOL and rel_max(to_np(v[lo:lo + k]), rv) <= F32_TOL
        d, rd = to_np(theta[lo:lo + k]) - t0, rt - t0
        assert np.max(np.abs(d - rd)) <= F32_TOL * np.max(np.abs(rd)) + 1e-7 * np.max(np.abs(t0))
