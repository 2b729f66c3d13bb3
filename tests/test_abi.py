"""CPU-only checks of the C-ABI library: it builds, loads, exports every declared symbol, and rejects
bad arguments on the host before touching a device."""
import ctypes as C
import os
import re

import pytest

from paper_2108_01624_b200 import binding as b
from paper_2108_01624_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    builder.build()
    return b.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "dp.h")).read()
    names = re.findall(r"DP_API\s+[\w\s\*]+?\b(dp_\w+)\s*\(", header)
    assert len(names) >= 12
    assert sorted(names) == sorted(b.EXPORTS)
    for n in names:
        assert hasattr(lib, n)


def test_status_strings_and_version(lib):
    assert lib.dp_version() >= 100
    assert b.status_string(0) == "ok"
    for code in range(-7, 0):
        assert b.status_string(code) not in ("ok", "unknown status")
    assert b.status_string(-99) == "unknown status"


def test_struct_layout_matches_header():
    assert C.sizeof(b.dp_layer) == 8 * 4 + 5 * 8
    assert b.dp_layer.A.offset == 32 and b.dp_layer.acc_b.offset == 64


def test_host_side_argument_validation(lib):
    """Null pointers, bad sizes and non-finite scalars are refused before any launch."""
    ARG = -1
    assert lib.dp_clip_factors(None, 4, 1.0, None, None) == ARG
    assert lib.dp_clip_factors(256, 0, 1.0, 512, None) == ARG
    assert lib.dp_clip_factors(256, 4, -1.0, 512, None) == ARG
    assert lib.dp_clip_factors(256, 4, float("nan"), 512, None) == ARG
    assert lib.dp_clip_factors(258, 4, 1.0, 512, None) == -2          # misaligned fp32 pointer
    assert lib.dp_add_noise_and_scale(None, 8, 0, 1.0, 1.0, 4, 0, 0, None) == ARG
    assert lib.dp_add_noise_and_scale(256, 8, 0, float("inf"), 1.0, 4, 0, 0, None) == ARG
    assert lib.dp_add_noise_and_scale(256, 8, 0, 1.0, 0.0, 4, 0, 0, None) == ARG
    assert lib.dp_add_noise_and_scale(256, 8, 0, 1.0, 1.0, 0, 0, 0, None) == ARG
    assert lib.dp_add_noise_and_scale(256, -1, 0, 1.0, 1.0, 4, 0, 0, None) == ARG
    assert lib.dp_add_noise_and_scale(None, 0, 0, 1.0, 1.0, 4, 0, 0, None) == 0   # empty range is a no-op
    assert lib.dp_adamw_step(256, 256, 256, 256, 8, 1e-3, 0.9, 0.999, 1e-11, 0.0, 0, None) == ARG   # t < 1
    assert lib.dp_adamw_step(256, 256, 256, 256, 8, 1e-3, 1.0, 0.999, 1e-11, 0.0, 1, None) == ARG   # beta1 = 1
    assert lib.dp_adamw_step(None, 256, 256, 256, 8, 1e-3, 0.9, 0.999, 1e-11, 0.0, 1, None) == ARG
    assert lib.dp_adamw_step(None, None, None, None, 0, 1e-3, 0.9, 0.999, 1e-11, 0.0, 1, None) == 0
    assert lib.dp_philox_u32(None, 4, 0, 0, 0, None) == ARG
    assert lib.dp_token_equality_mask(None, 1, 1, None, None) == ARG
    # layer lists
    L = (b.dp_layer * 2)()
    assert lib.dp_per_example_sqnorms(None, 1, 256, 0, None, 0, None) == ARG
    assert lib.dp_per_example_sqnorms(C.cast(L, C.c_void_p), 0, 256, 0, None, 0, None) == ARG
    for k in range(2):
        L[k].kind, L[k].dtype, L[k].B, L[k].T, L[k].d_in, L[k].d_out = 0, 0, 4, 8, 16, 16
        L[k].A, L[k].G = 1024, 2048
    p = C.cast(L, C.c_void_p)
    assert lib.dp_per_example_sqnorms(p, 2, None, 0, None, 0, None) == ARG       # no output
    L[1].B = 5
    assert lib.dp_per_example_sqnorms(p, 2, 256, 0, None, 0, None) == ARG       # B differs between layers
    L[1].B = 4
    L[1].A = None
    assert lib.dp_per_example_sqnorms(p, 2, 256, 0, None, 0, None) == ARG       # linear layer without A
    L[1].A = 1026
    assert lib.dp_per_example_sqnorms(p, 2, 256, 0, None, 0, None) == -2        # fp32 A not 4-byte aligned
    L[1].A = 1024
    L[1].kind = 7
    assert lib.dp_per_example_sqnorms(p, 2, 256, 0, None, 0, None) == ARG       # unknown kind
    L[1].kind = 2
    assert lib.dp_per_example_sqnorms(p, 2, 256, 0, None, 0, None) == ARG       # embedding without ids
    L[1].kind = 0
    assert lib.dp_clipped_accumulate(p, 2, 256, None, 0, None) == ARG           # accumulators missing
    assert lib.dp_workspace_bytes(p, 2) == 0                                    # nothing here needs scratch
    L[0].has_bias = 1
    assert lib.dp_workspace_bytes(p, 2) >= 4 * 16 * 4                           # bias column sums [B, d_out]
    L[0].acc_w, L[0].acc_b, L[1].acc_w = 4096, 8192, 4096
    assert lib.dp_clipped_accumulate(p, 2, 256, None, 0, None) == -6            # workspace missing


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(ImportError):
        b.lib()


def _fake_bf16_linears(shapes, B, T):
    """Descriptors with made-up (aligned) device addresses: enough for the host-only planning calls."""
    L = (b.dp_layer * len(shapes))()
    for k, (d_in, d_out) in enumerate(shapes):
        L[k].kind, L[k].dtype, L[k].has_bias, L[k].B, L[k].T, L[k].d_in, L[k].d_out = 0, 1, 1, B, T, d_in, d_out
        L[k].A, L[k].G = 1 << 20, 1 << 21
    return L


def _schedule(lib, L, units, max_launches=8):
    n = len(L)
    start, launch = (C.c_int64 * n)(), (C.c_int32 * n)()
    splits, slots = (C.c_int32 * max_launches)(), (C.c_int64 * max_launches)()
    rc = lib.dp_accumulate_schedule(C.cast(L, C.c_void_p), n, units, C.cast(start, C.c_void_p), C.cast(launch, C.c_void_p),
                                    C.cast(splits, C.c_void_p), C.cast(slots, C.c_void_p), max_launches)
    return rc, list(start), list(launch), list(splits), list(slots)


def _tiles(d_in, d_out):
    return -(-d_out // 256) * -(-d_in // 512)


def test_accumulate_schedule_bert_large_packs_layers_into_waves(lib):
    """96 linears of BERT-Large on 74 CTA pairs: 2304 tiles in 32 waves, no layer straddling a wave, no overlap."""
    block = [(1024, 3072), (1024, 1024), (1024, 4096), (4096, 1024)]
    shapes = block * 24
    rc, start, launch, splits, slots = _schedule(lib, _fake_bf16_linears(shapes, 256, 128), 74)
    assert rc == 1 and splits[0] == 1 and slots[0] == 32 * 74
    taken = set()
    for (d_in, d_out), s0 in zip(shapes, start):
        g = _tiles(d_in, d_out)
        assert s0 >= 0 and s0 // 74 == (s0 + g - 1) // 74          # inside one wave
        items = set(range(s0, s0 + g))
        assert not (items & taken)
        taken |= items
    assert len(taken) == 2304 and max(taken) < slots[0]


def test_accumulate_schedule_splits_large_groups_and_launches(lib):
    # a layer with more tiles than a wave takes whole waves; the small one shares its last wave
    rc, start, launch, splits, slots = _schedule(lib, _fake_bf16_linears([(512, 256), (4096, 4096)], 2, 64), 74)
    assert rc == 1 and splits[0] == 1
    assert start[1] == 0 and start[0] == 128 and slots[0] == 2 * 74
    # few tiles: the example range is split (<= B, <= 8) until the wave is at least 85 % full
    rc, start, launch, splits, slots = _schedule(lib, _fake_bf16_linears([(512, 256)] * 3, 6, 64), 74)
    assert rc == 1 and splits[0] == 6 and slots[0] == 74 and sorted(start) == [0, 6, 12]
    # more than 96 tensor-core layers: a second launch with a schedule of its own
    rc, start, launch, splits, slots = _schedule(lib, _fake_bf16_linears([(64, 64)] * 130, 3, 32), 74)
    assert rc == 2 and launch[:96] == [0] * 96 and launch[96:] == [1] * 34
    assert splits[:2] == [2, 2] and slots[:2] == [3 * 74, 74]      # 192 items in 3 waves, 68 items in 1
    assert sorted(start[:96]) == [2 * k for k in range(96)] and sorted(start[96:]) == [2 * k for k in range(34)]
    # widths that are multiples of 8 go to the tensor-core GEMM (a 72 x 40 layer is one tile); others are left out
    L = _fake_bf16_linears([(64, 64), (72, 40), (68, 40)], 3, 32)
    rc, start, launch, _, _ = _schedule(lib, L, 74)
    assert rc == 1 and launch[:2] == [0, 0] and start[0] != start[1] and start[2] == -1 and launch[2] == -1
    # argument checks
    assert lib.dp_accumulate_schedule(C.cast(L, C.c_void_p), 2, 0, 256, 256, 256, 256, 1) == -1


def test_fused_cross_rank_update_argument_checks(lib):
    ptrs2 = (C.c_void_p * 2)(4096, 8192)
    p2 = C.cast(ptrs2, C.c_void_p)
    ok = dict(n_ranks=2, zero=1, n=8, off=0)
    def call(theta=256, m=512, v=768, acc=p2, th=None, n_ranks=2, n=8, off=0, lr=1e-3, t=1):
        return lib.dp_reduce_noise_adamw_step(theta, m, v, acc, th, n_ranks, 1, n, off, 1.0, 1.0, 4, 0, 0, lr, 0.9, 0.999,
                                              1e-11, 0.0, t, None)
    assert call(acc=None) == -1
    assert call(n_ranks=0) == -1 and call(n_ranks=17) == -1
    assert call(t=0) == -1 and call(lr=float("nan")) == -1
    assert call(n=0) == 0                                   # empty shard: nothing to do
    assert call(theta=None) == -1
    assert call(off=2) == -2                                # shard must start on a Philox block
    assert call(theta=260) == -2                            # 16-byte alignment of every pointer
    bad = (C.c_void_p * 2)(4096, 8196)
    assert call(acc=C.cast(bad, C.c_void_p)) == -2
    null = (C.c_void_p * 2)(4096, None)
    assert call(acc=C.cast(null, C.c_void_p)) == -1
