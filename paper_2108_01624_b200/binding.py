"""ctypes binding of libdp_b200.so: the same entry points as include/dp.h, taking torch tensors.

Argument marshalling only -- every step runs in the library's CUDA kernels.  There is no CPU or
PyTorch fallback: if the shared library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# DP_B200_LIB selects another build of the library (e.g. one compiled with experimental -D flags).
LIB_PATH = os.environ.get("DP_B200_LIB") or os.path.join(_HERE, "libdp_b200.so")

DP_OK = 0
DP_LINEAR, DP_LAYERNORM, DP_EMBEDDING = 0, 1, 2
DP_F32, DP_BF16 = 0, 1
DP_PATH_AUTO, DP_PATH_GRAM, DP_PATH_MATERIALIZED = 0, 1, 2
_KINDS = {"linear": DP_LINEAR, "layernorm": DP_LAYERNORM, "embedding": DP_EMBEDDING}

EXPORTS = ["dp_workspace_bytes", "dp_per_example_sqnorms", "dp_clip_factors", "dp_clipped_accumulate", "dp_clipped_accumulate_after_sqnorms", "dp_accumulate_schedule", "dp_reduce_noise_adamw_step",
           "dp_add_noise_and_scale", "dp_adamw_step", "dp_noise_scale_adamw_step", "dp_noise_scale_adamw_step_snr",
           "dp_clip_stats", "dp_philox_u32", "dp_shared_table_cross_sqnorms",
           "dp_token_equality_mask", "dp_layernorm_sqnorms_static", "dp_poll_status", "dp_last_timeout_info", "dp_launch_count",
           "dp_set_wait_limit_cycles", "dp_selftest_wait_timeout",
           "dp_status_string", "dp_version"]


class dp_layer(C.Structure):
    _fields_ = [("kind", C.c_int32), ("dtype", C.c_int32), ("path", C.c_int32), ("has_bias", C.c_int32),
                ("B", C.c_int32), ("T", C.c_int32), ("d_in", C.c_int32), ("d_out", C.c_int32),
                ("A", C.c_void_p), ("ids", C.c_void_p), ("G", C.c_void_p),
                ("acc_w", C.c_void_p), ("acc_b", C.c_void_p)]


class DpError(RuntimeError):
    def __init__(self, fn: str, code: int):
        self.code = code
        super().__init__(f"{fn} failed: {code} ({status_string(code)})")


_lib = None


def lib() -> C.CDLL:
    """Load the shared library (built by paper_2108_01624_b200.build); fails loudly when absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} not found: run `python -m paper_2108_01624_b200.build` (needs nvcc). "
                              "There is no fallback implementation.")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u64, f32, sz = C.c_void_p, C.c_int, C.c_int64, C.c_uint64, C.c_double, C.c_size_t
        L.dp_workspace_bytes.restype = sz
        L.dp_workspace_bytes.argtypes = [vp, i32]
        L.dp_per_example_sqnorms.argtypes = [vp, i32, vp, i32, vp, sz, vp]
        L.dp_clip_factors.argtypes = [vp, i32, f32, vp, vp]
        L.dp_clipped_accumulate.argtypes = [vp, i32, vp, vp, sz, vp]
        L.dp_clipped_accumulate_after_sqnorms.argtypes = [vp, i32, vp, vp, sz, vp]
        L.dp_accumulate_schedule.argtypes = [vp, i32, i32, vp, vp, vp, vp, i32]
        L.dp_add_noise_and_scale.argtypes = [vp, i64, i64, f32, f32, i64, u64, u64, vp]
        L.dp_adamw_step.argtypes = [vp, vp, vp, vp, i64, f32, f32, f32, f32, f32, i64, vp]
        L.dp_noise_scale_adamw_step.argtypes = [vp, vp, vp, vp, i32, i64, i64, f32, f32, i64, u64, u64,
                                                f32, f32, f32, f32, f32, i64, vp]
        L.dp_reduce_noise_adamw_step.argtypes = [vp, vp, vp, vp, vp, i32, i32, i64, i64, f32, f32, i64, u64, u64,
                                                 f32, f32, f32, f32, f32, i64, vp]
        L.dp_noise_scale_adamw_step_snr.argtypes = [vp, vp, vp, vp, i32, i64, i64, f32, f32, i64, u64, u64,
                                                    f32, f32, f32, f32, f32, i64, vp, vp]
        L.dp_clip_stats.argtypes = [vp, i32, vp, vp]
        L.dp_philox_u32.argtypes = [vp, i64, i64, u64, u64, vp]
        L.dp_token_equality_mask.argtypes = [vp, i32, i32, vp, vp]
        L.dp_shared_table_cross_sqnorms.argtypes = [vp, vp, i32, i32, vp, vp, i32, i32, i32, i32, vp, vp]
        L.dp_layernorm_sqnorms_static.argtypes = [vp, vp, i32, vp]
        L.dp_poll_status.argtypes = [vp]
        L.dp_set_wait_limit_cycles.argtypes = [C.c_longlong]
        L.dp_selftest_wait_timeout.argtypes = [vp]
        L.dp_status_string.restype = C.c_char_p
        L.dp_status_string.argtypes = [i32]
        L.dp_version.restype = i32
        L.dp_launch_count.restype = C.c_longlong
        for name in EXPORTS:
            getattr(L, name)          # AttributeError if the library does not export it
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().dp_status_string(int(code)).decode()


def _check(fn: str, code: int):
    if code != DP_OK:
        raise DpError(fn, code)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("device tensor expected")
    if not t.is_contiguous():
        raise ValueError("contiguous tensor expected")
    return t.data_ptr()


def _stream(stream=None) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


@dataclass
class Layer:
    """Python-side layer description; tensors live on the GPU."""
    kind: str
    G: torch.Tensor
    A: Optional[torch.Tensor] = None
    ids: Optional[torch.Tensor] = None
    acc_w: Optional[torch.Tensor] = None
    acc_b: Optional[torch.Tensor] = None
    has_bias: bool = False
    vocab: int = 0
    path: int = DP_PATH_AUTO


class LayerList:
    """A HOST array of dp_layer descriptors plus references that keep the tensors alive."""

    def __init__(self, layers: Sequence[Layer]):
        self.layers = list(layers)
        self.array = (dp_layer * len(self.layers))()
        for k, L in enumerate(self.layers):
            d = self.array[k]
            B, T, d_out = L.G.shape
            if L.G.dtype not in (torch.float32, torch.bfloat16):
                raise ValueError("A and G must be fp32 or bf16")
            d.kind = _KINDS[L.kind]
            d.dtype = DP_F32 if L.G.dtype == torch.float32 else DP_BF16
            d.path = int(L.path)
            d.has_bias = int(bool(L.has_bias))
            d.B, d.T, d.d_out = B, T, d_out
            if L.kind == "embedding":
                if L.ids is None or L.ids.dtype != torch.int32:
                    raise ValueError("embedding needs int32 ids")
                d.d_in = int(L.vocab)
            else:
                if L.A is None or L.A.dtype != L.G.dtype:
                    raise ValueError("A must have G's dtype")
                d.d_in = L.A.shape[2]
            d.A, d.ids, d.G = _ptr(L.A), _ptr(L.ids), _ptr(L.G)
            d.acc_w, d.acc_b = _ptr(L.acc_w), _ptr(L.acc_b)
            for acc in (L.acc_w, L.acc_b):
                if acc is not None and acc.dtype != torch.float32:
                    raise ValueError("accumulators are fp32")

    @property
    def ptr(self):
        return C.cast(self.array, C.c_void_p)

    def __len__(self):
        return len(self.layers)

    @property
    def B(self) -> int:
        return int(self.array[0].B)


def dp_version() -> int:
    return lib().dp_version()


def dp_workspace_bytes(layers: LayerList) -> int:
    return int(lib().dp_workspace_bytes(layers.ptr, len(layers)))


def alloc_workspace(layers: LayerList) -> Optional[torch.Tensor]:
    """Caller-owned scratch for the two layer-list calls (torch's allocator aligns to 512 bytes)."""
    n = dp_workspace_bytes(layers)
    dev = layers.layers[0].G.device
    return torch.empty(max(n, 256), dtype=torch.uint8, device=dev)


def dp_per_example_sqnorms(layers: LayerList, sqnorm: torch.Tensor, accumulate_into: bool = False,
                           workspace: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    ws_p, ws_n = (_ptr(workspace), workspace.numel() * workspace.element_size()) if workspace is not None else (None, 0)
    _check("dp_per_example_sqnorms",
           lib().dp_per_example_sqnorms(layers.ptr, len(layers), _ptr(sqnorm), int(accumulate_into), ws_p, ws_n,
                                        _stream(stream)))
    return sqnorm


def dp_shared_table_cross_sqnorms(emb: Layer, proj: Layer, sqnorm: torch.Tensor, stream=None) -> torch.Tensor:
    """sqnorm[i] += 2 <scatter_i, dlogits_i^T h_i> for a table trained through the embedding layer `emb` and the
    output projection `proj` (a linear layer whose A is dlogits [B, T_out, V] and whose G is h [B, T_out, d])."""
    B, T, d = emb.G.shape
    _, T_out, V = proj.A.shape
    if emb.ids is None or emb.ids.dtype != torch.int32 or proj.A.dtype != emb.G.dtype or proj.G.dtype != emb.G.dtype:
        raise ValueError("embedding ids (int32) and one dtype for G_emb, dlogits and h expected")
    if proj.G.shape != (B, T_out, d) or int(emb.vocab) != V:
        raise ValueError("the projection must map [B, T_out, V] x [B, T_out, d] onto the embedding's [V, d] table")
    dtype = DP_F32 if emb.G.dtype == torch.float32 else DP_BF16
    _check("dp_shared_table_cross_sqnorms",
           lib().dp_shared_table_cross_sqnorms(_ptr(emb.ids), _ptr(emb.G), B, T, _ptr(proj.A), _ptr(proj.G), T_out, d, V,
                                               dtype, _ptr(sqnorm), _stream(stream)))
    return sqnorm


def dp_clip_factors(sqnorm: torch.Tensor, C_: float, clip: torch.Tensor, stream=None) -> torch.Tensor:
    _check("dp_clip_factors", lib().dp_clip_factors(_ptr(sqnorm), sqnorm.numel(), float(C_), _ptr(clip), _stream(stream)))
    return clip


def dp_clipped_accumulate(layers: LayerList, clip: torch.Tensor, workspace: Optional[torch.Tensor] = None,
                          stream=None) -> None:
    ws_p, ws_n = (_ptr(workspace), workspace.numel() * workspace.element_size()) if workspace is not None else (None, 0)
    _check("dp_clipped_accumulate",
           lib().dp_clipped_accumulate(layers.ptr, len(layers), _ptr(clip), ws_p, ws_n, _stream(stream)))


def dp_clipped_accumulate_after_sqnorms(layers: LayerList, clip: torch.Tensor, workspace: Optional[torch.Tensor] = None,
                                        stream=None) -> None:
    """dp_clipped_accumulate for the call that directly follows dp_per_example_sqnorms over the same `layers`
    and `workspace`: the LayerNorm column sums left there are reused instead of being recomputed."""
    ws_p, ws_n = (_ptr(workspace), workspace.numel() * workspace.element_size()) if workspace is not None else (None, 0)
    _check("dp_clipped_accumulate_after_sqnorms",
           lib().dp_clipped_accumulate_after_sqnorms(layers.ptr, len(layers), _ptr(clip), ws_p, ws_n, _stream(stream)))


def dp_accumulate_schedule(layers: LayerList, units: int, max_launches: int = 16) -> dict:
    """Host-only view of the accumulate GEMM's work schedule on a device with `units` CTA pairs: per layer the first
    work item and the launch it belongs to (-1: the layer takes another path), per launch the number of example
    ranges a tile is split into and the number of item slots."""
    n = len(layers)
    start, launch = (C.c_int64 * n)(), (C.c_int32 * n)()
    splits, slots = (C.c_int32 * max_launches)(), (C.c_int64 * max_launches)()
    rc = lib().dp_accumulate_schedule(layers.ptr, n, int(units), C.cast(start, C.c_void_p), C.cast(launch, C.c_void_p),
                                      C.cast(splits, C.c_void_p), C.cast(slots, C.c_void_p), max_launches)
    if rc < 0:
        raise DpError("dp_accumulate_schedule", rc)
    return {"item_start": list(start), "launch": list(launch), "splits": list(splits)[:rc], "slots": list(slots)[:rc]}


def dp_add_noise_and_scale(acc: torch.Tensor, sigma: float, C_: float, batch_size: int, seed: int, step: int,
                           elem_offset: int = 0, stream=None) -> torch.Tensor:
    _check("dp_add_noise_and_scale",
           lib().dp_add_noise_and_scale(_ptr(acc), acc.numel(), int(elem_offset), float(sigma), float(C_),
                                        int(batch_size), int(seed), int(step), _stream(stream)))
    return acc


def dp_adamw_step(theta, m, v, g, lr, beta1, beta2, xi, weight_decay, t, stream=None) -> None:
    _check("dp_adamw_step",
           lib().dp_adamw_step(_ptr(theta), _ptr(m), _ptr(v), _ptr(g), theta.numel(), float(lr), float(beta1),
                               float(beta2), float(xi), float(weight_decay), int(t), _stream(stream)))


def dp_noise_scale_adamw_step(theta, m, v, acc, zero_acc, sigma, C_, batch_size, seed, step, lr, beta1, beta2,
                              xi, weight_decay, t, elem_offset: int = 0, stream=None) -> None:
    _check("dp_noise_scale_adamw_step",
           lib().dp_noise_scale_adamw_step(_ptr(theta), _ptr(m), _ptr(v), _ptr(acc), int(bool(zero_acc)),
                                           theta.numel(), int(elem_offset), float(sigma), float(C_),
                                           int(batch_size), int(seed), int(step), float(lr), float(beta1),
                                           float(beta2), float(xi), float(weight_decay), int(t), _stream(stream)))


def dp_noise_scale_adamw_step_snr(theta, m, v, acc, zero_acc, sigma, C_, batch_size, seed, step, lr, beta1, beta2,
                                  xi, weight_decay, t, sq_sums: torch.Tensor, elem_offset: int = 0, stream=None) -> None:
    """sq_sums: float64 device tensor [2], accumulated into (sum acc^2, sum (sigma C z)^2)."""
    if sq_sums.dtype != torch.float64 or sq_sums.numel() != 2:
        raise ValueError("sq_sums must be a float64 tensor with 2 elements")
    _check("dp_noise_scale_adamw_step_snr",
           lib().dp_noise_scale_adamw_step_snr(_ptr(theta), _ptr(m), _ptr(v), _ptr(acc), int(bool(zero_acc)),
                                               theta.numel(), int(elem_offset), float(sigma), float(C_),
                                               int(batch_size), int(seed), int(step), float(lr), float(beta1),
                                               float(beta2), float(xi), float(weight_decay), int(t),
                                               _ptr(sq_sums), _stream(stream)))


def dp_reduce_noise_adamw_step(theta, m, v, acc_shards, theta_shards, zero_acc, sigma, C_, batch_size, seed, step, lr,
                               beta1, beta2, xi, weight_decay, t, elem_offset: int = 0, stream=None) -> None:
    """Fused cross-rank sum + noise + AdamW on one shard.  acc_shards: one entry per rank, the shard inside that
    rank's accumulator (a tensor, or a raw device address for peer-mapped memory); theta_shards: the shard inside
    every rank's replica of theta, entries may be None (or the whole argument None) to skip the write."""
    def addr(x):
        return 0 if x is None else (int(x) if isinstance(x, int) else x.data_ptr())
    R = len(acc_shards)
    acc_arr = (C.c_void_p * R)(*[addr(a) for a in acc_shards])
    th_arr = None if theta_shards is None else (C.c_void_p * R)(*[addr(x) for x in theta_shards])
    _check("dp_reduce_noise_adamw_step",
           lib().dp_reduce_noise_adamw_step(_ptr(theta), _ptr(m), _ptr(v), C.cast(acc_arr, C.c_void_p),
                                            None if th_arr is None else C.cast(th_arr, C.c_void_p), R,
                                            int(bool(zero_acc)), theta.numel(), int(elem_offset), float(sigma),
                                            float(C_), int(batch_size), int(seed), int(step), float(lr), float(beta1),
                                            float(beta2), float(xi), float(weight_decay), int(t), _stream(stream)))


def dp_clip_stats(clip: torch.Tensor, out: torch.Tensor, stream=None) -> torch.Tensor:
    _check("dp_clip_stats", lib().dp_clip_stats(_ptr(clip), clip.numel(), _ptr(out), _stream(stream)))
    return out


def dp_philox_u32(out: torch.Tensor, elem_offset: int, seed: int, step: int, stream=None) -> torch.Tensor:
    """out: int32 tensor (bit pattern of the uint32 words)."""
    _check("dp_philox_u32", lib().dp_philox_u32(_ptr(out), out.numel(), int(elem_offset), int(seed), int(step),
                                                _stream(stream)))
    return out


def dp_token_equality_mask(ids: torch.Tensor, mask: torch.Tensor, stream=None) -> torch.Tensor:
    B, T = ids.shape
    _check("dp_token_equality_mask", lib().dp_token_equality_mask(_ptr(ids), B, T, _ptr(mask), _stream(stream)))
    return mask


STATIC_SCRATCH_FLOATS = 1 << 20


def dp_layernorm_sqnorms_static(layers: LayerList, sqnorm: torch.Tensor, accumulate_into: bool = False,
                                stream=None) -> torch.Tensor:
    """Norms of the single LayerNorm layer in `layers` with the library's fixed scratch (no workspace)."""
    if len(layers) != 1:
        raise ValueError("exactly one LayerNorm layer expected")
    _check("dp_layernorm_sqnorms_static",
           lib().dp_layernorm_sqnorms_static(layers.ptr, _ptr(sqnorm), int(accumulate_into), _stream(stream)))
    return sqnorm


def dp_last_timeout_info():
    info = (C.c_int * 5)()
    _check("dp_last_timeout_info", lib().dp_last_timeout_info(info))
    return list(info)


def dp_launch_count() -> int:
    return int(lib().dp_launch_count())


def dp_poll_status(stream=None) -> int:
    return int(lib().dp_poll_status(_stream(stream)))


def dp_set_wait_limit_cycles(cycles: int) -> None:
    """Limit of every bounded device-side wait on the current device (<= 0: the default of 4e9 SM cycles)."""
    _check("dp_set_wait_limit_cycles", lib().dp_set_wait_limit_cycles(int(cycles)))


def dp_selftest_wait_timeout(stream=None) -> None:
    """Enqueues the kernel whose waits nobody satisfies; dp_poll_status reports DP_ERR_TIMEOUT afterwards."""
    _check("dp_selftest_wait_timeout", lib().dp_selftest_wait_timeout(_stream(stream)))

