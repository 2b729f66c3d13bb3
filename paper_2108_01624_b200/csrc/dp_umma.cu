// tcgen05 / TMEM / TMA kernels for bf16 linear layers (sm_100a).
//
//   k_gram_sqnorm       per-example squared norm by the token-Gram identity
//                       |A_i^T G_i|_F^2 + |1^T G_i|^2 = < A_i A_i^T + [bias] 1 1^T , G_i G_i^T >, for T <= 128.
//                       Both 128x128 fp32 Grams live in TMEM (2 x 128 columns, double-buffered); operands are
//                       K-major 128x64 tiles, two per TMA copy.  For a token embedding the input is one-hot, so
//                       A_i A_i^T is the token-id equality mask: only G_i G_i^T is formed on the tensor cores and
//                       the epilogue multiplies it by [id_t == id_s] (integer compares; any T).
//   k_gram_sqnorm_short the same for T <= 112 with copies as high as the example is long (T rounded up to 16) and as many
//                       64-feature groups per copy as fit a ring slot, and 128 x T' x 16 UMMAs.
//   k_gram_sqnorm_wide  the same identity for T > 128: a row block against two column blocks per item
//                       (128x256 UMMAs), upper triangle of the block grid only.
//   k_tile_sqnorm_pair  the materialised-tile norm on CTA pairs: 256 (d_out) x 256 (d_in) tiles of ONE example's
//                       A_i^T G_i (one 256x256x16 UMMA per 16 tokens, both operands MN-major straight from the
//                       row-major activations), squared and summed in the epilogue; the tile never leaves TMEM.
//   k_accum_pair        the clipped sum acc_w += sum_i c_i A_i^T G_i on CTA pairs (cta_group::2): 256 x 512
//                       tiles, the per-example factor applied to the G rows in shared memory by the worker
//                       warps, which also form the bias column sums, so A and G are read from HBM once.
//
// All are persistent kernels (grid = number of SMs) over a work list decoded on the device from
// per-layer tile counts; roles are warp-specialised (TMA producer / MMA issuer / epilogue or worker warps).
#include <cuda.h>

#include <algorithm>
#include <vector>

#include "dp_internal.h"
#include "dp_ptx.cuh"

namespace dpk {
using namespace ptx;

constexpr int kMaxLayers = kUmmaMaxLayers;

// Tunables (overridable with -D for experiments; the defaults are what was measured best).
#ifndef DP_ACCUM_ALIGN
#define DP_ACCUM_ALIGN 1                // accumulate kernel: soft per-wave alignment of the CTA pairs
#endif
#ifndef DP_ACCUM_READY
// accumulate kernel: how the worker warps of the odd CTA hand a rescaled G stage to the UMMA issuer in the even CTA
//   0  every warp: fence.proxy.async, then a plain remote mbarrier.arrive (16 arrivals per stage)
//   1  every warp: fence.proxy.async, fence.acq_rel.cluster, plain remote arrive (16 arrivals per stage)
//   2  the eight warps of a CTA meet at a named barrier and ONE thread (rotating over the warps) arrives with
//      release semantics at cluster scope (2 arrivals per stage); the issuer acquires at cluster scope
#define DP_ACCUM_READY 0
#endif
#ifndef DP_ACCUM_A_REUSE
#define DP_ACCUM_A_REUSE 1             // accumulate kernel: the two UMMAs of a k-step share the G tile through the operand
                                       // collector (16.03-16.13 against 16.11-16.19 ms per launch sustained, six alternating runs)
#endif
#ifndef DP_TMA_L2_PROMOTION
#define DP_TMA_L2_PROMOTION 2          // 0 none, 1 128 B, 2 256 B
#endif

struct alignas(64) UmmaLayer {
  CUtensorMap mapG;   // [B, T, d_out] bf16
  CUtensorMap mapA;   // [B, T, d_in]  bf16
  float* acc_w;
  float* acc_b;
  const int32_t* ids;     // embedding layers (Gram kernel): token ids [B, T]; the id-equality mask replaces A A^T
  int d_out, d_in;        // embedding: d_in = 0 (there is no A operand to stream)
  int item_start;         // first work item of this layer within the launch
  int partial_base;       // first per-example partial slot of this layer
  uint16_t tiles_m, tiles_n;   // tile kernels: tiles over d_out and over d_in
  uint8_t has_bias, is_emb;
  uint8_t rag_g, rag_a;   // the width of G / A is not a multiple of 64: its map is the 3-D one (one 64-feature group per copy)
  uint8_t pad[16];        // to 320 bytes (a multiple of the tensor maps' 64-byte alignment)
};
static_assert(sizeof(UmmaLayer) == 320, "UmmaLayer grew: 96 of them must fit the kernel parameter block");

struct UmmaParams {
  UmmaLayer L[kMaxLayers];
  int n_layers, total_items, B, T;
  int splits;             // accumulate: number of example ranges a tile is split into
  int box_rows, box_groups;   // short-example Gram kernel: token rows and 64-feature groups of one copy
  int partial_stride;
  unsigned int* wave_sync;  // accumulate: arrival counter of the soft per-wave alignment (zeroed before the launch)
  long long align_limit;    // accumulate: longest wait at a wave boundary, in SM cycles (a few tile durations)
  const float* clip;
  float* partial;
  int* status;
};
static_assert(sizeof(UmmaParams) <= 32000, "kernel parameter block too large");

__device__ __forceinline__ int find_layer(const UmmaParams& P, int item) {
  int l = 0;
  while (l + 1 < P.n_layers && item >= P.L[l + 1].item_start) ++l;
  return l;
}

__device__ __forceinline__ uint8_t* align1024(uint8_t* p) {
  return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~uintptr_t(1023));
}

// One operand tile of `groups` 64-feature groups (each `group_bytes` apart in shared memory), token rows from
// `row`, features from `f0` (a multiple of 64), example `ex`.  Widths that are multiples of 64 use the 4-D view of
// the tensor (one copy for all groups).  Other widths (multiples of 8) cannot: a 64-feature group that overhangs
// the row would run into the next token, so their map is the plain (feature, token, example) view, whose copies
// are bounded by the width and read zeros beyond it, one copy per group.
__device__ __forceinline__ void load_groups(uint8_t* dst, const CUtensorMap* map, uint64_t* bar, bool ragged, int groups,
                                            int group_bytes, int f0, int row, int ex) {
  if (!ragged) {
    tma_load_4d(dst, map, bar, 0, row, f0 / 64, ex);
  } else {
    for (int g = 0; g < groups; ++g) tma_load_3d(dst + g * group_bytes, map, bar, f0 + 64 * g, row, ex);
  }
}

// =================================================================================================
// Gram kernel
// =================================================================================================
constexpr int G_GROUPS = 2;                      // 64-feature tiles per TMA copy and ring slot
constexpr int G_SLOTS = 6;                       // (7 slots, or L2 prefetch of the tiles ahead of the ring: measured, no gain)
constexpr int G_TILE_BYTES = 128 * 128;          // 128 tokens x 64 bf16 features, 128-byte swizzle
constexpr int G_SLOT_BYTES = G_GROUPS * G_TILE_BYTES;
constexpr int G_THREADS = 192;                   // warp 0: TMA, warp 1: MMA, warps 2..5: epilogue
constexpr uint32_t G_IDESC = idesc_bf16_f32(128, 128, false, false);

struct GramCtl {
  uint64_t full[G_SLOTS], empty[G_SLOTS], tmem_full[2], tmem_empty[2], drain;
  uint32_t tmem_base;
  int abort;
};
constexpr int G_SMEM = 1024 + G_SLOTS * G_SLOT_BYTES + (int)sizeof(GramCtl);
static_assert(G_SMEM <= 232448, "over the shared memory of one CTA");

// item -> (layer, example, token-block pair r <= c)
__device__ __forceinline__ void gram_decode(const UmmaParams& P, int item, int npairs, int nblk, int& l, int& i, int& pair,
                                            int& r, int& c) {
  l = find_layer(P, item);
  const int rem = item - P.L[l].item_start;
  i = rem / npairs;
  pair = rem - i * npairs;
  int p = pair;
  r = 0;
  while (p >= nblk - r) { p -= nblk - r; ++r; }
  c = r + p;
}

__global__ void __launch_bounds__(G_THREADS, 1) k_gram_sqnorm(const __grid_constant__ UmmaParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = align1024(smem_raw);
  GramCtl* S = reinterpret_cast<GramCtl*>(tiles + G_SLOTS * G_SLOT_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &S->abort;

  if (threadIdx.x == 0) {
    for (int s = 0; s < G_SLOTS; ++s) { mbar_init(&S->full[s], 1); mbar_init(&S->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&S->tmem_full[b], 1); mbar_init(&S->tmem_empty[b], 4); }
    mbar_init(&S->drain, 1);
    S->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&S->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = S->tmem_base;
  const int nblk = (P.T + 127) / 128, npairs = nblk * (nblk + 1) / 2;
  // A box is always 128 tokens high and two 64-feature groups wide: rows beyond T and a group beyond the layer's
  // width are outside the tensor and arrive as zeros.  One copy instruction per 32 KB keeps the producer (whose
  // copies cost a fixed time each) well ahead of the 7 TB/s the ring can stream.

  if (warp == 0) {
    if (lane == 0) {   // ---------------- TMA producer ----------------
      uint32_t it = 0;
      bool alive = true;
      for (int item = blockIdx.x; item < P.total_items && alive; item += gridDim.x) {
        int l, i, pair, r, c;
        gram_decode(P, item, npairs, nblk, l, i, pair, r, c);
        const UmmaLayer& L = P.L[l];
        for (int which = 0; which < 2 && alive; ++which) {
          const CUtensorMap* map = which ? &L.mapG : &L.mapA;
          const int d = which ? L.d_out : L.d_in;
          for (int k0 = 0; k0 < d && alive; k0 += 64 * G_GROUPS) {
            for (int half = 0; half < (r == c ? 1 : 2); ++half) {
              const uint32_t slot = it % G_SLOTS, ph = (it / G_SLOTS) & 1u;
              if (!mbar_wait(&S->empty[slot], ph ^ 1u, abort_flag, P.status)) { alive = false; break; }
              mbar_arrive_expect_tx(&S->full[slot], (uint32_t)G_SLOT_BYTES);
              load_groups(tiles + slot * G_SLOT_BYTES, map, &S->full[slot], which ? L.rag_g : L.rag_a, G_GROUPS,
                          G_TILE_BYTES, k0, (half ? c : r) * 128, i);
              ++it;
            }
          }
        }
      }
      // Leave no copy in flight: every issued slot must have landed before shared memory is released.
      const uint32_t pending = it < (uint32_t)G_SLOTS ? it : (uint32_t)G_SLOTS;
      for (uint32_t k = 0; k < pending; ++k) {
        const uint32_t j = it - 1 - k;
        mbar_wait_drain(&S->full[j % G_SLOTS], (j / G_SLOTS) & 1u, P.status);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {   // ---------------- MMA issuer ----------------
      uint32_t it = 0, tile_it = 0;
      bool alive = true;
      for (int item = blockIdx.x; item < P.total_items && alive; item += gridDim.x, ++tile_it) {
        int l, i, pair, r, c;
        gram_decode(P, item, npairs, nblk, l, i, pair, r, c);
        const UmmaLayer& L = P.L[l];
        const uint32_t buf = tile_it & 1u, tph = (tile_it >> 1) & 1u;
        if (!mbar_wait(&S->tmem_empty[buf], tph ^ 1u, abort_flag, P.status)) { alive = false; break; }
        tc_fence_after();
        for (int which = 0; which < 2 && alive; ++which) {
          const int d = which ? L.d_out : L.d_in;
          const uint32_t d_tmem = tmem_base + buf * 256u + (uint32_t)which * 128u;
          for (int k0 = 0; k0 < d; k0 += 64 * G_GROUPS) {
            const uint32_t sr = it % G_SLOTS, pr = (it / G_SLOTS) & 1u;
            ++it;
            if (!mbar_wait(&S->full[sr], pr, abort_flag, P.status)) { alive = false; break; }
            uint32_t sc = sr;
            if (r != c) {
              sc = it % G_SLOTS;
              const uint32_t pc = (it / G_SLOTS) & 1u;
              ++it;
              if (!mbar_wait(&S->full[sc], pc, abort_flag, P.status)) { alive = false; break; }
            }
            tc_fence_after();
            const uint32_t ar = smem_u32(tiles + sr * G_SLOT_BYTES), ac = smem_u32(tiles + sc * G_SLOT_BYTES);
#pragma unroll
            for (int g = 0; g < G_GROUPS; ++g) {
              if (k0 + 64 * g < d) {                   // a group beyond the layer's width holds zeros: skip it
#pragma unroll
                for (int k4 = 0; k4 < 4; ++k4) {
                  umma_bf16(d_tmem, smem_desc_sw128(ar + g * G_TILE_BYTES + k4 * 32, 16, 1024),
                            smem_desc_sw128(ac + g * G_TILE_BYTES + k4 * 32, 16, 1024), G_IDESC, (k0 | g | k4) ? 1u : 0u);
                }
              }
            }
            umma_commit(&S->empty[sr]);
            if (r != c) umma_commit(&S->empty[sc]);
          }
        }
        if (alive) umma_commit(&S->tmem_full[buf]);
      }
      // Drain: all issued MMAs must have completed before TMEM and shared memory are released.
      umma_commit(&S->drain);
      mbar_wait_drain(&S->drain, 0u, P.status);
    }
  } else {   // ---------------- epilogue warps 2..5 ----------------
    const uint32_t q = (uint32_t)warp & 3u;
    uint32_t tile_it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < P.total_items; item += gridDim.x, ++tile_it) {
      int l, i, pair, r, c;
      gram_decode(P, item, npairs, nblk, l, i, pair, r, c);
      const UmmaLayer& L = P.L[l];
      const uint32_t buf = tile_it & 1u, tph = (tile_it >> 1) & 1u;
      if (alive) alive = __all_sync(0xffffffffu, mbar_wait(&S->tmem_full[buf], tph, abort_flag, P.status));
      if (!alive) continue;
      tc_fence_after();
      const float bias1 = L.has_bias ? 1.0f : 0.0f;
      float sum = 0.0f;
      if (L.is_emb) {
        // first factor = [id_t == id_s]; rows and columns beyond T meet zero entries of G G^T
        const int32_t* idrow = L.ids + (size_t)i * P.T;
        const int trow = r * 128 + (int)q * 32 + lane;
        const int32_t my_id = trow < P.T ? __ldg(idrow + trow) : -1;
#pragma unroll 1
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t qv[32];
          tmem_ld_32x32(tmem_base + ((q * 32u) << 16) + buf * 256u + 128u + (uint32_t)ch * 32u, qv);
          tmem_ld_wait();
          const int s0 = c * 128 + ch * 32;
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const int32_t other = (s0 + j < P.T) ? __ldg(idrow + s0 + j) : -2;
            sum += (other == my_id) ? __uint_as_float(qv[j]) : 0.0f;
          }
        }
      } else {
#pragma unroll 1
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t pv[32], qv[32];
          const uint32_t ta = tmem_base + ((q * 32u) << 16) + buf * 256u + (uint32_t)ch * 32u;
          tmem_ld_32x32(ta, pv);
          tmem_ld_32x32(ta + 128u, qv);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) sum = fmaf(__uint_as_float(pv[j]) + bias1, __uint_as_float(qv[j]), sum);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&S->tmem_empty[buf]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_down_sync(0xffffffffu, sum, o);
      if (lane == 0)
        P.partial[(size_t)i * P.partial_stride + L.partial_base + pair * 4 + (int)q] = (r == c) ? sum : 2.0f * sum;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// =================================================================================================
// Gram kernel for short examples (T <= 112: the masked positions of a masked-LM head, a pooler's single token)
//
// The same identity and roles as k_gram_sqnorm with one token block per example, but a copy is `rows` tokens high
// (T rounded up to 16) and carries as many 64-feature groups as fit the 32 KB ring slot, so that a short example
// does not pay for 128-token boxes of mostly zero fill (the copies, whose cost is per instruction and per byte
// written to shared memory, set the pace there), and the UMMAs are 128 x rows x 16.  Only the first `rows` rows
// of a tile are written; the UMMA's M operand reads 128, so accumulator rows from `rows` on hold whatever the
// ring held before and the epilogue leaves the lanes of tokens beyond T out.  Columns below `rows` are clean
// (tokens between T and `rows` arrive as zeros).
// =================================================================================================
// The M operand of a UMMA spans 128 rows (16 KB) from the start of a group, which for the last groups of a slot
// reaches into the next slot and, for the last slot, beyond the ring: a pad of one tile keeps those reads inside the
// CTA's shared memory (what they return feeds accumulator rows that nobody reads).
constexpr int G_SMEM_SHORT = 1024 + G_SLOTS * G_SLOT_BYTES + G_TILE_BYTES + (int)sizeof(GramCtl);
static_assert(G_SMEM_SHORT <= 232448, "over the shared memory of one CTA");

__global__ void __launch_bounds__(G_THREADS, 1) k_gram_sqnorm_short(const __grid_constant__ UmmaParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = align1024(smem_raw);
  GramCtl* S = reinterpret_cast<GramCtl*>(tiles + G_SLOTS * G_SLOT_BYTES + G_TILE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &S->abort;

  if (threadIdx.x == 0) {
    for (int s = 0; s < G_SLOTS; ++s) { mbar_init(&S->full[s], 1); mbar_init(&S->empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&S->tmem_full[b], 1); mbar_init(&S->tmem_empty[b], 4); }
    mbar_init(&S->drain, 1);
    S->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&S->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = S->tmem_base;
  const int rows = P.box_rows, groups = P.box_groups;      // rows: a multiple of 16 below 128; groups * rows <= 256
  const int group_bytes = rows * 128;
  const uint32_t slot_tx = (uint32_t)(groups * group_bytes);

  if (warp == 0) {
    if (lane == 0) {   // ---------------- TMA producer ----------------
      uint32_t it = 0;
      bool alive = true;
      for (int item = blockIdx.x; item < P.total_items && alive; item += gridDim.x) {
        const int l = find_layer(P, item), i = item - P.L[l].item_start;
        const UmmaLayer& L = P.L[l];
        for (int which = 0; which < 2 && alive; ++which) {
          const CUtensorMap* map = which ? &L.mapG : &L.mapA;
          const int d = which ? L.d_out : L.d_in;
          for (int k0 = 0; k0 < d; k0 += 64 * groups) {
            const uint32_t slot = it % G_SLOTS, ph = (it / G_SLOTS) & 1u;
            if (!mbar_wait(&S->empty[slot], ph ^ 1u, abort_flag, P.status, 31, (int)it)) { alive = false; break; }
            mbar_arrive_expect_tx(&S->full[slot], slot_tx);
            load_groups(tiles + slot * G_SLOT_BYTES, map, &S->full[slot], which ? L.rag_g : L.rag_a, groups, group_bytes,
                        k0, 0, i);
            ++it;
          }
        }
      }
      const uint32_t pending = it < (uint32_t)G_SLOTS ? it : (uint32_t)G_SLOTS;
      for (uint32_t k = 0; k < pending; ++k) {
        const uint32_t j = it - 1 - k;
        mbar_wait_drain(&S->full[j % G_SLOTS], (j / G_SLOTS) & 1u, P.status);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {   // ---------------- MMA issuer ----------------
      const uint32_t idesc = idesc_bf16_f32(128, rows, false, false);
      uint32_t it = 0, tile_it = 0;
      bool alive = true;
      for (int item = blockIdx.x; item < P.total_items && alive; item += gridDim.x, ++tile_it) {
        const int l = find_layer(P, item);
        const UmmaLayer& L = P.L[l];
        const uint32_t buf = tile_it & 1u, tph = (tile_it >> 1) & 1u;
        if (!mbar_wait(&S->tmem_empty[buf], tph ^ 1u, abort_flag, P.status, 32, (int)tile_it)) { alive = false; break; }
        tc_fence_after();
        for (int which = 0; which < 2 && alive; ++which) {
          const int d = which ? L.d_out : L.d_in;
          const uint32_t d_tmem = tmem_base + buf * 256u + (uint32_t)which * 128u;
          for (int k0 = 0; k0 < d; k0 += 64 * groups) {
            const uint32_t sr = it % G_SLOTS, pr = (it / G_SLOTS) & 1u;
            ++it;
            if (!mbar_wait(&S->full[sr], pr, abort_flag, P.status, 33, (int)it)) { alive = false; break; }
            tc_fence_after();
            const uint32_t a0 = smem_u32(tiles + sr * G_SLOT_BYTES);
            for (int g = 0; g < groups && k0 + 64 * g < d; ++g) {
#pragma unroll
              for (int k4 = 0; k4 < 4; ++k4) {
                const uint64_t desc = smem_desc_sw128(a0 + g * group_bytes + k4 * 32, 16, 1024);
                umma_bf16(d_tmem, desc, desc, idesc, (k0 | g | k4) ? 1u : 0u);
              }
            }
            umma_commit(&S->empty[sr]);
          }
        }
        if (alive) umma_commit(&S->tmem_full[buf]);
      }
      umma_commit(&S->drain);
      mbar_wait_drain(&S->drain, 0u, P.status);
    }
  } else {   // ---------------- epilogue warps 2..5 ----------------
    const uint32_t q = (uint32_t)warp & 3u;
    const int trow = (int)q * 32 + lane;
    uint32_t tile_it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < P.total_items; item += gridDim.x, ++tile_it) {
      const int l = find_layer(P, item), i = item - P.L[l].item_start;
      const UmmaLayer& L = P.L[l];
      const uint32_t buf = tile_it & 1u, tph = (tile_it >> 1) & 1u;
      if (alive) alive = __all_sync(0xffffffffu, mbar_wait(&S->tmem_full[buf], tph, abort_flag, P.status, 34, (int)tile_it));
      if (!alive) continue;
      tc_fence_after();
      const float bias1 = L.has_bias ? 1.0f : 0.0f;
      const int32_t* idrow = L.is_emb ? L.ids + (size_t)i * P.T : nullptr;
      const int32_t my_id = (L.is_emb && trow < P.T) ? __ldg(idrow + trow) : -1;
      float sum = 0.0f;
      if ((int)q * 32 < rows) {                       // warps whose lanes all lie beyond the box have nothing to add
#pragma unroll 1
        for (int ch = 0; ch * 32 < rows; ++ch) {
          uint32_t pv[32], qv[32];
          const uint32_t ta = tmem_base + ((q * 32u) << 16) + buf * 256u + (uint32_t)ch * 32u;
          if (!L.is_emb) tmem_ld_32x32(ta, pv);
          tmem_ld_32x32(ta + 128u, qv);
          tmem_ld_wait();
          if (trow < P.T) {                            // lanes of tokens beyond T hold stale accumulator rows
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int s = ch * 32 + j;
              if (s < P.T) {
                if (L.is_emb) sum += (__ldg(idrow + s) == my_id) ? __uint_as_float(qv[j]) : 0.0f;
                else sum = fmaf(__uint_as_float(pv[j]) + bias1, __uint_as_float(qv[j]), sum);
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&S->tmem_empty[buf]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_down_sync(0xffffffffu, sum, o);
      if (lane == 0) P.partial[(size_t)i * P.partial_stride + L.partial_base + (int)q] = sum;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// =================================================================================================
// Gram kernel for examples longer than one token block (T > 128, linear layers)
//
// With several 128-token blocks the Gram of an example is a grid of nblk x nblk blocks, of which the upper
// triangle is computed.  An item here is a row block r and TWO neighbouring column blocks (c0, c0 + 1), one
// 128 x 256 x 16 UMMA per 16 features: per 64-feature stage the SM receives the row tile (16 KB, not needed
// when r = c0: the first half of the column tile is the row tile) and the column tile (32 KB) for 512 tensor
// cycles, where the one-block-pair kernel above needs two 16 KB tiles per 256 cycles (and its 128 x 128 UMMAs read
// shared memory at the full 128 B/clk).  The last column block of a row with an odd count runs alone (N = 128).
// TMEM holds P = A_r A_c^T (256 columns) and Q = G_r G_c^T (256 columns), one buffer each; the pipeline is kept
// full by splitting the epilogue: as soon as P is complete the eight epilogue warps copy it to registers (128
// per thread) and release its columns, so the UMMAs of the next item's P overlap this item's Q and product-sum.
// =================================================================================================
// Shared memory is a ring of 16 KB units; a stage takes the units it needs (row tile 1, column tile 2 or 1), so
// the stages of an item whose row tile is also its first column tile occupy 32 KB instead of 48 KB and more of
// them are in flight.  A stage never straddles the end of the ring: the units left there are skipped.
#ifndef DP_WIDE_UNITS
#define DP_WIDE_UNITS 14
#endif
constexpr int W_UNITS = DP_WIDE_UNITS;
constexpr int W_UNIT_BYTES = 128 * 128;                 // 128 tokens x 64 bf16 features, 128-byte swizzle
constexpr int W_BARS = 16;                              // stage barriers (more than stages can be in flight)
static_assert(W_UNITS >= 3 && W_UNITS < W_BARS, "a stage of three units must fit, and every stage in flight needs a barrier");
constexpr int W_THREADS = 320;                          // warp 0 TMA, warp 1 UMMA issue, warps 2..9 epilogue
constexpr int kWideMaxLayers = 48;

struct alignas(64) WideLayer {
  CUtensorMap rowA, colA, rowG, colG;   // [B, T, d] bf16 as (feature, token, example); boxes 64 x 128 and 64 x 256
  int d_out, d_in;
  int item_start, partial_base;
  int has_bias;
  int pad[11];
};
static_assert(sizeof(WideLayer) == 576, "WideLayer: 48 of them must fit the kernel parameter block");

struct WideParams {
  WideLayer L[kWideMaxLayers];
  int n_layers, total_items, B, T;
  int partial_stride, pad;
  float* partial;
  int* status;
};
static_assert(sizeof(WideParams) <= 32000, "kernel parameter block too large");

struct WideCtl {
  uint64_t full[W_BARS], empty[W_BARS], x_full, x_empty, y_full, y_empty, drain;
  uint32_t tmem_base;
  int abort;
};
constexpr int W_SMEM = 1024 + W_UNITS * W_UNIT_BYTES + (int)sizeof(WideCtl);
static_assert(W_SMEM <= 232448, "over the shared memory of one CTA");

// items of one example: for every row block r the column blocks r, r+1, ... in pairs
__host__ __device__ inline int wide_items(int nblk) {
  int n = 0;
  for (int r = 0; r < nblk; ++r) n += (nblk - r + 1) / 2;
  return n;
}

struct WideItem { int l, i, idx, r, c0, ncol; };

__device__ __forceinline__ WideItem wide_decode(const WideParams& P, int item, int per_example, int nblk) {
  WideItem t;
  t.l = 0;
  while (t.l + 1 < P.n_layers && item >= P.L[t.l + 1].item_start) ++t.l;
  const int rem = item - P.L[t.l].item_start;
  t.i = rem / per_example;
  t.idx = rem - t.i * per_example;
  int p = t.idx;
  t.r = 0;
  while (p >= (nblk - t.r + 1) / 2) { p -= (nblk - t.r + 1) / 2; ++t.r; }
  t.c0 = t.r + 2 * p;
  t.ncol = (nblk - t.c0) < 2 ? (nblk - t.c0) : 2;
  return t;
}

__global__ void __launch_bounds__(W_THREADS, 1) k_gram_sqnorm_wide(const __grid_constant__ WideParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = align1024(smem_raw);
  WideCtl* S = reinterpret_cast<WideCtl*>(tiles + W_UNITS * W_UNIT_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &S->abort;

  if (threadIdx.x == 0) {
    for (int s = 0; s < W_BARS; ++s) { mbar_init(&S->full[s], 1); mbar_init(&S->empty[s], 1); }
    mbar_init(&S->x_full, 1);
    mbar_init(&S->y_full, 1);
    mbar_init(&S->x_empty, 8);
    mbar_init(&S->y_empty, 8);
    mbar_init(&S->drain, 1);
    S->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc(&S->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = S->tmem_base;
  const int nblk = (P.T + 127) / 128, per_example = wide_items(nblk);

  if (warp == 0) {
    if (lane == 0) {   // ---------------- TMA producer ----------------
      // Stage n uses barrier n % W_BARS; stages [tail, n) are in flight or unread, `foot` holds the units each of
      // them took (those skipped at the end of the ring included); they are released in order.
      uint32_t n = 0, tail = 0;
      int pos = 0, free_units = W_UNITS;
      uint8_t foot[W_BARS];
      bool alive = true;
      for (int item = blockIdx.x; item < P.total_items && alive; item += gridDim.x) {
        const WideItem t = wide_decode(P, item, per_example, nblk);
        const WideLayer& L = P.L[t.l];
        const bool diag = t.c0 == t.r;
        // a lone column block is fetched with the 128-token box; rows beyond T arrive as zeros either way
        const int u = (diag ? 0 : 1) + (t.ncol == 2 ? 2 : 1);
        for (int which = 0; which < 2 && alive; ++which) {
          const CUtensorMap* rowmap = which ? &L.rowG : &L.rowA;
          const CUtensorMap* colmap = t.ncol == 2 ? (which ? &L.colG : &L.colA) : rowmap;
          const int d = which ? L.d_out : L.d_in;
          for (int k0 = 0; k0 < d && alive; k0 += 64) {
            const int skip = pos + u > W_UNITS ? W_UNITS - pos : 0;
            while (free_units < skip + u) {
              if (!mbar_wait(&S->empty[tail % W_BARS], (tail / W_BARS) & 1u, abort_flag, P.status, 21, (int)tail)) {
                alive = false;
                break;
              }
              free_units += foot[tail % W_BARS];
              ++tail;
            }
            if (!alive) break;
            if (skip) pos = 0;
            uint8_t* st = tiles + pos * W_UNIT_BYTES;
            uint64_t* bar = &S->full[n % W_BARS];
            mbar_arrive_expect_tx(bar, (uint32_t)(u * W_UNIT_BYTES));
            if (!diag) tma_load_3d(st, rowmap, bar, k0, t.r * 128, t.i);
            tma_load_3d(st + (diag ? 0 : W_UNIT_BYTES), colmap, bar, k0, t.c0 * 128, t.i);
            foot[n % W_BARS] = (uint8_t)(skip + u);
            free_units -= skip + u;
            pos += u;
            if (pos == W_UNITS) pos = 0;
            ++n;
          }
        }
      }
      // Leave no copy in flight: every stage not yet released must have landed before shared memory is given up.
      for (uint32_t j = tail; j < n; ++j) mbar_wait_drain(&S->full[j % W_BARS], (j / W_BARS) & 1u, P.status);
    }
  } else if (warp == 1) {
    if (lane == 0) {   // ---------------- MMA issuer ----------------
      constexpr uint32_t IDESC_N256 = idesc_bf16_f32(128, 256, false, false);
      constexpr uint32_t IDESC_N128 = idesc_bf16_f32(128, 128, false, false);
      uint32_t n = 0, tile_it = 0;
      int pos = 0;
      bool alive = true;
      for (int item = blockIdx.x; item < P.total_items && alive; item += gridDim.x, ++tile_it) {
        const WideItem t = wide_decode(P, item, per_example, nblk);
        const WideLayer& L = P.L[t.l];
        const bool diag = t.c0 == t.r;
        const int u = (diag ? 0 : 1) + (t.ncol == 2 ? 2 : 1);
        const uint32_t idesc = t.ncol == 2 ? IDESC_N256 : IDESC_N128;
        const uint32_t tph = tile_it & 1u;
        for (int which = 0; which < 2 && alive; ++which) {
          if (!mbar_wait(which ? &S->y_empty : &S->x_empty, tph ^ 1u, abort_flag, P.status, 22, (int)tile_it)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const int d = which ? L.d_out : L.d_in;
          const uint32_t d_tmem = tmem_base + (uint32_t)which * 256u;
          for (int k0 = 0; k0 < d; k0 += 64) {
            if (pos + u > W_UNITS) pos = 0;              // the same walk over the unit ring as the producer's
            const uint32_t rowb = smem_u32(tiles + pos * W_UNIT_BYTES);
            const uint32_t colb = diag ? rowb : rowb + W_UNIT_BYTES;
            pos += u;
            if (pos == W_UNITS) pos = 0;
            const uint32_t b = n % W_BARS, ph = (n / W_BARS) & 1u;
            ++n;
            if (!mbar_wait(&S->full[b], ph, abort_flag, P.status, 23, (int)n)) { alive = false; break; }
            tc_fence_after();
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4)
              umma_bf16(d_tmem, smem_desc_sw128(rowb + k4 * 32, 16, 1024), smem_desc_sw128(colb + k4 * 32, 16, 1024),
                        idesc, (k0 | k4) ? 1u : 0u);
            umma_commit(&S->empty[b]);
          }
          if (alive) umma_commit(which ? &S->y_full : &S->x_full);
        }
      }
      umma_commit(&S->drain);
      mbar_wait_drain(&S->drain, 0u, P.status);
    }
  } else {   // ---------------- epilogue warps 2..9: lanes [32 q, +32), column block h of the pair ----------------
    const uint32_t q = (uint32_t)warp & 3u;
    const int h = warp >= 6 ? 1 : 0;
    uint32_t tile_it = 0;
    bool alive = true;
    for (int item = blockIdx.x; item < P.total_items; item += gridDim.x, ++tile_it) {
      const WideItem t = wide_decode(P, item, per_example, nblk);
      const WideLayer& L = P.L[t.l];
      const uint32_t tph = tile_it & 1u;
      const bool active = h < t.ncol;
      const uint32_t tsrc = tmem_base + ((q * 32u) << 16) + (uint32_t)h * 128u;
      if (alive) alive = __all_sync(0xffffffffu, mbar_wait(&S->x_full, tph, abort_flag, P.status, 24, (int)tile_it));
      if (!alive) continue;
      tc_fence_after();
      uint32_t pv[4][32];
      if (active) {
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) tmem_ld_32x32(tsrc + (uint32_t)ch * 32u, pv[ch]);
        tmem_ld_wait();
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&S->x_empty);
      alive = __all_sync(0xffffffffu, mbar_wait(&S->y_full, tph, abort_flag, P.status, 25, (int)tile_it));
      if (!alive) continue;
      tc_fence_after();
      const float bias1 = L.has_bias ? 1.0f : 0.0f;
      float sum = 0.0f;
      if (active) {
#pragma unroll
        for (int ch = 0; ch < 4; ++ch) {
          uint32_t qv[32];
          tmem_ld_32x32(tsrc + 256u + (uint32_t)ch * 32u, qv);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 32; ++j) sum = fmaf(__uint_as_float(pv[ch][j]) + bias1, __uint_as_float(qv[j]), sum);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&S->y_empty);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_down_sync(0xffffffffu, sum, o);
      if (lane == 0)
        P.partial[(size_t)t.i * P.partial_stride + L.partial_base + t.idx * 8 + h * 4 + (int)q] =
            (t.c0 + h == t.r) ? sum : 2.0f * sum;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

struct TileItem { int l, m0, n0, e, slot; };
constexpr int T_THREADS = 320;                          // warp 0 TMA, warp 1 UMMA issue (or forwarding), warps 2..9 epilogue

// =================================================================================================
// Tile kernel on CTA pairs: 256 (d_out) x 256 (d_in) tiles of ONE example's A_i^T G_i (cta_group::2).
// CTA r of the pair streams G features [m0 + 128 r, +128) (its rows of the tile) and A features
// [n0 + 128 r, +128) (its half of the N operand): 64 KB per 128-token stage and CTA for 1024 tensor cycles, where
// a lone CTA with a 128 x 256 tile needs 96 KB (measured: 932 -> 964 TFLOP/s at T=128, 1000 -> 1080 at T=512).  Two 256-column TMEM accumulators per CTA: the square-sum of a
// tile overlaps the UMMAs of the next.  The odd CTA's warp 1 forwards "my stage has landed" to the even CTA,
// whose warp 1 issues the UMMAs for both.
// =================================================================================================
constexpr int Q_BK = 128;                               // tokens per stage: one box per operand covers 8 k-steps (64-token
                                                        // stages, twice as many, measured 5-10 % slower: a copy has a fixed cost)
constexpr int Q_STAGES = 3;
constexpr int Q_ATOM_BYTES = Q_BK * 128;                // Q_BK tokens x 64 bf16 features
constexpr int Q_HALF_BYTES = 2 * Q_ATOM_BYTES;          // 128 features
constexpr int Q_STAGE_BYTES = 2 * Q_HALF_BYTES;         // G rows + A half
struct TilePairCtl {
  uint64_t full[Q_STAGES], empty[Q_STAGES], ready[Q_STAGES], tmem_full[2], tmem_empty[2], drain;
  uint32_t tmem_base;
  int abort;
};
constexpr int Q_SMEM = 1024 + Q_STAGES * Q_STAGE_BYTES + (int)sizeof(TilePairCtl);
static_assert(Q_SMEM <= 232448, "over the shared memory of one CTA");

// tiles_m / tiles_n count 256-wide tiles here; 16 partial sums per tile
__device__ __forceinline__ TileItem tile_pair_decode(const UmmaParams& P, int item) {
  TileItem t;
  t.l = find_layer(P, item);
  const UmmaLayer& L = P.L[t.l];
  const int rem = item - L.item_start, tiles = L.tiles_m * L.tiles_n;
  t.e = rem / tiles;
  const int tile = rem - t.e * tiles;
  const int mt = tile / L.tiles_n;
  t.m0 = mt * 256;
  t.n0 = (tile - mt * L.tiles_n) * 256;
  t.slot = L.partial_base + tile * 16;
  return t;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(T_THREADS, 1)
k_tile_sqnorm_pair(const __grid_constant__ UmmaParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = align1024(smem_raw);
  TilePairCtl* S = reinterpret_cast<TilePairCtl*>(tiles + Q_STAGES * Q_STAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &S->abort;
  const uint32_t rank = cluster_ctarank();
  const int first_item = (int)cluster_id_x(), item_stride = (int)cluster_count_x();

  if (threadIdx.x == 0) {
    for (int s = 0; s < Q_STAGES; ++s) { mbar_init(&S->full[s], 1); mbar_init(&S->empty[s], 1); mbar_init(&S->ready[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&S->tmem_full[b], 1); mbar_init(&S->tmem_empty[b], 16); }
    mbar_init(&S->drain, 1);
    S->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc_pair(&S->tmem_base, 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();           // the peer's barriers are initialised before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = S->tmem_base;
  const int n_tb = (P.T + Q_BK - 1) / Q_BK;

  if (warp == 0) {
    if (lane == 0) {   // ---------------- TMA producer (each CTA, its own slices) ----------------
      uint32_t it = 0;
      bool alive = true;
      for (int item = first_item; item < P.total_items && alive; item += item_stride) {
        const TileItem t = tile_pair_decode(P, item);
        const UmmaLayer& L = P.L[t.l];
        for (int tb = 0; tb < n_tb; ++tb) {
          const uint32_t slot = it % Q_STAGES, ph = (it / Q_STAGES) & 1u;
          if (!mbar_wait(&S->empty[slot], ph ^ 1u, abort_flag, P.status, 41, (int)it)) { alive = false; break; }
          uint8_t* st = tiles + slot * Q_STAGE_BYTES;
          // two boxes of 64 features x Q_BK tokens x 2 feature groups; tokens beyond T and groups beyond the
          // layer's width arrive as zeros
          mbar_arrive_expect_tx(&S->full[slot], (uint32_t)Q_STAGE_BYTES);
          load_groups(st, &L.mapG, &S->full[slot], L.rag_g, 2, Q_ATOM_BYTES, t.m0 + 128 * (int)rank, tb * Q_BK, t.e);
          load_groups(st + Q_HALF_BYTES, &L.mapA, &S->full[slot], L.rag_a, 2, Q_ATOM_BYTES, t.n0 + 128 * (int)rank,
                      tb * Q_BK, t.e);
          ++it;
        }
      }
      const uint32_t pending = it < (uint32_t)Q_STAGES ? it : (uint32_t)Q_STAGES;
      for (uint32_t k = 0; k < pending; ++k) {
        const uint32_t j = it - 1 - k;
        mbar_wait_drain(&S->full[j % Q_STAGES], (j / Q_STAGES) & 1u, P.status);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 1) {   // ---------------- odd CTA: forward "stage landed" to the issuer ----------------
      uint32_t it = 0;
      bool alive = true;
      for (int item = first_item; item < P.total_items && alive; item += item_stride) {
        for (int tb = 0; tb < n_tb; ++tb, ++it) {
          const uint32_t slot = it % Q_STAGES, ph = (it / Q_STAGES) & 1u;
          if (!mbar_wait(&S->full[slot], ph, abort_flag, P.status, 46, (int)it)) { alive = false; break; }
          mbar_arrive_cluster(&S->ready[slot], 0u);
        }
      }
    } else if (lane == 0) {   // ---------------- even CTA: UMMA issuer ----------------
      constexpr uint32_t IDESC = idesc_bf16_f32(256, 256, true, true);
      uint32_t it = 0, tile_it = 0;
      bool alive = true;
      for (int item = first_item; item < P.total_items && alive; item += item_stride, ++tile_it) {
        const uint32_t buf = tile_it & 1u, tph = (tile_it >> 1) & 1u;
        if (!mbar_wait(&S->tmem_empty[buf], tph ^ 1u, abort_flag, P.status, 42, (int)tile_it)) { alive = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * 256u;
        uint32_t first = 0;
        for (int tb = 0; tb < n_tb; ++tb) {
          const uint32_t slot = it % Q_STAGES, ph = (it / Q_STAGES) & 1u;
          ++it;
          if (!mbar_wait(&S->full[slot], ph, abort_flag, P.status, 43, (int)it) ||
              !mbar_wait(&S->ready[slot], ph, abort_flag, P.status, 47, (int)it)) {
            alive = false;
            break;
          }
          tc_fence_after();
          const uint32_t am = smem_u32(tiles + slot * Q_STAGE_BYTES), an = am + Q_HALF_BYTES;
          const int left = P.T - tb * Q_BK, nk = left >= Q_BK ? Q_BK / 16 : (left + 15) >> 4;   // k-steps that hold tokens
#pragma unroll
          for (int k8 = 0; k8 < Q_BK / 16; ++k8) {
            if (k8 < nk)
              umma_bf16_pair(d_tmem, smem_desc_sw128(am + k8 * 2048, Q_ATOM_BYTES, 1024),
                             smem_desc_sw128(an + k8 * 2048, Q_ATOM_BYTES, 1024), IDESC, first | (uint32_t)k8);
          }
          first = 1;
          umma_commit_pair(&S->empty[slot], (uint16_t)3);
        }
        if (alive) umma_commit_pair(&S->tmem_full[buf], (uint16_t)3);
      }
      umma_commit_pair(&S->drain, (uint16_t)1);
      mbar_wait_drain(&S->drain, 0u, P.status);
    }
  } else {   // ---------------- epilogue warps 2..9: lanes [32 q, +32), accumulator columns [128 h, +128) ----------------
    const uint32_t q = (uint32_t)warp & 3u, h = warp >= 6 ? 1u : 0u;
    uint32_t tile_it = 0;
    bool alive = true;
    for (int item = first_item; item < P.total_items; item += item_stride, ++tile_it) {
      const TileItem t = tile_pair_decode(P, item);
      const uint32_t buf = tile_it & 1u, tph = (tile_it >> 1) & 1u;
      if (alive) alive = __all_sync(0xffffffffu, mbar_wait(&S->tmem_full[buf], tph, abort_flag, P.status, 44, (int)tile_it));
      if (!alive) continue;
      tc_fence_after();
      float sum = 0.0f;
#pragma unroll 1
      for (int ch = 0; ch < 4; ++ch) {
        uint32_t v[32];
        tmem_ld_32x32(tmem_base + ((q * 32u) << 16) + buf * 256u + h * 128u + (uint32_t)ch * 32u, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) sum = fmaf(__uint_as_float(v[j]), __uint_as_float(v[j]), sum);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(&S->tmem_empty[buf], 0u);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_down_sync(0xffffffffu, sum, o);
      if (lane == 0) P.partial[(size_t)t.e * P.partial_stride + t.slot + (int)(rank * 8u + h * 4u + q)] = sum;
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();           // neither CTA leaves while the other may still read its memory or signal it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

struct AccumItem { int l, m0, n0, e0, e1, nt; bool valid, narrow; };

// acc_w[(nb + j) * d_out + m] += v[j]: one lane owns row m (a d_out index), 32 columns per chunk.  The adds are
// reductions performed at the L2 (no read-back into the SM); an element has one owner per launch unless the
// example range is split, so the result does not depend on their order in the unsplit case.
__device__ __forceinline__ void accum_store_chunk(const UmmaLayer& L, int m, int nb, const uint32_t (&v)[32]) {
  if (m >= L.d_out || nb >= L.d_in) return;
  float* p = L.acc_w + (size_t)nb * L.d_out + m;
  const int nv = (L.d_in - nb) < 32 ? (L.d_in - nb) : 32;
#pragma unroll
  for (int j = 0; j < 32; ++j)
    if (j < nv) atomicAdd(p + (size_t)j * L.d_out, __uint_as_float(v[j]));
}

// =================================================================================================
// Clipped-accumulate kernel on CTA pairs (tcgen05 cta_group::2): a cluster of two CTAs owns one
// 256 (d_out) x 512 (d_in) output tile.  CTA r of the pair streams
//   G features [m0 + 128 r, +128)  -- the M rows whose accumulator lives in its own TMEM, and
//   A features [n0 + 256 r, +256)  -- its half of the N operand of both 256 x 256 x 16 UMMAs of a k-step
//                                     (the first 128 go to N-half 0, the second 128 to N-half 1),
// so per 1024 UMMA cycles an SM receives 48 KB instead of the 64 KB a lone CTA with a 256 x 256 tile needs, and
// its tensor core reads 64 KB of operands from shared memory instead of 96 KB (the other half of the N operand
// comes from the peer).  A lone CTA kept the tensor pipe 74 % busy, the pair 91-95 %.
// One thread of the even CTA issues the UMMAs for both; every CTA scales its own G rows by the clip factor
// in shared memory, sums its own bias columns and drains its own 128 x 512 accumulator.
//   in every CTA   : full[s] (own TMA), empty[s] and tmem_full (multicast commits of the issuer)
//   in the even CTA: ready[s] (16 worker warps of the pair have scaled stage s), tmem_empty (16 warps drained)
// Every waiter waits for every phase of its barrier in order and whoever re-arms a barrier is gated on all
// of its waiters (an mbarrier wait tells phases apart by parity only).  No TMA multicast is used.
// Column c of N-half j of a CTA's accumulator is A feature n0 + 256 (c / 128) + 128 j + c % 128.
// A tile with at most 256 A features left (the last one along d_in when d_in % 512 is in 1..256) is "narrow": CTA r
// streams features [n0 + 128 r, +128) as its N-half 0 and the second UMMA of every k-step is skipped.
// =================================================================================================
constexpr int P_BK = 64;                                // tokens per stage
constexpr int P_STAGES = 4;
constexpr int P_ATOM_BYTES = P_BK * 128;                // 64 tokens x 64 bf16 features
constexpr int P_M_BYTES = 2 * P_ATOM_BYTES;             // this CTA's 128 features of d_out (G)
constexpr int P_N_BYTES = 4 * P_ATOM_BYTES;             // this CTA's 256 features of d_in (A)
constexpr int P_STAGE_BYTES = P_M_BYTES + P_N_BYTES;    // 48 KB
constexpr int P_THREADS = 320;                          // warp 0 TMA, warp 1 UMMA issue, warps 2..9 workers

struct PairCtl {
  uint64_t full[P_STAGES], empty[P_STAGES], ready[P_STAGES], tmem_full, tmem_empty, drain;
  uint32_t tmem_base;
  int abort;
  float colsum[16][128];
};
constexpr int P_SMEM = 1024 + P_STAGES * P_STAGE_BYTES + (int)sizeof(PairCtl);

__device__ __forceinline__ AccumItem pair_decode(const UmmaParams& P, int item) {
  AccumItem t;
  t.l = find_layer(P, item);
  const UmmaLayer& L = P.L[t.l];
  const int rem = item - L.item_start, tiles = L.tiles_m * L.tiles_n;
  const int split = rem / tiles, tile = rem - split * tiles;
  t.valid = item >= L.item_start && split < P.splits;     // the slots of a wave that no layer fills are idle
  const int mt = tile / L.tiles_n;
  t.nt = tile - mt * L.tiles_n;
  t.m0 = mt * 256;
  t.n0 = t.nt * 512;
  t.narrow = L.d_in - t.n0 <= 256;     // at most 256 of the tile's 512 A features exist: one N-half carries them all
  t.e0 = (int)((long long)split * P.B / P.splits);
  t.e1 = (int)((long long)(split + 1) * P.B / P.splits);
  return t;
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(P_THREADS, 1)
k_accum_pair(const __grid_constant__ UmmaParams P) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* tiles = align1024(smem_raw);
  PairCtl* S = reinterpret_cast<PairCtl*>(tiles + P_STAGES * P_STAGE_BYTES);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &S->abort;
  const uint32_t rank = cluster_ctarank();
  const int first_item = (int)cluster_id_x(), item_stride = (int)cluster_count_x();
  constexpr uint32_t IDESC = idesc_bf16_f32(256, 256, true, true);

  if (threadIdx.x == 0) {
    for (int s = 0; s < P_STAGES; ++s) {
      mbar_init(&S->full[s], 1);
      mbar_init(&S->empty[s], 1);
      mbar_init(&S->ready[s], DP_ACCUM_READY == 2 ? 2 : 16);
    }
    mbar_init(&S->tmem_full, 1);
    mbar_init(&S->tmem_empty, 16);
    mbar_init(&S->drain, 1);
    S->abort = 0;
    fence_mbar_init();
  }
  if (warp == 1) { tmem_alloc_pair(&S->tmem_base, 512); tmem_relinquish_pair(); }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();           // the peer's barriers are initialised before anyone signals them
  tc_fence_after();
  const uint32_t tmem_base = S->tmem_base;
  const int n_tb = (P.T + P_BK - 1) / P_BK;

  if (warp == 0) {
    if (lane == 0) {   // ---------------- TMA producer (each CTA, its own slices) ----------------
      uint32_t it = 0;
      bool alive = true;
      bool align = P.wave_sync != nullptr;
      uint32_t wave = 0;
      for (int item = first_item; item < P.total_items && alive; item += item_stride, ++wave) {
        // Soft alignment: the tiles of a wave share operand blocks, which reach L2 once only if the pairs stream
        // them at the same time.  Every CTA announces that it has reached wave w and waits, for a bounded time,
        // until all have; a CTA that gives up once stops waiting altogether (the result does not depend on it).
        if (align && wave > 0) {
          atomicAdd(P.wave_sync, 1u);
          const unsigned int target = wave * gridDim.x;
          const long long t0 = clock64();
          while (*reinterpret_cast<volatile unsigned int*>(P.wave_sync) < target) {
            __nanosleep(200);
            if (clock64() - t0 > P.align_limit) { align = false; break; }
          }
        }
        const AccumItem t = pair_decode(P, item);
        if (!t.valid) continue;
        const UmmaLayer& L = P.L[t.l];
        const int mh = t.m0 + 128 * (int)rank, nh = t.n0 + (t.narrow ? 128 : 256) * (int)rank;
        for (int e = t.e0; e < t.e1 && alive; ++e) {
          for (int tb = 0; tb < n_tb; ++tb) {
            const uint32_t slot = it % P_STAGES, ph = (it / P_STAGES) & 1u;
            if (!mbar_wait(&S->empty[slot], ph ^ 1u, abort_flag, P.status, 11, (int)it)) { alive = false; break; }
            uint8_t* st = tiles + slot * P_STAGE_BYTES;
            // two boxes of 64 features x 64 tokens x (2 | 4) feature groups; tokens beyond T and feature groups
            // beyond the layer's width are outside the tensor and arrive as zeros
            mbar_arrive_expect_tx(&S->full[slot], (uint32_t)P_STAGE_BYTES);
            load_groups(st, &L.mapG, &S->full[slot], L.rag_g, 2, P_ATOM_BYTES, mh, tb * P_BK, e);
            load_groups(st + P_M_BYTES, &L.mapA, &S->full[slot], L.rag_a, 4, P_ATOM_BYTES, nh, tb * P_BK, e);
            ++it;
          }
        }
      }
      const uint32_t pending = it < (uint32_t)P_STAGES ? it : (uint32_t)P_STAGES;
      for (uint32_t k = 0; k < pending; ++k) {
        const uint32_t j = it - 1 - k;
        mbar_wait_drain(&S->full[j % P_STAGES], (j / P_STAGES) & 1u, P.status);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {   // ---------------- UMMA issuer (even CTA only) ----------------
      uint32_t it = 0, tile_it = 0;
      bool alive = true;
      for (int item = first_item; item < P.total_items && alive; item += item_stride) {
        const AccumItem t = pair_decode(P, item);
        if (!t.valid) continue;
        if (!mbar_wait(&S->tmem_empty, (tile_it & 1u) ^ 1u, abort_flag, P.status, 12, (int)tile_it)) { alive = false; break; }
        tc_fence_after();
        uint32_t acc = 0;
        for (int e = t.e0; e < t.e1 && alive; ++e) {
          for (int tb = 0; tb < n_tb; ++tb) {
            const uint32_t slot = it % P_STAGES, ph = (it / P_STAGES) & 1u;
            ++it;
            if (!mbar_wait<0, DP_ACCUM_READY != 0>(&S->ready[slot], ph, abort_flag, P.status, 13, (int)it)) {
              alive = false;
              break;
            }
            tc_fence_after();
            const uint32_t am = smem_u32(tiles + slot * P_STAGE_BYTES), an = am + P_M_BYTES;
            const int left = P.T - tb * P_BK;
            if (left >= P_BK && !t.narrow) {
#pragma unroll
              for (int k4 = 0; k4 < P_BK / 16; ++k4) {
                const uint64_t adesc = smem_desc_sw128(am + k4 * 2048, P_ATOM_BYTES, 1024);
#if DP_ACCUM_A_REUSE
                umma_bf16_pair_a_reuse<true>(tmem_base, adesc, smem_desc_sw128(an + k4 * 2048, P_ATOM_BYTES, 1024), IDESC,
                                             acc | (uint32_t)k4);
                umma_bf16_pair_a_reuse<false>(tmem_base + 256u, adesc,
                                              smem_desc_sw128(an + 2 * P_ATOM_BYTES + k4 * 2048, P_ATOM_BYTES, 1024), IDESC,
                                              acc | (uint32_t)k4);
#else
#pragma unroll
                for (int j = 0; j < 2; ++j)
                  umma_bf16_pair(tmem_base + (uint32_t)j * 256u, adesc,
                                 smem_desc_sw128(an + j * 2 * P_ATOM_BYTES + k4 * 2048, P_ATOM_BYTES, 1024), IDESC,
                                 acc | (uint32_t)k4);
#endif
              }
            } else {                                   // ragged last stage or narrow tile: only the UMMAs that carry data
              const int nk = left >= P_BK ? P_BK / 16 : (left + 15) >> 4, nj = t.narrow ? 1 : 2;
#pragma unroll 1
              for (int k4 = 0; k4 < nk; ++k4) {
                const uint64_t adesc = smem_desc_sw128(am + k4 * 2048, P_ATOM_BYTES, 1024);
                for (int j = 0; j < nj; ++j)
                  umma_bf16_pair(tmem_base + (uint32_t)j * 256u, adesc,
                                 smem_desc_sw128(an + j * 2 * P_ATOM_BYTES + k4 * 2048, P_ATOM_BYTES, 1024), IDESC,
                                 acc | (uint32_t)k4);
              }
            }
            acc = 1;
            umma_commit_pair(&S->empty[slot], (uint16_t)3);
          }
        }
        if (alive) umma_commit_pair(&S->tmem_full, (uint16_t)3);
        ++tile_it;
      }
      umma_commit_pair(&S->drain, (uint16_t)1);
      mbar_wait_drain(&S->drain, 0u, P.status);
    }
  } else {   // ---------------- warps 2..9: scale this CTA's G rows (and sum its bias columns), then drain ----------------
    const uint32_t q = (uint32_t)warp & 3u;
    const int h = warp >= 6 ? 1 : 0;                  // which N-half (256 accumulator columns) this warp drains
    const int tt = threadIdx.x - 64;                  // 0..255
    const int ta = tt >> 7, kk = (tt & 127) >> 3, jp = tt & 7;   // atom, token row & 15, physical 16-byte chunk
    const int jl = jp ^ (kk & 7);                     // logical chunk under the 128-byte swizzle
    uint32_t it = 0, tile_it = 0;
    bool alive = true;
    for (int item = first_item; item < P.total_items; item += item_stride) {
      const AccumItem t = pair_decode(P, item);
      if (!t.valid) continue;
      const UmmaLayer& L = P.L[t.l];
      const bool need_bias = L.has_bias && t.nt == 0;
      float col[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) col[u] = 0.0f;
      for (int e = t.e0; e < t.e1; ++e) {
        const float cf = alive ? __ldg(P.clip + e) : 1.0f;
        // c = c_hi + c_lo in bf16: fma(x, c_hi, x*c_lo) keeps the factor to ~2^-17 with two packed instructions; the
        // small term is the one rounded first, so the only rounding that counts is the final one to bf16 (2^-9)
        const __nv_bfloat16 chi = __float2bfloat16_rn(cf);
        const __nv_bfloat162 chi2 = __halves2bfloat162(chi, chi);
        const __nv_bfloat16 clo = __float2bfloat16_rn(cf - __bfloat162float(chi));
        const __nv_bfloat162 clo2 = __halves2bfloat162(clo, clo);
        for (int tb = 0; tb < n_tb; ++tb) {
          const uint32_t slot = it % P_STAGES, ph = (it / P_STAGES) & 1u;
          ++it;
          if (alive && !mbar_wait(&S->full[slot], ph, abort_flag, P.status, 14, (int)it)) alive = false;
#if DP_ACCUM_READY != 2
          if (!alive) continue;
#endif
          if (alive && (cf != 1.0f || need_bias)) {
            uint8_t* base = tiles + slot * P_STAGE_BYTES + ta * P_ATOM_BYTES + kk * 128 + jp * 16;
#pragma unroll
            for (int i4 = 0; i4 < P_BK / 16; ++i4) {   // rows kk, kk+16, ... of atom ta
              uint4* p = reinterpret_cast<uint4*>(base + i4 * 2048);
              uint4 w = *p;
              uint32_t x[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
              for (int u = 0; u < 4; ++u) {
                if (need_bias) {
                  col[2 * u] = fmaf(__uint_as_float(x[u] << 16), cf, col[2 * u]);
                  col[2 * u + 1] = fmaf(__uint_as_float(x[u] & 0xffff0000u), cf, col[2 * u + 1]);
                }
                const __nv_bfloat162 xv = *reinterpret_cast<const __nv_bfloat162*>(&x[u]);
                const __nv_bfloat162 yv = __hfma2(xv, chi2, __hmul2(xv, clo2));
                x[u] = *reinterpret_cast<const uint32_t*>(&yv);
              }
              if (cf != 1.0f) *p = make_uint4(x[0], x[1], x[2], x[3]);
            }
            fence_proxy_async_smem();
          }
#if DP_ACCUM_READY == 2
          // one barrier per stage: all 256 workers have rescaled their share (and agree on whether anyone gave up)
          {
            uint32_t all_alive;
            asm volatile(
                "{\n"
                ".reg .pred p, q;\n"
                "setp.ne.b32 q, %1, 0;\n"
                "bar.red.and.pred p, 3, 256, q;\n"
                "selp.u32 %0, 1, 0, p;\n"
                "}\n"
                : "=r"(all_alive)
                : "r"((uint32_t)alive)
                : "memory");
            alive = all_alive != 0;
          }
          if (alive && tt == (int)((it & 7u) << 5)) mbar_arrive_cluster_release(&S->ready[slot], 0u);
#elif DP_ACCUM_READY == 1
          __syncwarp();
          if (lane == 0) {
            fence_acq_rel_cluster();
            mbar_arrive_cluster(&S->ready[slot], 0u);
          }
#else
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster(&S->ready[slot], 0u);
#endif
        }
      }
      if (need_bias) {      // uniform over the 256 worker threads; executed even after an abort
#pragma unroll
        for (int u = 0; u < 8; ++u) S->colsum[kk][ta * 64 + jl * 8 + u] = col[u];
        asm volatile("bar.sync 2, 256;" ::: "memory");
        const int mcol = t.m0 + 128 * (int)rank + tt;
        if (alive && tt < 128 && mcol < L.d_out) {
          float sacc = 0.0f;
#pragma unroll
          for (int r = 0; r < 16; ++r) sacc += S->colsum[r][tt];
          atomicAdd(L.acc_b + mcol, sacc);
        }
        asm volatile("bar.sync 2, 256;" ::: "memory");
      }
      // ---- drain this CTA's accumulator: lanes [32 q, +32), columns [256 h, +256)
      const uint32_t tph = tile_it & 1u;
      ++tile_it;
      if (alive) alive = __all_sync(0xffffffffu, mbar_wait(&S->tmem_full, tph, abort_flag, P.status, 15, (int)tile_it));
      if (!alive) continue;
      tc_fence_after();
      const int m = t.m0 + 128 * (int)rank + (int)q * 32 + lane;
      // narrow tile: N-half 0 alone holds features n0 + 128 (c / 128) + c % 128; N-half 1 was never written
      if (!(t.narrow && h)) {
        // two register buffers: the TMEM load of chunk ch + 1 is in flight while chunk ch goes out as L2 reductions
        uint32_t v[2][32];
        const uint32_t tsrc = tmem_base + ((q * 32u) << 16) + (uint32_t)h * 256u;
        const int nstep = t.narrow ? 128 : 256;
        tmem_ld_32x32(tsrc, v[0]);
#pragma unroll
        for (int ch = 0; ch < 8; ++ch) {
          tmem_ld_wait();
          if (ch + 1 < 8) tmem_ld_32x32(tsrc + (uint32_t)(ch + 1) * 32u, v[(ch + 1) & 1]);
          accum_store_chunk(L, m, t.n0 + nstep * (ch >> 2) + 128 * h + (ch & 3) * 32, v[ch & 1]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(&S->tmem_empty, 0u);
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();           // neither CTA leaves while the other may still read its memory or signal it
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem_base, 512);
  }
}

// =================================================================================================
// Host side: tensor maps, work lists, launches
// =================================================================================================
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is resolved at run time so that the library loads on machines without a driver.
static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor [B, T, d] viewed as (x = 64 features, y = token, a = 64-feature group, z = example);
// box = 64 x box_rows x groups x 1, 128-byte swizzle, out-of-range elements read as zero.
static bool encode_map4(CUtensorMap* map, const void* base, int B, int T, int d, int box_rows, int groups) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {64u, (cuuint64_t)T, (cuuint64_t)(d / 64), (cuuint64_t)B};
  const cuuint64_t strides[3] = {(cuuint64_t)d * 2, 128u, (cuuint64_t)T * d * 2};
  const cuuint32_t box[4] = {64u, (cuuint32_t)box_rows, (cuuint32_t)groups, 1u};
  const cuuint32_t estr[4] = {1u, 1u, 1u, 1u};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            DP_TMA_L2_PROMOTION == 0 ? CU_TENSOR_MAP_L2_PROMOTION_NONE
            : DP_TMA_L2_PROMOTION == 1 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// bf16 tensor [B, T, d] as (x = feature, y = token, z = example); box = 64 features x box_rows tokens of one
// example, 128-byte swizzle, out-of-range elements read as zero.
static bool encode_map3(CUtensorMap* map, const void* base, int B, int T, int d, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)T, (cuuint64_t)B};
  const cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)T * d * 2};
  const cuuint32_t box[3] = {64u, (cuuint32_t)box_rows, 1u};
  const cuuint32_t estr[3] = {1u, 1u, 1u};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
            DP_TMA_L2_PROMOTION == 0 ? CU_TENSOR_MAP_L2_PROMOTION_NONE
            : DP_TMA_L2_PROMOTION == 1 ? CU_TENSOR_MAP_L2_PROMOTION_L2_128B : CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool umma_supported(const dp_layer& L) {
  // widths must be multiples of 8: a token row is then a multiple of 16 bytes, which the tensor maps require
  if (L.kind == DP_EMBEDDING) {   // mask-Gram norm only (the accumulate is a scatter, not a contraction)
    return L.dtype == DP_BF16 && L.d_out % 8 == 0 && (reinterpret_cast<uintptr_t>(L.G) & 15u) == 0 &&
           (long long)L.T * L.d_out * 2 < (1ll << 40);
  }
  if (L.kind != DP_LINEAR || L.dtype != DP_BF16) return false;
  if (L.d_in % 8 != 0 || L.d_out % 8 != 0) return false;
  if ((reinterpret_cast<uintptr_t>(L.A) | reinterpret_cast<uintptr_t>(L.G)) & 15u) return false;
  if ((long long)L.T * (L.d_in > L.d_out ? L.d_in : L.d_out) * 2 >= (1ll << 40)) return false;
  return true;
}

static int gram_pairs(int T) { const int nb = (T + 127) / 128; return nb * (nb + 1) / 2; }
static int tile_count(const dp_layer& L) { return ceil_div(L.d_out, 256) * ceil_div(L.d_in, 256); }
static int tile_partials(const dp_layer& L) { return 16 * tile_count(L); }
// Gram layers with more than one token block run on the two-column-block kernel (linear layers only: the
// id-equality mask of an embedding is applied by the one-block-pair kernel).
static bool gram_wide(const dp_layer& L) { return L.kind == DP_LINEAR && L.T > 128; }
// fp32 partial sums per example that a layer's norm kernel writes
static int sqnorm_partials(const dp_layer& L, bool gram) {
  if (!gram) return tile_partials(L);
  return gram_wide(L) ? 8 * wide_items((L.T + 127) / 128) : 4 * gram_pairs(L.T);
}

size_t umma_sqnorm_partials_per_example(const dp_layer* layers, const int* idx, int n, const int* use_gram) {
  size_t c = 0;
  for (int k = 0; k < n; ++k) c += (size_t)sqnorm_partials(layers[idx[k]], use_gram[k] != 0);
  return c;
}

// Per-device facts, looked up once for each device a process drives (one process may drive several GPUs).
constexpr int kMaxDevices = 64;
static int current_device() {
  int dev = 0;
  return (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < kMaxDevices) ? dev : -1;
}

static int sm_count() {
  static int sms[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0) return 148;
  if (!sms[dev]) {
    int n = 0;
    cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
    sms[dev] = n > 0 ? n : 148;
  }
  return sms[dev];
}

template <typename K>
static bool ensure_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// The opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of a kernel.
static bool sqnorm_kernels_ready();
static bool accum_kernel_ready();

// groups_g / groups_a: 64-feature groups that a box of the G / A map spans.
// A box may be taller than T or span more groups than the layer has: what lies outside the tensor is zero-filled.
static bool fill_layer(UmmaLayer& U, const dp_layer& L, int box_rows, int groups_g, int groups_a) {
  const bool emb = L.kind == DP_EMBEDDING;
  U.rag_g = L.d_out % 64 != 0;
  U.rag_a = !emb && L.d_in % 64 != 0;
  if (!(U.rag_g ? encode_map3(&U.mapG, L.G, L.B, L.T, L.d_out, box_rows)
                : encode_map4(&U.mapG, L.G, L.B, L.T, L.d_out, box_rows, groups_g))) return false;
  if (emb) U.mapA = U.mapG;      // never used: an embedding streams no A operand (d_in = 0 below)
  else if (!(U.rag_a ? encode_map3(&U.mapA, L.A, L.B, L.T, L.d_in, box_rows)
                     : encode_map4(&U.mapA, L.A, L.B, L.T, L.d_in, box_rows, groups_a))) return false;
  U.acc_w = L.acc_w;
  U.acc_b = L.acc_b;
  U.ids = emb ? L.ids : nullptr;
  U.d_out = L.d_out;
  U.d_in = emb ? 0 : L.d_in;
  U.tiles_m = (uint16_t)ceil_div(L.d_out, 128);
  U.tiles_n = (uint16_t)ceil_div(L.d_in, 256);
  U.has_bias = emb ? 0 : L.has_bias;
  U.is_emb = emb ? 1 : 0;
  for (uint8_t& x : U.pad) x = 0;
  return true;
}

static bool sqnorm_kernels_ready() {
  static signed char state[kMaxDevices] = {};     // 0 unknown, 1 ready, -1 failed
  const int dev = current_device();
  if (dev < 0) return false;
  if (!state[dev])
    state[dev] = (ensure_smem(k_gram_sqnorm, G_SMEM) && ensure_smem(k_gram_sqnorm_short, G_SMEM_SHORT) &&
                  ensure_smem(k_gram_sqnorm_wide, W_SMEM) &&
                  ensure_smem(k_tile_sqnorm_pair, Q_SMEM)) ? 1 : -1;
  return state[dev] > 0;
}

static bool accum_kernel_ready() {
  static signed char state[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0) return false;
  if (!state[dev]) state[dev] = ensure_smem(k_accum_pair, P_SMEM) ? 1 : -1;
  return state[dev] > 0;
}

int launch_umma_sqnorms(const dp_layer* layers, const int* idx, int n, const int* use_gram, float* partial,
                        int partial_stride, int partial_base, int* status, cudaStream_t s) {
  if (n <= 0) return DP_OK;
  const int B = layers[idx[0]].B, T = layers[idx[0]].T;
  if (!sqnorm_kernels_ready()) return DP_ERR_CUDA;
  // Partial slots are assigned in the caller's layer order, whichever kernel fills them.
  std::vector<int> base(n);
  int pos = partial_base;
  for (int k = 0; k < n; ++k) {
    base[k] = pos;
    pos += sqnorm_partials(layers[idx[k]], use_gram[k] != 0);
  }
  {   // Gram layers with several token blocks, widest first: items go to the CTAs round-robin, so the last,
      // partly filled round then holds the shortest items
    const int per_example = wide_items((T + 127) / 128);
    std::vector<int> wide;
    for (int k = 0; k < n; ++k)
      if (use_gram[k] && gram_wide(layers[idx[k]])) wide.push_back(k);
    std::stable_sort(wide.begin(), wide.end(), [&](int a, int b) {
      return layers[idx[a]].d_in + layers[idx[a]].d_out > layers[idx[b]].d_in + layers[idx[b]].d_out;
    });
    size_t w = 0;
    while (w < wide.size()) {
      WideParams P;
      P.n_layers = 0;
      long long items = 0;
      for (; w < wide.size() && P.n_layers < kWideMaxLayers; ++w) {
        const int k = wide[w];
        const dp_layer& L = layers[idx[k]];
        const long long add = (long long)B * per_example;
        if (items + add > 0x7fffffffll) break;
        WideLayer& W = P.L[P.n_layers];
        if (!encode_map3(&W.rowA, L.A, B, T, L.d_in, 128) || !encode_map3(&W.colA, L.A, B, T, L.d_in, 256) ||
            !encode_map3(&W.rowG, L.G, B, T, L.d_out, 128) || !encode_map3(&W.colG, L.G, B, T, L.d_out, 256))
          return DP_ERR_CUDA;
        W.d_out = L.d_out;
        W.d_in = L.d_in;
        W.item_start = (int)items;
        W.partial_base = base[k];
        W.has_bias = L.has_bias;
        for (int& x : W.pad) x = 0;
        items += add;
        ++P.n_layers;
      }
      if (P.n_layers == 0) return DP_ERR_UNSUPPORTED;     // one layer alone has more items than an int holds
      P.total_items = (int)items;
      P.B = B;
      P.T = T;
      P.partial_stride = partial_stride;
      P.pad = 0;
      P.partial = partial;
      P.status = status;
      const int grid = P.total_items < sm_count() ? P.total_items : sm_count();
      k_gram_sqnorm_wide<<<grid, W_THREADS, W_SMEM, s>>>(P);
      if (counted(1) != cudaSuccess) return DP_ERR_CUDA;
    }
  }
  // Short examples (one token block that is mostly empty): copies of T rounded up to 16 token rows, as many feature
  // groups per copy as fit a ring slot
  const int short_rows = T <= 112 ? ((T + 15) / 16) * 16 : 0;
  const int short_groups = short_rows ? 256 / short_rows : 0;
  for (int pass = 0; pass < 2; ++pass) {             // pass 0: one-block-pair Gram layers, pass 1: materialised tiles
    const bool gram = pass == 0;
    int k = 0;
    while (k < n) {
      UmmaParams P;
      P.n_layers = 0;
      long long items = 0;
      for (; k < n && P.n_layers < kMaxLayers; ++k) {
        if ((use_gram[k] != 0) != gram) continue;
        if (gram && gram_wide(layers[idx[k]])) continue;
        const dp_layer& L = layers[idx[k]];
        const long long add = (long long)B * (gram ? gram_pairs(T) : tile_count(L));
        if (items + add > 0x7fffffffll) break;
        UmmaLayer& U = P.L[P.n_layers];
        if (!(gram ? fill_layer(U, L, short_rows ? short_rows : 128, short_rows ? short_groups : G_GROUPS,
                                short_rows ? short_groups : G_GROUPS)
                   : fill_layer(U, L, Q_BK, 2, 2)))
          return DP_ERR_CUDA;
        if (!gram) {
          U.tiles_m = (uint16_t)ceil_div(L.d_out, 256);
          U.tiles_n = (uint16_t)ceil_div(L.d_in, 256);
        }
        U.item_start = (int)items;
        U.partial_base = base[k];
        items += add;
        ++P.n_layers;
      }
      if (P.n_layers == 0) continue;
      P.total_items = (int)items;
      P.B = B;
      P.T = T;
      P.splits = 1;
      P.partial_stride = partial_stride;
      P.clip = nullptr;
      P.wave_sync = nullptr;
      P.align_limit = 0;
      P.partial = partial;
      P.status = status;
      const int grid = P.total_items < sm_count() ? P.total_items : sm_count();
      P.box_rows = short_rows;
      P.box_groups = short_groups;
      if (gram && short_rows) {
        k_gram_sqnorm_short<<<grid, G_THREADS, G_SMEM_SHORT, s>>>(P);
      } else if (gram) {
        k_gram_sqnorm<<<grid, G_THREADS, G_SMEM, s>>>(P);
      } else {
        const int units = sm_count() / 2;
        k_tile_sqnorm_pair<<<2 * (P.total_items < units ? P.total_items : units), T_THREADS, Q_SMEM, s>>>(P);
      }
      if (counted(1) != cudaSuccess) return DP_ERR_CUDA;
    }
  }
  return DP_OK;
}

// Work items are laid out in waves of `units` slots (one slot per CTA pair and wave; pair p runs slot p of
// every wave).  The tiles of a layer share operand blocks, so a layer's items are kept inside one wave where they
// fit (first-fit over the layers in decreasing size); slots that no layer fills stay idle.
static long long pack_waves(const std::vector<long long>& group, int units, std::vector<long long>& start) {
  const int n = (int)group.size();
  std::vector<int> order(n);
  for (int k = 0; k < n; ++k) order[k] = k;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return group[a] > group[b]; });
  std::vector<long long> fill;    // used slots per wave
  start.assign(n, 0);
  for (int k : order) {
    const long long g = group[k];
    size_t w = 0;
    if (g >= units) {
      w = fill.size();            // whole waves of its own; others may share its last one
    } else {
      while (w < fill.size() && fill[w] + g > units) ++w;
    }
    if (w == fill.size()) fill.push_back(0);
    start[k] = (long long)w * units + fill[w];
    long long left = g;
    while (left > 0) {
      if (w == fill.size()) fill.push_back(0);
      const long long take = left < units - fill[w] ? left : units - fill[w];
      fill[w] += take;
      left -= take;
      ++w;
    }
  }
  return (long long)fill.size() * units;
}

// The schedule of one accumulate launch over layers idx[0..n): the number of example ranges every tile is split
// into, the first work item of every layer, and (returned) the number of item slots = waves x units.
long long umma_accumulate_schedule(const dp_layer* layers, const int* idx, int n, int units, int* splits_out,
                                   std::vector<long long>& start) {
  const int B = layers[idx[0]].B;
  long long tiles = 0;
  for (int k = 0; k < n; ++k) {
    const dp_layer& L = layers[idx[k]];
    tiles += (long long)ceil_div(L.d_out, 256) * ceil_div(L.d_in, 512);
  }
  // Split the example range when the tiles alone cannot fill the machine: pick the smallest split count
  // (<= 8, <= B) whose last wave is at least 85% full.  Split tiles combine through fp32 atomics.
  int splits = 1;
  if (tiles < 4ll * units) {
    double best = 0.0;
    for (int sp = 1; sp <= 8 && sp <= B; ++sp) {
      const long long it = tiles * sp;
      const double eff = (double)it / (double)((it + units - 1) / units * units);
      if (eff > best + 1e-9) { best = eff; splits = sp; }
      if (eff >= 0.85) { splits = sp; break; }
    }
  }
  std::vector<long long> group(n);
  for (int k = 0; k < n; ++k) {
    const dp_layer& L = layers[idx[k]];
    group[k] = (long long)ceil_div(L.d_out, 256) * ceil_div(L.d_in, 512) * splits;
  }
  *splits_out = splits;
  return pack_waves(group, units, start);
}

int launch_umma_accumulate(const dp_layer* layers, const int* idx, int n, const float* clip, int* status,
                           unsigned int* wave_sync, cudaStream_t s) {
  if (n <= 0) return DP_OK;
  const int B = layers[idx[0]].B, T = layers[idx[0]].T;
  if (!accum_kernel_ready()) return DP_ERR_CUDA;
  const int bk = P_BK;
  const int units = sm_count() / 2;      // CTA pairs that work on tiles side by side
  for (int k0 = 0; k0 < n; k0 += kMaxLayers) {
    const int nl = (n - k0) < kMaxLayers ? (n - k0) : kMaxLayers;
    int splits = 1;
    std::vector<long long> start;
    const long long span = umma_accumulate_schedule(layers, idx + k0, nl, units, &splits, start);
    if (span > 0x7fffffffll) return DP_ERR_UNSUPPORTED;
    std::vector<int> by_start(nl);
    for (int k = 0; k < nl; ++k) by_start[k] = k;
    std::sort(by_start.begin(), by_start.end(), [&](int a, int b) { return start[a] < start[b]; });
    UmmaParams P;
    for (int j = 0; j < nl; ++j) {
      const dp_layer& L = layers[idx[k0 + by_start[j]]];
      UmmaLayer& U = P.L[j];
      if (!fill_layer(U, L, bk, 2, 4)) return DP_ERR_CUDA;
      U.tiles_m = (uint16_t)ceil_div(L.d_out, 256);
      U.tiles_n = (uint16_t)ceil_div(L.d_in, 512);
      U.item_start = (int)start[by_start[j]];
      U.partial_base = 0;
    }
    P.n_layers = nl;
    P.total_items = (int)span;
    P.B = B;
    P.T = T;
    P.splits = splits;
    P.partial_stride = 0;
    P.wave_sync = (DP_ACCUM_ALIGN && span > units) ? wave_sync : nullptr;     // a single wave needs no alignment
    // A pair with an idle slot waits one tile duration (about 1100 cycles per 64-token stage); twice that plus a
    // margin tells a late CTA from one that is not resident at all.
    P.align_limit = 2ll * (long long)B * ceil_div(T, bk) * 2000ll + 2000000ll;
    P.clip = clip;
    P.partial = nullptr;
    P.status = status;
    if (P.wave_sync && cudaMemsetAsync(P.wave_sync, 0, sizeof(unsigned int), s) != cudaSuccess) return DP_ERR_CUDA;
    k_accum_pair<<<2 * units, P_THREADS, P_SMEM, s>>>(P);     // the item stride of the kernel is the cluster count
    if (counted(1) != cudaSuccess) return DP_ERR_CUDA;
  }
  return DP_OK;
}

// ---------------------------------------------------------------------------------------------
// Wait limit and its self-test
// ---------------------------------------------------------------------------------------------
int set_wait_limit_cycles(long long cycles) {
  if (cycles <= 0) cycles = kDefaultWaitLimitCycles;
  return cudaMemcpyToSymbol(g_wait_limit_cycles, &cycles, sizeof(cycles)) == cudaSuccess ? DP_OK : DP_ERR_CUDA;
}

// One CTA whose two waiters poll a barrier that nobody ever arrives on, through the same bounded wait as the
// pipelines: the first to run out records the timeout and raises the CTA's abort flag, the other leaves by its own
// limit or by the flag, and the kernel returns.
__global__ void __launch_bounds__(64) k_selftest_wait(int* status) {
  __shared__ uint64_t bar;
  __shared__ int abort_word;
  volatile int* abort_flag = &abort_word;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_word = 0;
    fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) mbar_wait(&bar, 0u, abort_flag, status, 99, 7);
  if (threadIdx.x == 32) mbar_wait<64>(&bar, 0u, abort_flag, status, 98, 8);
  __syncthreads();
}

int launch_selftest_wait(int* status, cudaStream_t s) {
  k_selftest_wait<<<1, 64, 0, s>>>(status);
  return counted(1) == cudaSuccess ? DP_OK : DP_ERR_CUDA;
}

}  // namespace dpk
