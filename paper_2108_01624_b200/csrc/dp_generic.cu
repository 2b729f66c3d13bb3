// CUDA-core kernels that accept any shape and either dtype (fp32 or bf16 inputs, fp32 arithmetic).
// They carry the fp32 configurations, LayerNorm and embedding layers (which are bandwidth-bound
// reductions, not contractions), bias terms, and bf16 linear layers whose shape the tensor-core
// kernels exclude.  Every reduction runs in a fixed order, so results are reproducible.
#include "dp_internal.h"

// Tunables of the column-sum kernel (overridable with -D for experiments).
#ifndef DP_COLSUMS_MINBLOCKS
#define DP_COLSUMS_MINBLOCKS 2          // resident CTAs per SM asked of the compiler (caps the registers per thread)
#endif
#ifndef DP_COLSUMS_UNROLL
#define DP_COLSUMS_UNROLL 8             // token rows whose loads are issued together (8 with 2 CTAs per SM measured
                                        // best: 6.15 against 6.31 ms for the norm pass; 3 or 4 CTAs with 2 or 4 rows: no gain)
#endif

namespace dpk {

constexpr int kColsumsUnroll = DP_COLSUMS_UNROLL;

template <typename T> __device__ __forceinline__ float ldf(const T* p);
template <> __device__ __forceinline__ float ldf<float>(const float* p) { return __ldg(p); }
template <> __device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(*p);
}

// Sum over the block, result valid in thread 0.  Fixed tree => deterministic.
__device__ __forceinline__ float block_sum(float x, float* red /*[32]*/) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
  const int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  __syncthreads();
  if (l == 0) red[w] = x;
  __syncthreads();
  if (w == 0) {
    x = (l < nw) ? red[l] : 0.0f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_down_sync(0xffffffffu, x, o);
  }
  return x;
}

// ---------------------------------------------------------------------------------------------
// Linear layer, materialised per-example gradient: sum of squares of A_i^T G_i (+ bias column sums).
// One CTA per example; 64x64 output tiles, 4x4 per thread, token chunks of 16 staged in shared memory.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
k_lin_sqnorm_mat(const T* __restrict__ A, const T* __restrict__ G, int Tn, int d_in, int d_out, int has_bias,
                 float* __restrict__ sqnorm) {
  __shared__ float As[16][64 + 1];
  __shared__ float Gs[16][64 + 1];
  __shared__ float red[32];
  const int i = blockIdx.x;
  const T* Ai = A + (size_t)i * Tn * d_in;
  const T* Gi = G + (size_t)i * Tn * d_out;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float total = 0.0f;
  for (int p0 = 0; p0 < d_in; p0 += 64) {
    for (int q0 = 0; q0 < d_out; q0 += 64) {
      float acc[4][4] = {};
      for (int t0 = 0; t0 < Tn; t0 += 16) {
        for (int e = threadIdx.x; e < 16 * 64; e += 256) {
          const int t = e >> 6, c = e & 63;
          As[t][c] = (t0 + t < Tn && p0 + c < d_in) ? ldf(Ai + (size_t)(t0 + t) * d_in + p0 + c) : 0.0f;
          Gs[t][c] = (t0 + t < Tn && q0 + c < d_out) ? ldf(Gi + (size_t)(t0 + t) * d_out + q0 + c) : 0.0f;
        }
        __syncthreads();
#pragma unroll
        for (int t = 0; t < 16; ++t) {
          float a[4], g[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) { a[u] = As[t][ty * 4 + u]; g[u] = Gs[t][tx * 4 + u]; }
#pragma unroll
          for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int w = 0; w < 4; ++w) acc[u][w] = fmaf(a[u], g[w], acc[u][w]);
        }
        __syncthreads();
      }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int w = 0; w < 4; ++w) total = fmaf(acc[u][w], acc[u][w], total);
    }
  }
  if (has_bias) {
    for (int q = threadIdx.x; q < d_out; q += 256) {
      float s = 0.0f;
      for (int t = 0; t < Tn; ++t) s += ldf(Gi + (size_t)t * d_out + q);
      total = fmaf(s, s, total);
    }
  }
  total = block_sum(total, red);
  if (threadIdx.x == 0) sqnorm[i] += total;
}

// ---------------------------------------------------------------------------------------------
// Linear layer, token-Gram identity: sum_{t,s} (<a_t,a_s> + [bias]) * <g_t,g_s>.
// One CTA per example; 16x16 token pairs per tile, feature chunks of 32 staged in shared memory.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
k_lin_sqnorm_gram(const T* __restrict__ A, const T* __restrict__ G, int Tn, int d_in, int d_out, int has_bias,
                  float* __restrict__ sqnorm) {
  __shared__ float Xt[16][32 + 1];
  __shared__ float Xs[16][32 + 1];
  __shared__ float red[32];
  const int i = blockIdx.x;
  const T* Ai = A + (size_t)i * Tn * d_in;
  const T* Gi = G + (size_t)i * Tn * d_out;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float total = 0.0f;
  for (int t0 = 0; t0 < Tn; t0 += 16) {
    for (int s0 = 0; s0 < Tn; s0 += 16) {
      float pq[2] = {0.0f, 0.0f};
#pragma unroll
      for (int which = 0; which < 2; ++which) {
        const T* X = which ? Gi : Ai;
        const int d = which ? d_out : d_in;
        float dot = 0.0f;
        for (int k0 = 0; k0 < d; k0 += 32) {
          for (int e = threadIdx.x; e < 16 * 32; e += 256) {
            const int r = e >> 5, c = e & 31;
            Xt[r][c] = (t0 + r < Tn && k0 + c < d) ? ldf(X + (size_t)(t0 + r) * d + k0 + c) : 0.0f;
            Xs[r][c] = (s0 + r < Tn && k0 + c < d) ? ldf(X + (size_t)(s0 + r) * d + k0 + c) : 0.0f;
          }
          __syncthreads();
#pragma unroll
          for (int c = 0; c < 32; ++c) dot = fmaf(Xt[ty][c], Xs[tx][c], dot);
          __syncthreads();
        }
        pq[which] = dot;
      }
      if (t0 + ty < Tn && s0 + tx < Tn) total = fmaf(pq[0] + (has_bias ? 1.0f : 0.0f), pq[1], total);
    }
  }
  total = block_sum(total, red);
  if (threadIdx.x == 0) sqnorm[i] += total;
}

template <typename T>
static cudaError_t lin_sqnorm_t(const dp_layer& L, bool gram, float* sqnorm, cudaStream_t s) {
  const T* A = static_cast<const T*>(L.A);
  const T* G = static_cast<const T*>(L.G);
  if (gram) k_lin_sqnorm_gram<T><<<L.B, 256, 0, s>>>(A, G, L.T, L.d_in, L.d_out, L.has_bias, sqnorm);
  else      k_lin_sqnorm_mat<T><<<L.B, 256, 0, s>>>(A, G, L.T, L.d_in, L.d_out, L.has_bias, sqnorm);
  return counted(1);
}
cudaError_t launch_linear_sqnorm_generic(const dp_layer& L, bool gram, float* sqnorm, cudaStream_t s) {
  return L.dtype == DP_F32 ? lin_sqnorm_t<float>(L, gram, sqnorm, s) : lin_sqnorm_t<__nv_bfloat16>(L, gram, sqnorm, s);
}

// ---------------------------------------------------------------------------------------------
// Linear layer, clipped accumulate: acc_w[p,q] += sum_r clip[r / T] * A[r,p] * G[r,q], r over all B*T rows.
// One CTA per 64x64 output tile (single owner => plain read-modify-write, fixed summation order).
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
k_lin_accum(const T* __restrict__ A, const T* __restrict__ G, const float* __restrict__ clip, int rows, int Tn,
            int d_in, int d_out, float* __restrict__ acc_w) {
  __shared__ float As[16][64 + 1];
  __shared__ float Gs[16][64 + 1];
  const int q0 = blockIdx.x * 64, p0 = blockIdx.y * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  for (int r0 = 0; r0 < rows; r0 += 16) {
    for (int e = threadIdx.x; e < 16 * 64; e += 256) {
      const int r = e >> 6, c = e & 63;
      const bool ok = r0 + r < rows;
      const float cf = ok ? __ldg(clip + (r0 + r) / Tn) : 0.0f;
      As[r][c] = (ok && p0 + c < d_in) ? cf * ldf(A + (size_t)(r0 + r) * d_in + p0 + c) : 0.0f;
      Gs[r][c] = (ok && q0 + c < d_out) ? ldf(G + (size_t)(r0 + r) * d_out + q0 + c) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int r = 0; r < 16; ++r) {
      float a[4], g[4];
#pragma unroll
      for (int u = 0; u < 4; ++u) { a[u] = As[r][ty * 4 + u]; g[u] = Gs[r][tx * 4 + u]; }
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int w = 0; w < 4; ++w) acc[u][w] = fmaf(a[u], g[w], acc[u][w]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int u = 0; u < 4; ++u)
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const int p = p0 + ty * 4 + u, q = q0 + tx * 4 + w;
      if (p < d_in && q < d_out) acc_w[(size_t)p * d_out + q] += acc[u][w];
    }
}

cudaError_t launch_linear_accum_generic(const dp_layer& L, const float* clip, cudaStream_t s) {
  dim3 grid(ceil_div(L.d_out, 64), ceil_div(L.d_in, 64));
  if (L.dtype == DP_F32)
    k_lin_accum<float><<<grid, 256, 0, s>>>(static_cast<const float*>(L.A), static_cast<const float*>(L.G), clip,
                                            L.B * L.T, L.T, L.d_in, L.d_out, L.acc_w);
  else
    k_lin_accum<__nv_bfloat16><<<grid, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(L.A),
                                                    static_cast<const __nv_bfloat16*>(L.G), clip, L.B * L.T, L.T,
                                                    L.d_in, L.d_out, L.acc_w);
  return counted(1);
}

// ---------------------------------------------------------------------------------------------
// Per-example column sums over tokens (LayerNorm gain/bias gradients; linear bias gradient).
//   WITH_X: out[i][0..d) = sum_t X[i,t,:]*G[i,t,:], out[i][d..2d) = sum_t G[i,t,:]
//   else  : out[i][0..d) = sum_t G[i,t,:]
// One CTA per example: 128 column lanes (VEC columns each, 16-byte loads) x 4 token groups.
// ---------------------------------------------------------------------------------------------
template <typename T, int VEC> struct VecLoad;
template <> struct VecLoad<float, 4> {
  static __device__ __forceinline__ void ld(const float* p, float* o) {
    const float4 v = __ldg(reinterpret_cast<const float4*>(p));
    o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
  }
};
template <> struct VecLoad<__nv_bfloat16, 8> {
  static __device__ __forceinline__ void ld(const __nv_bfloat16* p, float* o) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      o[2 * k] = __uint_as_float(w[k] << 16);
      o[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
    }
  }
};
template <typename T> struct VecLoad<T, 1> {
  static __device__ __forceinline__ void ld(const T* p, float* o) { o[0] = ldf(p); }
};

template <typename T, int VEC, bool WITH_X>
__device__ __forceinline__ void
k_colsums_body(const T* __restrict__ X, const T* __restrict__ G, int Tn, int d, float* __restrict__ out) {
  __shared__ float sh[3][128][2 * VEC];
  const int i = blockIdx.x;
  const int lane = threadIdx.x & 127, tg = threadIdx.x >> 7;
  const T* Gi = G + (size_t)i * Tn * d;
  const T* Xi = WITH_X ? X + (size_t)i * Tn * d : nullptr;
  float* oi = out + (size_t)i * (WITH_X ? 2 : 1) * d;
  for (int c0 = 0; c0 < d; c0 += 128 * VEC) {
    const int col = c0 + lane * VEC;
    float sx[VEC], sg[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) { sx[k] = 0.0f; sg[k] = 0.0f; }
    if (col < d) {
#pragma unroll kColsumsUnroll
      for (int t = tg; t < Tn; t += 4) {
        float g[VEC], x[VEC];
        VecLoad<T, VEC>::ld(Gi + (size_t)t * d + col, g);
        if (WITH_X) VecLoad<T, VEC>::ld(Xi + (size_t)t * d + col, x);
#pragma unroll
        for (int k = 0; k < VEC; ++k) {
          sg[k] += g[k];
          if (WITH_X) sx[k] = fmaf(x[k], g[k], sx[k]);
        }
      }
    }
    __syncthreads();
    if (tg > 0) {
#pragma unroll
      for (int k = 0; k < VEC; ++k) { sh[tg - 1][lane][k] = sg[k]; sh[tg - 1][lane][VEC + k] = sx[k]; }
    }
    __syncthreads();
    if (tg == 0 && col < d) {
#pragma unroll
      for (int k = 0; k < VEC; ++k) {
        float a = sg[k], b = sx[k];
#pragma unroll
        for (int w = 0; w < 3; ++w) { a += sh[w][lane][k]; b += sh[w][lane][VEC + k]; }
        if (WITH_X) { oi[col + k] = b; oi[d + col + k] = a; } else { oi[col + k] = a; }
      }
    }
  }
}

// ---- batched over layers: one launch covers every LayerNorm (or bias) task of a call ------------------------
constexpr int kMaxColTasks = 64;
struct ColTask {
  const void* X;     // normalised input (WITH_X) or nullptr
  const void* G;
  float* out;        // [B][width] per-example column sums
  float* acc0;       // accumulate target of columns [0, d)
  float* acc1;       // accumulate target of columns [d, 2d) (WITH_X only)
  int d, width;
};
struct ColBatch {
  ColTask t[kMaxColTasks];
  int n, B, T, pad;
};

template <typename T, int VEC, bool WITH_X>
__global__ void __launch_bounds__(512, DP_COLSUMS_MINBLOCKS) k_colsums_b(const __grid_constant__ ColBatch P) {
  const ColTask& t = P.t[blockIdx.y];
  k_colsums_body<T, VEC, WITH_X>(static_cast<const T*>(t.X), static_cast<const T*>(t.G), P.T, t.d, t.out);
}

// sqnorm[i] += sum over tasks and columns of out[i][j]^2 (fixed order).
__global__ void __launch_bounds__(256) k_rows_sqsum_b(const __grid_constant__ ColBatch P, float* __restrict__ sqnorm) {
  __shared__ float red[32];
  float tot = 0.0f;
  for (int k = 0; k < P.n; ++k) {
    const float* w = P.t[k].out + (size_t)blockIdx.x * P.t[k].width;
    for (int j = threadIdx.x; j < P.t[k].width; j += 256) tot = fmaf(w[j], w[j], tot);
  }
  tot = block_sum(tot, red);
  if (threadIdx.x == 0) sqnorm[blockIdx.x] += tot;
}

// acc[j] += sum_i clip[i] * out[i][j] for task blockIdx.y; 64 columns x 4 example groups per CTA.
__global__ void __launch_bounds__(256)
k_weighted_rows_sum_b(const __grid_constant__ ColBatch P, const float* __restrict__ clip) {
  __shared__ float sh[4][64];
  const ColTask& t = P.t[blockIdx.y];
  const int c = threadIdx.x & 63, g = threadIdx.x >> 6;
  const int j = blockIdx.x * 64 + c;
  float a = 0.0f;
  if (j < t.width)
    for (int i = g; i < P.B; i += 4) a = fmaf(__ldg(clip + i), t.out[(size_t)i * t.width + j], a);
  sh[g][c] = a;
  __syncthreads();
  if (g == 0 && j < t.width) {
    const float v = (sh[0][c] + sh[1][c]) + (sh[2][c] + sh[3][c]);
    if (j < t.d) t.acc0[j] += v; else t.acc1[j - t.d] += v;
  }
}

// variant key of a task: dtype, vector width, with_x
static int col_variant(const dp_layer& L, bool with_x) {
  const int d = L.d_out;
  const bool al = ((reinterpret_cast<uintptr_t>(L.G) | (with_x ? reinterpret_cast<uintptr_t>(L.A) : 0)) & 15u) == 0;
  int v;
  if (L.dtype == DP_F32) v = (al && d % 4 == 0) ? 0 : 1; else v = (al && d % 8 == 0) ? 2 : 3;
  return v * 2 + (with_x ? 1 : 0);
}

template <typename T, int VEC>
static void colsums_b_launch(const ColBatch& P, bool with_x, cudaStream_t s) {
  dim3 grid(P.B, P.n);
  if (with_x) k_colsums_b<T, VEC, true><<<grid, 512, 0, s>>>(P); else k_colsums_b<T, VEC, false><<<grid, 512, 0, s>>>(P);
}

static ColTask make_task(const ColTaskHost& h) {
  const dp_layer& L = *h.L;
  ColTask t;
  t.X = h.with_x ? L.A : nullptr;
  t.G = L.G;
  t.out = h.out;
  t.d = L.d_out;
  t.width = (h.with_x ? 2 : 1) * L.d_out;
  t.acc0 = h.with_x ? L.acc_w : L.acc_b;
  t.acc1 = h.with_x ? L.acc_b : nullptr;
  return t;
}

cudaError_t launch_colsums_batched(const ColTaskHost* tasks, int n, cudaStream_t s) {
  // group by kernel variant, at most kMaxColTasks per launch
  for (int variant = 0; variant < 8; ++variant) {
    ColBatch P;
    P.n = 0;
    for (int k = 0; k <= n; ++k) {
      const bool take = k < n && col_variant(*tasks[k].L, tasks[k].with_x) == variant;
      if (take) {
        P.t[P.n++] = make_task(tasks[k]);
        P.B = tasks[k].L->B;
        P.T = tasks[k].L->T;
      }
      if (P.n == kMaxColTasks || (k == n && P.n > 0)) {
        const bool wx = variant & 1;
        switch (variant >> 1) {
          case 0: colsums_b_launch<float, 4>(P, wx, s); break;
          case 1: colsums_b_launch<float, 1>(P, wx, s); break;
          case 2: colsums_b_launch<__nv_bfloat16, 8>(P, wx, s); break;
          default: colsums_b_launch<__nv_bfloat16, 1>(P, wx, s); break;
        }
        const cudaError_t e = counted(1);
        if (e != cudaSuccess) return e;
        P.n = 0;
      }
    }
  }
  return cudaSuccess;
}

template <typename F>
static cudaError_t for_each_batch(const ColTaskHost* tasks, int n, F launch) {
  for (int k0 = 0; k0 < n; k0 += kMaxColTasks) {
    ColBatch P;
    P.n = (n - k0) < kMaxColTasks ? (n - k0) : kMaxColTasks;
    for (int k = 0; k < P.n; ++k) P.t[k] = make_task(tasks[k0 + k]);
    P.B = tasks[k0].L->B;
    P.T = tasks[k0].L->T;
    launch(P);
    const cudaError_t e = counted(1);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_rows_sqsum_batched(const ColTaskHost* tasks, int n, float* sqnorm, cudaStream_t s) {
  return for_each_batch(tasks, n, [&](const ColBatch& P) { k_rows_sqsum_b<<<P.B, 256, 0, s>>>(P, sqnorm); });
}

cudaError_t launch_weighted_rows_sum_batched(const ColTaskHost* tasks, int n, const float* clip, cudaStream_t s) {
  return for_each_batch(tasks, n, [&](const ColBatch& P) {
    int wmax = 0;
    for (int k = 0; k < P.n; ++k) wmax = P.t[k].width > wmax ? P.t[k].width : wmax;
    dim3 grid(ceil_div(wmax, 64), P.n);
    k_weighted_rows_sum_b<<<grid, 256, 0, s>>>(P, clip);
  });
}

__global__ void k_fill_zero(float* __restrict__ p, long long n) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < n; k += stride) p[k] = 0.0f;
}
cudaError_t launch_fill_zero(float* p, long long n, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  long long b = (n + 255) / 256;
  if (b > 148 * 8) b = 148 * 8;
  k_fill_zero<<<(int)b, 256, 0, s>>>(p, n);
  return counted(1);
}

// sqnorm[i] += sum_{j<count} partial[i*stride + j] in a fixed order.
__global__ void __launch_bounds__(256)
k_reduce_partials(const float* __restrict__ partial, int stride, int count, float* __restrict__ sqnorm) {
  __shared__ float red[32];
  const float* p = partial + (size_t)blockIdx.x * stride;
  float t = 0.0f;
  for (int j = threadIdx.x; j < count; j += 256) t += p[j];
  t = block_sum(t, red);
  if (threadIdx.x == 0) sqnorm[blockIdx.x] += t;
}
cudaError_t launch_reduce_partials(const float* partial, int B, int count, float* sqnorm, cudaStream_t s) {
  if (count <= 0) return cudaSuccess;
  k_reduce_partials<<<B, 256, 0, s>>>(partial, count, count, sqnorm);
  return counted(1);
}

// ---------------------------------------------------------------------------------------------
// Token embedding.  The per-example gradient has one row per DISTINCT id: the sum of the G rows
// whose ids are equal (the one-hot input makes A_i A_i^T the id-equality mask, so the squared norm
// sum_{t,s} [id_t == id_s] <G_t, G_s> is the sum over distinct ids of |sum of their rows|^2).
// One CTA per example.  leader[t] = first token with the same id (integer compares only).
// Norm kernel: sqnorm[i] += sum over leaders of |row sum|^2 (used when the Gram kernel's mask mode does not apply).
// Ids outside [0, V) are skipped and reported through the status word.
// ---------------------------------------------------------------------------------------------
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
k_embedding_sqnorm(const int32_t* __restrict__ ids, const T* __restrict__ G, int Tn, int V, int d,
                   float* __restrict__ out, int* __restrict__ status) {
  extern __shared__ int sh_i[];          // ids[T], leader[T]
  __shared__ float red[32];
  int* sid = sh_i;
  int* leader = sh_i + Tn;
  const int i = blockIdx.x;
  const T* Gi = G + (size_t)i * Tn * d;
  for (int t = threadIdx.x; t < Tn; t += blockDim.x) sid[t] = ids[(size_t)i * Tn + t];
  __syncthreads();
  for (int t = threadIdx.x; t < Tn; t += blockDim.x) {
    const int id = sid[t];
    int l = t;
    if (id < 0 || id >= V) {
      l = -1;
      atomicCAS(status, STATUS_OK, STATUS_BAD_ID);
    } else {
      for (int s = 0; s < t; ++s) if (sid[s] == id) { l = s; break; }
    }
    leader[t] = l;
  }
  __syncthreads();
  float total = 0.0f;
  for (int col = threadIdx.x * VEC; col < d; col += blockDim.x * VEC) {
    for (int l = 0; l < Tn; ++l) {
      if (leader[l] != l) continue;
      float sum[VEC];
#pragma unroll
      for (int k = 0; k < VEC; ++k) sum[k] = 0.0f;
      for (int s = l; s < Tn; ++s) {
        if (leader[s] != l) continue;
        float g[VEC];
        VecLoad<T, VEC>::ld(Gi + (size_t)s * d + col, g);
#pragma unroll
        for (int k = 0; k < VEC; ++k) sum[k] += g[k];
      }
#pragma unroll
      for (int k = 0; k < VEC; ++k) total = fmaf(sum[k], sum[k], total);
    }
  }
  total = block_sum(total, red);
  if (threadIdx.x == 0) out[i] += total;
}

// Accumulate, one warp per token: a warp whose token is the first of its id within the example (the leader) sums
// the example's rows with that id and adds clip[i] times the sum to acc[id] (fp32 atomics: rows of different
// examples collide, above all on the frequent ids).  grid = (B, ceil(T / 8)), 8 warps per block.
template <typename T, int VEC>
__global__ void __launch_bounds__(256)
k_embedding_accum(const int32_t* __restrict__ ids, const T* __restrict__ G, int Tn, int V, int d,
                  const float* __restrict__ clip, float* __restrict__ out, int* __restrict__ status, int vec_red) {
  extern __shared__ int sid[];           // ids[T] of this example
  const int i = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int t = threadIdx.x; t < Tn; t += blockDim.x) sid[t] = ids[(size_t)i * Tn + t];
  __syncthreads();
  const int t = blockIdx.y * 8 + warp;
  if (t >= Tn) return;
  const int id = sid[t];
  if (id < 0 || id >= V) {
    if (lane == 0) atomicCAS(status, STATUS_OK, STATUS_BAD_ID);
    return;
  }
  bool earlier = false;
  for (int s = lane; s < t; s += 32) earlier |= sid[s] == id;
  if (__any_sync(0xffffffffu, earlier)) return;      // not the leader of its id
  const T* Gi = G + (size_t)i * Tn * d;
  const float ci = __ldg(clip + i);
  float* dst = out + (size_t)id * d;
  for (int col0 = 0; col0 < d; col0 += 32 * VEC) {     // warp-uniform trip count: the ballots below need every lane
    const int col = col0 + lane * VEC;
    const bool in = col < d;
    float sum[VEC];
#pragma unroll
    for (int k = 0; k < VEC; ++k) sum[k] = 0.0f;
    for (int s0 = t & ~31; s0 < Tn; s0 += 32) {
      const int s = s0 + lane;
      unsigned m = __ballot_sync(0xffffffffu, s >= t && s < Tn && sid[s] == id);
      while (m) {
        const int b = __ffs(m) - 1;
        m &= m - 1;
        if (in) {
          float g[VEC];
          VecLoad<T, VEC>::ld(Gi + (size_t)(s0 + b) * d + col, g);
#pragma unroll
          for (int k = 0; k < VEC; ++k) sum[k] += g[k];
        }
      }
    }
    if (in) {
      if (VEC % 4 == 0 && vec_red) {        // 16-byte reductions: a quarter of the atomic operations at the L2
#pragma unroll
        for (int k = 0; k < VEC; k += 4)
          asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst + col + k), "f"(ci * sum[k]),
                       "f"(ci * sum[k + 1]), "f"(ci * sum[k + 2]), "f"(ci * sum[k + 3]) : "memory");
      } else {
#pragma unroll
        for (int k = 0; k < VEC; ++k) atomicAdd(dst + col + k, ci * sum[k]);
      }
    }
  }
}

cudaError_t launch_embedding_sqnorm(const dp_layer& L, float* sqnorm, int* status, cudaStream_t s) {
  const int d = L.d_out, V = L.d_in;
  const size_t sh = 2 * (size_t)L.T * sizeof(int);
  const bool al = (reinterpret_cast<uintptr_t>(L.G) & 15u) == 0;
  if (L.dtype == DP_F32) {
    const float* G = static_cast<const float*>(L.G);
    if (al && d % 4 == 0) k_embedding_sqnorm<float, 4><<<L.B, 256, sh, s>>>(L.ids, G, L.T, V, d, sqnorm, status);
    else                  k_embedding_sqnorm<float, 1><<<L.B, 256, sh, s>>>(L.ids, G, L.T, V, d, sqnorm, status);
  } else {
    const __nv_bfloat16* G = static_cast<const __nv_bfloat16*>(L.G);
    if (al && d % 8 == 0) k_embedding_sqnorm<__nv_bfloat16, 8><<<L.B, 128, sh, s>>>(L.ids, G, L.T, V, d, sqnorm, status);
    else                  k_embedding_sqnorm<__nv_bfloat16, 1><<<L.B, 256, sh, s>>>(L.ids, G, L.T, V, d, sqnorm, status);
  }
  return counted(1);
}
cudaError_t launch_embedding_accum(const dp_layer& L, const float* clip, int* status, cudaStream_t s) {
  const int d = L.d_out, V = L.d_in;
  const size_t sh = (size_t)L.T * sizeof(int);
  const dim3 grid((unsigned)L.B, (unsigned)((L.T + 7) / 8));
  const bool al = (reinterpret_cast<uintptr_t>(L.G) & 15u) == 0;
  const int vr = ((reinterpret_cast<uintptr_t>(L.acc_w) & 15u) == 0 && d % 4 == 0) ? 1 : 0;   // rows of the table 16-byte aligned
  if (L.dtype == DP_F32) {
    const float* G = static_cast<const float*>(L.G);
    if (al && d % 4 == 0) k_embedding_accum<float, 4><<<grid, 256, sh, s>>>(L.ids, G, L.T, V, d, clip, L.acc_w, status, vr);
    else                  k_embedding_accum<float, 1><<<grid, 256, sh, s>>>(L.ids, G, L.T, V, d, clip, L.acc_w, status, vr);
  } else {
    const __nv_bfloat16* G = static_cast<const __nv_bfloat16*>(L.G);
    if (al && d % 8 == 0) k_embedding_accum<__nv_bfloat16, 8><<<grid, 256, sh, s>>>(L.ids, G, L.T, V, d, clip, L.acc_w, status, vr);
    else                  k_embedding_accum<__nv_bfloat16, 1><<<grid, 256, sh, s>>>(L.ids, G, L.T, V, d, clip, L.acc_w, status, vr);
  }
  return counted(1);
}

// ---------------------------------------------------------------------------------------------
// Cross term of a table shared by a token embedding and an output projection: example i's gradient for the table
// is scatter_i + dlogits_i^T h_i, and <scatter_i, dlogits_i^T h_i> = sum_{t,s} dlogits[s, id_t] <h[s,:], G_emb[t,:]>.
// One CTA per example walks the T_out x T grid of token pairs in 64 x 64 blocks (a 4 x 4 micro-tile per thread,
// the feature dimension staged through shared memory 32 at a time) and weighs every inner product with the
// gathered output gradient.  Fixed order of summation: the result does not depend on the launch.
// ---------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(256)
k_shared_table_cross(const int32_t* __restrict__ ids, const T* __restrict__ Gemb, const T* __restrict__ dlogits,
                     const T* __restrict__ H, int Tn, int Tout, int d, int V, float* __restrict__ sqnorm,
                     int* __restrict__ status) {
  __shared__ float Hs[64][33], Gs[64][33];
  __shared__ float red[32];
  const int i = blockIdx.x;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const T* Hi = H + (size_t)i * Tout * d;
  const T* Gi = Gemb + (size_t)i * Tn * d;
  const T* Di = dlogits + (size_t)i * Tout * V;
  const int32_t* idi = ids + (size_t)i * Tn;
  float total = 0.0f;
  for (int s0 = 0; s0 < Tout; s0 += 64) {
    for (int t0 = 0; t0 < Tn; t0 += 64) {
      float acc[4][4];
#pragma unroll
      for (int u = 0; u < 4; ++u)
#pragma unroll
        for (int v = 0; v < 4; ++v) acc[u][v] = 0.0f;
      for (int k0 = 0; k0 < d; k0 += 32) {
        for (int e = threadIdx.x; e < 64 * 32; e += 256) {
          const int r = e >> 5, c = e & 31;
          const bool kin = k0 + c < d;
          Hs[r][c] = (kin && s0 + r < Tout) ? ldf(Hi + (size_t)(s0 + r) * d + k0 + c) : 0.0f;
          Gs[r][c] = (kin && t0 + r < Tn) ? ldf(Gi + (size_t)(t0 + r) * d + k0 + c) : 0.0f;
        }
        __syncthreads();
#pragma unroll 8
        for (int c = 0; c < 32; ++c) {
          float a[4], bb[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) { a[u] = Hs[ty * 4 + u][c]; bb[u] = Gs[tx * 4 + u][c]; }
#pragma unroll
          for (int u = 0; u < 4; ++u)
#pragma unroll
            for (int v = 0; v < 4; ++v) acc[u][v] = fmaf(a[u], bb[v], acc[u][v]);
        }
        __syncthreads();
      }
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        const int t = t0 + tx * 4 + v;
        if (t >= Tn) continue;
        const int id = idi[t];
        if (id < 0 || id >= V) {                     // skipped and reported, like the embedding kernels
          atomicCAS(status, STATUS_OK, STATUS_BAD_ID);
          continue;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int sx = s0 + ty * 4 + u;
          if (sx < Tout) total = fmaf(acc[u][v], ldf(Di + (size_t)sx * V + id), total);
        }
      }
    }
  }
  total = block_sum(total, red);
  if (threadIdx.x == 0) sqnorm[i] += 2.0f * total;
}

cudaError_t launch_shared_table_cross(const int32_t* ids, const void* G_emb, int B, int T, const void* dlogits,
                                      const void* h, int T_out, int d, int V, int dtype, float* sqnorm, int* status,
                                      cudaStream_t s) {
  if (dtype == DP_F32)
    k_shared_table_cross<float><<<B, 256, 0, s>>>(ids, static_cast<const float*>(G_emb), static_cast<const float*>(dlogits),
                                                  static_cast<const float*>(h), T, T_out, d, V, sqnorm, status);
  else
    k_shared_table_cross<__nv_bfloat16><<<B, 256, 0, s>>>(ids, static_cast<const __nv_bfloat16*>(G_emb),
                                                          static_cast<const __nv_bfloat16*>(dlogits),
                                                          static_cast<const __nv_bfloat16*>(h), T, T_out, d, V, sqnorm,
                                                          status);
  return counted(1);
}

}  // namespace dpk
