// Streaming kernels: clip factors, Philox4x32-10 noise + scaling, AdamW, and the fused pass.
// All are bandwidth-bound: one thread owns one Philox block (4 consecutive elements, one 16-byte
// vector per array), loads are fully coalesced, and the grid is a multiple of the SM count.
#include "dp_internal.h"

namespace dpk {

// ---------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): ten rounds of
//   (hi0,lo0) = M0*c0, (hi1,lo1) = M1*c2, c <- (hi1^c1^k0, lo1, hi0^c3^k1, lo0), key += (W0,W1).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(M0, c.x), lo0 = M0 * c.x;
    const uint32_t hi1 = __umulhi(M1, c.z), lo1 = M1 * c.z;
    c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    k0 += W0;
    k1 += W1;
  }
  return c;
}

__device__ __forceinline__ uint4 philox_block(unsigned long long j, const NoiseArgs& na) {
  return philox4x32_10(make_uint4((uint32_t)j, (uint32_t)(j >> 32), na.step0, na.step1), na.key0, na.key1);
}

// Box-Muller on one word pair.  The uniforms are exact binary32 values:
//   u1 = fl(x_a * 2^-32 + 2^-33) in (0,1],  u2 = fl(x_b * 2^-32) in [0,1].
// The logarithm is the accurate one (near u1 = 1 an approximate log would be off by more than the radius itself);
// the root and the sine / cosine may be the hardware approximations: the normals then carry an absolute error of
// about 3e-6 (|z| <= 6.76 times 5e-7) instead of 1e-7.
#ifndef DP_STREAM_FAST_MATH
#define DP_STREAM_FAST_MATH 1     // hardware approximations for sqrt, sin/cos and the AdamW division: about a quarter fewer
                                  // instructions per element; 0 selects sqrtf, sincospif and IEEE division
#endif
__device__ __forceinline__ float fast_sqrt(float x) {
#if DP_STREAM_FAST_MATH
  float y;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
#else
  return sqrtf(x);
#endif
}
__device__ __forceinline__ void box_muller(uint32_t xa, uint32_t xb, float& z_even, float& z_odd) {
  const float u1 = fmaf(__uint2float_rn(xa), 0x1p-32f, 0x1p-33f);
  const float u2 = __uint2float_rn(xb) * 0x1p-32f;
  const float r = fast_sqrt(-2.0f * logf(u1));
  float sn, cs;
#if DP_STREAM_FAST_MATH
  // angle 2 pi u2 folded to [-pi, pi) before the hardware sine / cosine (absolute error about 5e-7 there)
  const float ang = 6.283185307179586f * (u2 - (u2 >= 0.5f ? 1.0f : 0.0f));
  sn = __sinf(ang);
  cs = __cosf(ang);
#else
  sincospif(2.0f * u2, &sn, &cs);
#endif
  z_even = r * cs;
  z_odd = r * sn;
}

__device__ __forceinline__ float4 normals4(unsigned long long j, const NoiseArgs& na) {
  const uint4 x = philox_block(j, na);
  float4 z;
  box_muller(x.x, x.y, z.x, z.y);
  box_muller(x.z, x.w, z.z, z.w);
  return z;
}

__device__ __forceinline__ float adam_update(float& th, float& m, float& v, float g, const AdamArgs& a) {
  m = a.beta1 * m + a.one_m_beta1 * g;
  v = a.beta2 * v + a.one_m_beta2 * g * g;
  const float mh = m * a.bias1;
  const float vh = v * a.bias2;
#if DP_STREAM_FAST_MATH
  th = th - a.lr * (__fdividef(mh, fast_sqrt(vh) + a.xi) + a.wd * th);
#else
  th = th - a.lr * (mh / (sqrtf(vh) + a.xi) + a.wd * th);
#endif
  return th;
}

// ---------------------------------------------------------------------------------------------
// clip factors
// ---------------------------------------------------------------------------------------------
__global__ void k_clip_factors(const float* __restrict__ sqnorm, int B, float C, float* __restrict__ clip) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < B) {
    const float n = sqnorm[i];
    clip[i] = (n > 0.0f) ? fminf(1.0f, C / sqrtf(n)) : 1.0f;
  }
}

cudaError_t launch_clip_factors(const float* sqnorm, int B, float C, float* clip, cudaStream_t s) {
  k_clip_factors<<<ceil_div(B, 256), 256, 0, s>>>(sqnorm, B, C, clip);
  return counted(1);
}

// ---------------------------------------------------------------------------------------------
// The streaming pass.  MODE 0: noise+scale in place.  MODE 1: AdamW from g.  MODE 2: fused.
// Thread work item = Philox block j (elements 4j .. 4j+3 of the flat parameter vector); the local
// index of element e is e - elem_offset.  VEC: elem_offset % 4 == 0 and all pointers 16-byte
// aligned, so a block is one float4 of each array; otherwise elements are handled one by one.
// ---------------------------------------------------------------------------------------------
template <int MODE, bool VEC>
__global__ void __launch_bounds__(256)
k_stream(float* __restrict__ theta, float* __restrict__ m, float* __restrict__ v, float* __restrict__ acc,
         const float* __restrict__ g_in, int zero_acc, long long n, unsigned long long j0,
         unsigned long long n_blocks, NoiseArgs na, AdamArgs aa, double* __restrict__ sq_sums) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  float s_sig = 0.0f, s_noi = 0.0f;      // sum acc^2 and sum (sigma C z)^2 of this thread (gradient-SNR terms)
  for (unsigned long long b = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; b < n_blocks; b += stride) {
    const unsigned long long j = j0 + b;
    const long long k0 = (long long)(4ull * j) - na.elem_offset;   // local index of lane 0
    if (VEC && k0 >= 0 && k0 + 4 <= n) {
      float4 gv;
      if (MODE != 1) {
        const float4 a4 = *reinterpret_cast<const float4*>(acc + k0);
        const float4 z = normals4(j, na);
        if (sq_sums) {
          s_sig += a4.x * a4.x + a4.y * a4.y + a4.z * a4.z + a4.w * a4.w;
          const float nx = na.sigmaC * z.x, ny = na.sigmaC * z.y, nz = na.sigmaC * z.z, nw = na.sigmaC * z.w;
          s_noi += nx * nx + ny * ny + nz * nz + nw * nw;
        }
        gv.x = (a4.x + na.sigmaC * z.x) * na.inv_n;
        gv.y = (a4.y + na.sigmaC * z.y) * na.inv_n;
        gv.z = (a4.z + na.sigmaC * z.z) * na.inv_n;
        gv.w = (a4.w + na.sigmaC * z.w) * na.inv_n;
      } else {
        gv = *reinterpret_cast<const float4*>(g_in + k0);
      }
      if (MODE == 0) {
        *reinterpret_cast<float4*>(acc + k0) = gv;
      } else {
        float4 t4 = *reinterpret_cast<const float4*>(theta + k0);
        float4 m4 = *reinterpret_cast<const float4*>(m + k0);
        float4 v4 = *reinterpret_cast<const float4*>(v + k0);
        adam_update(t4.x, m4.x, v4.x, gv.x, aa);
        adam_update(t4.y, m4.y, v4.y, gv.y, aa);
        adam_update(t4.z, m4.z, v4.z, gv.z, aa);
        adam_update(t4.w, m4.w, v4.w, gv.w, aa);
        *reinterpret_cast<float4*>(theta + k0) = t4;
        *reinterpret_cast<float4*>(m + k0) = m4;
        *reinterpret_cast<float4*>(v + k0) = v4;
        if (MODE == 2 && zero_acc) *reinterpret_cast<float4*>(acc + k0) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    } else {
      float z[4] = {0.f, 0.f, 0.f, 0.f};
      if (MODE != 1) {
        const float4 z4 = normals4(j, na);
        z[0] = z4.x; z[1] = z4.y; z[2] = z4.z; z[3] = z4.w;
      }
#pragma unroll
      for (int l = 0; l < 4; ++l) {
        const long long k = k0 + l;
        if (k < 0 || k >= n) continue;
        float gv;
        if (MODE != 1) {
          const float a1 = acc[k], n1 = na.sigmaC * z[l];
          if (sq_sums) { s_sig += a1 * a1; s_noi += n1 * n1; }
          gv = (a1 + n1) * na.inv_n;
        } else {
          gv = g_in[k];
        }
        if (MODE == 0) {
          acc[k] = gv;
        } else {
          float t1 = theta[k], m1 = m[k], v1 = v[k];
          adam_update(t1, m1, v1, gv, aa);
          theta[k] = t1; m[k] = m1; v[k] = v1;
          if (MODE == 2 && zero_acc) acc[k] = 0.0f;
        }
      }
    }
  }
  if (MODE != 1 && sq_sums) {      // uniform branch: one double atomic per block and quantity
    __shared__ double red[2][8];
    double a = (double)s_sig, b = (double)s_noi;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      a += __shfl_down_sync(0xffffffffu, a, o);
      b += __shfl_down_sync(0xffffffffu, b, o);
    }
    if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = a; red[1][threadIdx.x >> 5] = b; }
    __syncthreads();
    if (threadIdx.x == 0) {
      double ta = 0.0, tb = 0.0;
#pragma unroll
      for (int w = 0; w < 8; ++w) { ta += red[0][w]; tb += red[1][w]; }
      atomicAdd(sq_sums, ta);
      atomicAdd(sq_sums + 1, tb);
    }
  }
}

static int stream_grid(unsigned long long n_blocks) {
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const unsigned long long want = (n_blocks + 255) / 256;
  const unsigned long long cap = (unsigned long long)sms * 16;   // 8 resident CTAs of 256 threads, two rounds
  unsigned long long g = want < cap ? want : cap;
  if (g >= (unsigned long long)sms) g = g / sms * sms;           // whole waves
  return (int)(g ? g : 1);
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <int MODE>
static cudaError_t launch_stream(float* theta, float* m, float* v, float* acc, const float* g, int zero_acc,
                                 long long n, const NoiseArgs& na, const AdamArgs& aa, cudaStream_t s,
                                 double* sq_sums = nullptr) {
  if (n <= 0) return cudaSuccess;
  const unsigned long long j0 = (unsigned long long)na.elem_offset >> 2;
  const unsigned long long j1 = ((unsigned long long)na.elem_offset + (unsigned long long)n + 3ull) >> 2;
  const unsigned long long nb = j1 - j0;
  bool vec = (na.elem_offset & 3) == 0;
  if (MODE != 1) vec = vec && aligned16(acc);
  if (MODE == 1) vec = vec && aligned16(g);
  if (MODE != 0) vec = vec && aligned16(theta) && aligned16(m) && aligned16(v);
  const int grid = stream_grid(nb);
  if (vec) k_stream<MODE, true><<<grid, 256, 0, s>>>(theta, m, v, acc, g, zero_acc, n, j0, nb, na, aa, sq_sums);
  else     k_stream<MODE, false><<<grid, 256, 0, s>>>(theta, m, v, acc, g, zero_acc, n, j0, nb, na, aa, sq_sums);
  return counted(1);
}

cudaError_t launch_noise_scale(float* acc, long long n, const NoiseArgs& na, cudaStream_t s) {
  AdamArgs aa = {};
  return launch_stream<0>(nullptr, nullptr, nullptr, acc, nullptr, 0, n, na, aa, s);
}
cudaError_t launch_adamw(float* theta, float* m, float* v, const float* g, long long n, const AdamArgs& aa,
                         cudaStream_t s) {
  NoiseArgs na = {};
  return launch_stream<1>(theta, m, v, nullptr, g, 0, n, na, aa, s);
}
cudaError_t launch_noise_adamw(float* theta, float* m, float* v, float* acc, int zero_acc, long long n,
                               const NoiseArgs& na, const AdamArgs& aa, cudaStream_t s, double* sq_sums) {
  return launch_stream<2>(theta, m, v, acc, nullptr, zero_acc, n, na, aa, s, sq_sums);
}

// ---------------------------------------------------------------------------------------------
// Macro-batch end of the data-parallel scheme in one pass over one shard of the flat vector:
//   g = (sum over ranks of acc_r + sigma C z) / N, AdamW on this rank's theta / m / v, the new theta written into
//   every rank's replica, every rank's accumulator shard zeroed.
// The ranks' buffers are reached through plain loads and stores on peer-mapped addresses (no multicast, no
// waiting on another rank inside the kernel: the caller orders the launches against the accumulate kernels of all
// ranks).  The sum runs over the ranks in index order, so it does not depend on which rank computes it.
// ---------------------------------------------------------------------------------------------
struct PeerSet {
  float* acc[kMaxRanks];       // shard start in rank r's accumulator
  float* theta[kMaxRanks];     // shard start in rank r's parameter replica (nullptr: not written)
  int n_ranks;
};

__global__ void __launch_bounds__(256)
k_reduce_update(float* __restrict__ theta, float* __restrict__ m, float* __restrict__ v, const PeerSet P, int zero_acc,
                long long n, unsigned long long j0, unsigned long long n_blocks, NoiseArgs na, AdamArgs aa) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  for (unsigned long long b = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; b < n_blocks; b += stride) {
    const unsigned long long j = j0 + b;
    const long long k0 = (long long)(4ull * j) - na.elem_offset;   // local index of lane 0 (a multiple of 4)
    const float4 z = normals4(j, na);
    if (k0 >= 0 && k0 + 4 <= n) {
      float4 a4 = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int r = 0; r < P.n_ranks; ++r) {
        const float4 x = *reinterpret_cast<const float4*>(P.acc[r] + k0);
        a4.x += x.x; a4.y += x.y; a4.z += x.z; a4.w += x.w;
      }
      float4 t4 = *reinterpret_cast<const float4*>(theta + k0);
      float4 m4 = *reinterpret_cast<const float4*>(m + k0);
      float4 v4 = *reinterpret_cast<const float4*>(v + k0);
      adam_update(t4.x, m4.x, v4.x, (a4.x + na.sigmaC * z.x) * na.inv_n, aa);
      adam_update(t4.y, m4.y, v4.y, (a4.y + na.sigmaC * z.y) * na.inv_n, aa);
      adam_update(t4.z, m4.z, v4.z, (a4.z + na.sigmaC * z.z) * na.inv_n, aa);
      adam_update(t4.w, m4.w, v4.w, (a4.w + na.sigmaC * z.w) * na.inv_n, aa);
      *reinterpret_cast<float4*>(theta + k0) = t4;
      *reinterpret_cast<float4*>(m + k0) = m4;
      *reinterpret_cast<float4*>(v + k0) = v4;
      for (int r = 0; r < P.n_ranks; ++r) {
        if (P.theta[r] && P.theta[r] != theta) *reinterpret_cast<float4*>(P.theta[r] + k0) = t4;
        if (zero_acc) *reinterpret_cast<float4*>(P.acc[r] + k0) = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    } else {
      const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
      for (int l = 0; l < 4; ++l) {
        const long long k = k0 + l;
        if (k < 0 || k >= n) continue;
        float a1 = 0.0f;
        for (int r = 0; r < P.n_ranks; ++r) a1 += P.acc[r][k];
        float t1 = theta[k], m1 = m[k], v1 = v[k];
        adam_update(t1, m1, v1, (a1 + na.sigmaC * zz[l]) * na.inv_n, aa);
        theta[k] = t1; m[k] = m1; v[k] = v1;
        for (int r = 0; r < P.n_ranks; ++r) {
          if (P.theta[r] && P.theta[r] != theta) P.theta[r][k] = t1;
          if (zero_acc) P.acc[r][k] = 0.0f;
        }
      }
    }
  }
}

cudaError_t launch_reduce_update(float* theta, float* m, float* v, float* const* acc_of_rank,
                                 float* const* theta_of_rank, int n_ranks, int zero_acc, long long n,
                                 const NoiseArgs& na, const AdamArgs& aa, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  PeerSet P;
  P.n_ranks = n_ranks;
  for (int r = 0; r < kMaxRanks; ++r) {
    P.acc[r] = r < n_ranks ? acc_of_rank[r] : nullptr;
    P.theta[r] = (r < n_ranks && theta_of_rank) ? theta_of_rank[r] : nullptr;
  }
  const unsigned long long j0 = (unsigned long long)na.elem_offset >> 2;
  const unsigned long long j1 = ((unsigned long long)na.elem_offset + (unsigned long long)n + 3ull) >> 2;
  k_reduce_update<<<stream_grid(j1 - j0), 256, 0, s>>>(theta, m, v, P, zero_acc, n, j0, j1 - j0, na, aa);
  return counted(1);
}

// out[0] = fraction of examples with clip < 1, out[1] = mean clip factor.  One block, fixed order.
__global__ void __launch_bounds__(256) k_clip_stats(const float* __restrict__ clip, int B, float* __restrict__ out) {
  __shared__ float red[2][8];
  float cnt = 0.0f, sum = 0.0f;
  for (int i = threadIdx.x; i < B; i += 256) {
    const float c = clip[i];
    cnt += (c < 1.0f) ? 1.0f : 0.0f;
    sum += c;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    cnt += __shfl_down_sync(0xffffffffu, cnt, o);
    sum += __shfl_down_sync(0xffffffffu, sum, o);
  }
  if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = cnt; red[1][threadIdx.x >> 5] = sum; }
  __syncthreads();
  if (threadIdx.x == 0) {
    float a = 0.0f, b = 0.0f;
    for (int w = 0; w < 8; ++w) { a += red[0][w]; b += red[1][w]; }
    out[0] = a / (float)B;
    out[1] = b / (float)B;
  }
}
cudaError_t launch_clip_stats(const float* clip, int B, float* out, cudaStream_t s) {
  k_clip_stats<<<1, 256, 0, s>>>(clip, B, out);
  return counted(1);
}

// ---------------------------------------------------------------------------------------------
// Test utilities
// ---------------------------------------------------------------------------------------------
__global__ void k_philox_u32(uint32_t* __restrict__ out, long long n, NoiseArgs na) {
  const long long stride = (long long)gridDim.x * blockDim.x;
  for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < n; k += stride) {
    const unsigned long long e = (unsigned long long)(na.elem_offset + k);
    const uint4 x = philox_block(e >> 2, na);
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
    out[k] = w[e & 3];
  }
}
cudaError_t launch_philox_u32(uint32_t* out, long long n, const NoiseArgs& na, cudaStream_t s) {
  if (n <= 0) return cudaSuccess;
  long long blocks = (n + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  k_philox_u32<<<(int)blocks, 256, 0, s>>>(out, n, na);
  return counted(1);
}

__global__ void k_equality_mask(const int32_t* __restrict__ ids, int T, uint8_t* __restrict__ mask) {
  const int i = blockIdx.x;
  const int32_t* row = ids + (size_t)i * T;
  uint8_t* out = mask + (size_t)i * T * T;
  for (int p = threadIdx.x; p < T * T; p += blockDim.x) out[p] = (row[p / T] == row[p % T]) ? 1 : 0;
}
cudaError_t launch_equality_mask(const int32_t* ids, int B, int T, uint8_t* mask, cudaStream_t s) {
  k_equality_mask<<<B, 256, 0, s>>>(ids, T, mask);
  return counted(1);
}

}  // namespace dpk
