// Internal declarations shared by the translation units of libdp_b200.so.
// Host-side launchers only; the C ABI in include/dp.h is implemented in dp_api.cu.
#pragma once

#include <vector>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/dp.h"

namespace dpk {

// ---- small helpers -------------------------------------------------------------------------
static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Launch accounting: every kernel launch of the library is counted (read back by dp_launch_count).
void note_launch(int n);
static inline cudaError_t counted(int n) { note_launch(n); return cudaGetLastError(); }

// Sticky device status word values (written with atomicCAS(0 -> code), first error wins).
enum : int { STATUS_OK = 0, STATUS_TIMEOUT = 1, STATUS_BAD_ID = 2 };

// ---- streaming kernels (dp_stream.cu) --------------------------------------------------------
struct NoiseArgs {
  float sigmaC;       // sigma * C
  float inv_n;        // 1 / batch_size
  uint32_t key0, key1;   // lo32(seed), hi32(seed)
  uint32_t step0, step1; // lo32(step), hi32(step)
  long long elem_offset;
};
struct AdamArgs {
  float lr, beta1, beta2, one_m_beta1, one_m_beta2, bias1, bias2, xi, wd;  // bias = 1/(1-beta^t)
};
cudaError_t launch_clip_factors(const float* sqnorm, int B, float C, float* clip, cudaStream_t s);
cudaError_t launch_noise_scale(float* acc, long long n, const NoiseArgs& na, cudaStream_t s);
cudaError_t launch_adamw(float* theta, float* m, float* v, const float* g, long long n, const AdamArgs& aa,
                         cudaStream_t s);
// sq_sums (optional, device double[2]): adds sum(acc^2) and sum((sigma C z)^2), the gradient-SNR terms.
cudaError_t launch_noise_adamw(float* theta, float* m, float* v, float* acc, int zero_acc, long long n,
                               const NoiseArgs& na, const AdamArgs& aa, cudaStream_t s, double* sq_sums = nullptr);
// Fused cross-rank sum + noise + AdamW + replica update on one shard (elem_offset % 4 == 0, 16-byte aligned pointers).
constexpr int kMaxRanks = 16;
cudaError_t launch_reduce_update(float* theta, float* m, float* v, float* const* acc_of_rank,
                                 float* const* theta_of_rank, int n_ranks, int zero_acc, long long n,
                                 const NoiseArgs& na, const AdamArgs& aa, cudaStream_t s);
cudaError_t launch_clip_stats(const float* clip, int B, float* out, cudaStream_t s);
cudaError_t launch_philox_u32(uint32_t* out, long long n, const NoiseArgs& na, cudaStream_t s);
cudaError_t launch_equality_mask(const int32_t* ids, int B, int T, uint8_t* mask, cudaStream_t s);

// ---- CUDA-core kernels for any shape and dtype (dp_generic.cu) ---------------------------------
// Per-example squared norms; each adds into sqnorm[i] (one writer per example, launches are ordered).
cudaError_t launch_linear_sqnorm_generic(const dp_layer& L, bool gram, float* sqnorm, cudaStream_t s);
cudaError_t launch_linear_accum_generic(const dp_layer& L, const float* clip, cudaStream_t s);
// Column-sum tasks, batched over layers.  A task yields out[B][width]: for a LayerNorm (with_x) the gain part
// sum_t x*G then the bias part sum_t G (width 2d); for a linear bias (no x) sum_t G (width d_out).
struct ColTaskHost { const dp_layer* L; bool with_x; float* out; };
cudaError_t launch_colsums_batched(const ColTaskHost* tasks, int n, cudaStream_t s);
// sqnorm[i] += sum over tasks, columns of out[i][j]^2.
cudaError_t launch_rows_sqsum_batched(const ColTaskHost* tasks, int n, float* sqnorm, cudaStream_t s);
// LayerNorm: acc_w += sum_i clip_i * gain part, acc_b += ... bias part.  Linear bias: acc_b += sum_i clip_i * out[i].
cudaError_t launch_weighted_rows_sum_batched(const ColTaskHost* tasks, int n, const float* clip, cudaStream_t s);
// Embedding by grouping equal ids inside an example.
cudaError_t launch_embedding_sqnorm(const dp_layer& L, float* sqnorm, int* status, cudaStream_t s);
cudaError_t launch_embedding_accum(const dp_layer& L, const float* clip, int* status, cudaStream_t s);
// sqnorm[i] += 2 <scatter_i, dlogits_i^T h_i> for a table shared by an embedding and an output projection.
cudaError_t launch_shared_table_cross(const int32_t* ids, const void* G_emb, int B, int T, const void* dlogits,
                                      const void* h, int T_out, int d, int V, int dtype, float* sqnorm, int* status,
                                      cudaStream_t s);
cudaError_t launch_fill_zero(float* p, long long n, cudaStream_t s);
// sqnorm[i] (+)= sum of partial[i * stride + j], j < count, in a fixed order.
cudaError_t launch_reduce_partials(const float* partial, int B, int count, float* sqnorm, cudaStream_t s);

// ---- tcgen05 / TMA kernels for bf16 layers (dp_umma.cu) ----------------------------------------
// A layer qualifies when dtype is bf16, d_in and d_out are multiples of 8 and pointers are 16-byte aligned.
bool umma_supported(const dp_layer& L);
// Number of fp32 partial sums the squared-norm kernels write for these layers (per example).
// The partial buffer is [B][count] and is summed by launch_reduce_partials.
size_t umma_sqnorm_partials_per_example(const dp_layer* layers, const int* idx, int n, const int* use_gram);
int launch_umma_sqnorms(const dp_layer* layers, const int* idx, int n, const int* use_gram, float* partial,
                        int partial_stride, int partial_base, int* status, cudaStream_t s);
// Host-side schedule of one accumulate launch (at most kUmmaMaxLayers layers): splits of the example range, first
// work item per layer; returns the number of item slots (waves x units).
constexpr int kUmmaMaxLayers = 96;
long long umma_accumulate_schedule(const dp_layer* layers, const int* idx, int n, int units, int* splits_out,
                                   std::vector<long long>& start);
// acc_w (and acc_b: the bias column sums are formed in the same kernel) += sum_i clip[i] * A_i^T G_i; the clip
// factor is applied to the G tile inside the kernel.
// wave_sync: one zero-initialisable device word of scratch (the kernel's CTAs align their waves through it).
int launch_umma_accumulate(const dp_layer* layers, const int* idx, int n, const float* clip, int* status,
                           unsigned int* wave_sync, cudaStream_t s);

// Limit of every bounded device-side wait on the current device, in SM cycles (<= 0 restores the default).
int set_wait_limit_cycles(long long cycles);
// One CTA that waits, bounded, on a barrier nobody arrives on: records a timeout (site tag 98 or 99) and returns.
int launch_selftest_wait(int* status, cudaStream_t s);

}  // namespace dpk
