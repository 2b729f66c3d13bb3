/*
 * dp.h -- C ABI of the B200 (sm_100a) DP-SGD privatised-gradient step.
 *
 * The library implements the update of Algorithm 1 of "Large-Scale Differentially
 * Private BERT" (arXiv 2108.01624): per-example clipping of the whole-model gradient,
 * summation over the (micro)batches of a mega-batch (Section 5.3), one Gaussian draw
 * N(0, sigma^2 C^2 I) per macro-batch, division by the batch size, and the Adam update
 * with decoupled weight decay.  Per-example gradients are never written to memory:
 * a layer is described by its per-token inputs A and output-gradients G (Section 4.3:
 * the gradient of a fully connected layer is grad_s * x^T, summed over tokens).
 *
 * Conventions for every entry point
 *   - All data pointers are DEVICE pointers owned by the caller, unless marked HOST.
 *     The `layers` descriptor array itself is a HOST array and is read during the call.
 *   - Calls only enqueue work on `cuda_stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream).  They do not synchronise the host, except dp_poll_status.
 *   - The library allocates no device memory.  Kernels that need scratch take it from the
 *     caller's `workspace` (size from dp_workspace_bytes, 256-byte aligned).  The contents
 *     of the workspace carry no meaning between calls.
 *   - Return value: DP_OK (0) or a negative dp_status.  Arguments are validated on the
 *     host before anything is launched; nothing throws, aborts or traps.
 *   - Matrices are row-major with the feature index fastest.  bf16 tensors must be
 *     16-byte aligned; accumulators and optimizer state are fp32.
 *   - G must be the gradient of the PER-EXAMPLE loss (no 1/B folded in), because the clip
 *     of Algorithm 1 acts on grad L(theta; x_j) of a single example.
 */
#ifndef DP_B200_H_
#define DP_B200_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define DP_API __attribute__((visibility("default")))
#else
#define DP_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DP_OK = 0,
  DP_ERR_ARG = -1,         /* null pointer, non-positive size, non-finite scalar, bad enum */
  DP_ERR_ALIGN = -2,       /* pointer not aligned as required */
  DP_ERR_UNSUPPORTED = -3, /* valid request the library cannot run (e.g. forced path on a shape it excludes) */
  DP_ERR_CUDA = -4,        /* a CUDA runtime/driver call failed */
  DP_ERR_TIMEOUT = -5,     /* a bounded device-side wait ran out (reported by dp_poll_status) */
  DP_ERR_WORKSPACE = -6,   /* workspace missing, misaligned or too small */
  DP_ERR_BAD_ID = -7       /* a token id outside [0, V) was met and skipped (dp_poll_status) */
} dp_status;

typedef enum { DP_LINEAR = 0, DP_LAYERNORM = 1, DP_EMBEDDING = 2 } dp_kind;
typedef enum { DP_F32 = 0, DP_BF16 = 1 } dp_dtype;
/* How a layer's per-example squared norm is obtained.
 *   GRAM          <A_i A_i^T (+ 1 1^T with a bias), G_i G_i^T>  over T x T token Grams;
 *                 for an embedding the first factor is the token-id equality mask.
 *   MATERIALIZED  tiles of A_i^T G_i formed on chip, squared and summed; for an embedding,
 *                 rows with equal ids are summed first.
 *   AUTO          linear: the cheaper way.  On the CUDA-core kernels GRAM iff T * (d_in + d_out) <= d_in * d_out,
 *                 the flop count of either way.  On the tensor-core kernels (see below) by measured cost: GRAM for
 *                 T <= 128; beyond, GRAM iff the multiply-accumulates it executes, 128 * 128 * (d_in + d_out) per
 *                 block pair of the upper triangle of the ceil(T/128)^2 token blocks, are at most 1.75 times
 *                 T * d_in * d_out;
 *                 embedding: GRAM whenever the tensor-core kernel accepts the layer (bf16, d_out % 8 == 0). */
typedef enum { DP_PATH_AUTO = 0, DP_PATH_GRAM = 1, DP_PATH_MATERIALIZED = 2 } dp_path;
/* Which kernels a layer gets.  A bf16 LINEAR layer whose d_in and d_out are multiples of 8 (a token row is then a
 * multiple of 16 bytes) and whose A and G are 16-byte aligned runs on the tensor cores (norms and clipped sum); widths
 * that are also multiples of 64 take one tensor copy per operand tile, the others one copy per 64-feature group
 * (the group that overhangs the width is filled with zeros).  Every other linear layer (fp32, other widths) runs on
 * plain CUDA-core kernels, which give the same results and are far slower.  LAYERNORM and the EMBEDDING accumulate are
 * bandwidth-bound kernels for any width; they use 16-byte loads when d is a multiple of 8 (bf16) or 4 (fp32) and
 * the tensors are aligned. */

/* One trainable layer of one microbatch.  B and T must be equal across the layers of a call. */
typedef struct dp_layer {
  int32_t kind;      /* dp_kind */
  int32_t dtype;     /* dp_dtype of A and G */
  int32_t path;      /* dp_path (norms only; ignored for LAYERNORM) */
  int32_t has_bias;  /* LINEAR: a bias [d_out] is trained and acc_b is given */
  int32_t B, T;      /* examples in the microbatch, tokens per example */
  int32_t d_in;      /* LINEAR: input width.  LAYERNORM: d (= d_out).  EMBEDDING: vocabulary size V */
  int32_t d_out;     /* width of G */
  const void* A;     /* LINEAR: [B,T,d_in] layer input.  LAYERNORM: [B,T,d] normalised input.  EMBEDDING: NULL */
  const int32_t* ids;/* EMBEDDING: [B,T] token ids, 0 <= id < V.  Otherwise NULL */
  const void* G;     /* [B,T,d_out] output-gradient of the per-example loss */
  float* acc_w;      /* LINEAR: [d_in,d_out] = sum_i c_i A_i^T G_i.  LAYERNORM: gain [d].  EMBEDDING: [V,d_out].
                        Accumulated in place (+=).  May be NULL for dp_per_example_sqnorms. */
  float* acc_b;      /* LINEAR with bias: [d_out].  LAYERNORM: bias [d].  Otherwise NULL */
} dp_layer;

/* Bytes of scratch that dp_per_example_sqnorms / dp_clipped_accumulate need over these layers (per-example
 * column sums of the LayerNorm / bias terms and the partial sums of the tensor-core norm kernels); 0 on invalid
 * layers.  The two calls plan the same layout, so one buffer serves both. */
DP_API size_t dp_workspace_bytes(const dp_layer* layers /*HOST*/, int n_layers);

/* Squared L2 norm of every example's whole gradient over the given layers (Algorithm 1 clips
 * grad L(theta; x_j) as one vector; Section 4.3 gives the per-layer form).
 *   sqnorm[B] fp32.  accumulate_into = 0: overwritten; 1: added to (so a model can be passed
 *   in several calls).  The per-layer path follows dp_layer.path. */
DP_API int dp_per_example_sqnorms(const dp_layer* layers /*HOST*/, int n_layers, float* sqnorm, int accumulate_into,
                           void* workspace, size_t workspace_bytes, void* cuda_stream);

/* c_i = min(1, C / sqrt(sqnorm_i)), c_i = 1 when sqnorm_i = 0: the factor of clip(., C) in
 * Algorithm 1.  C > 0. */
DP_API int dp_clip_factors(const float* sqnorm, int B, double C, float* clip, void* cuda_stream);

/* acc += sum_i clip_i * g_i for every layer: the sum of clipped gradients of Algorithm 1,
 * accumulated over microbatches as in Section 5.3.  clip[B] fp32 from dp_clip_factors. */
DP_API int dp_clipped_accumulate(const dp_layer* layers /*HOST*/, int n_layers, const float* clip,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* The same sum, for the usual sequence norms -> clip factors -> accumulate of one microbatch: the per-example
 * column sums of the LayerNorm terms (sum_t G and sum_t G*xhat, Section 4.3) are taken from `workspace`, where
 * the latest dp_per_example_sqnorms call left them, instead of being formed again from G and xhat.  The caller
 * guarantees that that call ran on the same stream over the same layer list (same order, shapes and tensors,
 * unchanged since) with the same workspace, and that nothing wrote the workspace in between; the library
 * cannot check this.  Results are bit-identical to dp_clipped_accumulate. */
DP_API int dp_clipped_accumulate_after_sqnorms(const dp_layer* layers /*HOST*/, int n_layers, const float* clip,
                                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/* Host-only, launches nothing: the work schedule that dp_clipped_accumulate uses for those linear layers of the list
 * that go to the tensor-core GEMM, on a device with `units` CTA pairs (SM count / 2).  A layer of d_in x d_out has
 * ceil(d_out/256) * ceil(d_in/512) tiles, each split into splits[k] example ranges; pair p runs item p of every
 * wave of `units` items.  item_start[l] = first item of layer l within its launch (-1: the layer takes another
 * path), launch[l] = index of that launch, splits[k] and slots[k] (= waves * units) per launch k < max_launches.
 * Returns the number of launches (>= 0) or a negative status. */
DP_API int dp_accumulate_schedule(const dp_layer* layers /*HOST*/, int n_layers, int units, int64_t* item_start /*HOST*/,
                           int32_t* launch /*HOST*/, int32_t* splits /*HOST*/, int64_t* slots /*HOST*/, int max_launches);

/* acc <- (acc + sigma * C * z) / batch_size in place, z ~ N(0, I): the g_t line of Algorithm 1.
 * z_e depends only on (seed, step, e) with e = elem_offset + index: Philox4x32-10 block e >> 2 with
 * counter (lo(e>>2), hi(e>>2), lo(step), hi(step)) and key (lo(seed), hi(seed)); Box-Muller on the word
 * pairs (x0,x1), (x2,x3).  n >= 0 elements; sigma >= 0, C > 0, batch_size > 0. */
DP_API int dp_add_noise_and_scale(float* acc, int64_t n, int64_t elem_offset, double sigma, double C,
                           int64_t batch_size, uint64_t seed, uint64_t step, void* cuda_stream);

/* Adam with bias correction and decoupled weight decay (Algorithm 1):
 *   m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;
 *   theta <- theta - lr * ( (m/(1-b1^t)) / (sqrt(v/(1-b2^t)) + xi) + weight_decay * theta ),  t >= 1.
 * Scalars are doubles so that 1-beta and the bias corrections 1/(1-beta^t) are formed on the host in double
 * precision before being rounded once to fp32 for the kernel. */
DP_API int dp_adamw_step(float* theta, float* m, float* v, const float* g, int64_t n, double lr, double beta1,
                  double beta2, double xi, double weight_decay, int64_t t, void* cuda_stream);

/* The two calls above in one pass over memory (same arithmetic, same Philox indexing): reads acc, theta,
 * m, v and writes theta, m, v; with zero_acc != 0 it also clears acc for the next macro-batch. */
DP_API int dp_noise_scale_adamw_step(float* theta, float* m, float* v, float* acc, int zero_acc, int64_t n,
                              int64_t elem_offset, double sigma, double C, int64_t batch_size, uint64_t seed,
                              uint64_t step, double lr, double beta1, double beta2, double xi, double weight_decay,
                              int64_t t, void* cuda_stream);

/* dp_noise_scale_adamw_step that also accumulates the two squared norms of the gradient-SNR diagnostic of
 * Section 5.2.1 (norm of the aggregated clipped gradient over norm of the noise vector) in the same pass:
 *   sq_sums[0] += sum_e acc_e^2,   sq_sums[1] += sum_e (sigma C z_e)^2      (device double[2], 8-byte aligned).
 * The caller zeroes sq_sums before the first tensor of a macro-batch; SNR = sqrt(sq_sums[0] / sq_sums[1]).
 * Block sums are combined with fp64 atomics, so the last bits depend on the launch. */
DP_API int dp_noise_scale_adamw_step_snr(float* theta, float* m, float* v, float* acc, int zero_acc, int64_t n,
                                         int64_t elem_offset, double sigma, double C, int64_t batch_size,
                                         uint64_t seed, uint64_t step, double lr, double beta1, double beta2,
                                         double xi, double weight_decay, int64_t t, double* sq_sums,
                                         void* cuda_stream);

/* Data-parallel end of a macro-batch in one pass (the gradient reduction that Section 5.3's large batches
 * amortise, fused with the g_t ... theta_t lines of Algorithm 1).  Every rank holds a full fp32 accumulator and a
 * full replica of theta; rank k owns the shard [elem_offset, elem_offset + n) of the flat vector and calls this
 * with pointers to the START OF THAT SHARD:
 *   theta, m, v        this rank's own shard (read and written);
 *   acc_of_rank[r]     the shard inside rank r's accumulator, r < n_ranks <= 16 (HOST array of device pointers
 *                      that this GPU can load from and store to: its own memory or peer-mapped memory);
 *   theta_of_rank[r]   the shard inside rank r's replica, or NULL entries / a NULL array to skip the write.
 * Computes g = (sum_r acc_r + sigma C z) / batch_size with the sum taken in rank order and z keyed by the global
 * element index (so the result is that of the single-GPU fused call on the summed accumulator), applies AdamW,
 * stores the new theta into every replica given and, if zero_acc, zeroes the shard of every accumulator.
 * The kernel waits for nobody: the caller orders it after all ranks' accumulate calls and orders any reader of
 * theta or writer of the accumulators on any rank after it (a barrier between the ranks on both sides).
 * elem_offset must be a multiple of 4 and every pointer 16-byte aligned (DP_ERR_ALIGN otherwise). */
DP_API int dp_reduce_noise_adamw_step(float* theta, float* m, float* v, float* const* acc_of_rank /*HOST*/,
                                      float* const* theta_of_rank /*HOST or NULL*/, int n_ranks, int zero_acc,
                                      int64_t n, int64_t elem_offset, double sigma, double C, int64_t batch_size,
                                      uint64_t seed, uint64_t step, double lr, double beta1, double beta2, double xi,
                                      double weight_decay, int64_t t, void* cuda_stream);

/* Clipping statistics of a microbatch (the other diagnostic that accompanies the gradient-SNR curves of
 * Section 5.2.1): out[0] = fraction of examples with clip_i < 1, out[1] = mean clip_i.  out: device float[2]. */
DP_API int dp_clip_stats(const float* clip, int B, float* out, void* cuda_stream);

/* A table trained through two layers: the token embedding and an output projection onto the same table.
 * (Section 4.3 names the word-piece embedding; the model of Section 4 is BERT-Large, whose masked-LM head
 * projects onto that table, logits[s, v] = <h[s, :], E[v, :]>; the paper does not restate this.)  Example i's gradient
 * for the table is then ONE tensor, scatter_i + dlogits_i^T h_i, and Algorithm 1's clip acts on the norm of that sum:
 * the two parts' squared norms, plus twice their inner product.  Pass the embedding as a DP_EMBEDDING layer and the
 * projection as a DP_LINEAR layer without bias whose A is dlogits [B, T_out, V] (d_in = V) and whose G is the
 * projection's input h [B, T_out, d] (d_out = d), both with acc_w = the table's [V, d] accumulator (each in a call
 * with its own token count, the second with accumulate_into = 1): dp_per_example_sqnorms then adds the two parts
 * and dp_clipped_accumulate sums both into the table.  This call adds the inner product,
 *   sqnorm[i] += 2 * sum_{t < T} sum_{s < T_out} dlogits[i, s, ids[i, t]] * <h[i, s, :], G_emb[i, t, :]>,
 * and must run before dp_clip_factors.  ids int32 [B, T]; G_emb [B, T, d]; dlogits [B, T_out, V]; h [B, T_out, d];
 * all three of `dtype` (DP_F32 or DP_BF16), row-major, device pointers owned by the caller; sqnorm fp32 [B].
 * fp32 accumulation in a fixed order.  A token id outside [0, V) is skipped and reported by dp_poll_status
 * (DP_ERR_BAD_ID).  DP_ERR_ARG on null pointers or non-positive sizes, DP_ERR_ALIGN on pointers not aligned to
 * their element size. */
DP_API int dp_shared_table_cross_sqnorms(const int32_t* ids, const void* G_emb, int B, int T, const void* dlogits,
                                         const void* h, int T_out, int d, int V, int dtype, float* sqnorm,
                                         void* cuda_stream);

/* Test utility: out[k] = the raw Philox word of element elem_offset + k (lane (e & 3) of block e >> 2). */
DP_API int dp_philox_u32(uint32_t* out, int64_t n_words, int64_t elem_offset, uint64_t seed, uint64_t step,
                  void* cuda_stream);

/* Test utility: mask[i,t,s] = (ids[i,t] == ids[i,s]) as bytes, the first factor of the embedding Gram. */
DP_API int dp_token_equality_mask(const int32_t* ids, int B, int T, uint8_t* mask, void* cuda_stream);

/* Floats of fixed device scratch behind dp_layernorm_sqnorms_static (4 MiB, held by every GPU that loads the
 * library until the process exits). */
#define DP_STATIC_SCRATCH_FLOATS (1u << 20)

/* (No counterpart in the paper: a variant for callers that cannot supply scratch memory.)
 * Squared L2 norms of ONE LayerNorm layer's per-example gain and bias gradients, like dp_per_example_sqnorms
 * restricted to that layer, but with the per-example column sums kept in a fixed array inside the library
 * instead of a caller-provided workspace.  It exists for callers that cannot call cudaMalloc -- code running
 * under a memory manager that owns the whole device, or where cudaMalloc's device-wide synchronisation is not
 * acceptable -- and it calls no cudaMalloc, cudaFree or allocating library routine itself.
 *   layer   HOST pointer to one dp_layer of kind DP_LAYERNORM (A = normalised input, G, B, T, d as usual;
 *           accumulators ignored).  Inputs and the output stay caller-owned device memory.
 *   sqnorm  [B] fp32, overwritten (accumulate_into = 0) or added to (1).
 * Limit: B * 2 * d <= DP_STATIC_SCRATCH_FLOATS, otherwise DP_ERR_WORKSPACE (nothing is launched).
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with that device
 * current); make that first call before any stream capture begins.
 * All calls on a device share the one array, which keeps the previous call's contents; every call overwrites
 * the part it reads, so nothing needs clearing, but two calls that overlap on the GPU (different streams) race
 * on it: serialise them. */
DP_API int dp_layernorm_sqnorms_static(const dp_layer* layer /*HOST*/, float* sqnorm, int accumulate_into,
                                       void* cuda_stream);

/* Waits for the stream, then returns and clears the sticky device-side status (DP_OK, DP_ERR_TIMEOUT
 * or DP_ERR_BAD_ID).  Device code never traps: a wait that runs out or an id out of range is recorded
 * here and the offending work is skipped. */
DP_API int dp_poll_status(void* cuda_stream);

/* Diagnostic: after dp_poll_status returned DP_ERR_TIMEOUT, info[0..4] = {wait site tag, block index, stage or
 * tile counter, barrier parity, thread index} of the first bounded device-side wait that gave up (HOST array).
 * Synchronises the device. */
DP_API int dp_last_timeout_info(int info[5]);

/* Every device-side wait of the tensor-core kernels (on a TMA copy, a tensor-core commit, another warp) gives up after
 * a limit, 4e9 SM clock cycles (2 to 3 s) by default; the kernel then records DP_ERR_TIMEOUT, skips the rest of its
 * work and returns.  This sets the limit for the CURRENT device (cycles <= 0 restores the default); it synchronises
 * with the device and must not be called while kernels of the library are running.  Meant for tests and for callers
 * that prefer an earlier error over a longer stall. */
DP_API int dp_set_wait_limit_cycles(long long cycles);

/* Self-test of that mechanism: enqueues one small kernel whose waiters poll a barrier that nobody arrives on.  They
 * give up at the limit, the kernel returns, and dp_poll_status then reports DP_ERR_TIMEOUT with
 * dp_last_timeout_info()[0] = 98 or 99 (the two wait sites of the self-test).  Nothing else is affected. */
DP_API int dp_selftest_wait_timeout(void* cuda_stream);

/* Number of kernels this library has launched in the calling process so far (host-side counter). */
DP_API long long dp_launch_count(void);

DP_API const char* dp_status_string(int status);
DP_API int dp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* DP_B200_H_ */
