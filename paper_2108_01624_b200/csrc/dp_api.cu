// C ABI (include/dp.h): argument validation, workspace layout and dispatch to the kernels.
#include <atomic>
#include <cmath>
#include <vector>

#include "dp_internal.h"

namespace dpk {

// [0] sticky status code; [1..5] where the first bounded wait gave up (tag, block, aux, parity, thread).
__device__ int g_status_word[8] = {0, 0, 0, 0, 0, 0, 0, 0};

static std::atomic<long long> g_launches{0};
void note_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Device address of the status word for the current device (looked up once per device).
static int* status_ptr() {
  static int* cache[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!cache[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_status_word) != cudaSuccess) return nullptr;
    cache[dev] = static_cast<int*>(p);
  }
  return cache[dev];
}

static size_t elem_size(int dtype) { return dtype == DP_F32 ? 4 : 2; }
static bool misaligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) != 0; }

// Shape/pointer checks shared by the two layer-list entry points.
static int validate_layers(const dp_layer* layers, int n_layers, bool need_acc) {
  if (!layers || n_layers <= 0) return DP_ERR_ARG;
  const int B = layers[0].B, T = layers[0].T;
  if (B <= 0 || T <= 0) return DP_ERR_ARG;
  for (int l = 0; l < n_layers; ++l) {
    const dp_layer& L = layers[l];
    if (L.B != B || L.T != T) return DP_ERR_ARG;
    if (L.kind != DP_LINEAR && L.kind != DP_LAYERNORM && L.kind != DP_EMBEDDING) return DP_ERR_ARG;
    if (L.dtype != DP_F32 && L.dtype != DP_BF16) return DP_ERR_ARG;
    if (L.path != DP_PATH_AUTO && L.path != DP_PATH_GRAM && L.path != DP_PATH_MATERIALIZED) return DP_ERR_ARG;
    if (L.d_in <= 0 || L.d_out <= 0 || !L.G) return DP_ERR_ARG;
    if ((long long)B * T * (long long)(L.d_out > L.d_in && L.kind != DP_EMBEDDING ? L.d_out : L.d_in) <= 0) return DP_ERR_ARG;
    if (misaligned(L.G, elem_size(L.dtype))) return DP_ERR_ALIGN;
    if (L.kind == DP_EMBEDDING) {
      if (!L.ids) return DP_ERR_ARG;
      if (misaligned(L.ids, 4)) return DP_ERR_ALIGN;
    } else {
      if (!L.A) return DP_ERR_ARG;
      if (misaligned(L.A, elem_size(L.dtype))) return DP_ERR_ALIGN;
      if (L.kind == DP_LAYERNORM && L.d_in != L.d_out) return DP_ERR_ARG;
    }
    if (need_acc) {
      if (!L.acc_w || misaligned(L.acc_w, 4)) return L.acc_w ? DP_ERR_ALIGN : DP_ERR_ARG;
      const bool wants_b = (L.kind == DP_LINEAR && L.has_bias) || L.kind == DP_LAYERNORM;
      if (wants_b && !L.acc_b) return DP_ERR_ARG;
      if (L.acc_b && misaligned(L.acc_b, 4)) return DP_ERR_ALIGN;
    }
  }
  return DP_OK;
}

// AUTO: the path with the lower cost.  On the CUDA-core kernels the cost is the flop count of either way.  On the
// tensor-core kernels it is measured: up to 128 tokens the Gram kernel is bound by reading A and G once and beat
// the tile kernel at every width tried (64 to 1024); beyond, it executes 128 x 128 x (d_in + d_out)
// multiply-accumulates per block pair of the upper triangle and came out ahead whenever that count stayed under
// about 1.75 times the tile kernel's T x d_in x d_out (whose tiles re-read A and G through L2 for every tile row
// and column): T from 256 to 4096, widths from 256 to 4096, one mispick of 13 % among fifteen shapes.
static bool use_gram(const dp_layer& L) {
  if (L.path == DP_PATH_GRAM) return true;
  if (L.path == DP_PATH_MATERIALIZED) return false;
  if (L.kind == DP_LINEAR && umma_supported(L)) {
    if (L.T <= 128) return true;
    const long long nblk = (L.T + 127) / 128;
    const double gram = 128.0 * 128.0 * (double)(nblk * (nblk + 1) / 2) * (double)(L.d_in + L.d_out);
    const double tiles = (double)L.T * (double)L.d_in * (double)L.d_out;
    return gram <= 1.75 * tiles;
  }
  return (long long)L.T * (L.d_in + L.d_out) <= (long long)L.d_in * L.d_out;
}

// Workspace layout: [per-example column sums of every LayerNorm / bias task | partial sums of the tensor-core
// norm kernels | wave-alignment counter of the accumulate GEMM].  The two layer-list calls plan the same layout, so one workspace serves both.
struct WsPlan {
  size_t colsum_bytes = 0;
  size_t partial_bytes = 0;    // B * partials_per_example floats
  int partials_per_example = 0;
  std::vector<int> umma_idx;   // layers handled by the tensor-core kernels
  std::vector<int> umma_gram;  // 1: Gram path, 0: materialised tiles
  std::vector<size_t> col_off; // per layer: byte offset of its column-sum block (or SIZE_MAX if it has none)
  std::vector<int> lin_idx;    // tensor-core layers that are linear (the accumulate GEMM takes only these)
  size_t sync_bytes = 0;       // accumulate GEMM: wave-alignment counter
  size_t sync_off() const { return align_up(colsum_bytes, 256) + align_up(partial_bytes, 256); }
  size_t total() const { return sync_off() + sync_bytes; }
};

static WsPlan plan_workspace(const dp_layer* layers, int n_layers) {
  WsPlan p;
  const size_t B = layers[0].B;
  p.col_off.assign(n_layers, (size_t)-1);
  for (int l = 0; l < n_layers; ++l) {
    const dp_layer& L = layers[l];
    size_t need = 0;
    if (L.kind == DP_LAYERNORM) need = B * 2 * (size_t)L.d_out * sizeof(float);
    if (L.kind == DP_LINEAR && L.has_bias) need = B * (size_t)L.d_out * sizeof(float);
    if (need) {
      p.col_off[l] = p.colsum_bytes;
      p.colsum_bytes += align_up(need, 256);
    }
    if (L.kind == DP_LINEAR && umma_supported(L)) {
      p.umma_idx.push_back(l);
      p.umma_gram.push_back(use_gram(L) ? 1 : 0);
    } else if (L.kind == DP_EMBEDDING && L.path != DP_PATH_MATERIALIZED && umma_supported(L)) {
      p.umma_idx.push_back(l);     // norms only: token-id equality mask times G G^T in the Gram kernel
      p.umma_gram.push_back(1);
    }
  }
  if (!p.umma_idx.empty()) {
    p.partials_per_example = (int)umma_sqnorm_partials_per_example(layers, p.umma_idx.data(), (int)p.umma_idx.size(),
                                                                   p.umma_gram.data());
    p.partial_bytes = B * (size_t)p.partials_per_example * sizeof(float);
  }
  for (int l : p.umma_idx)
    if (layers[l].kind == DP_LINEAR) p.lin_idx.push_back(l);
  if (!p.lin_idx.empty()) p.sync_bytes = 256;
  return p;
}

static int check_ws(const WsPlan& p, void* ws, size_t bytes) {
  if (p.total() == 0) return DP_OK;
  if (!ws || misaligned(ws, 256) || bytes < p.total()) return DP_ERR_WORKSPACE;
  return DP_OK;
}

#define DP_CUDA(expr) do { if ((expr) != cudaSuccess) return DP_ERR_CUDA; } while (0)

}  // namespace dpk

using namespace dpk;

extern "C" {

size_t dp_workspace_bytes(const dp_layer* layers, int n_layers) {
  if (validate_layers(layers, n_layers, false) != DP_OK) return 0;
  return plan_workspace(layers, n_layers).total();
}


int dp_per_example_sqnorms(const dp_layer* layers, int n_layers, float* sqnorm, int accumulate_into,
                           void* workspace, size_t workspace_bytes, void* cuda_stream) {
  int rc = validate_layers(layers, n_layers, false);
  if (rc != DP_OK) return rc;
  if (!sqnorm) return DP_ERR_ARG;
  if (misaligned(sqnorm, 4)) return DP_ERR_ALIGN;
  const WsPlan plan = plan_workspace(layers, n_layers);
  if ((rc = check_ws(plan, workspace, workspace_bytes)) != DP_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int* status = status_ptr();
  if (!status) return DP_ERR_CUDA;
  float* partial = reinterpret_cast<float*>(static_cast<char*>(workspace) + align_up(plan.colsum_bytes, 256));
  const int B = layers[0].B;
  if (!accumulate_into) DP_CUDA(launch_fill_zero(sqnorm, B, s));
  // Tensor-core layers first (one persistent launch per path), then the bandwidth-bound layers.
  if (!plan.umma_idx.empty()) {
    rc = launch_umma_sqnorms(layers, plan.umma_idx.data(), (int)plan.umma_idx.size(), plan.umma_gram.data(), partial,
                             plan.partials_per_example, 0, status, s);
    if (rc != DP_OK) return rc;
    DP_CUDA(launch_reduce_partials(partial, B, plan.partials_per_example, sqnorm, s));
  }
  // Bandwidth-bound layers: LayerNorm column sums (and the bias part of materialised-tile layers) in one
  // batched launch, then one reduction; generic linear layers and embeddings one launch each.
  std::vector<ColTaskHost> tasks;
  size_t u = 0;
  for (int l = 0; l < n_layers; ++l) {
    const dp_layer& L = layers[l];
    float* out = plan.col_off[l] == (size_t)-1 ? nullptr
                                                : reinterpret_cast<float*>(static_cast<char*>(workspace) + plan.col_off[l]);
    if (u < plan.umma_idx.size() && plan.umma_idx[u] == l) {
      // The materialised-tile kernel covers the weight gradient only; the bias part |sum_t G_i[t,:]|^2 is a
      // column sum (the Gram kernel has it built in as the +1 on the token Gram of A).
      if (!plan.umma_gram[u] && L.has_bias) tasks.push_back({&L, false, out});
      ++u;
      continue;
    }
    if (L.kind == DP_LINEAR) {
      DP_CUDA(launch_linear_sqnorm_generic(L, use_gram(L), sqnorm, s));
    } else if (L.kind == DP_LAYERNORM) {
      tasks.push_back({&L, true, out});
    } else {
      DP_CUDA(launch_embedding_sqnorm(L, sqnorm, status, s));
    }
  }
  if (!tasks.empty()) {
    DP_CUDA(launch_colsums_batched(tasks.data(), (int)tasks.size(), s));
    DP_CUDA(launch_rows_sqsum_batched(tasks.data(), (int)tasks.size(), sqnorm, s));
  }
  return DP_OK;
}

int dp_clip_factors(const float* sqnorm, int B, double C, float* clip, void* cuda_stream) {
  if (!sqnorm || !clip || B <= 0) return DP_ERR_ARG;
  if (!(C > 0.0) || !std::isfinite(C)) return DP_ERR_ARG;
  if (misaligned(sqnorm, 4) || misaligned(clip, 4)) return DP_ERR_ALIGN;
  DP_CUDA(launch_clip_factors(sqnorm, B, (float)C, clip, static_cast<cudaStream_t>(cuda_stream)));
  return DP_OK;
}

// reuse_colsums: the LayerNorm column sums are already in the workspace (left by dp_per_example_sqnorms).
static int clipped_accumulate(const dp_layer* layers, int n_layers, const float* clip, void* workspace,
                              size_t workspace_bytes, void* cuda_stream, bool reuse_colsums) {
  int rc = validate_layers(layers, n_layers, true);
  if (rc != DP_OK) return rc;
  if (!clip) return DP_ERR_ARG;
  if (misaligned(clip, 4)) return DP_ERR_ALIGN;
  const WsPlan plan = plan_workspace(layers, n_layers);
  if ((rc = check_ws(plan, workspace, workspace_bytes)) != DP_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  int* status = status_ptr();
  if (!status) return DP_ERR_CUDA;
  if (!plan.lin_idx.empty()) {
    unsigned int* wave_sync = reinterpret_cast<unsigned int*>(static_cast<char*>(workspace) + plan.sync_off());
    rc = launch_umma_accumulate(layers, plan.lin_idx.data(), (int)plan.lin_idx.size(), clip, status, wave_sync, s);
    if (rc != DP_OK) return rc;
  }
  std::vector<ColTaskHost> tasks, fresh;     // all column-sum tasks / those whose sums must be formed now
  size_t u = 0;
  for (int l = 0; l < n_layers; ++l) {
    const dp_layer& L = layers[l];
    float* out = plan.col_off[l] == (size_t)-1 ? nullptr
                                                : reinterpret_cast<float*>(static_cast<char*>(workspace) + plan.col_off[l]);
    const bool on_umma = u < plan.umma_idx.size() && plan.umma_idx[u] == l;
    if (on_umma) ++u;
    if (L.kind == DP_LINEAR) {
      if (!on_umma) DP_CUDA(launch_linear_accum_generic(L, clip, s));
      if (L.has_bias && !on_umma) {    // the tensor-core GEMM adds its own bias column sums
        tasks.push_back({&L, false, out});
        fresh.push_back({&L, false, out});    // the norm pass does not leave these behind
      }
    } else if (L.kind == DP_LAYERNORM) {
      tasks.push_back({&L, true, out});
      if (!reuse_colsums) fresh.push_back({&L, true, out});
    } else {
      DP_CUDA(launch_embedding_accum(L, clip, status, s));
    }
  }
  if (!fresh.empty()) DP_CUDA(launch_colsums_batched(fresh.data(), (int)fresh.size(), s));
  if (!tasks.empty()) DP_CUDA(launch_weighted_rows_sum_batched(tasks.data(), (int)tasks.size(), clip, s));
  return DP_OK;
}

int dp_accumulate_schedule(const dp_layer* layers, int n_layers, int units, int64_t* item_start, int32_t* launch,
                           int32_t* splits, int64_t* slots, int max_launches) {
  int rc = validate_layers(layers, n_layers, false);
  if (rc != DP_OK) return rc;
  if (units <= 0 || !item_start || !launch || !splits || !slots || max_launches <= 0) return DP_ERR_ARG;
  const WsPlan plan = plan_workspace(layers, n_layers);
  for (int l = 0; l < n_layers; ++l) { item_start[l] = -1; launch[l] = -1; }
  const int n = (int)plan.lin_idx.size();
  int n_launch = 0;
  for (int k0 = 0; k0 < n; k0 += kUmmaMaxLayers, ++n_launch) {
    if (n_launch >= max_launches) return DP_ERR_ARG;
    const int nl = (n - k0) < kUmmaMaxLayers ? (n - k0) : kUmmaMaxLayers;
    std::vector<long long> start;
    int sp = 1;
    slots[n_launch] = umma_accumulate_schedule(layers, plan.lin_idx.data() + k0, nl, units, &sp, start);
    splits[n_launch] = sp;
    for (int k = 0; k < nl; ++k) {
      item_start[plan.lin_idx[k0 + k]] = start[k];
      launch[plan.lin_idx[k0 + k]] = n_launch;
    }
  }
  return n_launch;
}

int dp_clipped_accumulate(const dp_layer* layers, int n_layers, const float* clip, void* workspace,
                          size_t workspace_bytes, void* cuda_stream) {
  return clipped_accumulate(layers, n_layers, clip, workspace, workspace_bytes, cuda_stream, false);
}

int dp_clipped_accumulate_after_sqnorms(const dp_layer* layers, int n_layers, const float* clip, void* workspace,
                                        size_t workspace_bytes, void* cuda_stream) {
  return clipped_accumulate(layers, n_layers, clip, workspace, workspace_bytes, cuda_stream, true);
}

static int make_noise_args(int64_t n, int64_t elem_offset, double sigma, double C, int64_t batch_size, uint64_t seed,
                           uint64_t step, NoiseArgs* na) {
  if (n < 0 || elem_offset < 0 || batch_size <= 0) return DP_ERR_ARG;
  if (!std::isfinite(sigma) || sigma < 0.0 || !std::isfinite(C) || !(C > 0.0)) return DP_ERR_ARG;
  na->sigmaC = (float)(sigma * C);
  na->inv_n = (float)(1.0 / (double)batch_size);
  na->key0 = (uint32_t)seed;
  na->key1 = (uint32_t)(seed >> 32);
  na->step0 = (uint32_t)step;
  na->step1 = (uint32_t)(step >> 32);
  na->elem_offset = elem_offset;
  return DP_OK;
}

static int make_adam_args(double lr, double b1, double b2, double xi, double wd, int64_t t, AdamArgs* aa) {
  if (t < 1) return DP_ERR_ARG;
  if (!std::isfinite(lr) || !std::isfinite(xi) || !std::isfinite(wd) || xi < 0.0) return DP_ERR_ARG;
  if (!(b1 >= 0.0 && b1 < 1.0) || !(b2 >= 0.0 && b2 < 1.0)) return DP_ERR_ARG;
  aa->lr = (float)lr; aa->beta1 = (float)b1; aa->beta2 = (float)b2; aa->xi = (float)xi; aa->wd = (float)wd;
  aa->one_m_beta1 = (float)(1.0 - b1);
  aa->one_m_beta2 = (float)(1.0 - b2);
  aa->bias1 = (float)(1.0 / (1.0 - std::pow(b1, (double)t)));
  aa->bias2 = (float)(1.0 / (1.0 - std::pow(b2, (double)t)));
  return DP_OK;
}

int dp_add_noise_and_scale(float* acc, int64_t n, int64_t elem_offset, double sigma, double C, int64_t batch_size,
                           uint64_t seed, uint64_t step, void* cuda_stream) {
  NoiseArgs na;
  int rc = make_noise_args(n, elem_offset, sigma, C, batch_size, seed, step, &na);
  if (rc != DP_OK) return rc;
  if (n == 0) return DP_OK;
  if (!acc) return DP_ERR_ARG;
  if (misaligned(acc, 4)) return DP_ERR_ALIGN;
  DP_CUDA(launch_noise_scale(acc, n, na, static_cast<cudaStream_t>(cuda_stream)));
  return DP_OK;
}

int dp_adamw_step(float* theta, float* m, float* v, const float* g, int64_t n, double lr, double beta1, double beta2,
                  double xi, double weight_decay, int64_t t, void* cuda_stream) {
  AdamArgs aa;
  if (n < 0) return DP_ERR_ARG;
  int rc = make_adam_args(lr, beta1, beta2, xi, weight_decay, t, &aa);
  if (rc != DP_OK) return rc;
  if (n == 0) return DP_OK;
  if (!theta || !m || !v || !g) return DP_ERR_ARG;
  if (misaligned(theta, 4) || misaligned(m, 4) || misaligned(v, 4) || misaligned(g, 4)) return DP_ERR_ALIGN;
  DP_CUDA(launch_adamw(theta, m, v, g, n, aa, static_cast<cudaStream_t>(cuda_stream)));
  return DP_OK;
}

int dp_noise_scale_adamw_step(float* theta, float* m, float* v, float* acc, int zero_acc, int64_t n,
                              int64_t elem_offset, double sigma, double C, int64_t batch_size, uint64_t seed,
                              uint64_t step, double lr, double beta1, double beta2, double xi, double weight_decay,
                              int64_t t, void* cuda_stream) {
  NoiseArgs na;
  AdamArgs aa;
  int rc = make_noise_args(n, elem_offset, sigma, C, batch_size, seed, step, &na);
  if (rc != DP_OK) return rc;
  if ((rc = make_adam_args(lr, beta1, beta2, xi, weight_decay, t, &aa)) != DP_OK) return rc;
  if (n == 0) return DP_OK;
  if (!theta || !m || !v || !acc) return DP_ERR_ARG;
  if (misaligned(theta, 4) || misaligned(m, 4) || misaligned(v, 4) || misaligned(acc, 4)) return DP_ERR_ALIGN;
  DP_CUDA(launch_noise_adamw(theta, m, v, acc, zero_acc, n, na, aa, static_cast<cudaStream_t>(cuda_stream)));
  return DP_OK;
}

int dp_noise_scale_adamw_step_snr(float* theta, float* m, float* v, float* acc, int zero_acc, int64_t n,
                                  int64_t elem_offset, double sigma, double C, int64_t batch_size, uint64_t seed,
                                  uint64_t step, double lr, double beta1, double beta2, double xi,
                                  double weight_decay, int64_t t, double* sq_sums, void* cuda_stream) {
  NoiseArgs na;
  AdamArgs aa;
  int rc = make_noise_args(n, elem_offset, sigma, C, batch_size, seed, step, &na);
  if (rc != DP_OK) return rc;
  if ((rc = make_adam_args(lr, beta1, beta2, xi, weight_decay, t, &aa)) != DP_OK) return rc;
  if (!sq_sums) return DP_ERR_ARG;
  if (misaligned(sq_sums, 8)) return DP_ERR_ALIGN;
  if (n == 0) return DP_OK;
  if (!theta || !m || !v || !acc) return DP_ERR_ARG;
  if (misaligned(theta, 4) || misaligned(m, 4) || misaligned(v, 4) || misaligned(acc, 4)) return DP_ERR_ALIGN;
  DP_CUDA(launch_noise_adamw(theta, m, v, acc, zero_acc, n, na, aa, static_cast<cudaStream_t>(cuda_stream), sq_sums));
  return DP_OK;
}

int dp_reduce_noise_adamw_step(float* theta, float* m, float* v, float* const* acc_of_rank,
                               float* const* theta_of_rank, int n_ranks, int zero_acc, int64_t n, int64_t elem_offset,
                               double sigma, double C, int64_t batch_size, uint64_t seed, uint64_t step, double lr,
                               double beta1, double beta2, double xi, double weight_decay, int64_t t,
                               void* cuda_stream) {
  NoiseArgs na;
  AdamArgs aa;
  int rc = make_noise_args(n, elem_offset, sigma, C, batch_size, seed, step, &na);
  if (rc != DP_OK) return rc;
  if ((rc = make_adam_args(lr, beta1, beta2, xi, weight_decay, t, &aa)) != DP_OK) return rc;
  if (n_ranks < 1 || n_ranks > kMaxRanks || !acc_of_rank) return DP_ERR_ARG;
  if (n == 0) return DP_OK;
  if (!theta || !m || !v) return DP_ERR_ARG;
  if ((elem_offset & 3) != 0 || misaligned(theta, 16) || misaligned(m, 16) || misaligned(v, 16)) return DP_ERR_ALIGN;
  for (int r = 0; r < n_ranks; ++r) {
    if (!acc_of_rank[r]) return DP_ERR_ARG;
    if (misaligned(acc_of_rank[r], 16)) return DP_ERR_ALIGN;
    if (theta_of_rank && theta_of_rank[r] && misaligned(theta_of_rank[r], 16)) return DP_ERR_ALIGN;
  }
  DP_CUDA(launch_reduce_update(theta, m, v, acc_of_rank, theta_of_rank, n_ranks, zero_acc, n, na, aa,
                               static_cast<cudaStream_t>(cuda_stream)));
  return DP_OK;
}

int dp_clip_stats(const float* clip, int B, float* out, void* cuda_stream) {
  if (!clip || !out || B <= 0) return DP_ERR_ARG;
  if (misaligned(clip, 4) || misaligned(out, 4)) return DP_ERR_ALIGN;
  DP_CUDA(launch_clip_stats(clip, B, out, static_cast<cudaStream_t>(cuda_stream)));
  return DP_OK;
}

int dp_philox_u32(uint32_t* out, int64_t n_words, int64_t elem_offset, uint64_t seed, uint64_t step,
                  void* cuda_stream) {
  if (n_words < 0 || elem_offset < 0) return DP_ERR_ARG;
  if (n_words == 0) return DP_OK;
  if (!out) return DP_ERR_ARG;
  if (misaligned(out, 4)) return DP_ERR_ALIGN;
  NoiseArgs na = {};
  na.key0 = (uint32_t)seed; na.key1 = (uint32_t)(seed >> 32);
  na.step0 = (uint32_t)step; na.step1 = (uint32_t)(step >> 32);
  na.elem_offset = elem_offset;
  DP_CUDA(launch_philox_u32(out, n_words, na, static_cast<cudaStream_t>(cuda_stream)));
  return DP_OK;
}

int dp_shared_table_cross_sqnorms(const int32_t* ids, const void* G_emb, int B, int T, const void* dlogits,
                                  const void* h, int T_out, int d, int V, int dtype, float* sqnorm, void* cuda_stream) {
  if (!ids || !G_emb || !dlogits || !h || !sqnorm) return DP_ERR_ARG;
  if (B <= 0 || T <= 0 || T_out <= 0 || d <= 0 || V <= 0) return DP_ERR_ARG;
  if (dtype != DP_F32 && dtype != DP_BF16) return DP_ERR_ARG;
  const size_t es = dtype == DP_F32 ? 4 : 2;
  if (misaligned(ids, 4) || misaligned(sqnorm, 4) || misaligned(G_emb, es) || misaligned(dlogits, es) || misaligned(h, es))
    return DP_ERR_ALIGN;
  int* status = status_ptr();
  if (!status) return DP_ERR_CUDA;
  DP_CUDA(launch_shared_table_cross(ids, G_emb, B, T, dlogits, h, T_out, d, V, dtype, sqnorm, status,
                                    static_cast<cudaStream_t>(cuda_stream)));
  return DP_OK;
}

int dp_token_equality_mask(const int32_t* ids, int B, int T, uint8_t* mask, void* cuda_stream) {
  if (!ids || !mask || B <= 0 || T <= 0) return DP_ERR_ARG;
  if (misaligned(ids, 4)) return DP_ERR_ALIGN;
  DP_CUDA(launch_equality_mask(ids, B, T, mask, static_cast<cudaStream_t>(cuda_stream)));
  return DP_OK;
}

int dp_poll_status(void* cuda_stream) {
  int* status = status_ptr();
  if (!status) return DP_ERR_CUDA;
  DP_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
  int h = 0;
  DP_CUDA(cudaMemcpy(&h, status, sizeof(int), cudaMemcpyDeviceToHost));
  if (h != STATUS_OK) DP_CUDA(cudaMemset(status, 0, sizeof(int)));
  if (h == STATUS_TIMEOUT) return DP_ERR_TIMEOUT;
  if (h == STATUS_BAD_ID) return DP_ERR_BAD_ID;
  return DP_OK;
}

int dp_last_timeout_info(int info[5]) {
  int* status = status_ptr();
  if (!status || !info) return DP_ERR_ARG;
  DP_CUDA(cudaMemcpy(info, status + 1, 5 * sizeof(int), cudaMemcpyDeviceToHost));
  return DP_OK;
}

int dp_set_wait_limit_cycles(long long cycles) { return set_wait_limit_cycles(cycles); }

int dp_selftest_wait_timeout(void* cuda_stream) {
  int* status = status_ptr();
  if (!status) return DP_ERR_CUDA;
  return launch_selftest_wait(status, static_cast<cudaStream_t>(cuda_stream));
}

const char* dp_status_string(int status) {
  switch (status) {
    case DP_OK: return "ok";
    case DP_ERR_ARG: return "invalid argument";
    case DP_ERR_ALIGN: return "misaligned pointer";
    case DP_ERR_UNSUPPORTED: return "unsupported request";
    case DP_ERR_CUDA: return "CUDA call failed";
    case DP_ERR_TIMEOUT: return "device-side wait timed out";
    case DP_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case DP_ERR_BAD_ID: return "token id out of range";
    default: return "unknown status";
  }
}

long long dp_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int dp_version(void) { return 100; }

}  // extern "C"
