// dp_layernorm_sqnorms_static: the LayerNorm squared-norm pass with its scratch in a fixed device array.
//
// Some callers have no way to hand the library a workspace: they run under a memory manager that has
// already claimed the device (a framework's caching allocator, a serving process with a fixed arena) or in
// a place where cudaMalloc's device-wide synchronisation is not acceptable, and they cannot call cudaMalloc
// themselves.  For them this one entry point keeps the per-example column sums in a file-scope device array
// instead of caller-provided scratch.  Every GPU that loads the library holds the array until exit.
#include "dp_internal.h"

namespace dpk {

// [B][2d] fp32 column sums (gain part, then bias part) of one LayerNorm layer.
static __device__ __align__(256) float g_ln_scratch[DP_STATIC_SCRATCH_FLOATS];

// In host code the array's name stands for the symbol, not for a device address; the address has to be
// asked for, once per device, with that device current.
static float* ln_scratch_ptr(int* rc) {
  static float* cache[64] = {};
  int dev = 0;
  *rc = DP_ERR_CUDA;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  if (!cache[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_ln_scratch) != cudaSuccess || !p) return nullptr;
    cache[dev] = p;
  }
  *rc = DP_OK;
  return cache[dev];
}

}  // namespace dpk

using namespace dpk;

extern "C" int dp_layernorm_sqnorms_static(const dp_layer* layer, float* sqnorm, int accumulate_into,
                                           void* cuda_stream) {
  if (!layer || !sqnorm) return DP_ERR_ARG;
  const dp_layer& L = *layer;
  if (L.kind != DP_LAYERNORM || (L.dtype != DP_F32 && L.dtype != DP_BF16)) return DP_ERR_ARG;
  if (L.B <= 0 || L.T <= 0 || L.d_out <= 0 || L.d_in != L.d_out || !L.A || !L.G) return DP_ERR_ARG;
  const size_t esz = L.dtype == DP_F32 ? 4 : 2;
  if ((reinterpret_cast<uintptr_t>(L.A) | reinterpret_cast<uintptr_t>(L.G)) & (esz - 1)) return DP_ERR_ALIGN;
  if (reinterpret_cast<uintptr_t>(sqnorm) & 3u) return DP_ERR_ALIGN;
  if ((unsigned long long)L.B * 2ull * (unsigned long long)L.d_out > (unsigned long long)DP_STATIC_SCRATCH_FLOATS)
    return DP_ERR_WORKSPACE;   // beyond the fixed scratch: use dp_per_example_sqnorms with a workspace
  int rc;
  float* scratch = ln_scratch_ptr(&rc);
  if (!scratch) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  if (!accumulate_into && launch_fill_zero(sqnorm, L.B, s) != cudaSuccess) return DP_ERR_CUDA;
  // The column sums are fully overwritten before they are read, so nothing in the array needs clearing.
  const ColTaskHost task = {&L, true, scratch};
  if (launch_colsums_batched(&task, 1, s) != cudaSuccess) return DP_ERR_CUDA;
  if (launch_rows_sqsum_batched(&task, 1, sqnorm, s) != cudaSuccess) return DP_ERR_CUDA;
  return DP_OK;
}
