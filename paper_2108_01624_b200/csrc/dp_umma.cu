// placeholder until the tcgen05 kernels land
#include "dp_internal.h"
namespace dpk {
bool umma_supported(const dp_layer&) { return false; }
bool umma_accumulates_bias() { return false; }
size_t umma_sqnorm_partials_per_example(const dp_layer*, const int*, int, const int*) { return 0; }
int launch_umma_sqnorms(const dp_layer*, const int*, int, const int*, float*, int, int, int*, cudaStream_t) { return DP_ERR_UNSUPPORTED; }
int launch_umma_accumulate(const dp_layer*, const int*, int, const float*, int*, cudaStream_t) { return DP_ERR_UNSUPPORTED; }
}
