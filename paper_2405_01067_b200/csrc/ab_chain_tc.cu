// Fused tensor-core chain (placeholder until the tcgen05 kernels land): reports "not supported"
// so every shape takes the general kernels.
#include "ab_common.cuh"

namespace ab {
bool chain_tc_supported(int64_t, int, int, int, int, int, int, const void*, const void*, const void*, const void*) { return false; }
size_t chain_tc_forward_ws(int64_t, int, int, int) { return 0; }
size_t chain_tc_backward_ws(int64_t, int, int, int) { return 0; }
int chain_tc_forward(const void*, const void*, const void*, void*, void*, int64_t, int, int, int, int, int, void*, size_t, cudaStream_t) { return AB_ERR_UNSUPPORTED; }
int chain_tc_backward(const void*, const void*, const void*, const void*, const void*, void*, float*, float*, int64_t, int, int, int, int, int, void*, size_t, cudaStream_t) { return AB_ERR_UNSUPPORTED; }
}  // namespace ab
