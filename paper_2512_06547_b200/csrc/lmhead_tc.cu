// placeholder until the tensor-core kernels land
#include "lmhead_internal.cuh"
namespace a3po {
bool lmhead_tc_supported(const void*, const void*, long long, int, int) { return false; }
int lmhead_tc_fwd_splits(long long, int) { return 1; }
int lmhead_fwd_tc(const void*, const void*, const int32_t*, long long, int, int, float, int, SoftmaxPartial*, float*,
                  float*, uint32_t*, cudaStream_t) { return A3PO_ERR_UNSUPPORTED; }
size_t lmhead_tc_bwd_ws_bytes(long long, long long, int, int) { return 0; }
int lmhead_bwd_tc(const void*, const void*, const int32_t*, const float*, const float*, long long, int, int, float,
                  void*, float*, int, void*, size_t, long long, uint32_t*, cudaStream_t) { return A3PO_ERR_UNSUPPORTED; }
}
