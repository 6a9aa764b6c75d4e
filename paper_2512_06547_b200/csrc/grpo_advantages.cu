// GRPO advantages: group reward normalisation, broadcast to the tokens of each sequence.
//
// Sec. 4.1 of the paper estimates advantages "using group reward normalization" without a
// formula; the usual one is taken: for the `group_size` responses of one prompt,
//     A_i = (R_i - mean) / (std + norm_eps),   std = population standard deviation,
// and every token of sequence i carries A_i.  Two tiny HBM-bound kernels.

#include "a3po_common.cuh"

namespace a3po {
namespace {

constexpr int kGrpoThreads = 256;

// One thread per group (groups are a handful of sequences).
__global__ void __launch_bounds__(kGrpoThreads)
grpo_group_kernel(const float* __restrict__ rewards, int n_groups, int group, float norm_eps,
                  float* __restrict__ adv_seq) {
  const int gidx = blockIdx.x * blockDim.x + threadIdx.x;
  if (gidx >= n_groups) return;
  const float* r = rewards + static_cast<long long>(gidx) * group;
  float mean = 0.f;
  for (int i = 0; i < group; ++i) mean += r[i];
  mean /= static_cast<float>(group);
  float var = 0.f;
  for (int i = 0; i < group; ++i) {
    const float d = r[i] - mean;
    var = fmaf(d, d, var);
  }
  const float inv = 1.0f / (sqrtf(var / static_cast<float>(group)) + norm_eps);
  for (int i = 0; i < group; ++i) adv_seq[static_cast<long long>(gidx) * group + i] = (r[i] - mean) * inv;
}

__global__ void __launch_bounds__(kGrpoThreads)
broadcast_per_sequence_kernel(const float* __restrict__ per_seq, const int32_t* __restrict__ cu_seqlens, int b,
                              long long n, float* __restrict__ per_token) {
  const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= n) return;
  int lo = 0, hi = b;  // last sequence whose first row is <= t
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (static_cast<long long>(cu_seqlens[mid]) <= t) lo = mid; else hi = mid;
  }
  per_token[t] = per_seq[lo];
}

}  // namespace
}  // namespace a3po

extern "C" {

size_t a3po_grpo_workspace_bytes(int B) { return B > 0 ? a3po::round_up(sizeof(float) * static_cast<size_t>(B), 256) : 256; }

int a3po_grpo_advantages(const float* rewards, int B, int group_size, const int32_t* cu_seqlens, int64_t N,
                         float norm_eps, float* adv, void* ws, size_t ws_bytes, void* stream_) {
  using namespace a3po;
  if (B < 0 || N < 0 || group_size <= 0 || (B % group_size) != 0 || !(norm_eps >= 0.f)) return A3PO_ERR_INVALID_ARG;
  if (B > 0 && (!rewards || !cu_seqlens)) return A3PO_ERR_INVALID_ARG;
  if (N > 0 && (!adv || B == 0)) return A3PO_ERR_INVALID_ARG;
  if (!ws || !aligned_to(ws, 256) || ws_bytes < a3po_grpo_workspace_bytes(B)) return A3PO_ERR_WORKSPACE;
  if (sm_count() <= 0) return A3PO_ERR_NO_DEVICE;
  if (B == 0 || N == 0) return A3PO_OK;
  cudaStream_t stream = as_stream(stream_);
  float* adv_seq = static_cast<float*>(ws);
  const int n_groups = B / group_size;
  A3PO_LAUNCH(kKGrpo, stream, (grpo_group_kernel<<<(n_groups + kGrpoThreads - 1) / kGrpoThreads, kGrpoThreads, 0, stream>>>(
                                  rewards, n_groups, group_size, norm_eps, adv_seq)));
  A3PO_RETURN_IF(after_launch());
  const unsigned blocks = static_cast<unsigned>((N + kGrpoThreads - 1) / kGrpoThreads);
  A3PO_LAUNCH(kKGrpo, stream, (broadcast_per_sequence_kernel<<<blocks, kGrpoThreads, 0, stream>>>(adv_seq, cu_seqlens, B,
                                                                                                N, adv)));
  return after_launch();
}

}  // extern "C"
