// dz from logits kept by the forward (no recomputation of the LM head in the backward).
//
// The saving forward leaves u[row, v] = z * log2(e) / T - ref[row, tile] (fp16) and ref (fp32).
// For every row that takes part in the backward (compact row c of the backward's row space):
//     p        = exp2(u + ref - lse * log2(e))                    softmax probability
//     dz[c, v] = (g / T) * (1[v == y] - p)                        bf16
// One streaming pass: 2 bytes read and 2 bytes written per logit.  Rows from the kept count up
// to the next multiple of 128 are written as zeros (the GEMMs read whole row tiles).

#include <cuda_fp16.h>

#include "a3po_common.cuh"
#include "lmhead_internal.cuh"

namespace a3po {
namespace {

constexpr int kDzThreads = 256;
constexpr int kColsPerLoad = 8;                          // one 16-byte load of fp16
constexpr int kLoadsPerThread = 2;                       // independent loads in flight per thread
constexpr int kHalfSeg = kDzThreads * kColsPerLoad;      // 2048 columns
constexpr int kSegCols = kHalfSeg * kLoadsPerThread;     // 4096 columns per block iteration
constexpr int kTileCols = 256;                           // column tile of the saving forward

__device__ __forceinline__ uint4 dz_piece(const uint4 raw, float shift, float g, int y, long long col0) {
  const __half2* h2 = reinterpret_cast<const __half2*>(&raw);
  float d[kColsPerLoad];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 f = __half22float2(h2[j]);
    d[2 * j] = -g * fast_exp2(f.x + shift);
    d[2 * j + 1] = -g * fast_exp2(f.y + shift);
  }
  if (y >= col0 && y < col0 + kColsPerLoad) {
#pragma unroll
    for (int j = 0; j < kColsPerLoad; ++j)
      if (col0 + j == y) d[j] += g;
  }
  __nv_bfloat162 b0 = __floats2bfloat162_rn(d[0], d[1]), b1 = __floats2bfloat162_rn(d[2], d[3]);
  __nv_bfloat162 b2 = __floats2bfloat162_rn(d[4], d[5]), b3 = __floats2bfloat162_rn(d[6], d[7]);
  uint4 out;
  out.x = *reinterpret_cast<uint32_t*>(&b0);
  out.y = *reinterpret_cast<uint32_t*>(&b1);
  out.z = *reinterpret_cast<uint32_t*>(&b2);
  out.w = *reinterpret_cast<uint32_t*>(&b3);
  return out;
}

__global__ void __launch_bounds__(kDzThreads)
dz_from_saved_kernel(const __half* __restrict__ u, const float* __restrict__ ref, long long vpad, int n_tiles, int v,
                     const int* __restrict__ fwd_pos, const int* __restrict__ idx, const int* __restrict__ count,
                     const int32_t* __restrict__ targets_c, const float* __restrict__ lse_c,
                     const float* __restrict__ g_c, float inv_t, long long cap, __nv_bfloat16* __restrict__ dz) {
  const long long kept = *count;
  long long rows = (kept + 127) / 128 * 128;
  if (rows > cap) rows = cap;
  const int segs = static_cast<int>((vpad + kSegCols - 1) / kSegCols);
  const long long items = rows * segs;
  for (long long item = blockIdx.x; item < items; item += gridDim.x) {
    const long long c = item / segs;
    const int seg = static_cast<int>(item % segs);
    const long long col_a = static_cast<long long>(seg) * kSegCols + threadIdx.x * kColsPerLoad;
    const long long col_b = col_a + kHalfSeg;
    const bool in_a = col_a < vpad, in_b = col_b < vpad;
    uint4 out_a = make_uint4(0u, 0u, 0u, 0u), out_b = out_a;
    const float g = (c < kept) ? g_c[c] * inv_t : 0.f;
    if (g != 0.f) {
      const long long orig = idx[c];                                  // row of the batch
      const long long src = fwd_pos ? fwd_pos[orig] : orig;           // its row in the forward's row space
      const __half* urow = u + src * vpad;
      uint4 raw_a = out_a, raw_b = out_a;
      if (in_a) raw_a = __ldcs(reinterpret_cast<const uint4*>(urow + col_a));
      if (in_b) raw_b = __ldcs(reinterpret_cast<const uint4*>(urow + col_b));
      const float lse2 = lse_c[c] * kLog2e;
      const int y = min(max(targets_c[c], 0), v - 1);
      const float* rrow = ref + src * n_tiles;
      if (in_a) out_a = dz_piece(raw_a, rrow[col_a / kTileCols] - lse2, g, y, col_a);
      if (in_b) out_b = dz_piece(raw_b, rrow[col_b / kTileCols] - lse2, g, y, col_b);
    }
    if (in_a) __stcs(reinterpret_cast<uint4*>(dz + c * vpad + col_a), out_a);
    if (in_b) __stcs(reinterpret_cast<uint4*>(dz + c * vpad + col_b), out_b);
  }
}

}  // namespace

int dz_from_saved(const void* saved, long long saved_rows, int v, const int* fwd_pos, const CompactBuffers& bwd,
                  float inv_t, void* dz, cudaStream_t stream) {
  const long long vpad = static_cast<long long>(round_up(static_cast<size_t>(v), 8));
  const int n_tiles = (v + kTileCols - 1) / kTileCols;
  const __half* u = static_cast<const __half*>(saved);
  const float* ref = reinterpret_cast<const float*>(static_cast<const char*>(saved) +
                                                    round_up(static_cast<size_t>(saved_rows) * vpad * 2, 256));
  const int blocks = sm_count() * 8;
  A3PO_LAUNCH(kKDzSaved, stream, (dz_from_saved_kernel<<<blocks, kDzThreads, 0, stream>>>(
                                     u, ref, vpad, n_tiles, v, fwd_pos, bwd.idx, bwd.count, bwd.targets_c, bwd.lse_c,
                                     bwd.g_c, inv_t, bwd.cap, static_cast<__nv_bfloat16*>(dz))));
  return after_launch();
}

}  // namespace a3po
