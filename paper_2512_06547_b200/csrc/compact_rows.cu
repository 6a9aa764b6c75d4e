// Row compaction for the tensor-core LM-head kernels.
//
// Rows that do not take part in a call (masked rows in the forward, rows whose upstream
// gradient is exactly zero in the backward: padding and clipped tokens) are work the method
// avoids.  TMA loads need dense operand tiles, so the kept rows of `hidden` are gathered into a
// compact buffer and the GEMM kernels run on the compact row space; the number of kept rows stays
// on the device (no host synchronisation) and the kernels size their work from it.
//
//   count kernel   : kept rows per block of the row range
//   offsets kernel : exclusive scan of the block counts, total -> *count
//   fill kernel    : pos[orig] = compact index or -1, idx[compact] = orig, compact copies of the
//                    per-row scalars (targets, lse, g); g is zero beyond the kept rows
//   gather kernel  : hidden_c[c, :] = hidden[idx[c], :], zero rows up to the next multiple of 128
//   scatter kernel : grad_hidden[t, :] = grad_hidden_c[pos[t], :] or 0

#include "a3po_common.cuh"
#include "lmhead_internal.cuh"

namespace a3po {
namespace {

constexpr int kCompactThreads = 256;
constexpr int kMaxCompactBlocks = 4096;

__device__ __forceinline__ bool keep_row(const uint8_t* row_mask, const float* g, long long t) {
  bool k = true;
  if (row_mask) k = row_mask[t] != 0;
  if (g) k = k && (g[t] != 0.f);
  return k;
}

__global__ void __launch_bounds__(kCompactThreads)
compact_count_kernel(const uint8_t* __restrict__ row_mask, const float* __restrict__ g, long long n,
                     long long rows_per_block, int* __restrict__ block_counts) {
  const long long lo = static_cast<long long>(blockIdx.x) * rows_per_block;
  const long long hi = (lo + rows_per_block < n) ? lo + rows_per_block : n;
  int c = 0;
  for (long long t = lo + threadIdx.x; t < hi; t += kCompactThreads) c += keep_row(row_mask, g, t) ? 1 : 0;
  c = static_cast<int>(warp_sum(static_cast<long long>(c)));
  __shared__ int sh[kCompactThreads / kWarp];
  if (threadIdx.x % kWarp == 0) sh[threadIdx.x / kWarp] = c;
  __syncthreads();
  if (threadIdx.x == 0) {
    int total = 0;
    for (int w = 0; w < kCompactThreads / kWarp; ++w) total += sh[w];
    block_counts[blockIdx.x] = total;
  }
}

// One block: exclusive scan of up to kMaxCompactBlocks counts.
__global__ void __launch_bounds__(1024)
compact_offsets_kernel(const int* __restrict__ block_counts, int blocks, int* __restrict__ block_offsets,
                       int* __restrict__ count) {
  __shared__ int sh[1024];
  constexpr int kPer = kMaxCompactBlocks / 1024;
  int local[kPer];
  int sum = 0;
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int b = threadIdx.x * kPer + i;
    local[i] = (b < blocks) ? block_counts[b] : 0;
    sum += local[i];
  }
  sh[threadIdx.x] = sum;
  __syncthreads();
  for (int off = 1; off < 1024; off <<= 1) {  // Hillis-Steele inclusive scan
    const int v = (threadIdx.x >= off) ? sh[threadIdx.x - off] : 0;
    __syncthreads();
    sh[threadIdx.x] += v;
    __syncthreads();
  }
  int run = sh[threadIdx.x] - sum;  // exclusive prefix of this thread's group
#pragma unroll
  for (int i = 0; i < kPer; ++i) {
    const int b = threadIdx.x * kPer + i;
    if (b < blocks) block_offsets[b] = run;
    run += local[i];
  }
  if (threadIdx.x == 1023) *count = sh[1023];
}

__global__ void __launch_bounds__(kCompactThreads)
compact_fill_kernel(const uint8_t* __restrict__ row_mask, const float* __restrict__ g,
                    const int32_t* __restrict__ targets, const float* __restrict__ lse, long long n, long long cap,
                    long long rows_per_block, const int* __restrict__ block_offsets, const int* __restrict__ count,
                    int* __restrict__ pos, int* __restrict__ idx, int32_t* __restrict__ targets_c,
                    float* __restrict__ lse_c, float* __restrict__ g_c) {
  const long long lo = static_cast<long long>(blockIdx.x) * rows_per_block;
  const long long hi = (lo + rows_per_block < n) ? lo + rows_per_block : n;
  __shared__ int warp_base[kCompactThreads / kWarp];
  __shared__ int running;
  if (threadIdx.x == 0) running = block_offsets[blockIdx.x];
  __syncthreads();
  const int lane = threadIdx.x % kWarp, warp = threadIdx.x / kWarp;
  for (long long base = lo; base < hi; base += kCompactThreads) {
    const long long t = base + threadIdx.x;
    const bool k = (t < hi) && keep_row(row_mask, g, t);
    const unsigned ballot = __ballot_sync(0xffffffffu, k);
    if (lane == 0) warp_base[warp] = __popc(ballot);
    __syncthreads();
    int before = running;
    for (int w = 0; w < warp; ++w) before += warp_base[w];
    const int c = before + __popc(ballot & ((1u << lane) - 1u));
    if (t < hi) pos[t] = k ? c : -1;
    if (k) {
      idx[c] = static_cast<int>(t);
      targets_c[c] = targets[t];
      if (lse_c) lse_c[c] = lse[t];
      if (g_c) g_c[c] = g[t];
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      int total = 0;
      for (int w = 0; w < kCompactThreads / kWarp; ++w) total += warp_base[w];
      running += total;
    }
    __syncthreads();
  }
  // rows of the compact space that hold no token: zero upstream gradient, harmless target
  const long long kept = *count;
  const long long stride = static_cast<long long>(gridDim.x) * kCompactThreads;
  for (long long c = kept + static_cast<long long>(blockIdx.x) * kCompactThreads + threadIdx.x; c < cap; c += stride) {
    if (g_c) g_c[c] = 0.f;
    if (lse_c) lse_c[c] = 0.f;
    targets_c[c] = 0;
    idx[c] = 0;
  }
}

// One warp per compact row; rows in [count, round_up(count, 128)) are written as zeros so that
// partial tiles of the GEMMs see finite data.
__global__ void __launch_bounds__(kCompactThreads)
gather_rows_kernel(const __nv_bfloat16* __restrict__ hidden, int h, const int* __restrict__ idx,
                   const int* __restrict__ count, long long offset, long long rows,
                   __nv_bfloat16* __restrict__ dst) {
  long long kept = static_cast<long long>(*count) - offset;   // kept rows inside [offset, offset + rows)
  kept = kept < 0 ? 0 : (kept > rows ? rows : kept);
  long long fill_to = (kept + 127) / 128 * 128;
  if (fill_to > rows) fill_to = rows;
  const int lane = threadIdx.x % kWarp;
  const long long warps = static_cast<long long>(gridDim.x) * (kCompactThreads / kWarp);
  const int vec_per_row = h / 8;  // 16-byte pieces
  for (long long r = static_cast<long long>(blockIdx.x) * (kCompactThreads / kWarp) + threadIdx.x / kWarp; r < fill_to;
       r += warps) {
    uint4* out = reinterpret_cast<uint4*>(dst + r * h);
    if (r < kept) {
      const uint4* src = reinterpret_cast<const uint4*>(hidden + static_cast<long long>(idx[offset + r]) * h);
      for (int j = lane; j < vec_per_row; j += kWarp) out[j] = __ldg(src + j);
    } else {
      for (int j = lane; j < vec_per_row; j += kWarp) out[j] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

__global__ void __launch_bounds__(kCompactThreads)
scatter_rows_kernel(const __nv_bfloat16* __restrict__ src_c, int h, const int* __restrict__ pos, long long n,
                    __nv_bfloat16* __restrict__ dst) {
  const int lane = threadIdx.x % kWarp;
  const long long warps = static_cast<long long>(gridDim.x) * (kCompactThreads / kWarp);
  const int vec_per_row = h / 8;
  for (long long t = static_cast<long long>(blockIdx.x) * (kCompactThreads / kWarp) + threadIdx.x / kWarp; t < n;
       t += warps) {
    const int c = pos[t];
    uint4* out = reinterpret_cast<uint4*>(dst + t * h);
    if (c >= 0) {
      const uint4* in = reinterpret_cast<const uint4*>(src_c + static_cast<long long>(c) * h);
      for (int j = lane; j < vec_per_row; j += kWarp) out[j] = in[j];
    } else {
      for (int j = lane; j < vec_per_row; j += kWarp) out[j] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

}  // namespace

long long compact_capacity(long long n) { return (n + 127) / 128 * 128; }

size_t compact_ws_bytes(long long n, int h, bool backward) {
  const size_t cap = static_cast<size_t>(compact_capacity(n));
  size_t b = 256 /*count*/ + 2 * round_up(sizeof(int) * kMaxCompactBlocks, 256);
  b += round_up(sizeof(int) * static_cast<size_t>(n), 256);       // pos
  b += 2 * round_up(sizeof(int) * cap, 256);                       // idx, targets_c
  b += round_up(cap * static_cast<size_t>(h) * 2, 256);           // hidden_c
  if (backward) {
    b += 2 * round_up(sizeof(float) * cap, 256);                   // lse_c, g_c
    b += round_up(cap * static_cast<size_t>(h) * 2, 256);         // grad_hidden_c
  }
  return b + 256;
}

bool compact_carve(void* ws, size_t ws_bytes, long long n, int h, bool backward, CompactBuffers* out, size_t* used) {
  Arena arena(ws, ws_bytes);
  const size_t cap = static_cast<size_t>(compact_capacity(n));
  out->cap = static_cast<long long>(cap);
  out->count = arena.take<int>(1);
  out->block_counts = arena.take<int>(kMaxCompactBlocks);
  out->block_offsets = arena.take<int>(kMaxCompactBlocks);
  out->pos = arena.take<int>(static_cast<size_t>(n));
  out->idx = arena.take<int>(cap);
  out->targets_c = arena.take<int32_t>(cap);
  out->hidden_c = arena.take<__nv_bfloat16>(cap * static_cast<size_t>(h));
  out->lse_c = nullptr;
  out->g_c = nullptr;
  out->grad_hidden_c = nullptr;
  if (backward) {
    out->lse_c = arena.take<float>(cap);
    out->g_c = arena.take<float>(cap);
    out->grad_hidden_c = arena.take<__nv_bfloat16>(cap * static_cast<size_t>(h));
  }
  if (!arena.ok()) return false;
  *used = round_up(arena.used, 256);
  return true;
}

int compact_index(const int32_t* targets, const uint8_t* row_mask, const float* g, const float* lse, long long n,
                  const CompactBuffers& cb, cudaStream_t stream) {
  long long rows_per_block = (n + kMaxCompactBlocks - 1) / kMaxCompactBlocks;
  rows_per_block = (rows_per_block + kCompactThreads - 1) / kCompactThreads * kCompactThreads;
  if (rows_per_block < kCompactThreads) rows_per_block = kCompactThreads;
  const int blocks = static_cast<int>((n + rows_per_block - 1) / rows_per_block);
  A3PO_LAUNCH(kKCompact, stream, (compact_count_kernel<<<blocks, kCompactThreads, 0, stream>>>(
                                     row_mask, g, n, rows_per_block, cb.block_counts)));
  A3PO_RETURN_IF(after_launch());
  A3PO_LAUNCH(kKCompact, stream, (compact_offsets_kernel<<<1, 1024, 0, stream>>>(cb.block_counts, blocks,
                                                                                 cb.block_offsets, cb.count)));
  A3PO_RETURN_IF(after_launch());
  A3PO_LAUNCH(kKCompact, stream, (compact_fill_kernel<<<blocks, kCompactThreads, 0, stream>>>(
                                     row_mask, g, targets, lse, n, cb.cap, rows_per_block, cb.block_offsets, cb.count,
                                     cb.pos, cb.idx, cb.targets_c, cb.lse_c, cb.g_c)));
  return after_launch();
}

int gather_rows_range(const void* hidden, int h, const int* idx, const int* count, long long offset, long long rows,
                      void* dst, cudaStream_t stream) {
  if (rows <= 0) return A3PO_OK;
  int gather_blocks = sm_count() * 8;
  const long long want = (rows + 7) / 8;
  if (gather_blocks > want) gather_blocks = static_cast<int>(want);
  A3PO_LAUNCH(kKCompact, stream, (gather_rows_kernel<<<gather_blocks, kCompactThreads, 0, stream>>>(
                                     static_cast<const __nv_bfloat16*>(hidden), h, idx, count, offset, rows,
                                     static_cast<__nv_bfloat16*>(dst))));
  return after_launch();
}

int compact_rows(const void* hidden, int h, const int32_t* targets, const uint8_t* row_mask, const float* g,
                 const float* lse, long long n, const CompactBuffers& cb, cudaStream_t stream) {
  A3PO_RETURN_IF(compact_index(targets, row_mask, g, lse, n, cb, stream));
  return gather_rows_range(hidden, h, cb.idx, cb.count, 0, cb.cap, cb.hidden_c, stream);
}

int scatter_rows(const void* src_c, int h, const int* pos, long long n, void* dst, cudaStream_t stream) {
  int blocks = sm_count() * 8;
  const long long want = (n + 7) / 8;
  if (blocks > want) blocks = static_cast<int>(want);
  if (blocks < 1) return A3PO_OK;
  A3PO_LAUNCH(kKCompact, stream, (scatter_rows_kernel<<<blocks, kCompactThreads, 0, stream>>>(
                                     static_cast<const __nv_bfloat16*>(src_c), h, pos, n,
                                     static_cast<__nv_bfloat16*>(dst))));
  return after_launch();
}

}  // namespace a3po
