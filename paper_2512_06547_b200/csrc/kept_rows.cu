// Per-row kernels of the backward that does not recompute the LM head.
//
// The keeping forward (lmhead_tc.cu) leaves, for each row that takes part, the probability ratios
//     q[r, v] = exp(z[r, v] - zy[r]) = p[r, v] / p[r, y_r]        bf16, 0 at the target column y_r
// and s[r] = sum_{v != y_r} q[r, v].  With p_y = 1 / (1 + s):
//     lse = zy + log1p(s)          logp = -log1p(s)          1 - p_y = s / (1 + s)
//     dz[r, v] = (g / T) (1[v = y] - p[r, v]) = a[r] * q'[r, v],   a = -g / (T (1 + s)),  q'[r, y] = -s
// so the two gradient contractions run on q' itself: grad_hidden = diag(a) (q' W) and
// grad_w = q'^T (diag(a) hidden).  Nothing here is a stream over the [rows, V] matrix: every kernel
// below touches O(rows * H) or O(rows) data.
//
// All kernels take the compact-row count from device memory and cover compact rows
// [offset, offset + rows); nothing ever reads it on the host.

#include "a3po_common.cuh"
#include "lmhead_internal.cuh"

namespace a3po {
namespace {

constexpr int kRowThreads = 256;
constexpr int kWarpsPerBlock = kRowThreads / kWarp;

// Rows of this launch that a GEMM launch over the same range may touch: the kept ones, rounded up to
// whole 128-row tiles, inside [offset, offset + rows).
__device__ __forceinline__ long long touched_rows(const int* count, long long offset, long long rows) {
  long long have = static_cast<long long>(*count) - offset;
  have = have < 0 ? 0 : have;
  long long up = (have + 127) / 128 * 128;
  return up > rows ? rows : up;
}

__device__ __forceinline__ float dot8(const uint4 a, const uint4 b, float acc) {
  const __nv_bfloat162* x = reinterpret_cast<const __nv_bfloat162*>(&a);
  const __nv_bfloat162* y = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float2 fx = __bfloat1622float2(x[j]);
    const float2 fy = __bfloat1622float2(y[j]);
    acc = fmaf(fx.x, fy.x, acc);
    acc = fmaf(fx.y, fy.y, acc);
  }
  return acc;
}

// One warp per row: zy = <hidden_c[c], W[y_c]> / T in fp32.
__global__ void __launch_bounds__(kRowThreads)
target_logit_kernel(const __nv_bfloat16* __restrict__ hidden_c, const __nv_bfloat16* __restrict__ w,
                    const int32_t* __restrict__ targets_c, const int* __restrict__ count, long long offset,
                    long long rows, int h, int v, float inv_t, float* __restrict__ zy) {
  const long long live = touched_rows(count, offset, rows);
  const int lane = threadIdx.x % kWarp;
  const long long warps = static_cast<long long>(gridDim.x) * kWarpsPerBlock;
  const int vec = h / 8;
  for (long long r = static_cast<long long>(blockIdx.x) * kWarpsPerBlock + threadIdx.x / kWarp; r < live; r += warps) {
    const long long c = offset + r;
    const int y = min(max(targets_c[c], 0), v - 1);
    const uint4* a = reinterpret_cast<const uint4*>(hidden_c + r * h);   // hidden_c starts at the launch's first row
    const uint4* b = reinterpret_cast<const uint4*>(w + static_cast<long long>(y) * h);
    float acc = 0.f;
    for (int j = lane; j < vec; j += kWarp) acc = dot8(__ldg(a + j), __ldg(b + j), acc);
    acc = warp_sum(acc);
    if (lane == 0) zy[c] = acc * inv_t;
  }
}

__global__ void __launch_bounds__(kRowThreads)
merge_kept_kernel(const float* __restrict__ part_s, const float* __restrict__ part_e, const float* __restrict__ zy,
                  const int* __restrict__ count, long long offset, long long rows, int splits, float inv_t,
                  float* __restrict__ sprime, float* __restrict__ logp, float* __restrict__ lse,
                  float* __restrict__ entropy, uint32_t* status) {
  const long long r = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (r >= rows) return;
  const long long c = offset + r;
  if (c >= *count) {
    sprime[c] = 0.f;
    logp[c] = 0.f;
    lse[c] = 0.f;
    if (entropy) entropy[c] = 0.f;
    return;
  }
  float s = 0.f, e = 0.f;
  for (int i = 0; i < splits; ++i) {   // fixed order: the same bits from run to run
    s += part_s[static_cast<long long>(i) * rows + r];
    if (part_e) e += part_e[static_cast<long long>(i) * rows + r];
  }
  // a ratio had to be clamped (or the sum overflowed): the row's target probability is below ~1e-37
  if (!(s < 1e37f) && status) atomicOr(status, A3PO_STATUS_KEPT_RANGE);
  const float l1p = log1pf(s);
  const float z = zy[c];
  sprime[c] = s;
  logp[c] = -l1p;
  lse[c] = z + l1p;
  // sum_v p_v z_v = p_y (z_y + sum_{v != y} q_v z_v), p_y = 1 / (1 + s); part_e holds raw (unscaled) logits
  if (entropy) entropy[c] = (z + l1p) - (z + e * inv_t) / (1.f + s);
}

__global__ void __launch_bounds__(kRowThreads)
gather_loss_inputs_kernel(const int* __restrict__ idx, const int* __restrict__ count, long long cap,
                          const float* __restrict__ behav, const int32_t* __restrict__ versions,
                          const float* __restrict__ adv, float* __restrict__ behav_c, int32_t* __restrict__ versions_c,
                          float* __restrict__ adv_c, uint8_t* __restrict__ mask_c, long long* __restrict__ n_valid) {
  const long long c = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  const long long kept = *count;
  if (c == 0) *n_valid = kept;
  if (c >= cap) return;
  if (c < kept) {
    const long long t = idx[c];
    behav_c[c] = behav[t];
    versions_c[c] = versions[t];
    adv_c[c] = adv[t];
    mask_c[c] = 1;
  } else {
    behav_c[c] = 0.f;
    versions_c[c] = 0;
    adv_c[c] = 0.f;
    mask_c[c] = 0;
  }
}

// Which rows of a launch's range take part in the backward, and how to make them contiguous by moving as few
// rows as possible.  Among the `live` rows of the range, K have a non-zero upstream gradient.  Positions
// 0 .. K-1 are the backward's rows: a position whose own row has g != 0 keeps it (perm[p] = p); the others
// ("holes", rows with g == 0: clipped tokens) are filled, in order, with the rows at positions >= K that
// have g != 0.  Only those rows have to be copied (move_src[i] -> move_dst[i]); a stable compaction would
// move almost every row.  One block; the sums involved are integer, so the plan is deterministic.
constexpr int kPlanThreads = 1024;
__global__ void __launch_bounds__(kPlanThreads)
plan_backward_rows_kernel(const float* __restrict__ g_c, const int* __restrict__ count, long long offset,
                          long long rows, int* __restrict__ bwd_count, int* __restrict__ n_moves,
                          int* __restrict__ perm, int* __restrict__ move_src, int* __restrict__ move_dst) {
  __shared__ int sh[kPlanThreads];
  __shared__ int s_nz_before_k;
  long long live = static_cast<long long>(*count) - offset;
  live = live < 0 ? 0 : (live > rows ? rows : live);
  const long long per = (live + kPlanThreads - 1) / kPlanThreads;
  long long lo = static_cast<long long>(threadIdx.x) * per;
  lo = lo > live ? live : lo;
  const long long hi = (lo + per > live) ? live : lo + per;
  const float* g = g_c + offset;
  int nz = 0;
  for (long long p = lo; p < hi; ++p) nz += (g[p] != 0.f) ? 1 : 0;
  sh[threadIdx.x] = nz;
  __syncthreads();
  for (int off = 1; off < kPlanThreads; off <<= 1) {  // Hillis-Steele inclusive scan
    const int add = (threadIdx.x >= off) ? sh[threadIdx.x - off] : 0;
    __syncthreads();
    sh[threadIdx.x] += add;
    __syncthreads();
  }
  const int before = sh[threadIdx.x] - nz;   // non-zero rows in front of this thread's segment
  const long long k = sh[kPlanThreads - 1];  // rows of the backward
  if (threadIdx.x == 0) s_nz_before_k = static_cast<int>(k);  // stands when no position >= k exists
  __syncthreads();
  if (lo <= k && k < hi) {                   // this segment holds position k: non-zero rows in front of it
    int c = before;
    for (long long p = lo; p < k; ++p) c += (g[p] != 0.f) ? 1 : 0;
    s_nz_before_k = c;
  }
  __syncthreads();
  const int nz_before_k = s_nz_before_k;
  int running = before;
  for (long long p = lo; p < hi; ++p) {
    const bool is_nz = g[p] != 0.f;
    if (p < k) {
      if (is_nz) perm[p] = static_cast<int>(p);
      else move_dst[p - running] = static_cast<int>(p);        // the (p - running)-th hole
    } else if (is_nz) {
      move_src[running - nz_before_k] = static_cast<int>(p);   // the matching filler
    }
    running += is_nz ? 1 : 0;
  }
  __threadfence_block();
  __syncthreads();
  const int holes = static_cast<int>(k) - nz_before_k;
  for (int i = threadIdx.x; i < holes; i += kPlanThreads) perm[move_dst[i]] = move_src[i];
  if (threadIdx.x == 0) {
    *bwd_count = static_cast<int>(k);
    *n_moves = holes;
  }
}

// q[move_dst[i], :] = q[move_src[i], :] for the planned moves (rows of one launch, pitch vpad).
constexpr int kMoveCols = kRowThreads * 8 * 2;   // columns per block iteration: two 16-byte pieces per thread
__global__ void __launch_bounds__(kRowThreads)
move_rows_kernel(__nv_bfloat16* __restrict__ q, long long vpad, const int* __restrict__ move_src,
                 const int* __restrict__ move_dst, const int* __restrict__ n_moves) {
  const int moves = *n_moves;
  const int segs = static_cast<int>((vpad + kMoveCols - 1) / kMoveCols);
  const long long items = static_cast<long long>(moves) * segs;
  for (long long item = blockIdx.x; item < items; item += gridDim.x) {
    const int i = static_cast<int>(item / segs);
    const long long col_a = static_cast<long long>(item % segs) * kMoveCols + threadIdx.x * 8;
    const long long col_b = col_a + kRowThreads * 8;
    const __nv_bfloat16* src = q + static_cast<long long>(move_src[i]) * vpad;
    __nv_bfloat16* dst = q + static_cast<long long>(move_dst[i]) * vpad;
    uint4 a = make_uint4(0u, 0u, 0u, 0u), b = a;
    if (col_a < vpad) a = __ldcs(reinterpret_cast<const uint4*>(src + col_a));
    if (col_b < vpad) b = __ldcs(reinterpret_cast<const uint4*>(src + col_b));
    if (col_a < vpad) *reinterpret_cast<uint4*>(dst + col_a) = a;
    if (col_b < vpad) *reinterpret_cast<uint4*>(dst + col_b) = b;
  }
}

// One warp per position of the launch.
__global__ void __launch_bounds__(kRowThreads)
prepare_kept_backward_kernel(const int* __restrict__ count, long long offset, long long rows,
                             const int* __restrict__ bwd_count, const int* __restrict__ perm, int h, int v,
                             long long vpad, float inv_t, const float* __restrict__ sprime,
                             const int32_t* __restrict__ targets_c, const float* __restrict__ g_c,
                             const float* __restrict__ g_batch, const int* __restrict__ idx,
                             const __nv_bfloat16* __restrict__ hidden_c, const __nv_bfloat16* __restrict__ hidden_batch,
                             float* __restrict__ row_scale, int* __restrict__ bwd_idx, __nv_bfloat16* __restrict__ q,
                             __nv_bfloat16* __restrict__ hs) {
  long long k;   // positions that hold a row of the backward
  if (bwd_count) {
    k = *bwd_count;
  } else {
    k = static_cast<long long>(*count) - offset;
    k = k < 0 ? 0 : (k > rows ? rows : k);
  }
  long long live = (k + 127) / 128 * 128;   // the GEMMs read whole 128-row tiles
  live = live > rows ? rows : live;
  const int lane = threadIdx.x % kWarp;
  const long long warps = static_cast<long long>(gridDim.x) * kWarpsPerBlock;
  const int vec = h / 8;
  for (long long p = static_cast<long long>(blockIdx.x) * kWarpsPerBlock + threadIdx.x / kWarp; p < live; p += warps) {
    uint4* dst = reinterpret_cast<uint4*>(hs + p * h);
    float a = 0.f;
    if (p < k) {
      const long long c = offset + (perm ? perm[p] : p);   // compact row that sits at this position
      const long long t = idx[c];
      const float g = g_c ? g_c[c] : g_batch[t];
      const float s = sprime[c];
      a = -(g * inv_t) / (1.f + s);
      if (!(fabsf(a) < 3.0e38f)) a = 0.f;   // a row the merge has flagged (non-finite sum): contributes nothing
      if (lane == 0) {
        const int y = min(max(targets_c[c], 0), v - 1);
        q[p * vpad + y] = __float2bfloat16_rn(-s);
        if (bwd_idx) bwd_idx[p] = static_cast<int>(t);
      }
      const uint4* src = reinterpret_cast<const uint4*>(hidden_c ? hidden_c + (c - offset) * h : hidden_batch + t * h);
      for (int j = lane; j < vec; j += kWarp) {
        const uint4 in = __ldg(src + j);
        const __nv_bfloat162* x = reinterpret_cast<const __nv_bfloat162*>(&in);
        uint4 out;
        __nv_bfloat162* o = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(x[e]);
          o[e] = __floats2bfloat162_rn(a * f.x, a * f.y);
        }
        dst[j] = out;
      }
    } else {
      for (int j = lane; j < vec; j += kWarp) dst[j] = make_uint4(0u, 0u, 0u, 0u);
    }
    if (lane == 0) row_scale[p] = a;
  }
}

__global__ void __launch_bounds__(kRowThreads)
scatter_rows_range_kernel(const __nv_bfloat16* __restrict__ src, int h, const int* __restrict__ bwd_idx,
                          const int* __restrict__ bwd_count, __nv_bfloat16* __restrict__ dst) {
  const long long live = *bwd_count;
  const int lane = threadIdx.x % kWarp;
  const long long warps = static_cast<long long>(gridDim.x) * kWarpsPerBlock;
  const int vec = h / 8;
  for (long long p = static_cast<long long>(blockIdx.x) * kWarpsPerBlock + threadIdx.x / kWarp; p < live; p += warps) {
    const uint4* in = reinterpret_cast<const uint4*>(src + p * h);
    uint4* out = reinterpret_cast<uint4*>(dst + static_cast<long long>(bwd_idx[p]) * h);
    for (int j = lane; j < vec; j += kWarp) out[j] = in[j];
  }
}

__global__ void __launch_bounds__(kRowThreads)
finish_scalars_kernel(const int* __restrict__ pos, long long n, const float* __restrict__ a_c, float* __restrict__ a,
                      const float* __restrict__ b_c, float* __restrict__ b, const float* __restrict__ c_c,
                      float* __restrict__ c, const float* __restrict__ d_c, float* __restrict__ d) {
  const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= n) return;
  const int p = pos[t];
  if (a) a[t] = p >= 0 ? a_c[p] : 0.f;
  if (b) b[t] = p >= 0 ? b_c[p] : 0.f;
  if (c) c[t] = p >= 0 ? c_c[p] : 0.f;
  if (d) d[t] = p >= 0 ? d_c[p] : 0.f;
}

// Rows of the batch that no backward row was scattered to: not kept by the forward, or zero upstream gradient.
__global__ void __launch_bounds__(kRowThreads)
zero_unkept_rows_kernel(const int* __restrict__ pos, const float* __restrict__ g_c, long long n, int h,
                        __nv_bfloat16* __restrict__ dst) {
  const int lane = threadIdx.x % kWarp;
  const long long warps = static_cast<long long>(gridDim.x) * kWarpsPerBlock;
  const int vec = h / 8;
  for (long long t = static_cast<long long>(blockIdx.x) * kWarpsPerBlock + threadIdx.x / kWarp; t < n; t += warps) {
    const int c = pos[t];
    if (c >= 0 && (g_c == nullptr || g_c[c] != 0.f)) continue;
    uint4* out = reinterpret_cast<uint4*>(dst + t * h);
    for (int j = lane; j < vec; j += kWarp) out[j] = make_uint4(0u, 0u, 0u, 0u);
  }
}

int row_grid(long long rows) {
  long long want = (rows + kWarpsPerBlock - 1) / kWarpsPerBlock;
  const long long cap = static_cast<long long>(sm_count()) * 8;
  if (want > cap) want = cap;
  return static_cast<int>(want < 1 ? 1 : want);
}

}  // namespace

int target_logits(const void* hidden_c, const void* w, const int32_t* targets_c, const int* count, long long offset,
                  long long rows, int h, int v, float inv_t, float* zy, cudaStream_t stream) {
  if (rows <= 0) return A3PO_OK;
  A3PO_LAUNCH(kKKeptRows, stream, (target_logit_kernel<<<row_grid(rows), kRowThreads, 0, stream>>>(
                                      static_cast<const __nv_bfloat16*>(hidden_c),
                                      static_cast<const __nv_bfloat16*>(w), targets_c, count, offset, rows, h, v,
                                      inv_t, zy)));
  return after_launch();
}

int merge_kept(const float* part_s, const float* part_e, const float* zy, const int* count, long long offset,
               long long rows, int splits, float inv_t, float* sprime, float* logp, float* lse, float* entropy,
               uint32_t* status, cudaStream_t stream) {
  if (rows <= 0) return A3PO_OK;
  const unsigned blocks = static_cast<unsigned>((rows + kRowThreads - 1) / kRowThreads);
  A3PO_LAUNCH(kKKeptRows, stream, (merge_kept_kernel<<<blocks, kRowThreads, 0, stream>>>(
                                      part_s, entropy ? part_e : nullptr, zy, count, offset, rows, splits, inv_t,
                                      sprime, logp, lse, entropy, status)));
  return after_launch();
}

int gather_loss_inputs(const int* idx, const int* count, long long cap, const float* behav, const int32_t* versions,
                       const float* adv, float* behav_c, int32_t* versions_c, float* adv_c, uint8_t* mask_c,
                       long long* n_valid, cudaStream_t stream) {
  const unsigned blocks = static_cast<unsigned>((cap + kRowThreads - 1) / kRowThreads);
  A3PO_LAUNCH(kKKeptRows, stream, (gather_loss_inputs_kernel<<<blocks < 1 ? 1 : blocks, kRowThreads, 0, stream>>>(
                                      idx, count, cap, behav, versions, adv, behav_c, versions_c, adv_c, mask_c,
                                      n_valid)));
  return after_launch();
}

int plan_backward_rows(const float* g_c, const int* count, long long offset, long long rows, int* bwd_count,
                       int* n_moves, int* perm, int* move_src, int* move_dst, void* q, int v, cudaStream_t stream) {
  if (rows <= 0) return A3PO_OK;
  A3PO_LAUNCH(kKKeptRows, stream, (plan_backward_rows_kernel<<<1, kPlanThreads, 0, stream>>>(
                                      g_c, count, offset, rows, bwd_count, n_moves, perm, move_src, move_dst)));
  A3PO_RETURN_IF(after_launch());
  const long long vpad = static_cast<long long>(round_up(static_cast<size_t>(v), 8));
  A3PO_LAUNCH(kKMoveRows, stream, (move_rows_kernel<<<sm_count() * 8, kRowThreads, 0, stream>>>(
                                      static_cast<__nv_bfloat16*>(q), vpad, move_src, move_dst, n_moves)));
  return after_launch();
}

int prepare_kept_backward(const int* count, long long offset, long long rows, const int* bwd_count, const int* perm,
                          int h, int v, float inv_t, const float* sprime, const int32_t* targets_c, const float* g_c,
                          const float* g_batch, const int* idx, const void* hidden_c, const void* hidden_batch,
                          float* row_scale, int* bwd_idx, void* q, void* hs, cudaStream_t stream) {
  if (rows <= 0) return A3PO_OK;
  const long long vpad = static_cast<long long>(round_up(static_cast<size_t>(v), 8));
  A3PO_LAUNCH(kKKeptRows, stream, (prepare_kept_backward_kernel<<<row_grid(rows), kRowThreads, 0, stream>>>(
                                      count, offset, rows, bwd_count, perm, h, v, vpad, inv_t, sprime, targets_c, g_c,
                                      g_batch, idx, static_cast<const __nv_bfloat16*>(hidden_c),
                                      static_cast<const __nv_bfloat16*>(hidden_batch), row_scale, bwd_idx,
                                      static_cast<__nv_bfloat16*>(q), static_cast<__nv_bfloat16*>(hs))));
  return after_launch();
}

int scatter_rows_range(const void* src, int h, const int* bwd_idx, const int* bwd_count, long long rows, void* dst,
                       cudaStream_t stream) {
  if (rows <= 0) return A3PO_OK;
  A3PO_LAUNCH(kKKeptRows, stream, (scatter_rows_range_kernel<<<row_grid(rows), kRowThreads, 0, stream>>>(
                                      static_cast<const __nv_bfloat16*>(src), h, bwd_idx, bwd_count,
                                      static_cast<__nv_bfloat16*>(dst))));
  return after_launch();
}

int finish_batch_outputs(const int* pos, long long n, const float* logp_c, float* logp, const float* lse_c, float* lse,
                         const float* g_c, float* grad_logp, const float* ent_c, float* entropy, void* grad_hidden,
                         int h, cudaStream_t stream) {
  if (n <= 0) return A3PO_OK;
  const unsigned blocks = static_cast<unsigned>((n + kRowThreads - 1) / kRowThreads);
  A3PO_LAUNCH(kKKeptRows, stream, (finish_scalars_kernel<<<blocks, kRowThreads, 0, stream>>>(
                                      pos, n, logp_c, logp, lse_c, lse, g_c, grad_logp, ent_c, entropy)));
  A3PO_RETURN_IF(after_launch());
  if (grad_hidden) {
    A3PO_LAUNCH(kKKeptRows, stream, (zero_unkept_rows_kernel<<<row_grid(n), kRowThreads, 0, stream>>>(
                                        pos, g_c, n, h, static_cast<__nv_bfloat16*>(grad_hidden))));
    A3PO_RETURN_IF(after_launch());
  }
  return A3PO_OK;
}

}  // namespace a3po
