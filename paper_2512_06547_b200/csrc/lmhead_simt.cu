// LM-head log-prob forward/backward on the FP32 pipes (FFMA tiles, fp32 accumulate).
//
// This is the full-precision path: fp32 hidden/W (tcgen05 has no fp32 x fp32 kind, and tf32
// inputs cannot meet a 1e-5 tolerance), and bf16 shapes the tensor-core path does not take.
// Same data flow as the tensor-core path: logits exist only as 64x64 register tiles; the
// forward keeps an online (max, sum-exp) per row and writes per-split partials that the merge
// kernel combines; the backward materialises dz for a chunk of rows and runs two contractions.

#include "a3po_common.cuh"
#include "lmhead_internal.cuh"

namespace a3po {
namespace {

constexpr int kTile = 64;
constexpr int kBK = 16;
constexpr int kSimtThreads = 256;

// acc[i][j] = sum_k hidden[row0 + ty*4 + i, k] * w[col0 + tx*4 + j, k]   (rows/cols out of range read 0)
template <typename T>
__device__ __forceinline__ void logits_tile(const T* __restrict__ hidden, const T* __restrict__ w, long long row0,
                                            int col0, long long n, int h, int v, float (&acc)[4][4],
                                            float (&as)[kBK][kTile + 4], float (&bs)[kBK][kTile + 4]) {
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < h; k0 += kBK) {
#pragma unroll
    for (int e = tid; e < kTile * kBK; e += kSimtThreads) {
      const int r = e / kBK, k = e % kBK;
      const long long gr = row0 + r;
      const int gc = col0 + r;
      const int gk = k0 + k;
      as[k][r] = (gr < n && gk < h) ? to_float(hidden[gr * h + gk]) : 0.f;
      bs[k][r] = (gc < v && gk < h) ? to_float(w[static_cast<long long>(gc) * h + gk]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kBK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = as[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
}

__device__ __forceinline__ float group16_max(float x) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float group16_sum(float x) {
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// grid = (row tiles, vocab splits).  Each block sweeps its vocab tiles with an online softmax.
template <typename T, bool ENT>
__global__ void __launch_bounds__(kSimtThreads)
lmhead_fwd_simt_kernel(const T* __restrict__ hidden, const T* __restrict__ w, const int32_t* __restrict__ targets,
                       long long n, int h, int v, float inv_t, int tiles_per_split, int n_tiles,
                       SoftmaxPartial* __restrict__ part, float* __restrict__ part_ent, float* __restrict__ zy) {
  __shared__ float as[kBK][kTile + 4];
  __shared__ float bs[kBK][kTile + 4];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const long long row0 = static_cast<long long>(blockIdx.x) * kTile;
  const int split = blockIdx.y;
  float m_run[4], s_run[4], e_run[4];
  int y[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m_run[i] = -INFINITY; s_run[i] = 0.f; e_run[i] = 0.f;
    const long long r = row0 + ty * 4 + i;
    int t = (r < n) ? targets[r] : 0;
    y[i] = min(max(t, 0), v - 1);
  }
  const int tile_lo = split * tiles_per_split;
  const int tile_hi = min(tile_lo + tiles_per_split, n_tiles);
  for (int tile = tile_lo; tile < tile_hi; ++tile) {
    const int col0 = tile * kTile;
    float acc[4][4];
    logits_tile<T>(hidden, w, row0, col0, n, h, v, acc, as, bs);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float z[4];
      float tmax = -INFINITY;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int c = col0 + tx * 4 + j;
        z[j] = (c < v) ? acc[i][j] * inv_t : -INFINITY;
        tmax = fmaxf(tmax, z[j]);
        if (c == y[i]) {
          const long long r = row0 + ty * 4 + i;
          if (r < n) zy[r] = z[j];
        }
      }
      tmax = group16_max(tmax);
      const float m_new = fmaxf(m_run[i], tmax);  // finite: every tile has at least one valid column
      float ssum = 0.f, esum = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float p = expf(z[j] - m_new);  // exp(-inf) = 0 for columns past V
        ssum += p;
        if (ENT) esum += (p > 0.f) ? p * z[j] : 0.f;
      }
      ssum = group16_sum(ssum);
      const float scale = expf(m_run[i] - m_new);  // 0 on the first tile
      s_run[i] = s_run[i] * scale + ssum;
      if (ENT) e_run[i] = e_run[i] * scale + group16_sum(esum);
      m_run[i] = m_new;
    }
  }
  if (tx == 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const long long r = row0 + ty * 4 + i;
      if (r < n) {
        part[static_cast<long long>(split) * n + r] = SoftmaxPartial{m_run[i], s_run[i]};
        if (ENT) part_ent[static_cast<long long>(split) * n + r] = e_run[i];
      }
    }
  }
}

// dz tile for rows [row_begin, row_begin + nc): ds[(r - row_begin) * v + c] (fp32).
template <typename T>
__global__ void __launch_bounds__(kSimtThreads)
lmhead_dz_simt_kernel(const T* __restrict__ hidden, const T* __restrict__ w, const int32_t* __restrict__ targets,
                      const float* __restrict__ lse, const float* __restrict__ grad_logp, long long row_begin,
                      long long row_end, int h, int v, float inv_t, float* __restrict__ ds) {
  __shared__ float as[kBK][kTile + 4];
  __shared__ float bs[kBK][kTile + 4];
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  const long long row0 = row_begin + static_cast<long long>(blockIdx.x) * kTile;
  const int col0 = blockIdx.y * kTile;
  float acc[4][4];
  logits_tile<T>(hidden, w, row0, col0, row_end, h, v, acc, as, bs);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long r = row0 + ty * 4 + i;
    if (r >= row_end) continue;
    const float g = grad_logp[r];
    const float l = lse[r];
    const int y = min(max(targets[r], 0), v - 1);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int c = col0 + tx * 4 + j;
      if (c < v) {
        const float p = expf(acc[i][j] * inv_t - l);
        const float dz = (g == 0.f) ? 0.f : g * ((c == y ? 1.f : 0.f) - p) * inv_t;
        ds[(r - row_begin) * v + c] = dz;
      }
    }
  }
}

// C[m, n] (+)= sum_k A(m, k) * B(k, n);  A(m,k) = a[m*a_rs + k*a_cs],  B(k,n) = b[k*b_rs + n]  (n contiguous)
template <typename TA, typename TB, typename TC, bool A_K_CONTIG>
__global__ void __launch_bounds__(kSimtThreads)
gemm_simt_kernel(const TA* __restrict__ a, long long a_rs, long long a_cs, const TB* __restrict__ b, long long b_rs,
                 TC* __restrict__ c, long long c_rs, long long m_dim, int n_dim, long long k_dim, int accumulate) {
  __shared__ float as[kBK][kTile + 4];
  __shared__ float bs[kBK][kTile + 4];
  const int tid = threadIdx.x, tx = tid % 16, ty = tid / 16;
  const long long m0 = static_cast<long long>(blockIdx.x) * kTile;
  const int n0 = blockIdx.y * kTile;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  for (long long k0 = 0; k0 < k_dim; k0 += kBK) {
#pragma unroll
    for (int e = tid; e < kTile * kBK; e += kSimtThreads) {
      int r, k;
      if (A_K_CONTIG) { r = e / kBK; k = e % kBK; } else { k = e / kTile; r = e % kTile; }
      const long long gm = m0 + r, gk = k0 + k;
      as[k][r] = (gm < m_dim && gk < k_dim) ? to_float(a[gm * a_rs + gk * a_cs]) : 0.f;
      const int kb = e / kTile, nb = e % kTile;
      const long long gkb = k0 + kb;
      const int gn = n0 + nb;
      bs[kb][nb] = (gkb < k_dim && gn < n_dim) ? to_float(b[gkb * b_rs + gn]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kBK; ++k) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = as[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long gm = m0 + ty * 4 + i;
    if (gm >= m_dim) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gn = n0 + tx * 4 + j;
      if (gn >= n_dim) continue;
      TC* dst = c + gm * c_rs + gn;
      float val = acc[i][j];
      if (accumulate) val += to_float(*dst);
      *dst = from_float<TC>(val);
    }
  }
}

template <typename T>
int fwd_impl(const T* hidden, const T* w, const int32_t* targets, long long n, int h, int v, float inv_t,
             int splits, SoftmaxPartial* part, float* part_ent, float* zy, cudaStream_t stream) {
  const int n_tiles = (v + kTile - 1) / kTile;
  const int tiles_per_split = (n_tiles + splits - 1) / splits;
  dim3 grid(static_cast<unsigned>((n + kTile - 1) / kTile), static_cast<unsigned>(splits));
  if (part_ent)
    A3PO_LAUNCH(kKSimtFwd, stream, (lmhead_fwd_simt_kernel<T, true><<<grid, kSimtThreads, 0, stream>>>(
                                       hidden, w, targets, n, h, v, inv_t, tiles_per_split, n_tiles, part, part_ent, zy)));
  else
    A3PO_LAUNCH(kKSimtFwd, stream, (lmhead_fwd_simt_kernel<T, false><<<grid, kSimtThreads, 0, stream>>>(
                                       hidden, w, targets, n, h, v, inv_t, tiles_per_split, n_tiles, part, nullptr, zy)));
  return after_launch();
}

template <typename T>
int bwd_impl(const T* hidden, const T* w, const int32_t* targets, const float* lse, const float* grad_logp,
             long long n, int h, int v, float inv_t, T* grad_hidden, float* grad_w, int accumulate,
             float* ds, long long chunk_rows, cudaStream_t stream) {
  const unsigned vt = static_cast<unsigned>((v + kTile - 1) / kTile);
  const unsigned ht = static_cast<unsigned>((h + kTile - 1) / kTile);
  if (n == 0 && !accumulate) {
    if (cudaMemsetAsync(grad_w, 0, sizeof(float) * static_cast<size_t>(v) * h, stream) != cudaSuccess)
      return A3PO_ERR_CUDA;
    return A3PO_OK;
  }
  for (long long r0 = 0; r0 < n; r0 += chunk_rows) {
    const long long r1 = (r0 + chunk_rows < n) ? r0 + chunk_rows : n;
    const long long nc = r1 - r0;
    const unsigned rt = static_cast<unsigned>((nc + kTile - 1) / kTile);
    A3PO_LAUNCH(kKSimtDz, stream, (lmhead_dz_simt_kernel<T><<<dim3(rt, vt), kSimtThreads, 0, stream>>>(
                                      hidden, w, targets, lse, grad_logp, r0, r1, h, v, inv_t, ds)));
    A3PO_RETURN_IF(after_launch());
    // grad_hidden[r0:r1, :] = dz @ W
    A3PO_LAUNCH(kKSimtGemm, stream, (gemm_simt_kernel<float, T, T, true><<<dim3(rt, ht), kSimtThreads, 0, stream>>>(
                                        ds, v, 1, w, h, grad_hidden + r0 * h, h, nc, h, v, 0)));
    A3PO_RETURN_IF(after_launch());
    // grad_w (+)= dz^T @ hidden[r0:r1, :]
    A3PO_LAUNCH(kKSimtGemm, stream,
                (gemm_simt_kernel<float, T, float, false><<<dim3(vt, ht), kSimtThreads, 0, stream>>>(
                    ds, 1, v, hidden + r0 * h, h, grad_w, h, v, h, nc, (accumulate || r0 > 0) ? 1 : 0)));
    A3PO_RETURN_IF(after_launch());
  }
  return A3PO_OK;
}

}  // namespace

int lmhead_fwd_simt(const void* hidden, const void* w, const int32_t* targets, long long n, int h, int v,
                    a3po_dtype dt, float inv_t, int splits, SoftmaxPartial* part, float* part_ent, float* zy,
                    cudaStream_t stream) {
  if (dt == A3PO_F32)
    return fwd_impl<float>(static_cast<const float*>(hidden), static_cast<const float*>(w), targets, n, h, v, inv_t,
                           splits, part, part_ent, zy, stream);
  return fwd_impl<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(hidden), static_cast<const __nv_bfloat16*>(w),
                                 targets, n, h, v, inv_t, splits, part, part_ent, zy, stream);
}

int lmhead_bwd_simt(const void* hidden, const void* w, const int32_t* targets, const float* lse,
                    const float* grad_logp, long long n, int h, int v, a3po_dtype dt, float inv_t, void* grad_hidden,
                    float* grad_w, int accumulate, float* ds, long long chunk_rows, cudaStream_t stream) {
  if (dt == A3PO_F32)
    return bwd_impl<float>(static_cast<const float*>(hidden), static_cast<const float*>(w), targets, lse, grad_logp, n,
                           h, v, inv_t, static_cast<float*>(grad_hidden), grad_w, accumulate, ds, chunk_rows, stream);
  return bwd_impl<__nv_bfloat16>(static_cast<const __nv_bfloat16*>(hidden), static_cast<const __nv_bfloat16*>(w),
                                 targets, lse, grad_logp, n, h, v, inv_t, static_cast<__nv_bfloat16*>(grad_hidden),
                                 grad_w, accumulate, ds, chunk_rows, stream);
}

}  // namespace a3po
