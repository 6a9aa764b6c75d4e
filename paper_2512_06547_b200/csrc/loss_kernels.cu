// A-3PO decoupled clipped loss: forward, backward and one-pass forward+backward.
//
// Eq. 2 (decoupled clipped objective) with the proximal anchor of Eq. 3 and the staleness
// coefficient of Eq. 4.  The path is a pure HBM stream: 17 bytes read per token (two fp32
// log-probs, an int32 version, an fp32 advantage, a uint8 mask) and, for the backward, 4 bytes
// written.  Each thread handles groups of four consecutive tokens with 128-bit loads (32-bit for
// the mask), two groups in flight per iteration; reductions go thread -> warp shuffle -> block
// -> per-block partial -> one finalising block, in a fixed order, so results do not change from
// run to run.
//
// An ABI call is ONE launch where the device allows it: the kernel is launched cooperatively and
// runs up to three phases separated by grid-wide barriers: count the mask (when the backward needs
// M and no forward statistics supply it), stream the tokens, and let block 0 sum the block
// partials in index order.  Where a cooperative launch is not possible (or not wanted: the
// static-scratch entry) the same phases run as separate launches.

#include <cooperative_groups.h>

#include <mutex>

#include "a3po_common.cuh"
#include "lmhead_internal.cuh"

namespace a3po {
namespace {

namespace cg = cooperative_groups;

constexpr int kLossThreads = 256;
constexpr int kBlocksPerSm = 4;   // resident blocks per SM at <= 64 registers per thread
constexpr int kMaxLossBlocks = 4096;

struct alignas(16) LossPartial {
  double sum;
  long long n_valid;
  long long n_clipped;
  float iw_max;
  float iw_min;
};

struct LossArgs {
  const float* logp;
  const float* behav;
  const int32_t* versions;  // per token (interpolated anchor)
  const float* prox;        // explicit proximal log-probs (EXPLICIT kernels), else unused
  const float* adv;
  const uint8_t* mask;
  long long n;
  int32_t current_version;
  float lo;  // 1 - eps
  float hi;  // 1 + eps
  int detach;
  const float* grad_loss;        // device scalar or null
  const long long* n_valid_ptr;  // device: M, for the backward coefficient
  float* grad_logp;
};

// Phases a cooperative launch of loss_kernel runs besides the token stream.
enum : int { kPhaseCountMask = 1, kPhaseFinalize = 2 };
struct LossPhases {
  int bits;
  long long* block_counts;  // kPhaseCountMask: per-block mask counts, then M in n_valid
  long long* n_valid;
  float* loss;              // kPhaseFinalize outputs
  a3po_stats* stats;
};

enum : int { kFwd = 0, kBwd = 1, kFwdBwd = 2 };

struct Acc {
  double sum = 0.0;
  int n_valid = 0;
  int n_clipped = 0;
  float iw_max = 0.f;      // valid tokens have iw > 0
  float iw_min = 3.4e38f;
};

// One token of Eq. 2-4.  iw and r are evaluated through the closed form of the theorem
// (r = w^alpha, iw = w^(1-alpha), w = exp(l_theta - l_behav)): the same function as the literal
// interpolation of Eq. 3 but conditioned on the small difference of the two log-probs.
// Staleness is exact for any pair of int32 versions: a signed compare decides d >= 1 and the
// unsigned difference is d itself in that case; d = 1 takes alpha = 1 without a reciprocal.
// EXPLICIT: the anchor is given (`ver` then carries the bits of log pi_prox), Eq. 2 as it stands:
// iw = exp(l_prox - l_behav), r = exp(l_theta - l_prox); the anchor is a constant in the backward.
template <int MODE, bool EXPLICIT>
__device__ __forceinline__ void token(float lt, float lb, int ver, float a, bool valid,
                                      const LossArgs& p, float coef, float& fsum, Acc& acc,
                                      float& grad) {
  float alpha = 1.0f, r, iw;
  if (EXPLICIT) {
    const float lp = __int_as_float(ver);
    r = fast_exp2((lt - lp) * kLog2e);
    iw = fast_exp2((lp - lb) * kLog2e);
  } else {
    const unsigned du = static_cast<unsigned>(p.current_version) - static_cast<unsigned>(ver);
    const bool interpolate = (ver < p.current_version) && (du > 1u);
    alpha = interpolate ? fast_rcp(static_cast<float>(du)) : 1.0f;
    const float d2 = (lt - lb) * kLog2e;
    const float ad2 = alpha * d2;
    r = fast_exp2(ad2);
    iw = fast_exp2(d2 - ad2);
  }
  const float s1 = r * a;
  const float s2 = fminf(fmaxf(r, p.lo), p.hi) * a;
  const bool act = s1 <= s2;
  const float obj = iw * fminf(s1, s2);
  if (MODE != kBwd) {
    fsum += valid ? obj : 0.f;
    acc.n_clipped += (valid && !act) ? 1 : 0;
    acc.iw_max = fmaxf(acc.iw_max, valid ? iw : 0.f);
    acc.iw_min = fminf(acc.iw_min, valid ? iw : 3.4e38f);
  }
  if (MODE != kFwd) {
    const float through = act ? iw * s1 : 0.f;
    const float dobj = (EXPLICIT || p.detach) ? through : fmaf(alpha, through - obj, obj);  // (1-a)*obj + a*through
    grad = valid ? coef * dobj : 0.f;
  }
}

template <int MODE, bool EXPLICIT>
__device__ __forceinline__ void group4(long long g, const LossArgs& p, float coef, Acc& acc) {
  const float4 lt = __ldcs(reinterpret_cast<const float4*>(p.logp) + g);
  const float4 lb = __ldcs(reinterpret_cast<const float4*>(p.behav) + g);
  const int4 ver = __ldcs(reinterpret_cast<const int4*>(EXPLICIT ? static_cast<const void*>(p.prox)
                                                                  : static_cast<const void*>(p.versions)) + g);
  const float4 a = __ldcs(reinterpret_cast<const float4*>(p.adv) + g);
  const unsigned m = __vcmpne4(__ldcs(reinterpret_cast<const unsigned*>(p.mask) + g), 0u);  // 0xff per valid token
  float fsum = 0.f;
  float4 gr;
  token<MODE, EXPLICIT>(lt.x, lb.x, ver.x, a.x, (m & 0x000000ffu) != 0, p, coef, fsum, acc, gr.x);
  token<MODE, EXPLICIT>(lt.y, lb.y, ver.y, a.y, (m & 0x0000ff00u) != 0, p, coef, fsum, acc, gr.y);
  token<MODE, EXPLICIT>(lt.z, lb.z, ver.z, a.z, (m & 0x00ff0000u) != 0, p, coef, fsum, acc, gr.z);
  token<MODE, EXPLICIT>(lt.w, lb.w, ver.w, a.w, (m & 0xff000000u) != 0, p, coef, fsum, acc, gr.w);
  if (MODE != kBwd) {
    acc.sum += static_cast<double>(fsum);
    acc.n_valid += __popc(m) >> 3;
  }
  if (MODE != kFwd) __stcs(reinterpret_cast<float4*>(p.grad_logp) + g, gr);
}

template <int MODE, bool EXPLICIT>
__device__ __forceinline__ void single(long long t, const LossArgs& p, float coef, Acc& acc) {
  float fsum = 0.f, gr = 0.f;
  const bool valid = p.mask[t] != 0;
  const int third = EXPLICIT ? __float_as_int(p.prox[t]) : p.versions[t];
  token<MODE, EXPLICIT>(p.logp[t], p.behav[t], third, p.adv[t], valid, p, coef, fsum, acc, gr);
  if (MODE != kBwd) {
    acc.sum += static_cast<double>(fsum);
    acc.n_valid += valid ? 1 : 0;
  }
  if (MODE != kFwd) p.grad_logp[t] = gr;
}

// Sums `count` per-block partials in a fixed order (every thread a strided subsequence, then a
// shared-memory tree): loss = -sum / max(M,1), plus the diagnostics.  Called by one whole block.
__device__ __forceinline__ void finalize_block(const LossPartial* partials, int count, float* loss,
                                               a3po_stats* stats, LossPartial* sh /*[kLossThreads]*/) {
  LossPartial mine{0.0, 0, 0, 0.f, 3.4e38f};
  for (int i = threadIdx.x; i < count; i += kLossThreads) {
    const uint4 lo = __ldcg(reinterpret_cast<const uint4*>(partials + i));       // written by other blocks
    const uint4 hi = __ldcg(reinterpret_cast<const uint4*>(partials + i) + 1);
    LossPartial q;
    memcpy(&q, &lo, 16);
    memcpy(reinterpret_cast<char*>(&q) + 16, &hi, 16);
    mine.sum += q.sum;
    mine.n_valid += q.n_valid;
    mine.n_clipped += q.n_clipped;
    mine.iw_max = fmaxf(mine.iw_max, q.iw_max);
    mine.iw_min = fminf(mine.iw_min, q.iw_min);
  }
  sh[threadIdx.x] = mine;
  __syncthreads();
  for (int s = kLossThreads / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) {
      sh[threadIdx.x].sum += sh[threadIdx.x + s].sum;
      sh[threadIdx.x].n_valid += sh[threadIdx.x + s].n_valid;
      sh[threadIdx.x].n_clipped += sh[threadIdx.x + s].n_clipped;
      sh[threadIdx.x].iw_max = fmaxf(sh[threadIdx.x].iw_max, sh[threadIdx.x + s].iw_max);
      sh[threadIdx.x].iw_min = fminf(sh[threadIdx.x].iw_min, sh[threadIdx.x + s].iw_min);
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const LossPartial t = sh[0];
    const long long m = t.n_valid;
    *loss = static_cast<float>(-t.sum / static_cast<double>(m > 0 ? m : 1));
    if (stats) {
      stats->n_valid = m;
      stats->n_clipped = t.n_clipped;
      stats->iw_max = m > 0 ? t.iw_max : 0.f;
      stats->iw_min = m > 0 ? t.iw_min : 0.f;
    }
  }
}

// This block's share of M = number of non-zero mask bytes (16 mask bytes per load where alignment
// allows, four loads in flight per thread); the block total goes to block_counts[blockIdx.x].
__device__ __forceinline__ int popc16(const uint4 m) {
  return (__popc(__vcmpne4(m.x, 0u)) + __popc(__vcmpne4(m.y, 0u)) + __popc(__vcmpne4(m.z, 0u)) +
          __popc(__vcmpne4(m.w, 0u))) >> 3;
}
__device__ __forceinline__ void count_mask_block(const uint8_t* mask, long long n, long long* block_counts,
                                                 long long* sh /*[kLossThreads / kWarp]*/) {
  long long count = 0;
  const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
  const bool vec = (reinterpret_cast<uintptr_t>(mask) & 15) == 0;
  long long done = 0;
  if (vec) {
    const long long groups = n >> 4;
    const uint4* m16 = reinterpret_cast<const uint4*>(mask);
    long long g = tid;
    for (; g + 3 * nthreads < groups; g += 4 * nthreads) {
      const uint4 a = __ldg(m16 + g), b = __ldg(m16 + g + nthreads), c = __ldg(m16 + g + 2 * nthreads),
                  d = __ldg(m16 + g + 3 * nthreads);
      count += popc16(a) + popc16(b) + popc16(c) + popc16(d);
    }
    for (; g < groups; g += nthreads) count += popc16(__ldg(m16 + g));
    done = groups << 4;
  }
  for (long long t = done + tid; t < n; t += nthreads) count += mask[t] != 0;
  count = warp_sum(count);
  if (threadIdx.x % kWarp == 0) sh[threadIdx.x / kWarp] = count;
  __syncthreads();
  if (threadIdx.x == 0) {
    long long total = 0;
    for (int w = 0; w < kLossThreads / kWarp; ++w) total += sh[w];
    block_counts[blockIdx.x] = total;
  }
}

// Sum of `count` block counts in a fixed order; called by one whole block.
__device__ __forceinline__ void sum_counts_block(const long long* block_counts, int count, long long* out,
                                                 long long* sh /*[kLossThreads]*/) {
  long long mine = 0;
  for (int i = threadIdx.x; i < count; i += kLossThreads) mine += __ldcg(block_counts + i);  // written by other blocks
  sh[threadIdx.x] = mine;
  __syncthreads();
  for (int s = kLossThreads / 2; s > 0; s >>= 1) {
    if (threadIdx.x < s) sh[threadIdx.x] += sh[threadIdx.x + s];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = sh[0];
}

// VEC = true needs 16-byte aligned fp32/int32 arrays and a 4-byte aligned mask.
// ph.bits != 0 only in a cooperative launch (the grid-wide barriers are legal there and nowhere else).
template <int MODE, bool VEC, bool EXPLICIT>
__global__ void __launch_bounds__(kLossThreads, kBlocksPerSm) loss_kernel(LossArgs p, LossPartial* partials,
                                                                          LossPhases ph) {
  __shared__ LossPartial sh[kLossThreads];
  __shared__ long long s_m;
  if (ph.bits & kPhaseCountMask) {
    // every block counts its share, then (one grid-wide barrier later) adds up all the shares itself, in index
    // order: the same M in every block without a second barrier
    long long* shc = reinterpret_cast<long long*>(sh);
    count_mask_block(p.mask, p.n, ph.block_counts, shc);
    cg::this_grid().sync();
    sum_counts_block(ph.block_counts, gridDim.x, &s_m, shc);
    __syncthreads();
    if (blockIdx.x == 0 && threadIdx.x == 0) *ph.n_valid = s_m;
  }
  float coef = 0.f;
  if (MODE != kFwd) {
    long long m = (ph.bits & kPhaseCountMask) ? s_m : *p.n_valid_ptr;
    float gl = p.grad_loss ? *p.grad_loss : 1.0f;
    coef = (m > 0) ? -gl / static_cast<float>(m) : 0.f;
  }
  Acc acc;
  const long long tid = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  const long long nthreads = static_cast<long long>(gridDim.x) * blockDim.x;
  if (VEC) {
    const long long groups = p.n >> 2;
    long long g = tid;
    for (; g + nthreads < groups; g += 2 * nthreads) {
      group4<MODE, EXPLICIT>(g, p, coef, acc);
      group4<MODE, EXPLICIT>(g + nthreads, p, coef, acc);
    }
    if (g < groups) group4<MODE, EXPLICIT>(g, p, coef, acc);
    const long long t = (groups << 2) + tid;  // ragged tail: at most three tokens
    if (t < p.n) single<MODE, EXPLICIT>(t, p, coef, acc);
  } else {
    for (long long t = tid; t < p.n; t += nthreads) single<MODE, EXPLICIT>(t, p, coef, acc);
  }
  if (MODE == kBwd) return;

  double sum = warp_sum(acc.sum);
  long long nv = warp_sum(static_cast<long long>(acc.n_valid));
  long long nc = warp_sum(static_cast<long long>(acc.n_clipped));
  float mx = warp_max(acc.iw_max);
  float mn = warp_min(acc.iw_min);
  const int lane = threadIdx.x % kWarp, warp = threadIdx.x / kWarp;
  __syncthreads();   // the count phase may have used the shared array
  if (lane == 0) sh[warp] = LossPartial{sum, nv, nc, mx, mn};
  __syncthreads();
  if (threadIdx.x == 0) {
    LossPartial out = sh[0];
    for (int w = 1; w < kLossThreads / kWarp; ++w) {
      out.sum += sh[w].sum;
      out.n_valid += sh[w].n_valid;
      out.n_clipped += sh[w].n_clipped;
      out.iw_max = fmaxf(out.iw_max, sh[w].iw_max);
      out.iw_min = fminf(out.iw_min, sh[w].iw_min);
    }
    partials[blockIdx.x] = out;
  }
  if (ph.bits & kPhaseFinalize) {
    cg::this_grid().sync();
    if (blockIdx.x == 0) finalize_block(partials, gridDim.x, ph.loss, ph.stats, sh);
  }
}

// The same phases as separate launches.
__global__ void __launch_bounds__(kLossThreads) loss_finalize_kernel(const LossPartial* partials,
                                                                    int count, float* loss,
                                                                    a3po_stats* stats) {
  __shared__ LossPartial sh[kLossThreads];
  finalize_block(partials, count, loss, stats, sh);
}

__global__ void __launch_bounds__(kLossThreads) mask_count_kernel(const uint8_t* mask, long long n,
                                                                 long long* block_counts) {
  __shared__ long long sh[kLossThreads / kWarp];
  count_mask_block(mask, n, block_counts, sh);
}

__global__ void __launch_bounds__(kLossThreads) mask_count_finalize_kernel(const long long* block_counts,
                                                                          int count, long long* out) {
  __shared__ long long sh[kLossThreads];
  sum_counts_block(block_counts, count, out, sh);
}

// Data-parallel mean: a shard with M_r valid tokens out of M in the whole job weighs M_r / M.
__global__ void dp_scale_kernel(const long long* m_local, const long long* m_global, const float* loss_local,
                                float* scale, float* weighted_loss) {
  const long long m = *m_global;
  const float sc = m > 0 ? static_cast<float>(static_cast<double>(*m_local) / static_cast<double>(m)) : 0.f;
  *scale = sc;
  if (loss_local) *weighted_loss = sc * *loss_local;
}

// versions given per sequence: write the per-token array the streaming kernels read.
__global__ void __launch_bounds__(kLossThreads) expand_versions_kernel(const int32_t* per_seq,
                                                                      const int32_t* cu_seqlens, int b,
                                                                      long long n, int32_t* per_token) {
  const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= n) return;
  int lo = 0, hi = b;  // find the last sequence whose start is <= t
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (static_cast<long long>(cu_seqlens[mid]) <= t) lo = mid; else hi = mid;
  }
  per_token[t] = per_seq[lo];
}

struct LossWs {
  LossPartial* partials;
  long long* block_counts;
  long long* n_valid;
  int32_t* versions;
};

size_t loss_ws_bytes(long long n) {
  return round_up(sizeof(LossPartial) * kMaxLossBlocks, 256) + round_up(sizeof(long long) * kMaxLossBlocks, 256) +
         256 + round_up(sizeof(int32_t) * static_cast<size_t>(n > 0 ? n : 0), 256) + 256;
}

int grid_for(long long n_items, int max_blocks = kMaxLossBlocks) {
  long long want = (n_items + kLossThreads - 1) / kLossThreads;
  long long cap = static_cast<long long>(sm_count()) * kBlocksPerSm;
  if (cap > max_blocks) cap = max_blocks;
  if (want > cap) want = cap;
  if (want < 1) want = 1;
  return static_cast<int>(want);
}

using LossKernel = void (*)(LossArgs, LossPartial*, LossPhases);

LossKernel pick_kernel(int mode, bool vec, bool explicit_anchor) {
#define A3PO_PICK(MODE)                                                                  \
  (explicit_anchor ? (vec ? loss_kernel<MODE, true, true> : loss_kernel<MODE, false, true>) \
                   : (vec ? loss_kernel<MODE, true, false> : loss_kernel<MODE, false, false>))
  if (mode == kFwd) return A3PO_PICK(kFwd);
  if (mode == kBwd) return A3PO_PICK(kBwd);
  return A3PO_PICK(kFwdBwd);
#undef A3PO_PICK
}

// Largest grid of `kernel` whose blocks are all resident at once on the current device (what a
// cooperative launch requires); 0 if the device cannot launch cooperatively.
int cooperative_capacity(LossKernel kernel) {
  int dev = -1, coop = 0, per_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kLossThreads, 0) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return per_sm * sm_count();
}

int kernel_id_of(int mode) { return mode == kFwd ? kKLossFwd : (mode == kBwd ? kKLossBwd : kKLossFwdBwd); }

// allow_single_launch = false keeps every phase in its own plain launch.
int run_loss(int mode, const float* logp, const float* behav, const float* prox, const int32_t* versions,
             int versions_per_seq,
             const int32_t* cu_seqlens, int b, int32_t current_version, const float* adv, const uint8_t* mask,
             long long n, float clip_eps, int detach, const float* grad_loss, const a3po_stats* fwd_stats,
             float* loss, a3po_stats* stats, float* grad_logp, void* ws, size_t ws_bytes, void* stream_,
             bool allow_single_launch = true) {
  if (n < 0 || !(clip_eps >= 0.f)) return A3PO_ERR_INVALID_ARG;
  if (n > 0 && (!logp || !behav || (!versions && !prox) || !adv || !mask)) return A3PO_ERR_INVALID_ARG;
  if (mode != kBwd && !loss) return A3PO_ERR_INVALID_ARG;
  if (mode != kFwd && n > 0 && !grad_logp) return A3PO_ERR_INVALID_ARG;
  if (!prox && versions_per_seq && n > 0 && (!cu_seqlens || b <= 0)) return A3PO_ERR_INVALID_ARG;
  if (!ws || !aligned_to(ws, 256) || ws_bytes < loss_ws_bytes(n)) return A3PO_ERR_WORKSPACE;
  if (!aligned_to(logp, 4) || !aligned_to(behav, 4) || !aligned_to(versions, 4) || !aligned_to(prox, 4) ||
      !aligned_to(adv, 4) ||
      !aligned_to(grad_logp, 4))
    return A3PO_ERR_UNSUPPORTED;
  if (sm_count() <= 0) return A3PO_ERR_NO_DEVICE;
  cudaStream_t stream = as_stream(stream_);

  Arena arena(ws, ws_bytes);
  LossWs w;
  w.partials = arena.take<LossPartial>(kMaxLossBlocks);
  w.block_counts = arena.take<long long>(kMaxLossBlocks);
  w.n_valid = arena.take<long long>(1);
  w.versions = arena.take<int32_t>(static_cast<size_t>(n));
  if (!arena.ok()) return A3PO_ERR_WORKSPACE;

  if (!prox && versions_per_seq && n > 0) {
    const int blocks = static_cast<int>((n + kLossThreads - 1) / kLossThreads);
    A3PO_LAUNCH(kKExpandVersions, stream,
                expand_versions_kernel<<<blocks, kLossThreads, 0, stream>>>(versions, cu_seqlens, b, n, w.versions));
    A3PO_RETURN_IF(after_launch());
    versions = w.versions;
  }

  LossArgs p;
  p.logp = logp; p.behav = behav; p.versions = versions; p.prox = prox; p.adv = adv; p.mask = mask; p.n = n;
  p.current_version = current_version;
  p.lo = 1.0f - clip_eps; p.hi = 1.0f + clip_eps;
  p.detach = detach;
  p.grad_loss = grad_loss;
  p.grad_logp = grad_logp;
  p.n_valid_ptr = nullptr;
  const bool need_count = mode != kFwd && !fwd_stats;
  if (mode != kFwd) p.n_valid_ptr = fwd_stats ? reinterpret_cast<const long long*>(&fwd_stats->n_valid) : w.n_valid;

  const bool vec = aligned_to(logp, 16) && aligned_to(behav, 16) && aligned_to(versions, 16) && aligned_to(prox, 16) &&
                   aligned_to(adv, 16) && aligned_to(mask, 4) && (mode == kFwd || aligned_to(grad_logp, 16));
  LossKernel kernel = pick_kernel(mode, vec, prox != nullptr);
  int blocks = grid_for(vec ? (n + 7) / 8 : n);
  LossPhases ph{0, w.block_counts, w.n_valid, loss, stats};
  if (need_count) ph.bits |= kPhaseCountMask;
  if (mode != kBwd) ph.bits |= kPhaseFinalize;

  // ---- one cooperative launch: [count the mask] -> stream -> [sum the partials]
  if (ph.bits != 0 && allow_single_launch) {
    const int cap = cooperative_capacity(kernel);
    if (cap >= 1) {
      if (blocks > cap) blocks = cap;
      void* kargs[] = {&p, &w.partials, &ph};
      cudaError_t err;
      {
        ProfileScope scope(kernel_id_of(mode), stream);
        err = cudaLaunchCooperativeKernel(reinterpret_cast<void*>(kernel), dim3(blocks), dim3(kLossThreads), kargs, 0,
                                          stream);
      }
      if (err == cudaSuccess) return after_launch();
      cudaGetLastError();  // not launchable this way here: fall through to the separate launches
      blocks = grid_for(vec ? (n + 7) / 8 : n);
    }
  }

  // ---- the same phases as separate launches
  if (need_count) {
    const int cb = grid_for((n + 15) / 16);
    A3PO_LAUNCH(kKMaskCount, stream, mask_count_kernel<<<cb, kLossThreads, 0, stream>>>(mask, n, w.block_counts));
    A3PO_RETURN_IF(after_launch());
    A3PO_LAUNCH(kKMaskCountFinalize, stream,
                mask_count_finalize_kernel<<<1, kLossThreads, 0, stream>>>(w.block_counts, cb, w.n_valid));
    A3PO_RETURN_IF(after_launch());
  }
  ph.bits = 0;
  A3PO_LAUNCH(kernel_id_of(mode), stream, (kernel<<<blocks, kLossThreads, 0, stream>>>(p, w.partials, ph)));
  A3PO_RETURN_IF(after_launch());
  if (mode != kBwd) {
    A3PO_LAUNCH(kKLossFinalize, stream,
                loss_finalize_kernel<<<1, kLossThreads, 0, stream>>>(w.partials, blocks, loss, stats));
    A3PO_RETURN_IF(after_launch());
  }
  return A3PO_OK;
}

}  // namespace

// ---- loss on a slice of tokens with M known, partials kept for a later finalize (row-chunked step)
size_t loss_partial_bytes() { return sizeof(LossPartial); }
int loss_max_partials() { return kMaxLossBlocks; }
int loss_blocks_for(long long n, int max_blocks) { return grid_for((n + 7) / 8, max_blocks); }

int loss_fwd_bwd_slice(const float* logp, const float* behav, const int32_t* versions, const float* adv,
                       const uint8_t* mask, long long n, int32_t current_version, float clip_eps,
                       const long long* n_valid, const float* grad_loss, float* grad_logp, void* partials, int blocks,
                       cudaStream_t stream) {
  LossArgs p;
  p.logp = logp; p.behav = behav; p.versions = versions; p.prox = nullptr; p.adv = adv; p.mask = mask; p.n = n;
  p.current_version = current_version;
  p.lo = 1.0f - clip_eps; p.hi = 1.0f + clip_eps;
  p.detach = 1;
  p.grad_loss = grad_loss;
  p.grad_logp = grad_logp;
  p.n_valid_ptr = n_valid;
  const bool vec = aligned_to(logp, 16) && aligned_to(behav, 16) && aligned_to(versions, 16) && aligned_to(adv, 16) &&
                   aligned_to(mask, 4) && aligned_to(grad_logp, 16);
  LossKernel kernel = pick_kernel(kFwdBwd, vec, false);
  LossPhases ph{0, nullptr, nullptr, nullptr, nullptr};
  A3PO_LAUNCH(kKLossFwdBwd, stream, (kernel<<<blocks, kLossThreads, 0, stream>>>(
                                        p, static_cast<LossPartial*>(partials), ph)));
  return after_launch();
}

int loss_finalize_partials(const void* partials, int count, float* loss, a3po_stats* stats, cudaStream_t stream) {
  A3PO_LAUNCH(kKLossFinalize, stream, loss_finalize_kernel<<<1, kLossThreads, 0, stream>>>(
                                          static_cast<const LossPartial*>(partials), count, loss, stats));
  return after_launch();
}

}  // namespace a3po

extern "C" {

size_t a3po_loss_workspace_bytes(int64_t N) { return a3po::loss_ws_bytes(N); }

int a3po_loss_fwd(const float* logp, const float* behav_logp, const int32_t* versions, int versions_per_seq,
                  const int32_t* cu_seqlens, int B, int32_t current_version, const float* adv,
                  const uint8_t* mask, int64_t N, float clip_eps, float* loss, a3po_stats* stats, void* ws,
                  size_t ws_bytes, void* stream) {
  return a3po::run_loss(a3po::kFwd, logp, behav_logp, nullptr, versions, versions_per_seq, cu_seqlens, B, current_version,
                        adv, mask, N, clip_eps, 1, nullptr, nullptr, loss, stats, nullptr, ws, ws_bytes, stream);
}

}  // extern "C"

// ---------------------------------------------------------------------------------------------------
// Loss forward without a caller workspace: the scratch lives in this library's device image.
// ---------------------------------------------------------------------------------------------------
namespace a3po {
namespace {

constexpr size_t static_round(size_t x) { return (x + 255) / 256 * 256; }
// Same layout as loss_ws_bytes(A3PO_LOSS_FWD_STATIC_MAX_TOKENS): block partials, block counts, M,
// expanded per-token versions (checked against loss_ws_bytes at run time).
constexpr size_t kStaticScratchBytes =
    static_round(sizeof(LossPartial) * kMaxLossBlocks) + static_round(sizeof(long long) * kMaxLossBlocks) + 256 +
    static_round(sizeof(int32_t) * static_cast<size_t>(A3PO_LOSS_FWD_STATIC_MAX_TOKENS)) + 256;

// One copy per GPU that loads the library, resident until the process exits.  In host code this
// name is only a handle for cudaGetSymbolAddress; it is not a device address.
static __device__ __align__(256) unsigned char g_static_loss_scratch[kStaticScratchBytes];

// Device address of the array on the current device, looked up once per device.
int static_loss_scratch(void** out) {
  static std::mutex mu;
  static void* cached[64];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return A3PO_ERR_NO_DEVICE;
  }
  std::lock_guard<std::mutex> lock(mu);
  if (!cached[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_loss_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return A3PO_ERR_CUDA;
    }
    cached[dev] = p;
  }
  *out = cached[dev];
  return A3PO_OK;
}

}  // namespace
}  // namespace a3po

extern "C" {

int a3po_loss_fwd_static(const float* logp, const float* behav_logp, const int32_t* versions, int versions_per_seq,
                         const int32_t* cu_seqlens, int B, int32_t current_version, const float* adv,
                         const uint8_t* mask, int64_t N, float clip_eps, float* loss, a3po_stats* stats,
                         void* stream) {
  if (N > A3PO_LOSS_FWD_STATIC_MAX_TOKENS) return A3PO_ERR_TOO_LARGE;
  if (N >= 0 && a3po::loss_ws_bytes(N) > a3po::kStaticScratchBytes) return A3PO_ERR_TOO_LARGE;
  if (a3po::sm_count() <= 0) return A3PO_ERR_NO_DEVICE;
  void* scratch = nullptr;
  A3PO_RETURN_IF(a3po::static_loss_scratch(&scratch));
  return a3po::run_loss(a3po::kFwd, logp, behav_logp, nullptr, versions, versions_per_seq, cu_seqlens, B, current_version,
                        adv, mask, N, clip_eps, 1, nullptr, nullptr, loss, stats, nullptr, scratch,
                        a3po::kStaticScratchBytes, stream, /*allow_single_launch=*/false);
}

int a3po_loss_bwd(const float* logp, const float* behav_logp, const int32_t* versions, int versions_per_seq,
                  const int32_t* cu_seqlens, int B, int32_t current_version, const float* adv,
                  const uint8_t* mask, int64_t N, float clip_eps, int detach_prox, const float* grad_loss,
                  const a3po_stats* fwd_stats, float* grad_logp, void* ws, size_t ws_bytes, void* stream) {
  return a3po::run_loss(a3po::kBwd, logp, behav_logp, nullptr, versions, versions_per_seq, cu_seqlens, B, current_version,
                        adv, mask, N, clip_eps, detach_prox, grad_loss, fwd_stats, nullptr, nullptr, grad_logp, ws,
                        ws_bytes, stream);
}

int a3po_loss_fwd_bwd(const float* logp, const float* behav_logp, const int32_t* versions, int versions_per_seq,
                      const int32_t* cu_seqlens, int B, int32_t current_version, const float* adv,
                      const uint8_t* mask, int64_t N, float clip_eps, int detach_prox, float* loss,
                      a3po_stats* stats, float* grad_logp, void* ws, size_t ws_bytes, void* stream) {
  return a3po::run_loss(a3po::kFwdBwd, logp, behav_logp, nullptr, versions, versions_per_seq, cu_seqlens, B,
                        current_version, adv, mask, N, clip_eps, detach_prox, nullptr, nullptr, loss, stats,
                        grad_logp, ws, ws_bytes, stream);
}

size_t a3po_mask_count_workspace_bytes(void) { return a3po::round_up(sizeof(long long) * a3po::kMaxLossBlocks, 256) + 256; }

int a3po_mask_count(const uint8_t* mask, int64_t N, int64_t* count, void* ws, size_t ws_bytes, void* stream_) {
  using namespace a3po;
  if (N < 0 || !count || (N > 0 && !mask)) return A3PO_ERR_INVALID_ARG;
  if (!ws || !aligned_to(ws, 256) || ws_bytes < a3po_mask_count_workspace_bytes()) return A3PO_ERR_WORKSPACE;
  if (sm_count() <= 0) return A3PO_ERR_NO_DEVICE;
  cudaStream_t stream = as_stream(stream_);
  long long* block_counts = static_cast<long long*>(ws);
  const int cb = grid_for((N + 15) / 16);
  A3PO_LAUNCH(kKMaskCount, stream, mask_count_kernel<<<cb, kLossThreads, 0, stream>>>(mask, N, block_counts));
  A3PO_RETURN_IF(after_launch());
  A3PO_LAUNCH(kKMaskCountFinalize, stream, mask_count_finalize_kernel<<<1, kLossThreads, 0, stream>>>(
                                               block_counts, cb, reinterpret_cast<long long*>(count)));
  return after_launch();
}

int a3po_dp_loss_scale(const int64_t* m_local, const int64_t* m_global, const float* loss_local, float* scale,
                       float* weighted_loss, void* stream_) {
  using namespace a3po;
  if (!m_local || !m_global || !scale || (loss_local && !weighted_loss)) return A3PO_ERR_INVALID_ARG;
  if (sm_count() <= 0) return A3PO_ERR_NO_DEVICE;
  cudaStream_t stream = as_stream(stream_);
  A3PO_LAUNCH(kKLossFinalize, stream, dp_scale_kernel<<<1, 1, 0, stream>>>(
                                          reinterpret_cast<const long long*>(m_local),
                                          reinterpret_cast<const long long*>(m_global), loss_local, scale,
                                          weighted_loss));
  return after_launch();
}

int a3po_decoupled_loss_fwd_bwd(const float* logp, const float* behav_logp, const float* prox_logp, const float* adv,
                                const uint8_t* mask, int64_t N, float clip_eps, float* loss, a3po_stats* stats,
                                float* grad_logp, void* ws, size_t ws_bytes, void* stream) {
  if (N > 0 && !prox_logp) return A3PO_ERR_INVALID_ARG;
  const int mode = grad_logp ? a3po::kFwdBwd : a3po::kFwd;
  static const float kNoTokens = 0.f;  // N == 0: run_loss still wants a non-null anchor to pick this variant
  return a3po::run_loss(mode, logp, behav_logp, prox_logp ? prox_logp : &kNoTokens, nullptr, 0, nullptr, 0, 0, adv,
                        mask, N, clip_eps, 1, nullptr, nullptr, loss, stats, grad_logp, ws, ws_bytes, stream);
}

}  // extern "C"
