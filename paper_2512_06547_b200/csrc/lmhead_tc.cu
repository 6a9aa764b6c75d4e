// LM-head log-prob forward/backward on the sm_100a tensor cores (bf16 in, fp32 accumulate).
//
// One persistent, warp-specialised kernel template does every contraction of the path,
//     C[M, N] = A[M, K] * B[N, K]^T,
// and differs only in its epilogue:
//   forward      A = hidden, B = W           online (max, sum-exp) per row + target gather
//   forward+keep same, and every probability is kept as a bf16 ratio to the target token's for a backward
//                without recomputation
//   dz           A = hidden, B = W           dz = g (1[v = y] - exp(z - lse)) -> bf16 chunk of rows
//   grad_hidden  A = dz,     B = W^T         bf16 store, optional per-row scale (W read in place, N-major)
//   grad_w       A = dz^T,   B = hidden^T    fp32 store/accumulate (both read in place, M-/N-major)
// (with kept probability ratios in place of dz the per-row factor of dz moves into the grad_hidden epilogue
// and into the hidden operand of grad_w)
//
// Per CTA (one per SM): warp 0 = TMA producer (one elected lane), warp 1 = tcgen05.mma issuer
// (one elected lane; it also owns the TMEM allocation), warps 2-5 = epilogue (one TMEM lane
// quarter each, one accumulator row per thread).  Operand tiles (128 x 64 and 256 x 64 bf16,
// 128-byte swizzle) move through a 4-stage shared-memory ring guarded by full/empty mbarriers;
// the 128 x 256 fp32 accumulator is double-buffered in TMEM (2 x 256 columns) so the epilogue
// of tile i overlaps the MMAs of tile i+1.  Output tiles (kept ratios, dz, gradients) leave through
// two swizzled shared-memory slabs and TMA tile stores.  The full logits matrix never exists: the
// plain forward keeps nothing, the keeping forward writes only the rows that take part, into scratch.
//
// Every mbarrier wait is bounded; on expiry the CTA raises A3PO_STATUS_WAIT_TIMEOUT in the
// caller's status word, releases its TMEM and exits.

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>

#include "a3po_common.cuh"
#include "lmhead_internal.cuh"
#include "sm100_ptx.cuh"

namespace a3po {
namespace {

using namespace ptx;

constexpr int BM = 128;
constexpr int BN = 256;
constexpr int BK = 64;
constexpr int kTcThreads = 192;
constexpr int kEpiChunk = 32;
constexpr uint32_t kABytes = BM * BK * 2;   // one 128-row A tile
constexpr uint32_t kBBytes = BN * BK * 2;
constexpr uint32_t kMnBlockBytes = 64 * BK * 2;  // one 64 (M/N) x 64 (k) box of an MN-major operand
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSlabBytes = BM * 128;  // output staging slab: 128 rows x 128 bytes
// MT = A tiles (of 128 rows) a CTA multiplies with each B tile.  MT = 1: a 128 x 256 output tile, two accumulators
// in TMEM so that the epilogue of one tile overlaps the MMAs of the next, 4-stage ring.  MT = 2: a 256 x 256 output
// tile (all 512 TMEM columns, one accumulator set, no epilogue overlap), 3-stage ring of 64 KB stages: a third fewer
// operand bytes per flop out of L2 and shared memory, for the contractions whose epilogue is negligible (K = V or
// K = rows, thousands of k-blocks per tile).
template <int MT> struct TileCfg {
  static constexpr int kStages = MT == 1 ? 4 : 3;
  static constexpr int kAccStages = 2 / MT;
  static constexpr uint32_t kAStage = MT * kABytes;
  static constexpr uint32_t kStageBytes = kAStage + kBBytes;
  static constexpr size_t kSmemBytes = 1024 /*alignment slack*/ + kStages * kStageBytes + 2 * kSlabBytes + 256 /*barriers*/;
};
// Row tiles per rasterisation group (see ItemMap) of the contractions whose items are single output tiles (the
// gradients).  Small groups win on B200: with 4 the 8B-shaped step takes 216 ms against 231 with 16 (1.5B-shaped:
// 10.7 against 11.2 ms), 3 and 6 are worse than 4 and 8; the kernels are energy bound under the board's power cap
// and fewer HBM re-reads of the operands are fewer joules.
constexpr int kGroupM = 4;
// The forward contractions (items sweep a range of column tiles) take large groups instead, see fwd_group_m().
constexpr long long kFwdGroupBytes = 40ll << 20;

// Work decomposition: an item is (row tile, vocabulary split); a split is a contiguous range of
// column tiles.  Items are ordered so that CTAs running at the same time share row tiles and
// column tiles through L2: groups of group_m row tiles, all splits of a group before the next.
struct ItemMap {
  int m_tiles;
  int n_tiles;
  int splits;
  int group_m;  // row tiles per rasterisation group
  long long items;
  // Optional device-side row count (compact row space): this launch covers rows
  // [dyn_offset, dyn_offset + dyn_cap) of it and really has clamp(*dyn_rows - dyn_offset, 0, dyn_cap).
  const int* dyn_rows;   // null: extents are the static ones above
  int dyn_is_k;          // 0: the rows are the M extent; 1: the rows are the K extent
  int zero_when_empty;   // dyn_is_k only: with no rows, store an all-zero output instead of doing nothing
  long long dyn_offset;
  long long dyn_cap;
  // Optional device-side choice between two launches of the same contraction with different tiles: this launch
  // does its work only if *select == select_value (the other one then exits at once).
  const int* select;
  int select_value;
  // Optional pacing of the CTAs of a launch (see Pace): ring of arrival counters, null = off.
  unsigned int* pace;
  int pace_period;  // k-blocks between two pacing points
  int pace_slack;   // how many pacing points a CTA may be ahead of the slowest one
};

struct Item {
  int m_tile;
  int split;
  int n_begin;
  int n_end;
};

__device__ __forceinline__ Item decode_item(const ItemMap& im, long long i) {
  const int kGroupM = im.group_m;
  const long long per_group = static_cast<long long>(kGroupM) * im.splits;
  const int full_groups = im.m_tiles / kGroupM;
  Item it;
  if (i < per_group * full_groups) {
    const int g = static_cast<int>(i / per_group);
    const int w = static_cast<int>(i % per_group);
    it.split = w / kGroupM;
    it.m_tile = g * kGroupM + w % kGroupM;
  } else {
    const int rem = im.m_tiles - full_groups * kGroupM;
    const int w = static_cast<int>(i - per_group * full_groups);
    it.split = w / rem;
    it.m_tile = full_groups * kGroupM + w % rem;
  }
  it.n_begin = static_cast<int>(static_cast<long long>(it.split) * im.n_tiles / im.splits);
  it.n_end = static_cast<int>(static_cast<long long>(it.split + 1) * im.n_tiles / im.splits);
  return it;
}

// Pacing.  The CTAs of a launch that run at the same time read the same operand tiles (that is what the item order
// arranges), but only the first reader of a tile takes it from HBM if the others follow before L2 has replaced
// it.  Nothing keeps a persistent CTA in step with the others over dozens of tiles, so they drift apart and the
// same bytes come out of HBM several times: on the 8B-shaped batch the gradient contractions read 100 GB per
// launch unpaced and 51 GB paced (the floor for 148 concurrent 256 x 256 tiles), 5-8 % of their time under the
// board's power cap.  Every kPacePeriod k-blocks the producer thread of each CTA counts itself in at a pacing
// point and does not run more than kPaceSlack points ahead of the slowest CTA.  It is advisory: no data depends
// on it, a wait gives up after kPaceWaitCycles and the CTA then skips a growing number of points (so CTAs that
// cannot be in step, e.g. because they started late, lose microseconds, not the kernel), and a CTA with nothing
// to load counts itself in for the points it will not reach.
// Counters of one launch: kPaceRing arrival counters (point g uses slot g mod kPaceRing; a slot counts up over the
// launch) followed by one counter of finished CTAs; the last CTA to finish zeroes all of them again, so a block of
// counters is zero whenever no launch is using it.
constexpr int kPaceRing = 32;
constexpr int kPaceBlockWords = 64;            // one launch's counters: ring + finished count, padded to 256 bytes
constexpr int kPaceBlocks = 32;                // handed out round-robin, so launches on different streams differ
constexpr int kPacePeriod = 16;
constexpr int kPaceSlack = 3;
constexpr long long kPaceWaitCycles = 40000;   // 20-40 us
struct Pace {
  unsigned int* slots = nullptr;
  unsigned int ctas = 0;
  int slack = 0;
  int skip = 0;
  int backoff = 8;
  unsigned int seen = 0;   // arrivals counted, one point ago, at the point this CTA has to wait for next
  long long next = 0;      // index of the next pacing point of this CTA

  __device__ __forceinline__ void arrive() {
    atomicAdd(&slots[next & (kPaceRing - 1)], 1u);
    ++next;
  }
  // The counter this CTA will compare at its next pacing point is read one point early (`seen`), so that the
  // producer does not sit out an L2 round trip at every point; a stale value can only be too small, and then the
  // loop below reads the counter afresh.
  __device__ __forceinline__ void arrive_and_wait() {
    const long long behind = next - slack;
    arrive();
    if (behind >= 0) {
      if (skip > 0) {
        --skip;
      } else {
        const unsigned int expected = static_cast<unsigned int>(behind / kPaceRing + 1) * ctas;
        if (seen < expected) {
          volatile unsigned int* slot = slots + (behind & (kPaceRing - 1));
          const long long t0 = clock64();
          bool late = false;
          while (*slot < expected) {
            if (clock64() - t0 > kPaceWaitCycles) { late = true; break; }
          }
          if (late) {
            skip = backoff;
            backoff = backoff < 4096 ? 2 * backoff : backoff;
          } else {
            backoff = 8;
          }
        } else {
          backoff = 8;
        }
      }
    }
    if (behind + 1 >= 0) seen = *(static_cast<volatile unsigned int*>(slots) + ((behind + 1) & (kPaceRing - 1)));
  }
  __device__ __forceinline__ void finish() {
    __threadfence();
    const unsigned int done = atomicAdd(&slots[kPaceRing], 1u);
    if (done + 1 == ctas) {
      for (int i = 0; i <= kPaceRing; ++i) slots[i] = 0u;
    }
  }
};

__device__ __forceinline__ float bits_to_float(uint32_t u) { return __uint_as_float(u); }

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 p = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&p);
}

// Waits on an mbarrier that never completes; the wait gives up after limit_ns and raises the
// status bit, exactly as a stuck pipeline stage would.
__global__ void wait_timeout_kernel(uint32_t* status, unsigned long long limit_ns) {
  __shared__ uint64_t bar;
  __shared__ uint32_t abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool completed = mbar_wait(&bar, 0, &abort_flag, limit_ns);
    if (!completed && status) atomicOr(status, A3PO_STATUS_WAIT_TIMEOUT);
  }
}

// ------------------------------------------------------------------------------------ tensor maps
using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static std::once_flag once;
  static EncodeTiledFn fn = nullptr;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  });
  return fn;
}


// Tensor map of an output matrix [rows, cols] (row-major, `pitch` elements per row, 2- or 4-byte
// elements) for slab stores: boxes of 128 rows x 128 bytes with the 128-byte swizzle.
int make_out_map(CUtensorMap* map, const void* base, int elt_bytes, long long cols, long long rows, long long pitch) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return A3PO_ERR_CUDA;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(pitch) * elt_bytes};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(128 / elt_bytes), static_cast<cuuint32_t>(BM)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, elt_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2,
                        const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? A3PO_OK : A3PO_ERR_CUDA;
}

// ------------------------------------------------------------------------------------ epilogues
// Each epilogue thread owns one accumulator row (`row` = global row of the A operand).
// begin(): per-item state; chunk(): 32 consecutive fp32 columns starting at global column `col0`;
// end(): per-item output.

struct SlabStore;  // output staging for TMA stores, defined below

template <bool ENT>
struct FwdEpilogue {
  static constexpr int kKernelId = kKTcFwd;
  struct Params {
    const int32_t* targets;
    long long n;
    int v;
    float scale_log2;  // inv_temperature * log2(e)
    float inv_t;
    SoftmaxPartial* part;
    float* part_ent;
    float* zy;
  };
  static int make_c_map(const Params&, CUtensorMap* map) {
    memset(map, 0, sizeof(*map));  // the forward stores nothing through the copy engine
    return A3PO_OK;
  }
  float m, s, e;
  int y;
  long long row;
  __device__ __forceinline__ void begin(const Params& p, long long row_) {
    row = row_;
    m = -INFINITY; s = 0.f; e = 0.f;
    y = -1;
    if (row < p.n) y = min(max(p.targets[row], 0), p.v - 1);
  }
  __device__ __forceinline__ void chunk(const Params& p, int /*tile_row0*/, int col0, uint32_t (&r)[kEpiChunk],
                                        SlabStore&) {
    if (col0 + kEpiChunk > p.v) {  // ragged vocabulary tail: columns past V do not exist
#pragma unroll
      for (int j = 0; j < kEpiChunk; ++j)
        if (col0 + j >= p.v) r[j] = 0xff800000u;  // -inf
    }
    float zmax = -INFINITY;
#pragma unroll
    for (int j = 0; j < kEpiChunk; ++j) zmax = fmaxf(zmax, bits_to_float(r[j]));
    const float xm = zmax * p.scale_log2;
    if (xm > m) {
      const float f = fast_exp2(m - xm);
      s *= f;
      if (ENT) e *= f;
      m = xm;
    }
    float acc = 0.f, ee = 0.f;
#pragma unroll
    for (int j = 0; j < kEpiChunk; ++j) {
      const float z = bits_to_float(r[j]);
      const float pj = fast_exp2(fmaf(z, p.scale_log2, -m));
      acc += pj;
      if (ENT) ee = fmaf(pj, pj > 0.f ? z : 0.f, ee);
    }
    s += acc;
    if (ENT) e = fmaf(ee, p.inv_t, e);
    if (y >= col0 && y < col0 + kEpiChunk) {
      float zyv = 0.f;
#pragma unroll
      for (int j = 0; j < kEpiChunk; ++j)
        if (col0 + j == y) zyv = bits_to_float(r[j]);
      p.zy[row] = zyv * p.inv_t;
    }
  }
  __device__ __forceinline__ void end(const Params& p, long long row, int split) {
    if (row < p.n) {
      p.part[static_cast<long long>(split) * p.n + row] = SoftmaxPartial{m * kLn2, s};
      if (ENT) p.part_ent[static_cast<long long>(split) * p.n + row] = e;
    }
  }
};

// Staging of output tiles for TMA stores.  The 128 epilogue threads fill a 128-row x 128-byte
// slab in shared memory (one row each, 128-byte swizzle), and one of them hands the slab to the
// copy engine, which writes it to global memory fully coalesced and clips it at the tensor's
// extents (ragged row / column tails need no guards).  Two slabs alternate so that filling one
// overlaps the copy of the other.
struct SlabStore {
  uint8_t* slab0;
  uint8_t* slab1;
  const CUtensorMap* map;
  int row_in_tile;
  bool issuer;
  uint32_t issued = 0;
  static constexpr int kBarrierId = 1;

  // Returns the slab to fill next; all epilogue threads call it together.
  __device__ __forceinline__ uint8_t* acquire() {
    if (issuer) bulk_wait_group_read<1>();  // the copy that used this slab two submissions ago has read it
    named_barrier_sync(kBarrierId, 128);
    return (issued & 1u) ? slab1 : slab0;
  }
  // 16-byte piece j (0..7) of this thread's row.
  __device__ __forceinline__ uint4* piece(uint8_t* s, int j) const {
    return reinterpret_cast<uint4*>(s + row_in_tile * 128 + ((j ^ (row_in_tile & 7)) << 4));
  }
  // Hands the filled slab to the copy engine: global tile origin (x, y) in elements.
  __device__ __forceinline__ void submit(uint8_t* s, int x, int y, bool in_range, bool reduce_add) {
    fence_proxy_async_smem();
    named_barrier_sync(kBarrierId, 128);
    if (issuer) {
      if (in_range) {
        if (reduce_add) tma_reduce_add_f32_2d(map, s, x, y);
        else tma_store_2d(map, s, x, y);
      }
      bulk_commit_group();
    }
    ++issued;
  }
  __device__ __forceinline__ void drain() {
    if (issuer) bulk_wait_group<0>();
  }
};

struct DzEpilogue {
  static constexpr int kKernelId = kKTcDz;
  struct Params {
    const int32_t* targets;   // indexed by global token row
    const float* lse;
    const float* grad_logp;
    long long row_begin;      // first token row of this chunk; A-operand row 0 == row_begin
    long long row_end;
    int v;
    int vpad;                 // row pitch of dz
    float scale_log2;
    float inv_t;
    __nv_bfloat16* dz;        // [chunk rows, vpad]
  };
  static int make_c_map(const Params& p, CUtensorMap* map) {
    return make_out_map(map, p.dz, /*bytes per element*/ 2, p.v, p.row_end - p.row_begin, p.vpad);
  }
  float g, l2;
  int y;
  uint8_t* cur;
  __device__ __forceinline__ void begin(const Params& p, long long row) {
    const long long t = p.row_begin + row;
    g = 0.f; l2 = INFINITY; y = -1;
    if (t < p.row_end) {
      g = p.grad_logp[t] * p.inv_t;
      if (g != 0.f) l2 = p.lse[t] * kLog2e;   // g == 0: exp2(-inf) = 0, the row contributes nothing
      y = min(max(p.targets[t], 0), p.v - 1);
    }
  }
  __device__ __forceinline__ void chunk(const Params& p, int tile_row0, int col0, uint32_t (&r)[kEpiChunk],
                                        SlabStore& st) {
    float d[kEpiChunk];
    const float ng = -g;
#pragma unroll
    for (int j = 0; j < kEpiChunk; ++j)
      d[j] = ng * fast_exp2(fmaf(bits_to_float(r[j]), p.scale_log2, -l2));
    if (y >= col0 && y < col0 + kEpiChunk) {
#pragma unroll
      for (int j = 0; j < kEpiChunk; ++j)
        if (col0 + j == y) d[j] += g;
    }
    // a slab holds 64 bf16 columns: two consecutive 32-column chunks
    const int half = (col0 >> 5) & 1;
    if (half == 0) cur = st.acquire();
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint4 u;
      u.x = pack_bf16x2(d[q * 8 + 0], d[q * 8 + 1]);
      u.y = pack_bf16x2(d[q * 8 + 2], d[q * 8 + 3]);
      u.z = pack_bf16x2(d[q * 8 + 4], d[q * 8 + 5]);
      u.w = pack_bf16x2(d[q * 8 + 6], d[q * 8 + 7]);
      *st.piece(cur, half * 4 + q) = u;
    }
    if (half == 1) st.submit(cur, col0 - 32, tile_row0, col0 - 32 < p.v, false);
  }
  __device__ __forceinline__ void end(const Params&, long long, int) {}
};

// Forward that also keeps the row's softmax for the backward, so that the backward need not recompute
// the logits.  The reference of row t is its own target logit zy (computed beforehand, one dot product
// per row), and what is kept is the probability ratio
//     q[t, v] = exp(z[t, v] - zy[t]) = p[t, v] / p[t, y_t]                  (bf16, 0 at v = y_t)
// A ratio is a floating-point number with bf16's uniform relative precision whatever its size, so
// peaked and flat rows are kept equally well, and every split of a row shares the one reference, so
// no running maximum, rescaling or extra sweep is needed.  The target column is left out of the sum:
//     s[t] = sum_{v != y_t} q[t, v],  lse = zy + log1p(s),  logp = -log1p(s),  1 - p_y = s / (1 + s),
// which stays accurate when p_y approaches 1.  The exponent is clamped at 126 (a ratio above 2^126
// means p_y < 1e-37; the merge flags such a row).
template <bool ENT>
struct KeepEpilogue {
  static constexpr int kKernelId = kKTcFwdKeep;
  struct Params {
    const int32_t* targets;   // [n] rows of this launch
    const float* zy;          // [n] target logit / T, natural-log units
    long long n;
    int v;
    int vpad;                 // row pitch of q
    float scale_log2;
    float inv_t;
    float* part_s;            // [splits][n] sum of the ratios over the split's columns, target left out
    float* part_e;            // [splits][n] sum of ratio * raw logit (entropy), or null
    __nv_bfloat16* q;         // [n, vpad]
  };
  static int make_c_map(const Params& p, CUtensorMap* map) { return make_out_map(map, p.q, 2, p.v, p.n, p.vpad); }
  float s, e, ref2;
  int y;
  uint8_t* cur;
  __device__ __forceinline__ void begin(const Params& p, long long row) {
    s = 0.f; e = 0.f; ref2 = 0.f;
    y = -1;
    if (row < p.n) {
      y = min(max(p.targets[row], 0), p.v - 1);
      ref2 = p.zy[row] * kLog2e;
    }
  }
  __device__ __forceinline__ void chunk(const Params& p, int tile_row0, int col0, uint32_t (&r)[kEpiChunk],
                                        SlabStore& st) {
    if (col0 + kEpiChunk > p.v) {
#pragma unroll
      for (int j = 0; j < kEpiChunk; ++j)
        if (col0 + j >= p.v) r[j] = 0xff800000u;  // -inf: columns past V do not exist
    }
    float q[kEpiChunk];
#pragma unroll
    for (int j = 0; j < kEpiChunk; ++j)
      q[j] = fast_exp2(fminf(fmaf(bits_to_float(r[j]), p.scale_log2, -ref2), 126.f));
    if (y >= col0 && y < col0 + kEpiChunk) {
#pragma unroll
      for (int j = 0; j < kEpiChunk; ++j)
        if (col0 + j == y) q[j] = 0.f;   // the target's own entry is written by the backward (-s)
    }
    float acc = 0.f, ee = 0.f;
#pragma unroll
    for (int j = 0; j < kEpiChunk; ++j) {
      acc += q[j];
      if (ENT) ee = fmaf(q[j], q[j] > 0.f ? bits_to_float(r[j]) : 0.f, ee);
    }
    s += acc;
    if (ENT) e += ee;
    const int half = (col0 >> 5) & 1;
    if (half == 0) cur = st.acquire();
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      uint4 w;
      w.x = pack_bf16x2(q[k * 8 + 0], q[k * 8 + 1]);
      w.y = pack_bf16x2(q[k * 8 + 2], q[k * 8 + 3]);
      w.z = pack_bf16x2(q[k * 8 + 4], q[k * 8 + 5]);
      w.w = pack_bf16x2(q[k * 8 + 6], q[k * 8 + 7]);
      *st.piece(cur, half * 4 + k) = w;
    }
    if (half == 1) st.submit(cur, col0 - 32, tile_row0, col0 - 32 < p.v, false);
  }
  __device__ __forceinline__ void end(const Params& p, long long row, int split) {
    if (row < p.n) {
      p.part_s[static_cast<long long>(split) * p.n + row] = s;
      if (ENT) p.part_e[static_cast<long long>(split) * p.n + row] = e;
    }
  }
};

struct StoreBf16Epilogue {
  static constexpr int kKernelId = kKTcGradHidden;
  struct Params {
    __nv_bfloat16* c;
    long long ldc;
    long long m_rows;
    int n_cols;  // multiple of 8
    const float* row_scale;  // [m_rows] factor applied to each output row, or null for none
  };
  static int make_c_map(const Params& p, CUtensorMap* map) {
    return make_out_map(map, p.c, 2, p.n_cols, p.m_rows, p.ldc);
  }
  uint8_t* cur;
  float sc;
  __device__ __forceinline__ void begin(const Params& p, long long row) {
    sc = (p.row_scale != nullptr && row < p.m_rows) ? p.row_scale[row] : 1.0f;
  }
  __device__ __forceinline__ void chunk(const Params& p, int tile_row0, int col0, uint32_t (&r)[kEpiChunk],
                                        SlabStore& st) {
    const int half = (col0 >> 5) & 1;
    if (half == 0) cur = st.acquire();
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      uint4 u;
      u.x = pack_bf16x2(sc * bits_to_float(r[q * 8 + 0]), sc * bits_to_float(r[q * 8 + 1]));
      u.y = pack_bf16x2(sc * bits_to_float(r[q * 8 + 2]), sc * bits_to_float(r[q * 8 + 3]));
      u.z = pack_bf16x2(sc * bits_to_float(r[q * 8 + 4]), sc * bits_to_float(r[q * 8 + 5]));
      u.w = pack_bf16x2(sc * bits_to_float(r[q * 8 + 6]), sc * bits_to_float(r[q * 8 + 7]));
      *st.piece(cur, half * 4 + q) = u;
    }
    if (half == 1) st.submit(cur, col0 - 32, tile_row0, col0 - 32 < p.n_cols, false);
  }
  __device__ __forceinline__ void end(const Params&, long long, int) {}
};

struct StoreF32Epilogue {
  static constexpr int kKernelId = kKTcGradW;
  struct Params {
    float* c;
    long long ldc;
    long long m_rows;
    int n_cols;  // multiple of 4
    int accumulate;  // add into c (performed by the copy engine's element-wise reduction) instead of overwriting
  };
  static int make_c_map(const Params& p, CUtensorMap* map) {
    return make_out_map(map, p.c, 4, p.n_cols, p.m_rows, p.ldc);
  }
  __device__ __forceinline__ void begin(const Params&, long long) {}
  __device__ __forceinline__ void chunk(const Params& p, int tile_row0, int col0, uint32_t (&r)[kEpiChunk],
                                        SlabStore& st) {
    uint8_t* s = st.acquire();  // 32 fp32 columns = one 128-byte slab row
#pragma unroll
    for (int q = 0; q < 8; ++q) *st.piece(s, q) = make_uint4(r[q * 4 + 0], r[q * 4 + 1], r[q * 4 + 2], r[q * 4 + 3]);
    st.submit(s, col0, tile_row0, col0 < p.n_cols, p.accumulate != 0);
  }
  __device__ __forceinline__ void end(const Params&, long long, int) {}
};

// AND of a predicate over the 128 epilogue threads (hardware barrier 2).
__device__ __forceinline__ bool all_epilogue_threads(bool pred) {
  uint32_t out;
  asm volatile(
      "{\n"
      ".reg .pred p, q;\n"
      "setp.ne.u32 q, %1, 0;\n"
      "bar.red.and.pred p, 2, 128, q;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(out)
      : "r"(static_cast<uint32_t>(pred))
      : "memory");
  return out != 0;
}

#ifdef A3PO_TUNING
// Tuning builds only: per-CTA start / end of every GEMM launch in wall-clock nanoseconds and SM cycles, written to
// a caller-provided buffer (a3po_tuning_set_trace), to read the finish-time spread of the CTAs and the SM clock a
// kernel really ran at.
struct TraceRecord {
  unsigned long long t_begin_ns, t_end_ns, cycles, items;
  // SM cycles each role spent waiting: producer on a free stage, MMA issuer on a filled stage, MMA issuer on a free
  // accumulator, epilogue (warp 2) on a finished accumulator
  unsigned long long wait_stage_free, wait_stage_full, wait_acc_free, wait_acc_full;
};
__device__ TraceRecord* g_trace = nullptr;
__device__ unsigned int g_trace_capacity = 0;
__device__ unsigned int g_trace_next = 0;
#endif

// ------------------------------------------------------------------------------------ the kernel
// A_MN / B_MN: the operand is read from a tensor whose contiguous index is M (resp. N) instead of
// K: it arrives as 64 x 64 boxes (64 M/N elements by 64 k) and is fed to the MMA as an MN-major
// shared-memory matrix, so no transposed copy of the operand ever has to exist in memory.
template <class Epi, bool A_MN, bool B_MN, int MT>
__global__ void __launch_bounds__(kTcThreads, 1)
gemm_tn_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_c, ItemMap im_static, int k_blocks_static,
               typename Epi::Params ep, uint32_t* status) {
  // Work extents: static, or derived from the device-resident row count (identical in every thread).
  ItemMap im = im_static;
  int k_blocks = k_blocks_static;
  bool zero_output = false;  // K extent is empty: the product is the zero matrix
  if (im.select != nullptr && *im.select != im.select_value) {
    im.items = 0;
    im.dyn_rows = nullptr;
  }
  if (im.dyn_rows != nullptr) {
    long long rows = static_cast<long long>(*im.dyn_rows) - im.dyn_offset;
    rows = rows < 0 ? 0 : (rows > im.dyn_cap ? im.dyn_cap : rows);
    if (im.dyn_is_k) {
      k_blocks = static_cast<int>((rows + BK - 1) / BK);
      if (k_blocks == 0) {
        if (im.zero_when_empty) zero_output = true;
        else im.items = 0;
      }
    } else {
      im.m_tiles = static_cast<int>((rows + BM * MT - 1) / (BM * MT));
      im.items = static_cast<long long>(im.m_tiles) * im.splits;
    }
  }
  using Cfg = TileCfg<MT>;
  constexpr int kStages = Cfg::kStages;
  constexpr int kAccStages = Cfg::kAccStages;
  constexpr uint32_t kAStage = Cfg::kAStage;
  constexpr uint32_t kStageBytes = Cfg::kStageBytes;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + kStages * kAStage;
  uint8_t* smem_slabs = smem + kStages * kStageBytes;  // two 16 KB output staging slabs
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_slabs + 2 * kSlabBytes);
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* tmem_full_bar = empty_bar + kStages;
  uint64_t* tmem_empty_bar = tmem_full_bar + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty_bar + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x / kWarp;
  const int lane = threadIdx.x % kWarp;
#ifdef A3PO_TUNING
  unsigned long long trace_t0 = 0, trace_c0 = 0;
  __shared__ unsigned long long trace_wait[4];
  unsigned long long waited = 0, waited2 = 0;
  if (threadIdx.x == 0) {
    trace_t0 = globaltimer_ns();
    trace_c0 = static_cast<unsigned long long>(clock64());
    trace_wait[0] = trace_wait[1] = trace_wait[2] = trace_wait[3] = 0;
  }
#define A3PO_TIMED_WAIT(acc, expr) [&] { const long long t_ = clock64(); const bool r_ = (expr); acc += clock64() - t_; return r_; }()
#else
#define A3PO_TIMED_WAIT(acc, expr) (expr)
  constexpr int waited = 0, waited2 = 0;
  (void)waited; (void)waited2;
#endif

  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(&full_bar[i], 1);
      mbar_init(&empty_bar[i], 1);
    }
    for (int i = 0; i < kAccStages; ++i) {
      mbar_init(&tmem_full_bar[i], 1);
      mbar_init(&tmem_empty_bar[i], 4);  // one arrival per epilogue warp
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, kTmemCols);
    tmem_relinquish_alloc_permit();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  bool ok = true;
  if (warp < 2 && zero_output) {
    // nothing to load or multiply: the epilogue warps write zeros
  } else if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (elect_one()) {
      int stage = 0;
      uint32_t phase = 0;
      // pacing points: every CTA of the launch passes the same number per wave of items, whether it has an item
      // in that wave (or a last column tile in its item) or not
      Pace pace;
      const bool paced = im.pace != nullptr && im.pace_period > 0 && im.items > 0 && k_blocks > 0;
      const int points_per_tile = paced ? (k_blocks + im.pace_period - 1) / im.pace_period : 0;
      const long long points_per_wave =
          static_cast<long long>((im.n_tiles + im.splits - 1) / im.splits) * points_per_tile;
      long long waves_done = 0;
      if (paced) {
        pace.slots = im.pace;
        pace.ctas = gridDim.x;
        pace.slack = im.pace_slack;
      }
      for (long long i = blockIdx.x; i < im.items && ok; i += gridDim.x) {
        const Item it = decode_item(im, i);
        for (int nt = it.n_begin; nt < it.n_end && ok; ++nt) {
          for (int kb = 0; kb < k_blocks; ++kb) {
            if (paced && kb % im.pace_period == 0) pace.arrive_and_wait();
            if (!A3PO_TIMED_WAIT(waited, mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag))) { ok = false; break; }
            mbar_arrive_expect_tx(&full_bar[stage], kStageBytes);
            uint8_t* sa = smem_a + stage * kAStage;
            uint8_t* sb = smem_b + stage * kBBytes;
            if (A_MN) {
#pragma unroll
              for (int j = 0; j < MT * BM / 64; ++j)
                tma_load_2d(sa + j * kMnBlockBytes, &map_a, &full_bar[stage], it.m_tile * (BM * MT) + j * 64, kb * BK);
            } else {
              tma_load_2d(sa, &map_a, &full_bar[stage], kb * BK, it.m_tile * (BM * MT));  // one box of MT * 128 rows
            }
            if (B_MN) {
#pragma unroll
              for (int j = 0; j < BN / 64; ++j)
                tma_load_2d(sb + j * kMnBlockBytes, &map_b, &full_bar[stage], nt * BN + j * 64, kb * BK);
            } else {
              tma_load_2d(sb, &map_b, &full_bar[stage], kb * BK, nt * BN);
            }
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
        }
        ++waves_done;
        if (paced)
          while (pace.next < waves_done * points_per_wave) pace.arrive();
      }
      if (paced) {
        const long long waves = (im.items + gridDim.x - 1) / gridDim.x;
        while (pace.next < waves * points_per_wave) pace.arrive();
        pace.finish();
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (elect_one()) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(BM, BN, A_MN, B_MN);
      // descriptor start-address step (16-byte units) per UMMA (K = 16): 32 bytes inside the swizzled
      // row for a K-major tile, two 1024-byte k-group atoms for an MN-major tile
      constexpr uint32_t a_step = A_MN ? (2 * 1024) >> 4 : 32 >> 4;
      constexpr uint32_t b_step = B_MN ? (2 * 1024) >> 4 : 32 >> 4;
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      for (long long i = blockIdx.x; i < im.items && ok; i += gridDim.x) {
        const Item it = decode_item(im, i);
        for (int nt = it.n_begin; nt < it.n_end && ok; ++nt) {
          if (!A3PO_TIMED_WAIT(waited2, mbar_wait(&tmem_empty_bar[acc], acc_phase ^ 1u, abort_flag))) { ok = false; break; }
          tcgen05_fence_after_sync();
          const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(acc * BN * MT);
          for (int kb = 0; kb < k_blocks; ++kb) {
            if (!A3PO_TIMED_WAIT(waited, mbar_wait(&full_bar[stage], phase, abort_flag))) { ok = false; break; }
            tcgen05_fence_after_sync();
            const uint32_t sa = smem_u32(smem_a + stage * kAStage);
            const uint32_t sb = smem_u32(smem_b + stage * kBBytes);
            const uint64_t desc_a = A_MN ? umma_desc_mn_major_sw128(sa, kMnBlockBytes) : umma_desc_k_major_sw128(sa);
            const uint64_t desc_b = B_MN ? umma_desc_mn_major_sw128(sb, kMnBlockBytes) : umma_desc_k_major_sw128(sb);
#pragma unroll
            for (int k = 0; k < BK / 16; ++k) {
#pragma unroll
              for (int mt = 0; mt < MT; ++mt)   // the A tiles of a stage lie kABytes apart (either major-ness)
                umma_bf16(tmem_d + static_cast<uint32_t>(mt * BN), desc_a + mt * (kABytes >> 4) + a_step * k,
                          desc_b + b_step * k, idesc, (kb | k) != 0 ? 1u : 0u);
            }
            umma_commit(&empty_bar[stage]);  // stage reusable once these MMAs have read it
            if (++stage == kStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) umma_commit(&tmem_full_bar[acc]);
          if (++acc == kAccStages) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps
    const int quarter = warp & 3;  // TMEM lanes this warp may read: 32*quarter .. +31
    const int row_in_tile = quarter * 32 + lane;
    int acc = 0;
    uint32_t acc_phase = 0;
    Epi epi;
    SlabStore st;
    st.slab0 = smem_slabs;
    st.slab1 = smem_slabs + kSlabBytes;
    st.map = &map_c;
    st.row_in_tile = row_in_tile;
    st.issuer = (threadIdx.x == 2 * kWarp);
    for (long long i = blockIdx.x; i < im.items && ok; i += gridDim.x) {
      const Item it = decode_item(im, i);
      const int item_row0 = it.m_tile * (BM * MT);
      if (MT == 1) epi.begin(ep, static_cast<long long>(item_row0) + row_in_tile);
      for (int nt = it.n_begin; nt < it.n_end && ok; ++nt) {
        // the four epilogue warps share named barriers further down: they must agree on giving up
        if (!zero_output) {
          ok = all_epilogue_threads(A3PO_TIMED_WAIT(waited, mbar_wait(&tmem_full_bar[acc], acc_phase, abort_flag)));
          if (!ok) break;
          tcgen05_fence_after_sync();
        }
#pragma unroll 1
        for (int mt = 0; mt < MT; ++mt) {
          const int tile_row0 = item_row0 + mt * BM;
          // epilogues of the MT = 2 kernels keep no state from one column tile to the next
          if (MT > 1) epi.begin(ep, static_cast<long long>(tile_row0) + row_in_tile);
          const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) +
                                 static_cast<uint32_t>(acc * BN * MT + mt * BN);
#pragma unroll 1
          for (int c = 0; c < BN / kEpiChunk; ++c) {
            uint32_t r[kEpiChunk];
            if (!zero_output) {
              tmem_ld_32x32(taddr + static_cast<uint32_t>(c * kEpiChunk), r);
              tmem_ld_wait();
            } else {
#pragma unroll
              for (int j = 0; j < kEpiChunk; ++j) r[j] = 0u;
            }
            epi.chunk(ep, tile_row0, nt * BN + c * kEpiChunk, r, st);
          }
        }
        if (!zero_output) {
          tcgen05_fence_before_sync();
          __syncwarp();
          if (lane == 0) mbar_arrive(&tmem_empty_bar[acc]);
          if (++acc == kAccStages) { acc = 0; acc_phase ^= 1u; }
        }
      }
      if (MT == 1 && ok) epi.end(ep, static_cast<long long>(item_row0) + row_in_tile, it.split);
    }
    st.drain();  // shared memory must stay valid until the copy engine has read every submitted slab
  }

#ifdef A3PO_TUNING
  if (lane == 0 || (warp < 2)) {
    if (warp == 0 && waited) trace_wait[0] = waited;
    if (warp == 1 && waited) trace_wait[1] = waited;
    if (warp == 1 && waited2) trace_wait[2] = waited2;
    if (warp == 2 && lane == 0) trace_wait[3] = waited;
  }
#endif
  if (!ok) {
    *abort_flag = 1;
    if (status) atomicOr(status, A3PO_STATUS_WAIT_TIMEOUT);
    __nanosleep(200000);  // let copies / MMAs already in flight drain before TMEM is released
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    tcgen05_fence_after_sync();
    tmem_dealloc(tmem_base, kTmemCols);
  }
#ifdef A3PO_TUNING
  if (threadIdx.x == 0 && g_trace != nullptr) {
    const unsigned int slot = atomicAdd(&g_trace_next, 1u);
    if (slot < g_trace_capacity) {
      unsigned long long mine = 0;
      for (long long i = blockIdx.x; i < im.items; i += gridDim.x) ++mine;
      g_trace[slot] = TraceRecord{trace_t0, globaltimer_ns(), static_cast<unsigned long long>(clock64()) - trace_c0,
                                  (static_cast<unsigned long long>(Epi::kKernelId) << 48) |
                                      (static_cast<unsigned long long>(blockIdx.x) << 32) | mine,
                                  trace_wait[0], trace_wait[1], trace_wait[2], trace_wait[3]};
    }
  }
#endif
}

// ------------------------------------------------------------------------------------ the pair kernel
// The same contraction with both operands K-major, run by pairs of CTAs on neighbouring SMs (clusters of two,
// tcgen05 cta_group::2).  A pair owns a 256-row output tile: each CTA loads its own 128 rows of A and only ITS
// half (128 of 256 rows) of every B tile, the leader's MMAs (M = 256) read both halves, and each CTA finds its
// 128 x 256 accumulator in its own tensor memory and runs the epilogue on it.  Per flop a CTA then pulls a third
// fewer operand bytes out of L2 and through shared memory than with a full B tile of its own, which is where the
// single-CTA kernel saturates when the SM clock is high.  Accumulators stay double-buffered (the epilogue of one
// tile overlaps the MMAs of the next), so this is the kernel for the epilogue-heavy forward contractions.
// Every CTA fetches its own tiles (no multicast).  Barriers: "stage filled" lives in the leader (both CTAs' loads
// signal it), "stage free" and "accumulator ready" exist in both CTAs (the leader's commit arrives on both),
// "accumulator free" lives in the leader and collects the eight epilogue warps of the pair.
constexpr int kPairStages = 6;
constexpr uint32_t kPairStageBytes = kABytes + kBBytes / 2;   // per CTA: 128 x 64 of A, 128 x 64 of B
constexpr size_t kPairSmemBytes = 1024 + kPairStages * kPairStageBytes + 2 * kSlabBytes + 256;

template <class Epi>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kTcThreads, 1)
gemm_pair_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
                 const __grid_constant__ CUtensorMap map_c, ItemMap im_static, int k_blocks,
                 typename Epi::Params ep, uint32_t* status) {
  constexpr int kPairRows = 2 * BM;
  ItemMap im = im_static;   // m_tiles counts 256-row pair tiles here
  if (im.dyn_rows != nullptr) {
    long long rows = static_cast<long long>(*im.dyn_rows) - im.dyn_offset;
    rows = rows < 0 ? 0 : (rows > im.dyn_cap ? im.dyn_cap : rows);
    im.m_tiles = static_cast<int>((rows + kPairRows - 1) / kPairRows);
    im.items = static_cast<long long>(im.m_tiles) * im.splits;
  }
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + kPairStages * kABytes;
  uint8_t* smem_slabs = smem + kPairStages * kPairStageBytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem_slabs + 2 * kSlabBytes);
  uint64_t* empty_bar = full_bar + kPairStages;
  uint64_t* tmem_full_bar = empty_bar + kPairStages;
  uint64_t* tmem_empty_bar = tmem_full_bar + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tmem_empty_bar + 2);
  volatile uint32_t* abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x / kWarp;
  const int lane = threadIdx.x % kWarp;
  const uint32_t rank = cluster_ctarank();         // 0 = leader
  const long long pair_id = blockIdx.x >> 1;
  const long long n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kPairStages; ++i) {
      mbar_init(&full_bar[i], 1);    // used in the leader only: its producer's arrive + the bytes of both CTAs
      mbar_init(&empty_bar[i], 1);   // one arrival: the leader's commit
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&tmem_full_bar[i], 1);
      mbar_init(&tmem_empty_bar[i], 8);  // used in the leader only: four epilogue warps in each CTA
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 0 && lane == 0) {
    prefetch_tensormap(&map_a);
    prefetch_tensormap(&map_b);
  }
  if (warp == 1) {   // the same warp in both CTAs, together
    tmem_alloc_pair(tmem_slot, kTmemCols);
    tmem_relinquish_alloc_permit_pair();
  }
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();   // the peer's barriers exist before anything signals them
  tcgen05_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  bool ok = true;
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer (both CTAs)
    if (elect_one()) {
      const uint32_t leader_full = map_to_cta(smem_u32(&full_bar[0]), 0);
      int stage = 0;
      uint32_t phase = 0;
      for (long long i = pair_id; i < im.items && ok; i += n_pairs) {
        const Item it = decode_item(im, i);
        const int row0 = it.m_tile * kPairRows + static_cast<int>(rank) * BM;
        for (int nt = it.n_begin; nt < it.n_end && ok; ++nt) {
          const int col0 = nt * BN + static_cast<int>(rank) * (BN / 2);
          for (int kb = 0; kb < k_blocks; ++kb) {
            if (!mbar_wait(&empty_bar[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
            if (rank == 0) mbar_arrive_expect_tx(&full_bar[stage], 2 * kPairStageBytes);
            const uint32_t bar = leader_full + static_cast<uint32_t>(stage * sizeof(uint64_t));
            tma_load_2d_pair(smem_a + stage * kABytes, &map_a, bar, kb * BK, row0);
            tma_load_2d_pair(smem_b + stage * (kBBytes / 2), &map_b, bar, kb * BK, col0);
            if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
          }
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer (leader only)
    if (rank == 0 && elect_one()) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(kPairRows, BN, false, false);
      int stage = 0;
      uint32_t phase = 0;
      int acc = 0;
      uint32_t acc_phase = 0;
      for (long long i = pair_id; i < im.items && ok; i += n_pairs) {
        const Item it = decode_item(im, i);
        for (int nt = it.n_begin; nt < it.n_end && ok; ++nt) {
          if (!mbar_wait(&tmem_empty_bar[acc], acc_phase ^ 1u, abort_flag)) { ok = false; break; }
          tcgen05_fence_after_sync();
          const uint32_t tmem_d = tmem_base + static_cast<uint32_t>(acc * BN);
          for (int kb = 0; kb < k_blocks; ++kb) {
            if (!mbar_wait(&full_bar[stage], phase, abort_flag)) { ok = false; break; }
            tcgen05_fence_after_sync();
            const uint64_t desc_a = umma_desc_k_major_sw128(smem_u32(smem_a + stage * kABytes));
            const uint64_t desc_b = umma_desc_k_major_sw128(smem_u32(smem_b + stage * (kBBytes / 2)));
#pragma unroll
            for (int k = 0; k < BK / 16; ++k)
              umma_bf16_pair(tmem_d, desc_a + 2 * k, desc_b + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
            umma_commit_pair(&empty_bar[stage], 3);   // both CTAs may refill the stage
            if (++stage == kPairStages) { stage = 0; phase ^= 1u; }
          }
          if (ok) umma_commit_pair(&tmem_full_bar[acc], 3);
          if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue warps (both CTAs)
    const int quarter = warp & 3;
    const int row_in_tile = quarter * 32 + lane;
    const uint32_t leader_tmem_empty = map_to_cta(smem_u32(&tmem_empty_bar[0]), 0);
    int acc = 0;
    uint32_t acc_phase = 0;
    Epi epi;
    SlabStore st;
    st.slab0 = smem_slabs;
    st.slab1 = smem_slabs + kSlabBytes;
    st.map = &map_c;
    st.row_in_tile = row_in_tile;
    st.issuer = (threadIdx.x == 2 * kWarp);
    for (long long i = pair_id; i < im.items && ok; i += n_pairs) {
      const Item it = decode_item(im, i);
      const int tile_row0 = it.m_tile * kPairRows + static_cast<int>(rank) * BM;
      epi.begin(ep, static_cast<long long>(tile_row0) + row_in_tile);
      for (int nt = it.n_begin; nt < it.n_end && ok; ++nt) {
        ok = all_epilogue_threads(mbar_wait(&tmem_full_bar[acc], acc_phase, abort_flag));
        if (!ok) break;
        tcgen05_fence_after_sync();
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + static_cast<uint32_t>(acc * BN);
#pragma unroll 1
        for (int c = 0; c < BN / kEpiChunk; ++c) {
          uint32_t r[kEpiChunk];
          tmem_ld_32x32(taddr + static_cast<uint32_t>(c * kEpiChunk), r);
          tmem_ld_wait();
          epi.chunk(ep, tile_row0, nt * BN + c * kEpiChunk, r, st);
        }
        tcgen05_fence_before_sync();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(leader_tmem_empty + static_cast<uint32_t>(acc * sizeof(uint64_t)));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (ok) epi.end(ep, static_cast<long long>(tile_row0) + row_in_tile, it.split);
    }
    st.drain();
  }

  if (!ok) {
    *abort_flag = 1;
    if (status) atomicOr(status, A3PO_STATUS_WAIT_TIMEOUT);
    __nanosleep(200000);
  }
  // neither CTA may leave (or give up its tensor memory) while the other can still read its shared memory or
  // signal its barriers
  tcgen05_fence_before_sync();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    tcgen05_fence_after_sync();
    tmem_dealloc_pair(tmem_base, kTmemCols);
  }
}

// ------------------------------------------------------------------------------------ host side
// One GEMM operand as it lies in memory (bf16, row-major with `pitch` elements per row).
//   K-major : tensor [mn_extent rows, k_extent cols]   -> boxes of tile_mn rows x 64 k
//   MN-major: tensor [k_extent rows, mn_extent cols]   -> boxes of 64 k rows x 64 M/N elements
// Out-of-range elements read as zero, which is what makes ragged M, N and K tails work.
struct Operand {
  const void* base;
  long long mn_extent;
  long long k_extent;
  long long pitch;
};

int make_map(CUtensorMap* map, const Operand& op, bool mn_major, int tile_mn) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return A3PO_ERR_CUDA;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(mn_major ? op.mn_extent : op.k_extent),
                              static_cast<cuuint64_t>(mn_major ? op.k_extent : op.mn_extent)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(op.pitch) * 2};
  const cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(mn_major ? BK : tile_mn)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(op.base), dims, strides, box,
                        estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? A3PO_OK : A3PO_ERR_CUDA;
}

// Tuning overrides (positive integers read from the environment) exist only in builds made with
// -DA3PO_TUNING, for sweeps; a normal build takes the defaults and reads no environment variable.
int tuning_override(const char* name, int fallback) {
#ifdef A3PO_TUNING
  const char* e = std::getenv(name);
  if (!e) return fallback;
  const int v = std::atoi(e);
  return v > 0 ? v : fallback;
#else
  (void)name;
  return fallback;
#endif
}

// Pacing counters (see Pace) live in the library's device image, 8 KB per GPU: all zero when the library is
// loaded, and every paced launch leaves its block zero again.  In host code the array's name is only a handle for
// cudaGetSymbolAddress.
__device__ __align__(256) unsigned int g_pace_counters[kPaceBlocks * kPaceBlockWords];
unsigned int* next_pace_block() {
  static std::mutex mu;
  static unsigned int* cached[64];
  static unsigned int turn[64];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return nullptr;
  }
  std::lock_guard<std::mutex> lock(mu);
  if (!cached[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_pace_counters) != cudaSuccess || !p) {
      cudaGetLastError();
      return nullptr;   // the launch then runs unpaced
    }
    cached[dev] = static_cast<unsigned int*>(p);
  }
  return cached[dev] + static_cast<size_t>(turn[dev]++ % kPaceBlocks) * kPaceBlockWords;
}

// Row tiles per group for the forward contractions.  With G row tiles per group the CTAs of a launch work on
// SMs / G vocabulary splits of the same G row tiles at a time (items are split-major inside a group): every W tile
// comes out of HBM once per G row tiles, and the G row tiles of the other operand (G x 128 x K x 2 bytes) have to
// stay in L2 while the column tiles are swept.  G = the largest of SMs, SMs/2, SMs/4, ... whose row tiles fit
// kFwdGroupBytes.  Measured on the 8B-shaped batch (K = 4096, 65,536 rows, paced CTAs), HBM bytes read by one
// launch: G = 4: 58 GB, 16: 50 GB, 37: 23 GB, 74: 155 GB (the row tiles no longer fit).
int fwd_group_m(long long k_extent) {
  const long long tile_bytes = static_cast<long long>(BM) * k_extent * 2;
  int g = sm_count();
  if (g <= 0) g = 148;
  while (g > kGroupM && g * tile_bytes > kFwdGroupBytes) g /= 2;
  return g > kGroupM ? g : kGroupM;
}

// Device-resident row count for a launch (see ItemMap).
struct DynRows {
  const int* rows = nullptr;
  int is_k = 0;
  int zero_when_empty = 0;
  long long offset = 0;
  long long cap = 0;
  const int* select = nullptr;
  int select_value = 0;
};

// C[M, N] = sum_k A[m, k] B[n, k];  splits = 0 means one column tile per work item.
template <class Epi, bool A_MN, bool B_MN, int MT = 1>
int launch_gemm(const Operand& a, const Operand& b, int splits, const typename Epi::Params& ep, const DynRows& dyn,
                uint32_t* status, cudaStream_t stream) {
  constexpr size_t kSmemBytes = TileCfg<MT>::kSmemBytes;
  CUtensorMap map_a, map_b, map_c;
  A3PO_RETURN_IF(make_map(&map_a, a, A_MN, BM * MT));
  A3PO_RETURN_IF(make_map(&map_b, b, B_MN, BN));
  A3PO_RETURN_IF(Epi::make_c_map(ep, &map_c));
  ItemMap im;
  im.m_tiles = static_cast<int>((a.mn_extent + BM * MT - 1) / (BM * MT));
  im.n_tiles = static_cast<int>((b.mn_extent + BN - 1) / BN);
  im.splits = splits > 0 ? splits : im.n_tiles;
  im.items = static_cast<long long>(im.m_tiles) * im.splits;
  // hidden x W^T with one tile per item (the recomputed dz) sweeps W like the forward does
  constexpr bool kForwardLike = !A_MN && !B_MN;
  im.group_m = splits > 0 ? tuning_override("A3PO_GROUP_M", fwd_group_m(a.k_extent))
               : kForwardLike ? tuning_override("A3PO_GROUP_M_DZ", fwd_group_m(a.k_extent))
                              : tuning_override("A3PO_GROUP_M_GRAD", kGroupM);
  im.dyn_rows = dyn.rows;
  im.dyn_is_k = dyn.is_k;
  im.zero_when_empty = dyn.zero_when_empty;
  im.dyn_offset = dyn.offset;
  im.dyn_cap = dyn.cap;
  im.select = dyn.select;
  im.select_value = dyn.select_value;
  im.pace_period = tuning_override("A3PO_PACE_PERIOD", kPacePeriod);
  im.pace_slack = tuning_override("A3PO_PACE_SLACK", kPaceSlack);
  if (im.pace_slack > kPaceRing / 2) im.pace_slack = kPaceRing / 2;   // a slot must not be reused while waited on
  im.pace = tuning_override("A3PO_PACE_OFF", 0) == 1 ? nullptr : next_pace_block();
  const int k_blocks = static_cast<int>((a.k_extent + BK - 1) / BK);
  auto kernel = gemm_tn_kernel<Epi, A_MN, B_MN, MT>;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemBytes)) !=
      cudaSuccess) {
    cudaGetLastError();
    return A3PO_ERR_CUDA;
  }
  long long grid = sm_count();
  if (grid > im.items) grid = im.items;
  if (grid < 1) return A3PO_OK;
  A3PO_LAUNCH(Epi::kKernelId, stream, (kernel<<<static_cast<unsigned>(grid), kTcThreads, kSmemBytes, stream>>>(
                                          map_a, map_b, map_c, im, k_blocks, ep, status)));
  return after_launch();
}

// Pairs of CTAs that can be resident at once (the kernel is persistent: one pair per two SMs).
template <class Epi>
int pair_capacity() {
  static std::mutex mu;
  static int cached[64];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return 0;
  }
  std::lock_guard<std::mutex> lock(mu);
  if (cached[dev] == 0) {
    auto kernel = gemm_pair_kernel<Epi>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kPairSmemBytes)) !=
        cudaSuccess) {
      cudaGetLastError();
      return 0;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(sm_count() / 2 * 2));
    cfg.blockDim = dim3(kTcThreads);
    cfg.dynamicSmemBytes = kPairSmemBytes;
    cudaLaunchAttribute attr;
    attr.id = cudaLaunchAttributeClusterDimension;
    attr.val.clusterDim.x = 2;
    attr.val.clusterDim.y = 1;
    attr.val.clusterDim.z = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    int clusters = 0;
    if (cudaOccupancyMaxActiveClusters(&clusters, kernel, &cfg) != cudaSuccess) {
      cudaGetLastError();
      clusters = -1;
    }
    cached[dev] = clusters > 0 ? clusters : -1;
#ifdef A3PO_TUNING
    fprintf(stderr, "[a3po tuning] CTA pairs resident at once: %d\n", clusters);
#endif
  }
  return cached[dev] > 0 ? cached[dev] : 0;
}

// C[M, N] = sum_k A[m, k] B[n, k], both K-major, on CTA pairs; `splits` vocabulary splits per 256-row pair tile.
template <class Epi>
int launch_pair_gemm(const Operand& a, const Operand& b, int splits, const typename Epi::Params& ep, const DynRows& dyn,
                     uint32_t* status, cudaStream_t stream) {
  const int pairs_max = pair_capacity<Epi>();
  if (pairs_max <= 0) return A3PO_ERR_UNSUPPORTED;
  CUtensorMap map_a, map_b, map_c;
  A3PO_RETURN_IF(make_map(&map_a, a, false, BM));
  A3PO_RETURN_IF(make_map(&map_b, b, false, BN / 2));
  A3PO_RETURN_IF(Epi::make_c_map(ep, &map_c));
  ItemMap im;
  im.m_tiles = static_cast<int>((a.mn_extent + 2 * BM - 1) / (2 * BM));
  im.n_tiles = static_cast<int>((b.mn_extent + BN - 1) / BN);
  im.splits = splits > 0 ? splits : im.n_tiles;
  im.items = static_cast<long long>(im.m_tiles) * im.splits;
  im.group_m = tuning_override("A3PO_GROUP_M", kGroupM);
  im.dyn_rows = dyn.rows;
  im.dyn_is_k = 0;
  im.zero_when_empty = 0;
  im.dyn_offset = dyn.offset;
  im.dyn_cap = dyn.cap;
  im.select = nullptr;
  im.select_value = 0;
  im.pace = nullptr;
  im.pace_period = 0;
  im.pace_slack = 0;
  const int k_blocks = static_cast<int>((a.k_extent + BK - 1) / BK);
  long long pairs = pairs_max;
  if (pairs > im.items) pairs = im.items;
  if (pairs < 1) return A3PO_OK;
  auto kernel = gemm_pair_kernel<Epi>;
  A3PO_LAUNCH(Epi::kKernelId, stream, (kernel<<<static_cast<unsigned>(2 * pairs), kTcThreads, kPairSmemBytes, stream>>>(
                                          map_a, map_b, map_c, im, k_blocks, ep, status)));
  return after_launch();
}

// Which tile a contraction over `rows` output rows and n_tiles column tiles should take.  The 256 x 256 tile moves a
// third fewer operand bytes per flop, but its work items are twice as coarse; with few items per SM the idle tail
// of the last wave costs more than that saves.  efficiency = items / (waves * SMs).
__host__ __device__ inline int choose_mt(long long rows, int n_tiles, int sms) {
  if (rows <= 0 || sms <= 0) return 2;
  const long long i1 = (rows + BM - 1) / BM * n_tiles, i2 = (rows + 2 * BM - 1) / (2 * BM) * n_tiles;
  const double e1 = static_cast<double>(i1) / static_cast<double>((i1 + sms - 1) / sms * sms);
  const double e2 = static_cast<double>(i2) / static_cast<double>((i2 + sms - 1) / sms * sms);
  return e2 >= 0.93 * e1 ? 2 : 1;
}

__global__ void choose_mt_kernel(const int* __restrict__ rows_ptr, long long offset, long long cap, int n_tiles,
                                 int sms, int* __restrict__ out) {
  long long rows = static_cast<long long>(*rows_ptr) - offset;
  rows = rows < 0 ? 0 : (rows > cap ? cap : rows);
  *out = choose_mt(rows, n_tiles, sms);
}

// The gradient contractions.  rows_are_m: the (possibly device-resident) row count is the M extent (grad_hidden),
// so the tile is chosen from it, on the device when it lives there (both variants are launched, one of them
// exits at once; `select` is a device int the choice is written to).  Otherwise (grad_w: M = V) the 256 x 256
// tile always pays.
template <class Epi, bool A_MN, bool B_MN>
int launch_grad_gemm(const Operand& a, const Operand& b, const typename Epi::Params& ep, DynRows dyn, bool rows_are_m,
                     int* select, uint32_t* status, cudaStream_t stream) {
  const int forced = tuning_override("A3PO_GRAD_MT", 0);
  const int n_tiles = static_cast<int>((b.mn_extent + BN - 1) / BN);
  int mt = 2;
  if (forced == 1 || forced == 2) {
    mt = forced;
  } else if (rows_are_m && dyn.rows != nullptr && select != nullptr) {
    A3PO_LAUNCH(kKCompact, stream, (choose_mt_kernel<<<1, 1, 0, stream>>>(dyn.rows, dyn.offset, dyn.cap, n_tiles,
                                                                          sm_count(), select)));
    A3PO_RETURN_IF(after_launch());
    dyn.select = select;
    dyn.select_value = 1;
    A3PO_RETURN_IF((launch_gemm<Epi, A_MN, B_MN, 1>(a, b, 0, ep, dyn, status, stream)));
    dyn.select_value = 2;
    return launch_gemm<Epi, A_MN, B_MN, 2>(a, b, 0, ep, dyn, status, stream);
  } else if (rows_are_m) {
    mt = choose_mt(a.mn_extent, n_tiles, sm_count());
  }
  if (mt == 1) return launch_gemm<Epi, A_MN, B_MN, 1>(a, b, 0, ep, dyn, status, stream);
  return launch_gemm<Epi, A_MN, B_MN, 2>(a, b, 0, ep, dyn, status, stream);
}

// Scratch of the backward: one bf16 dz chunk [chunk_rows, vpad].
size_t bwd_dz_bytes(long long chunk_rows, int v) {
  const size_t vpad = round_up(static_cast<size_t>(v), 8);
  return round_up(static_cast<size_t>(chunk_rows) * vpad * 2, 256);
}
// ... followed by one int (the tile choice of the chunk's grad_hidden launch)
size_t bwd_ws_layout(long long chunk_rows, int v) { return bwd_dz_bytes(chunk_rows, v) + 256; }

}  // namespace

#ifdef A3PO_TUNING
}  // namespace a3po
// Tuning builds only (not part of the ABI in include/): where the GEMM kernels record their per-CTA trace.
// `records` is a device buffer of `capacity` 64-byte records, or null to stop tracing; resets the write position.
extern "C" int a3po_tuning_set_trace(void* records, unsigned int capacity) {
  a3po::TraceRecord* p = static_cast<a3po::TraceRecord*>(records);
  unsigned int zero = 0;
  if (cudaMemcpyToSymbol(a3po::g_trace, &p, sizeof(p)) != cudaSuccess ||
      cudaMemcpyToSymbol(a3po::g_trace_capacity, &capacity, sizeof(capacity)) != cudaSuccess ||
      cudaMemcpyToSymbol(a3po::g_trace_next, &zero, sizeof(zero)) != cudaSuccess) {
    cudaGetLastError();
    return A3PO_ERR_CUDA;
  }
  return A3PO_OK;
}
extern "C" unsigned int a3po_tuning_trace_count() {
  unsigned int n = 0;
  if (cudaMemcpyFromSymbol(&n, a3po::g_trace_next, sizeof(n)) != cudaSuccess) cudaGetLastError();
  return n;
}
namespace a3po {
#endif

// Exercises the bounded wait the pipelines rely on: a barrier nothing ever arrives at.
int selftest_wait_timeout(uint32_t* status, unsigned timeout_ms, cudaStream_t stream) {
  A3PO_LAUNCH(kKSelfTest, stream, (wait_timeout_kernel<<<1, 32, 0, stream>>>(
                                      status, static_cast<unsigned long long>(timeout_ms) * 1000000ull)));
  return after_launch();
}

bool lmhead_tc_supported(const void* hidden, const void* w, long long n, int h, int v) {
  return n > 0 && h >= 8 && (h % 8) == 0 && v >= 1 && aligned_to(hidden, 16) && aligned_to(w, 16) &&
         n < (1ll << 31) - 256;
}

// Whether the forward contractions run on CTA pairs (gemm_pair_kernel).  Off: measured on B200 under its power
// cap (seconds-long loops on one GPU) the pair kernel sustains 1083 TFLOP/s against 1241 for the single-CTA
// kernel on the same forward, although its tensor pipe is busier when the clock is free (99 % against 90 % under
// the profiler).  A tuning build switches it on with A3PO_FWD_PAIR=1 for comparisons and for its parity test.
bool fwd_uses_pairs() {
  if (tuning_override("A3PO_FWD_PAIR", 2) != 1) return false;
  return pair_capacity<KeepEpilogue<false>>() > 0;
}

// Picks the number of vocabulary splits so that (row tiles x splits) items spread evenly over
// the workers (SMs, or CTA pairs with 256-row tiles; static round-robin) while every item still sweeps several
// column tiles.  With G row tiles per group and SMs / G splits in flight, a split count that is a multiple of
// SMs / G makes every full group a whole number of waves, so that the CTAs never hold the row tiles of two
// groups at once (8B-shaped batch, 65,536 rows: 23 GB read from HBM per launch against 47 GB with 13 splits).
int lmhead_tc_fwd_splits(long long n, int h, int v) {
  const bool pairs = fwd_uses_pairs();
  const int tile_rows = pairs ? 2 * BM : BM;
  const long long m_tiles = (n + tile_rows - 1) / tile_rows;
  const int n_tiles = (v + BN - 1) / BN;
  if (m_tiles <= 0) return 1;
  int workers = pairs ? pair_capacity<KeepEpilogue<false>>() : sm_count();
  if (workers <= 0) workers = pairs ? 74 : 148;
  const int forced = tuning_override("A3PO_FWD_SPLITS", 0);
  if (forced > 0) return forced < n_tiles ? (forced < 64 ? forced : 64) : n_tiles;
  const int s_max = n_tiles < 64 ? n_tiles : 64;
  int s_min = s_max < 8 ? s_max : 8;  // several splits in flight keep the row-tile working set inside L2
  int step = 1;
  if (!pairs) {
    const int group = tuning_override("A3PO_GROUP_M", fwd_group_m(h));
    if (group > kGroupM && m_tiles >= group && workers % group == 0 && workers / group <= s_max) step = workers / group;
  }
  int best = 0;
  double best_cost = 1e300;
  for (int s = (s_min + step - 1) / step * step; s <= s_max; s += step) {
    const long long items = m_tiles * s;
    const long long waves = (items + workers - 1) / workers;
    const long long tiles_per_item = (n_tiles + s - 1) / s;
    const double cost = static_cast<double>(waves) * (static_cast<double>(tiles_per_item) + 0.5);
    if (cost < best_cost - 1e-9) { best_cost = cost; best = s; }
  }
  return best > 0 ? best : s_min;
}

int lmhead_fwd_tc(const void* hidden, const void* w, const int32_t* targets, long long n, int h, int v, float inv_t,
                  int splits, SoftmaxPartial* part, float* part_ent, float* zy, const int* dyn_rows, uint32_t* status,
                  cudaStream_t stream) {
  const Operand a{hidden, n, h, h};
  const Operand b{w, v, h, h};
  DynRows dyn;
  dyn.rows = dyn_rows;
  dyn.cap = n;
  const bool pairs = fwd_uses_pairs();
  if (part_ent) {
    FwdEpilogue<true>::Params p{targets, n, v, inv_t * kLog2e, inv_t, part, part_ent, zy};
    if (pairs) return launch_pair_gemm<FwdEpilogue<true>>(a, b, splits, p, dyn, status, stream);
    return launch_gemm<FwdEpilogue<true>, false, false>(a, b, splits, p, dyn, status, stream);
  }
  FwdEpilogue<false>::Params p{targets, n, v, inv_t * kLog2e, inv_t, part, nullptr, zy};
  if (pairs) return launch_pair_gemm<FwdEpilogue<false>>(a, b, splits, p, dyn, status, stream);
  return launch_gemm<FwdEpilogue<false>, false, false>(a, b, splits, p, dyn, status, stream);
}

size_t lmhead_tc_kept_bytes(long long rows, int v) {
  const size_t vpad = round_up(static_cast<size_t>(v), 8);
  return round_up(static_cast<size_t>(rows > 0 ? rows : 0) * vpad * 2, 256);
}

int lmhead_fwd_keep_tc(const void* hidden, const void* w, const int32_t* targets, const float* zy, long long n, int h,
                       int v, float inv_t, int splits, float* part_s, float* part_e, void* q, const int* dyn_rows,
                       long long dyn_offset, uint32_t* status, cudaStream_t stream) {
  const Operand a{hidden, n, h, h};
  const Operand b{w, v, h, h};
  DynRows dyn;
  dyn.rows = dyn_rows;
  dyn.offset = dyn_offset;
  dyn.cap = n;
  const int vpad = static_cast<int>(round_up(static_cast<size_t>(v), 8));
  const bool pairs = fwd_uses_pairs();
  if (part_e) {
    KeepEpilogue<true>::Params p{targets, zy, n, v, vpad, inv_t * kLog2e, inv_t, part_s, part_e,
                                 static_cast<__nv_bfloat16*>(q)};
    if (pairs) return launch_pair_gemm<KeepEpilogue<true>>(a, b, splits, p, dyn, status, stream);
    return launch_gemm<KeepEpilogue<true>, false, false>(a, b, splits, p, dyn, status, stream);
  }
  KeepEpilogue<false>::Params p{targets, zy, n, v, vpad, inv_t * kLog2e, inv_t, part_s, nullptr,
                                static_cast<__nv_bfloat16*>(q)};
  if (pairs) return launch_pair_gemm<KeepEpilogue<false>>(a, b, splits, p, dyn, status, stream);
  return launch_gemm<KeepEpilogue<false>, false, false>(a, b, splits, p, dyn, status, stream);
}

size_t lmhead_tc_bwd_ws_bytes(long long chunk_rows, long long /*n*/, int /*h*/, int v) {
  return bwd_ws_layout(chunk_rows, v);
}

int lmhead_bwd_tc(const void* hidden_, const void* w_, const int32_t* targets, const float* lse,
                  const float* grad_logp, long long n, int h, int v, float inv_t, void* grad_hidden_, float* grad_w,
                  int accumulate, void* ws, size_t ws_bytes, long long chunk_rows, const int* dyn_rows,
                  uint32_t* status, cudaStream_t stream) {
  const __nv_bfloat16* hidden = static_cast<const __nv_bfloat16*>(hidden_);
  const __nv_bfloat16* w = static_cast<const __nv_bfloat16*>(w_);
  __nv_bfloat16* grad_hidden = static_cast<__nv_bfloat16*>(grad_hidden_);
  if (bwd_ws_layout(chunk_rows, v) > ws_bytes) return A3PO_ERR_WORKSPACE;
  __nv_bfloat16* dz = static_cast<__nv_bfloat16*>(ws);  // [chunk_rows, vpad]
  int* select = reinterpret_cast<int*>(static_cast<char*>(ws) + bwd_dz_bytes(chunk_rows, v));
  const int vpad = static_cast<int>(round_up(static_cast<size_t>(v), 8));

  for (long long r0 = 0; r0 < n; r0 += chunk_rows) {
    const long long r1 = (r0 + chunk_rows < n) ? r0 + chunk_rows : n;
    const long long nc = r1 - r0;
    const __nv_bfloat16* hid_c = hidden + r0 * h;
    // dz[t, v] for this chunk of rows, from recomputed logits:  A = hidden (K-major), B = W (K-major)
    DzEpilogue::Params dp{targets, lse, grad_logp, r0, r1, v, vpad, inv_t * kLog2e, inv_t, dz};
    DynRows dyn_m;  // dz and grad_hidden: the rows are the M extent
    dyn_m.rows = dyn_rows;
    dyn_m.offset = r0;
    dyn_m.cap = nc;
    DynRows dyn_k = dyn_m;  // grad_w: the rows are the K extent
    dyn_k.is_k = 1;
    dyn_k.zero_when_empty = (r0 == 0 && !accumulate) ? 1 : 0;
    A3PO_RETURN_IF((launch_gemm<DzEpilogue, false, false>(Operand{hid_c, nc, h, h}, Operand{w, v, h, h}, 0, dp,
                                                          dyn_m, status, stream)));
    // grad_hidden[t, j] = sum_v dz[t, v] W[v, j]:  A = dz (K = v contiguous), B = W read N-major
    StoreBf16Epilogue::Params hp{grad_hidden + r0 * h, h, nc, h, nullptr};
    A3PO_RETURN_IF((launch_grad_gemm<StoreBf16Epilogue, false, true>(Operand{dz, nc, v, vpad}, Operand{w, h, v, h}, hp,
                                                                     dyn_m, true, select, status, stream)));
    // grad_w[v, j] (+)= sum_t dz[t, v] hidden[t, j]:  A = dz read M-major, B = hidden read N-major (K = t)
    StoreF32Epilogue::Params wp{grad_w, h, v, h, (accumulate || r0 > 0) ? 1 : 0};
    A3PO_RETURN_IF((launch_grad_gemm<StoreF32Epilogue, true, true>(Operand{dz, v, nc, vpad}, Operand{hid_c, h, nc, h},
                                                                   wp, dyn_k, false, nullptr, status, stream)));
  }
  return A3PO_OK;
}

// The two contractions of the backward on kept probability ratios q [n, v^8] (rows of one launch of the
// keeping forward, `dyn_offset` rows into the compact row space whose size is *dyn_rows):
//   grad_hidden[r, :] = row_scale[r] * sum_v q[r, v] W[v, :]
//   grad_w[v, :]    (+)= sum_r q[r, v] hs[r, :]                 hs = row_scale * hidden, made by the caller
// which equal dz W and dz^T hidden for dz[r, v] = row_scale[r] q[r, v].
int lmhead_grad_hidden_from_kept_tc(const void* q_, const void* w_, const float* row_scale, long long n, int h, int v,
                                    void* grad_hidden_, const int* dyn_rows, long long dyn_offset, int* select,
                                    uint32_t* status, cudaStream_t stream) {
  const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(q_);
  const __nv_bfloat16* w = static_cast<const __nv_bfloat16*>(w_);
  const int vpad = static_cast<int>(round_up(static_cast<size_t>(v), 8));
  DynRows dyn_m;
  dyn_m.rows = dyn_rows;
  dyn_m.offset = dyn_offset;
  dyn_m.cap = n;
  StoreBf16Epilogue::Params hp{static_cast<__nv_bfloat16*>(grad_hidden_), h, n, h, row_scale};
  return launch_grad_gemm<StoreBf16Epilogue, false, true>(Operand{q, n, v, vpad}, Operand{w, h, v, h}, hp, dyn_m, true,
                                                          select, status, stream);
}

int lmhead_grad_w_from_kept_tc(const void* q_, const void* hs_, long long n, int h, int v, float* grad_w,
                               int accumulate, int zero_when_empty, const int* dyn_rows, long long dyn_offset,
                               uint32_t* status, cudaStream_t stream) {
  const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(q_);
  const __nv_bfloat16* hs = static_cast<const __nv_bfloat16*>(hs_);
  const int vpad = static_cast<int>(round_up(static_cast<size_t>(v), 8));
  DynRows dyn_k;
  dyn_k.rows = dyn_rows;
  dyn_k.offset = dyn_offset;
  dyn_k.cap = n;
  dyn_k.is_k = 1;
  dyn_k.zero_when_empty = zero_when_empty;
  StoreF32Epilogue::Params wp{grad_w, h, v, h, accumulate ? 1 : 0};
  return launch_grad_gemm<StoreF32Epilogue, true, true>(Operand{q, v, n, vpad}, Operand{hs, h, n, h}, wp, dyn_k, false,
                                                        nullptr, status, stream);
}

}  // namespace a3po
