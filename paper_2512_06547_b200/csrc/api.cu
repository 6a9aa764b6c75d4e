// C ABI of the LM-head log-prob calls, the whole-step host entry and library-wide helpers.

#include <atomic>
#include <cstring>
#include <mutex>
#include <utility>
#include <vector>

#include "a3po_common.cuh"
#include "lmhead_internal.cuh"

namespace a3po {

std::atomic<long long> g_launches{0};

// ---- optional CUDA-event profile of every launch -------------------------------------------------
namespace {
struct ProfileRecord {
  int kernel_id;
  cudaEvent_t start, stop;
};
std::mutex g_profile_mu;
std::atomic<int> g_profile_on{0};
std::vector<ProfileRecord> g_profile_records;
std::vector<cudaEvent_t> g_event_pool;

cudaEvent_t take_event() {
  if (!g_event_pool.empty()) {
    cudaEvent_t e = g_event_pool.back();
    g_event_pool.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  if (cudaEventCreate(&e) != cudaSuccess) {
    cudaGetLastError();
    return nullptr;
  }
  return e;
}
}  // namespace

// The scope owns its two events until the launch has been bracketed; only then does the finished
// record enter the list, so a concurrent a3po_profile_read never sees (or recycles) half a record.
ProfileScope::ProfileScope(int id, cudaStream_t s) : kernel_id(id), stream(s), start(nullptr), stop(nullptr) {
  if (!g_profile_on.load(std::memory_order_relaxed)) return;
  {
    std::lock_guard<std::mutex> lock(g_profile_mu);
    start = take_event();
    stop = take_event();
  }
  if (!start || !stop) {
    std::lock_guard<std::mutex> lock(g_profile_mu);
    if (start) g_event_pool.push_back(start);
    if (stop) g_event_pool.push_back(stop);
    start = stop = nullptr;
    return;
  }
  cudaEventRecord(start, stream);
}

ProfileScope::~ProfileScope() {
  if (!start) return;
  cudaEventRecord(stop, stream);
  std::lock_guard<std::mutex> lock(g_profile_mu);
  g_profile_records.push_back(ProfileRecord{kernel_id, start, stop});
}

int sm_count() {
  static std::mutex mu;
  static int cached[64];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) {
    cudaGetLastError();
    return 0;
  }
  std::lock_guard<std::mutex> lock(mu);
  if (cached[dev] == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      cudaGetLastError();
      return 0;
    }
    cached[dev] = sms;
  }
  return cached[dev];
}

namespace {

constexpr int kMergeThreads = 256;
constexpr int kSimtTile = 64;
constexpr long long kSimtChunkRows = 4096;
constexpr long long kTcChunkRows = 16384;

// Combines the per-split online-softmax partials of each row:
//   M = max_i m_i, S = sum_i s_i exp(m_i - M), lse = M + log S, logp = z_y - lse,
//   entropy = lse - (sum_i e_i exp(m_i - M)) / S   with e_i = sum_v exp(z_v - m_i) z_v.
__global__ void __launch_bounds__(kMergeThreads)
merge_partials_kernel(const SoftmaxPartial* __restrict__ part, const float* __restrict__ part_ent,
                      const float* __restrict__ zy, const int32_t* __restrict__ targets,
                      const uint8_t* __restrict__ row_mask, const int* __restrict__ pos, long long n, int v,
                      int splits, float* __restrict__ logp, float* __restrict__ lse, float* __restrict__ entropy,
                      uint32_t* status) {
  const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= n) return;
  const int y = targets[t];
  if ((y < 0 || y >= v) && status) atomicOr(status, A3PO_STATUS_TARGET_OUT_OF_RANGE);
  // c = row of the partials: the row itself, or its place in the compact row space (-1: not computed)
  const long long c = pos ? static_cast<long long>(pos[t]) : t;
  if ((row_mask && row_mask[t] == 0) || c < 0) {
    logp[t] = 0.f;
    lse[t] = 0.f;
    if (entropy) entropy[t] = 0.f;
    return;
  }
  float m = -INFINITY;
  for (int i = 0; i < splits; ++i) m = fmaxf(m, part[static_cast<long long>(i) * n + c].m);
  float s = 0.f, e = 0.f;
  for (int i = 0; i < splits; ++i) {
    const SoftmaxPartial q = part[static_cast<long long>(i) * n + c];
    const float scale = expf(q.m - m);
    s = fmaf(q.s, scale, s);
    if (entropy) e = fmaf(part_ent[static_cast<long long>(i) * n + c], scale, e);
  }
  const float l = m + logf(s);
  lse[t] = l;
  logp[t] = zy[c] - l;
  if (entropy) entropy[t] = l - e / s;
}

// ORs A3PO_STATUS_TARGET_OUT_OF_RANGE into *status if any target lies outside [0, v).
__global__ void __launch_bounds__(kMergeThreads)
flag_bad_targets_kernel(const int32_t* __restrict__ targets, long long n, int v, uint32_t* status) {
  const long long t = static_cast<long long>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= n) return;
  const int y = targets[t];
  if (y < 0 || y >= v) atomicOr(status, A3PO_STATUS_TARGET_OUT_OF_RANGE);
}

int flag_bad_targets(const int32_t* targets, long long n, int v, uint32_t* status, cudaStream_t stream) {
  if (!status || n <= 0) return A3PO_OK;
  const unsigned blocks = static_cast<unsigned>((n + kMergeThreads - 1) / kMergeThreads);
  A3PO_LAUNCH(kKMergePartials, stream, (flag_bad_targets_kernel<<<blocks, kMergeThreads, 0, stream>>>(targets, n, v,
                                                                                                      status)));
  return after_launch();
}

int simt_fwd_splits(long long n, int v) {
  const long long row_tiles = (n + kSimtTile - 1) / kSimtTile;
  const int n_tiles = (v + kSimtTile - 1) / kSimtTile;
  int sms = sm_count();
  if (sms <= 0) sms = 148;
  long long s = row_tiles > 0 ? (static_cast<long long>(sms) * 4 + row_tiles - 1) / row_tiles : 1;
  if (s > n_tiles) s = n_tiles;
  if (s > 64) s = 64;
  if (s < 1) s = 1;
  return static_cast<int>(s);
}

size_t fwd_ws_for(long long n, int splits) {
  const size_t rows = static_cast<size_t>(n > 0 ? n : 0);
  return round_up(rows * splits * sizeof(SoftmaxPartial), 256) + round_up(rows * splits * sizeof(float), 256) +
         round_up(rows * sizeof(float), 256) + 256;
}

bool use_tc(a3po_dtype dt, const void* hidden, const void* w, long long n, int h, int v) {
  return dt == A3PO_BF16 && lmhead_tc_supported(hidden, w, n, h, v);
}

size_t elt_size(a3po_dtype dt) { return dt == A3PO_F32 ? 4 : 2; }

size_t simt_bwd_ws(long long chunk_rows, int v) {
  return round_up(static_cast<size_t>(chunk_rows) * v * sizeof(float), 256) + 256;
}

long long clamp_chunk(long long want, long long n, long long quantum) {
  long long c = want;
  const long long n_up = (n + quantum - 1) / quantum * quantum;
  if (c > n_up) c = n_up;
  if (c < quantum) c = quantum;
  return c;
}

int check_lmhead_args(const void* hidden, const void* w, const int32_t* targets, long long n, int h, int v,
                      a3po_dtype dt, float inv_t) {
  if (n < 0 || h <= 0 || v <= 0 || !(inv_t > 0.f)) return A3PO_ERR_INVALID_ARG;
  if (dt != A3PO_F32 && dt != A3PO_BF16) return A3PO_ERR_UNSUPPORTED;
  if (!w || (n > 0 && (!hidden || !targets))) return A3PO_ERR_INVALID_ARG;
  if (!aligned_to(hidden, 16) || !aligned_to(w, 16) || !aligned_to(targets, 4)) return A3PO_ERR_UNSUPPORTED;
  if (sm_count() <= 0) return A3PO_ERR_NO_DEVICE;
  return A3PO_OK;
}

}  // namespace
}  // namespace a3po

using namespace a3po;

extern "C" {

const char* a3po_status_string(int code) {
  switch (code) {
    case A3PO_OK: return "ok";
    case A3PO_ERR_INVALID_ARG: return "invalid argument";
    case A3PO_ERR_UNSUPPORTED: return "unsupported dtype, shape or alignment";
    case A3PO_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case A3PO_ERR_CUDA: return "CUDA call or kernel launch failed";
    case A3PO_ERR_NO_DEVICE: return "no usable CUDA device is current";
    case A3PO_ERR_TOO_LARGE: return "N exceeds the fixed scratch of a3po_loss_fwd_static (A3PO_LOSS_FWD_STATIC_MAX_TOKENS)";
    default: return "unknown a3po status";
  }
}

int a3po_version(void) { return 2000; }

int a3po_selftest_wait_timeout(uint32_t* status, unsigned timeout_ms, void* stream) {
  if (!status || timeout_ms == 0 || timeout_ms > 2000) return A3PO_ERR_INVALID_ARG;
  if (sm_count() <= 0) return A3PO_ERR_NO_DEVICE;
  return selftest_wait_timeout(status, timeout_ms, as_stream(stream));
}

int64_t a3po_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char* a3po_kernel_name(int kernel_id) {
  static const char* names[kKernelIdCount] = {
      "loss_fwd", "loss_bwd", "loss_fwd_bwd", "loss_finalize", "mask_count", "mask_count_finalize",
      "expand_versions", "merge_partials", "lmhead_fwd_fp32pipe", "lmhead_dz_fp32pipe", "gemm_fp32pipe",
      "gemm_tn<fwd_logsoftmax>", "gemm_tn<dz>", "gemm_tn<grad_hidden>", "gemm_tn<grad_w>", "compact_rows", "grpo_advantages", "selftest",
      "gemm_tn<fwd_logsoftmax+keep>", "kept_rows", "h2d_copies", "move_kept_rows"};
  return (kernel_id >= 0 && kernel_id < kKernelIdCount) ? names[kernel_id] : "?";
}

int a3po_profile_enable(int on) {
  std::lock_guard<std::mutex> lock(g_profile_mu);
  g_profile_on.store(on ? 1 : 0);
  return A3PO_OK;
}

int a3po_profile_read(int max_entries, int* kernel_ids, float* milliseconds, int* count) {
  if (!count || max_entries < 0 || (max_entries > 0 && (!kernel_ids || !milliseconds))) return A3PO_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_profile_mu);
  int n = 0;
  int rc = A3PO_OK;
  for (const ProfileRecord& r : g_profile_records) {
    float ms = 0.f;
    if (cudaEventSynchronize(r.stop) != cudaSuccess || cudaEventElapsedTime(&ms, r.start, r.stop) != cudaSuccess) {
      cudaGetLastError();
      rc = A3PO_ERR_CUDA;
    } else if (n < max_entries) {
      kernel_ids[n] = r.kernel_id;
      milliseconds[n] = ms;
      ++n;
    }
    g_event_pool.push_back(r.start);
    g_event_pool.push_back(r.stop);
  }
  g_profile_records.clear();
  *count = n;
  return rc;
}

size_t a3po_token_logprobs_min_workspace_bytes(int64_t N, int H, int V, a3po_dtype dt, int is_bwd) {
  if (N < 0 || H <= 0 || V <= 0) return 0;
  if (!is_bwd) {
    size_t a = fwd_ws_for(N, simt_fwd_splits(N, V));
    if (dt == A3PO_BF16) {
      const size_t b = fwd_ws_for(N, lmhead_tc_fwd_splits(N, H, V));
      if (b > a) a = b;
    }
    return a;
  }
  size_t a = simt_bwd_ws(kSimtTile, V);
  if (dt == A3PO_BF16) {
    const size_t b = lmhead_tc_bwd_ws_bytes(128, N, H, V);
    if (b > a) a = b;
  }
  return a;
}

size_t a3po_token_logprobs_workspace_bytes(int64_t N, int H, int V, a3po_dtype dt, int is_bwd) {
  if (N < 0 || H <= 0 || V <= 0) return 0;
  // the recommended size adds room for the row compaction of the tensor-core path
  const size_t compact = (dt == A3PO_BF16 && N > 0) ? compact_ws_bytes(N, H, is_bwd != 0) : 0;
  if (!is_bwd) return a3po_token_logprobs_min_workspace_bytes(N, H, V, dt, 0) + compact;
  size_t a = simt_bwd_ws(clamp_chunk(kSimtChunkRows, N, kSimtTile), V);
  if (dt == A3PO_BF16) {
    const size_t b = lmhead_tc_bwd_ws_bytes(clamp_chunk(kTcChunkRows, N, 128), N, H, V) + compact;
    if (b > a) a = b;
  }
  return a;
}

int a3po_token_logprobs_fwd(const void* hidden, const void* w, const int32_t* targets, const uint8_t* row_mask,
                            int64_t N, int H, int V, a3po_dtype dt, float inv_temperature, float* logp, float* lse,
                            float* entropy, void* ws, size_t ws_bytes, uint32_t* status, void* stream_) {
  A3PO_RETURN_IF(check_lmhead_args(hidden, w, targets, N, H, V, dt, inv_temperature));
  if (N > 0 && (!logp || !lse)) return A3PO_ERR_INVALID_ARG;
  if (N == 0) return A3PO_OK;
  if (!ws || !aligned_to(ws, 256)) return A3PO_ERR_WORKSPACE;
  cudaStream_t stream = as_stream(stream_);
  const bool tc = use_tc(dt, hidden, w, N, H, V);
  const int splits = tc ? lmhead_tc_fwd_splits(N, H, V) : simt_fwd_splits(N, V);
  if (ws_bytes < fwd_ws_for(N, splits)) return A3PO_ERR_WORKSPACE;
  // Masked rows are skipped, not computed: with a row mask and enough workspace the kept rows are
  // gathered into a compact buffer and the kernels run on that (count stays on the device).
  CompactBuffers cb;
  bool compacted = false;
  size_t ws_off = 0;
  if (tc && row_mask && ws_bytes >= fwd_ws_for(N, splits) + compact_ws_bytes(N, H, false)) {
    if (!compact_carve(ws, ws_bytes, N, H, false, &cb, &ws_off)) return A3PO_ERR_WORKSPACE;
    compacted = true;
  }
  Arena arena(static_cast<char*>(ws) + ws_off, ws_bytes - ws_off);
  SoftmaxPartial* part = arena.take<SoftmaxPartial>(static_cast<size_t>(N) * splits);
  float* part_ent = arena.take<float>(static_cast<size_t>(N) * splits);
  float* zy = arena.take<float>(static_cast<size_t>(N));
  if (!arena.ok()) return A3PO_ERR_WORKSPACE;
  if (!entropy) part_ent = nullptr;
  if (compacted) {
    A3PO_RETURN_IF(compact_rows(hidden, H, targets, row_mask, nullptr, nullptr, N, cb, stream));
    A3PO_RETURN_IF(lmhead_fwd_tc(cb.hidden_c, w, cb.targets_c, N, H, V, inv_temperature, splits, part, part_ent, zy,
                                 cb.count, status, stream));
  } else if (tc) {
    A3PO_RETURN_IF(lmhead_fwd_tc(hidden, w, targets, N, H, V, inv_temperature, splits, part, part_ent, zy, nullptr,
                                 status, stream));
  } else {
    A3PO_RETURN_IF(lmhead_fwd_simt(hidden, w, targets, N, H, V, dt, inv_temperature, splits, part, part_ent, zy,
                                   stream));
  }
  const unsigned blocks = static_cast<unsigned>((N + kMergeThreads - 1) / kMergeThreads);
  A3PO_LAUNCH(kKMergePartials, stream, (merge_partials_kernel<<<blocks, kMergeThreads, 0, stream>>>(
                                           part, part_ent, zy, targets, row_mask, compacted ? cb.pos : nullptr, N, V,
                                           splits, logp, lse, entropy, status)));
  return after_launch();
}

int a3po_token_logprobs_bwd(const void* hidden, const void* w, const int32_t* targets, const float* lse,
                            const float* grad_logp, int64_t N, int H, int V, a3po_dtype dt, float inv_temperature,
                            void* grad_hidden, float* grad_w, int accumulate_grad_w, void* ws, size_t ws_bytes,
                            uint32_t* status, void* stream_) {
  A3PO_RETURN_IF(check_lmhead_args(hidden, w, targets, N, H, V, dt, inv_temperature));
  if (!grad_w || (N > 0 && (!lse || !grad_logp || !grad_hidden))) return A3PO_ERR_INVALID_ARG;
  if (!aligned_to(grad_hidden, 16) || !aligned_to(grad_w, 16)) return A3PO_ERR_UNSUPPORTED;
  if (!ws || !aligned_to(ws, 256)) return A3PO_ERR_WORKSPACE;
  cudaStream_t stream = as_stream(stream_);
  if (use_tc(dt, hidden, w, N, H, V) && N > 0) {
    // Rows with a zero upstream gradient (padding, clipped tokens) are skipped: with enough workspace
    // the other rows are gathered into a compact buffer first (their count stays on the device).
    CompactBuffers cb;
    size_t ws_off = 0;
    const bool compacted = ws_bytes >= compact_ws_bytes(N, H, true) + lmhead_tc_bwd_ws_bytes(128, N, H, V) &&
                           compact_carve(ws, ws_bytes, N, H, true, &cb, &ws_off);
    if (!compacted) ws_off = 0;
    void* ws_rest = static_cast<char*>(ws) + ws_off;
    const size_t rest_bytes = ws_bytes - ws_off;
    // largest chunk (multiple of 128 rows) whose scratch fits what is left of the caller's buffer
    long long chunk = clamp_chunk(kTcChunkRows, N, 128);
    while (chunk > 128 && lmhead_tc_bwd_ws_bytes(chunk, N, H, V) > rest_bytes) chunk -= 128;
    if (lmhead_tc_bwd_ws_bytes(chunk, N, H, V) > rest_bytes) return A3PO_ERR_WORKSPACE;
    if (!compacted)
      return lmhead_bwd_tc(hidden, w, targets, lse, grad_logp, N, H, V, inv_temperature, grad_hidden, grad_w,
                           accumulate_grad_w, ws_rest, rest_bytes, chunk, nullptr, status, stream);
    A3PO_RETURN_IF(compact_rows(hidden, H, targets, nullptr, grad_logp, lse, N, cb, stream));
    A3PO_RETURN_IF(lmhead_bwd_tc(cb.hidden_c, w, cb.targets_c, cb.lse_c, cb.g_c, N, H, V, inv_temperature,
                                 cb.grad_hidden_c, grad_w, accumulate_grad_w, ws_rest, rest_bytes, chunk, cb.count,
                                 status, stream));
    return scatter_rows(cb.grad_hidden_c, H, cb.pos, N, grad_hidden, stream);
  }
  if (ws_bytes < simt_bwd_ws(kSimtTile, V)) return A3PO_ERR_WORKSPACE;
  long long chunk = clamp_chunk(kSimtChunkRows, N, kSimtTile);
  const long long fit = static_cast<long long>((ws_bytes - 256) / (sizeof(float) * static_cast<size_t>(V)));
  if (chunk > fit) chunk = fit / kSimtTile * kSimtTile;
  if (chunk < kSimtTile) return A3PO_ERR_WORKSPACE;
  return lmhead_bwd_simt(hidden, w, targets, lse, grad_logp, N, H, V, dt, inv_temperature, grad_hidden, grad_w,
                         accumulate_grad_w, static_cast<float*>(ws), chunk, stream);
}

// ------------------------------------------------------------------------------------------------
// Whole step with per-step inputs in host memory.
// ------------------------------------------------------------------------------------------------
namespace {
struct StageLayout {
  size_t hidden, targets, behav, versions, adv, mask, logp, lse, grad_logp, loss, stats, total;
};
StageLayout stage_layout(long long n, int h, a3po_dtype dt) {
  StageLayout s;
  size_t off = 0;
  const size_t rows = static_cast<size_t>(n > 0 ? n : 0);
  auto take = [&](size_t bytes) { size_t o = off; off = round_up(off + bytes, 256); return o; };
  s.hidden = take(rows * h * elt_size(dt));
  s.targets = take(rows * 4);
  s.behav = take(rows * 4);
  s.versions = take(rows * 4);
  s.adv = take(rows * 4);
  s.mask = take(rows);
  s.logp = take(rows * 4);
  s.lse = take(rows * 4);
  s.grad_logp = take(rows * 4);
  s.loss = take(sizeof(float));
  s.stats = take(sizeof(a3po_stats));
  s.total = off;
  return s;
}
}  // namespace

size_t a3po_train_step_stage_bytes(int64_t N, int H, a3po_dtype dt) {
  if (N < 0 || H <= 0) return 0;
  return stage_layout(N, H, dt).total;
}

// ------------------------------------------------------------------------------------------------
// Forward that keeps its softmax / backward that uses it (no recomputation of the LM head).
// ------------------------------------------------------------------------------------------------
namespace {
// `kept` buffer: what the backward needs from the forward, all in the compact row space of the rows that took
// part: their number, the maps batch row <-> compact row, targets, the tail sums s, and the probability ratios q.
struct KeptLayout {
  size_t count, pos, idx, targets, sprime, q, total;
};
KeptLayout kept_layout(long long n, int v) {
  KeptLayout k;
  size_t off = 0;
  const size_t rows = static_cast<size_t>(n > 0 ? n : 0);
  const size_t cap = static_cast<size_t>(compact_capacity(n > 0 ? n : 0));
  auto take = [&](size_t bytes) { size_t o = off; off = round_up(off + bytes, 256); return o; };
  k.count = take(sizeof(int));
  k.pos = take(sizeof(int) * rows);
  k.idx = take(sizeof(int) * cap);
  k.targets = take(sizeof(int32_t) * cap);
  k.sprime = take(sizeof(float) * cap);
  k.q = take(lmhead_tc_kept_bytes(static_cast<long long>(cap), v));
  k.total = off;
  return k;
}

constexpr size_t kScanBytes = 2 * 4096 * sizeof(int);  // block counts + offsets of the compaction scan

size_t fwd_keep_ws_bytes(long long n, int h, int v) {
  const size_t cap = static_cast<size_t>(compact_capacity(n));
  const int splits = lmhead_tc_fwd_splits(static_cast<long long>(cap), h, v);
  return round_up(kScanBytes, 256) + round_up(cap * static_cast<size_t>(h) * 2, 256) /*hidden_c*/ +
         4 * round_up(sizeof(float) * cap, 256) /*zy, logp_c, lse_c, ent_c*/ +
         2 * round_up(sizeof(float) * cap * splits, 256) /*part_s, part_e*/ + 256;
}

size_t bwd_kept_ws_bytes(long long n, int h) {
  const size_t cap = static_cast<size_t>(compact_capacity(n));
  return round_up(sizeof(float) * cap, 256) /*row_scale*/ + 2 * round_up(cap * static_cast<size_t>(h) * 2, 256) +
         256 /*tile choice*/ + 256;
}
}  // namespace

size_t a3po_kept_bytes(int64_t N, int V) {
  if (N < 0 || V <= 0) return 0;
  return kept_layout(N, V).total + 256;
}

size_t a3po_token_logprobs_fwd_keep_workspace_bytes(int64_t N, int H, int V) {
  if (N < 0 || H <= 0 || V <= 0) return 0;
  return fwd_keep_ws_bytes(N, H, V);
}

size_t a3po_token_logprobs_bwd_kept_workspace_bytes(int64_t N, int H, int V) {
  if (N < 0 || H <= 0 || V <= 0) return 0;
  return bwd_kept_ws_bytes(N, H);
}

int a3po_token_logprobs_fwd_keep(const void* hidden, const void* w, const int32_t* targets, const uint8_t* row_mask,
                                 int64_t N, int H, int V, float inv_temperature, float* logp, float* lse,
                                 float* entropy, void* kept, size_t kept_bytes, void* ws, size_t ws_bytes,
                                 uint32_t* status, void* stream_) {
  A3PO_RETURN_IF(check_lmhead_args(hidden, w, targets, N, H, V, A3PO_BF16, inv_temperature));
  if (N > 0 && (!logp || !lse)) return A3PO_ERR_INVALID_ARG;
  if (N == 0) return A3PO_OK;
  if (!use_tc(A3PO_BF16, hidden, w, N, H, V)) return A3PO_ERR_UNSUPPORTED;
  if (!kept || !aligned_to(kept, 256) || kept_bytes < a3po_kept_bytes(N, V)) return A3PO_ERR_WORKSPACE;
  if (!ws || !aligned_to(ws, 256) || ws_bytes < fwd_keep_ws_bytes(N, H, V)) return A3PO_ERR_WORKSPACE;
  cudaStream_t stream = as_stream(stream_);
  const KeptLayout kl = kept_layout(N, V);
  char* kb = static_cast<char*>(kept);
  const long long cap = compact_capacity(N);
  const int splits = lmhead_tc_fwd_splits(cap, H, V);

  Arena arena(ws, ws_bytes);
  CompactBuffers cb;
  cb.cap = cap;
  cb.count = reinterpret_cast<int*>(kb + kl.count);
  cb.pos = reinterpret_cast<int*>(kb + kl.pos);
  cb.idx = reinterpret_cast<int*>(kb + kl.idx);
  cb.targets_c = reinterpret_cast<int32_t*>(kb + kl.targets);
  cb.block_counts = arena.take<int>(4096);
  cb.block_offsets = arena.take<int>(4096);
  cb.hidden_c = arena.take<__nv_bfloat16>(static_cast<size_t>(cap) * H);
  cb.lse_c = nullptr;
  cb.g_c = nullptr;
  cb.grad_hidden_c = nullptr;
  float* zy = arena.take<float>(static_cast<size_t>(cap));
  float* logp_c = arena.take<float>(static_cast<size_t>(cap));
  float* lse_c = arena.take<float>(static_cast<size_t>(cap));
  float* ent_c = arena.take<float>(static_cast<size_t>(cap));
  float* part_s = arena.take<float>(static_cast<size_t>(cap) * splits);
  float* part_e = arena.take<float>(static_cast<size_t>(cap) * splits);
  if (!arena.ok()) return A3PO_ERR_WORKSPACE;
  float* sprime = reinterpret_cast<float*>(kb + kl.sprime);
  void* q = kb + kl.q;

  A3PO_RETURN_IF(compact_rows(hidden, H, targets, row_mask, nullptr, nullptr, N, cb, stream));
  A3PO_RETURN_IF(target_logits(cb.hidden_c, w, cb.targets_c, cb.count, 0, cap, H, V, inv_temperature, zy, stream));
  A3PO_RETURN_IF(lmhead_fwd_keep_tc(cb.hidden_c, w, cb.targets_c, zy, cap, H, V, inv_temperature, splits, part_s,
                                    entropy ? part_e : nullptr, q, cb.count, 0, status, stream));
  A3PO_RETURN_IF(merge_kept(part_s, part_e, zy, cb.count, 0, cap, splits, inv_temperature, sprime, logp_c, lse_c,
                            entropy ? ent_c : nullptr, status, stream));
  A3PO_RETURN_IF(flag_bad_targets(targets, N, V, status, stream));
  return finish_batch_outputs(cb.pos, N, logp_c, logp, lse_c, lse, nullptr, nullptr, ent_c, entropy, nullptr, H,
                              stream);
}

int a3po_token_logprobs_bwd_kept(const void* hidden, const void* w, const int32_t* targets, const float* lse,
                                 const float* grad_logp, void* kept, size_t kept_bytes, int64_t N, int H, int V,
                                 float inv_temperature, void* grad_hidden, float* grad_w, int accumulate_grad_w,
                                 void* ws, size_t ws_bytes, uint32_t* status, void* stream_) {
  A3PO_RETURN_IF(check_lmhead_args(hidden, w, targets, N, H, V, A3PO_BF16, inv_temperature));
  if (!grad_w || (N > 0 && (!lse || !grad_logp || !grad_hidden))) return A3PO_ERR_INVALID_ARG;
  if (!aligned_to(grad_hidden, 16) || !aligned_to(grad_w, 16)) return A3PO_ERR_UNSUPPORTED;
  if (N == 0) {
    if (!accumulate_grad_w &&
        cudaMemsetAsync(grad_w, 0, sizeof(float) * static_cast<size_t>(V) * H, as_stream(stream_)) != cudaSuccess) {
      cudaGetLastError();
      return A3PO_ERR_CUDA;
    }
    return A3PO_OK;
  }
  if (!use_tc(A3PO_BF16, hidden, w, N, H, V)) return A3PO_ERR_UNSUPPORTED;
  if (!kept || !aligned_to(kept, 256) || kept_bytes < a3po_kept_bytes(N, V)) return A3PO_ERR_WORKSPACE;
  if (!ws || !aligned_to(ws, 256) || ws_bytes < bwd_kept_ws_bytes(N, H)) return A3PO_ERR_WORKSPACE;
  cudaStream_t stream = as_stream(stream_);
  const KeptLayout kl = kept_layout(N, V);
  char* kb = static_cast<char*>(kept);
  const long long cap = compact_capacity(N);
  const int* count = reinterpret_cast<const int*>(kb + kl.count);
  const int* pos = reinterpret_cast<const int*>(kb + kl.pos);
  const int* idx = reinterpret_cast<const int*>(kb + kl.idx);
  const int32_t* targets_c = reinterpret_cast<const int32_t*>(kb + kl.targets);
  const float* sprime = reinterpret_cast<const float*>(kb + kl.sprime);
  void* q = kb + kl.q;
  Arena arena(ws, ws_bytes);
  float* row_scale = arena.take<float>(static_cast<size_t>(cap));
  __nv_bfloat16* hs = arena.take<__nv_bfloat16>(static_cast<size_t>(cap) * H);
  __nv_bfloat16* ghc = arena.take<__nv_bfloat16>(static_cast<size_t>(cap) * H);
  int* select = arena.take<int>(1);
  if (!arena.ok()) return A3PO_ERR_WORKSPACE;

  // the target's entry of q and the per-row factor of dz, then the two contractions on q itself
  A3PO_RETURN_IF(prepare_kept_backward(count, 0, cap, nullptr, nullptr, H, V, inv_temperature, sprime, targets_c,
                                       nullptr, grad_logp, idx, nullptr, hidden, row_scale, nullptr, q, hs, stream));
  A3PO_RETURN_IF(lmhead_grad_hidden_from_kept_tc(q, w, row_scale, cap, H, V, ghc, count, 0, select, status, stream));
  A3PO_RETURN_IF(scatter_rows(ghc, H, pos, N, grad_hidden, stream));
  return lmhead_grad_w_from_kept_tc(q, hs, cap, H, V, grad_w, accumulate_grad_w, accumulate_grad_w ? 0 : 1, count, 0,
                                    status, stream);
}

// ------------------------------------------------------------------------------------------------
// Whole step in one call.
// ------------------------------------------------------------------------------------------------
namespace {
constexpr long long kStepChunkRows = 65536;     // rows of kept ratios the recommended workspace holds at a time
constexpr long long kStepMinChunkRows = 2048;   // below this the recomputing calls are used instead
constexpr int kStepMaxSplits = 64;

// Workspace of the step that keeps the forward's softmax for the backward, one chunk of compact rows at a time.
struct StepLayout {
  // whole batch
  size_t count, scan, pos, idx, targets_c, zy, sprime, logp_c, lse_c, g_c, ent_c, behav_c, adv_c,
      versions_c, mask_c, n_valid, partials;
  // one chunk
  size_t hidden_c, part_s, part_e, q, hs, ghc, perm, move_src, move_dst, bwd_idx, scale_p, bwd_count;
  size_t total;
};
StepLayout step_layout(long long n, int h, int v, long long chunk_rows) {
  StepLayout s;
  size_t off = 0;
  const size_t rows = static_cast<size_t>(n);
  const size_t cap = static_cast<size_t>(compact_capacity(n));
  const size_t rc = static_cast<size_t>(chunk_rows);
  auto take = [&](size_t bytes) { size_t o = off; off = round_up(off + bytes, 256); return o; };
  s.count = take(sizeof(int));
  s.scan = take(kScanBytes);
  s.pos = take(4 * rows);
  s.idx = take(4 * cap);
  s.targets_c = take(4 * cap);
  s.zy = take(4 * cap); s.sprime = take(4 * cap); s.logp_c = take(4 * cap); s.lse_c = take(4 * cap);
  s.g_c = take(4 * cap); s.ent_c = take(4 * cap); s.behav_c = take(4 * cap); s.adv_c = take(4 * cap);
  s.versions_c = take(4 * cap);
  s.mask_c = take(cap);
  s.n_valid = take(sizeof(long long));
  s.partials = take(loss_partial_bytes() * loss_max_partials());
  s.hidden_c = take(rc * static_cast<size_t>(h) * 2);   // the chunk's rows of hidden, gathered
  s.part_s = take(4 * rc * kStepMaxSplits);
  s.part_e = take(4 * rc * kStepMaxSplits);
  s.q = take(lmhead_tc_kept_bytes(chunk_rows, v));
  s.hs = take(rc * static_cast<size_t>(h) * 2);
  s.ghc = take(rc * static_cast<size_t>(h) * 2);
  s.perm = take(4 * rc); s.move_src = take(4 * rc); s.move_dst = take(4 * rc); s.bwd_idx = take(4 * rc);
  s.scale_p = take(4 * rc);
  s.bwd_count = take(4 * sizeof(int));   // rows of the chunk's backward, rows moved, tile choice of grad_hidden
  s.total = off;
  return s;
}
// Largest chunk (multiple of 128 rows, at most the compact capacity) whose scratch fits `ws_bytes`; 0 if the
// keeping path does not fit.
long long step_chunk_rows_for(size_t ws_bytes, long long n, int h, int v) {
  const long long cap = compact_capacity(n);
  const size_t fixed = step_layout(n, h, v, 0).total;
  if (ws_bytes <= fixed) return 0;
  const size_t per_128 = step_layout(n, h, v, 128).total - fixed;
  long long rc = static_cast<long long>((ws_bytes - fixed) / per_128) * 128;
  if (rc > cap) rc = cap;
  while (rc > 0 && step_layout(n, h, v, rc).total > ws_bytes) rc -= 128;
  const long long need = cap < kStepMinChunkRows ? cap : kStepMinChunkRows;
  return rc >= need ? rc : 0;
}
}  // namespace

size_t a3po_train_step_min_workspace_bytes(int64_t N, int H, int V, a3po_dtype dt) {
  if (N < 0 || H <= 0 || V <= 0) return 0;
  size_t a = a3po_token_logprobs_min_workspace_bytes(N, H, V, dt, 0);
  const size_t b = a3po_token_logprobs_min_workspace_bytes(N, H, V, dt, 1);
  const size_t c = a3po_loss_workspace_bytes(N);
  if (b > a) a = b;
  if (c > a) a = c;
  return a;
}

size_t a3po_train_step_workspace_bytes(int64_t N, int H, int V, a3po_dtype dt) {
  if (N < 0 || H <= 0 || V <= 0) return 0;
  size_t a = a3po_train_step_min_workspace_bytes(N, H, V, dt);
  if (dt == A3PO_BF16 && N > 0 && H % 8 == 0) {
    // the keeping path: kept ratios for one chunk of up to kStepChunkRows rows (about 2 V bytes per row) plus
    // buffers that scale with N x H; a caller may pass more and gets larger chunks (fewer launches)
    long long rc = compact_capacity(N);
    if (rc > kStepChunkRows) rc = kStepChunkRows;
    const size_t d = step_layout(N, H, V, rc).total;
    if (d > a) a = d;
  } else {
    size_t f = a3po_token_logprobs_workspace_bytes(N, H, V, dt, 0);
    const size_t b = a3po_token_logprobs_workspace_bytes(N, H, V, dt, 1);
    if (b > f) f = b;
    if (f > a) a = f;
  }
  return a;
}

int a3po_train_step(const void* hidden, const int32_t* targets, const float* behav_logp, const int32_t* versions,
                    const float* adv, const uint8_t* mask, int64_t N, int H, int V, a3po_dtype dt,
                    int32_t current_version, float clip_eps, float inv_temperature, const void* w, float* grad_w,
                    int accumulate_grad_w, void* grad_hidden, float* logp, float* lse, float* entropy,
                    float* grad_logp, float* loss, a3po_stats* stats, const float* loss_scale, void* ws,
                    size_t ws_bytes, uint32_t* status, void* stream_) {
  A3PO_RETURN_IF(check_lmhead_args(hidden, w, targets, N, H, V, dt, inv_temperature));
  if (!grad_w || !loss || !(clip_eps >= 0.f) ||
      (N > 0 && (!behav_logp || !versions || !adv || !mask || !grad_hidden || !logp || !lse || !grad_logp)))
    return A3PO_ERR_INVALID_ARG;
  if (!ws || !aligned_to(ws, 256)) return A3PO_ERR_WORKSPACE;
  const long long chunk_rows = (N > 0 && use_tc(dt, hidden, w, N, H, V) && aligned_to(grad_hidden, 16) &&
                                aligned_to(grad_w, 16))
                                   ? step_chunk_rows_for(ws_bytes, N, H, V)
                                   : 0;
  if (chunk_rows == 0) {
    // three independent calls; the backward recomputes the logits chunk by chunk
    A3PO_RETURN_IF(a3po_token_logprobs_fwd(hidden, w, targets, mask, N, H, V, dt, inv_temperature, logp, lse, entropy,
                                           ws, ws_bytes, status, stream_));
    if (loss_scale == nullptr) {
      A3PO_RETURN_IF(a3po_loss_fwd_bwd(logp, behav_logp, versions, 0, nullptr, 0, current_version, adv, mask, N,
                                       clip_eps, 1, loss, stats, grad_logp, ws, ws_bytes, stream_));
    } else {   // a weighted upstream gradient: forward and backward as two calls, the backward takes the weight
      A3PO_RETURN_IF(a3po_loss_fwd(logp, behav_logp, versions, 0, nullptr, 0, current_version, adv, mask, N, clip_eps,
                                   loss, stats, ws, ws_bytes, stream_));
      A3PO_RETURN_IF(a3po_loss_bwd(logp, behav_logp, versions, 0, nullptr, 0, current_version, adv, mask, N, clip_eps,
                                   1, loss_scale, stats, grad_logp, ws, ws_bytes, stream_));
    }
    return a3po_token_logprobs_bwd(hidden, w, targets, lse, grad_logp, N, H, V, dt, inv_temperature, grad_hidden,
                                   grad_w, accumulate_grad_w, ws, ws_bytes, status, stream_);
  }

  // ---- rows with mask != 0 are gathered once; then, per chunk of those rows: forward keeping the softmax ->
  // loss forward + backward (M is the number of gathered rows, known up front) -> the two gradient contractions
  cudaStream_t stream = as_stream(stream_);
  const StepLayout lay = step_layout(N, H, V, chunk_rows);
  if (lay.total > ws_bytes) return A3PO_ERR_WORKSPACE;
  char* base = static_cast<char*>(ws);
  const long long cap = compact_capacity(N);
  CompactBuffers cb;
  cb.cap = cap;
  cb.count = reinterpret_cast<int*>(base + lay.count);
  cb.block_counts = reinterpret_cast<int*>(base + lay.scan);
  cb.block_offsets = cb.block_counts + 4096;
  cb.pos = reinterpret_cast<int*>(base + lay.pos);
  cb.idx = reinterpret_cast<int*>(base + lay.idx);
  cb.targets_c = reinterpret_cast<int32_t*>(base + lay.targets_c);
  cb.hidden_c = reinterpret_cast<__nv_bfloat16*>(base + lay.hidden_c);
  cb.lse_c = nullptr;
  cb.g_c = nullptr;
  cb.grad_hidden_c = nullptr;
  auto f32 = [&](size_t off) { return reinterpret_cast<float*>(base + off); };
  float *zy = f32(lay.zy), *sprime = f32(lay.sprime), *logp_c = f32(lay.logp_c), *lse_c = f32(lay.lse_c);
  float *g_c = f32(lay.g_c), *ent_c = f32(lay.ent_c), *behav_c = f32(lay.behav_c), *adv_c = f32(lay.adv_c);
  float* scale_p = f32(lay.scale_p);
  int* perm = reinterpret_cast<int*>(base + lay.perm);
  int* move_src = reinterpret_cast<int*>(base + lay.move_src);
  int* move_dst = reinterpret_cast<int*>(base + lay.move_dst);
  int* bwd_idx = reinterpret_cast<int*>(base + lay.bwd_idx);
  int* bwd_count = reinterpret_cast<int*>(base + lay.bwd_count);
  int32_t* versions_c = reinterpret_cast<int32_t*>(base + lay.versions_c);
  uint8_t* mask_c = reinterpret_cast<uint8_t*>(base + lay.mask_c);
  long long* n_valid = reinterpret_cast<long long*>(base + lay.n_valid);
  char* partials = base + lay.partials;
  float *part_s = f32(lay.part_s), *part_e = f32(lay.part_e);
  void* q = base + lay.q;
  __nv_bfloat16* hs = reinterpret_cast<__nv_bfloat16*>(base + lay.hs);
  __nv_bfloat16* ghc = reinterpret_cast<__nv_bfloat16*>(base + lay.ghc);
  const __nv_bfloat16* hidden_c = cb.hidden_c;

  const int n_chunks = static_cast<int>((cap + chunk_rows - 1) / chunk_rows);
  int max_blocks = loss_max_partials() / n_chunks;
  if (max_blocks < 1) return A3PO_ERR_WORKSPACE;   // more than 4096 chunks: the workspace is far too small for N
  const int loss_blocks = loss_blocks_for(chunk_rows, max_blocks);

  A3PO_RETURN_IF(compact_index(targets, mask, nullptr, nullptr, N, cb, stream));
  A3PO_RETURN_IF(gather_loss_inputs(cb.idx, cb.count, cap, behav_logp, versions, adv, behav_c, versions_c, adv_c,
                                    mask_c, n_valid, stream));
  A3PO_RETURN_IF(flag_bad_targets(targets, N, V, status, stream));
  for (int i = 0; i < n_chunks; ++i) {
    const long long c0 = static_cast<long long>(i) * chunk_rows;
    const long long rows = (c0 + chunk_rows <= cap) ? chunk_rows : cap - c0;
    const int splits = lmhead_tc_fwd_splits(rows, H, V);
    A3PO_RETURN_IF(gather_rows_range(hidden, H, cb.idx, cb.count, c0, rows, cb.hidden_c, stream));
    A3PO_RETURN_IF(target_logits(hidden_c, w, cb.targets_c, cb.count, c0, rows, H, V, inv_temperature, zy, stream));
    A3PO_RETURN_IF(lmhead_fwd_keep_tc(hidden_c, w, cb.targets_c + c0, zy + c0, rows, H, V, inv_temperature,
                                      splits, part_s, entropy ? part_e : nullptr, q, cb.count, c0, status, stream));
    A3PO_RETURN_IF(merge_kept(part_s, part_e, zy, cb.count, c0, rows, splits, inv_temperature, sprime, logp_c, lse_c,
                              entropy ? ent_c : nullptr, status, stream));
    A3PO_RETURN_IF(loss_fwd_bwd_slice(logp_c + c0, behav_c + c0, versions_c + c0, adv_c + c0, mask_c + c0, rows,
                                      current_version, clip_eps, n_valid, loss_scale, g_c + c0,
                                      partials + static_cast<size_t>(i) * loss_blocks * loss_partial_bytes(),
                                      loss_blocks, stream));
    // the backward's rows: those with a non-zero gradient (clipped tokens drop out), made contiguous in q
    A3PO_RETURN_IF(plan_backward_rows(g_c, cb.count, c0, rows, bwd_count, bwd_count + 1, perm, move_src, move_dst, q,
                                      V, stream));
    A3PO_RETURN_IF(prepare_kept_backward(cb.count, c0, rows, bwd_count, perm, H, V, inv_temperature, sprime,
                                         cb.targets_c, g_c, nullptr, cb.idx, hidden_c, nullptr, scale_p, bwd_idx, q, hs,
                                         stream));
    A3PO_RETURN_IF(lmhead_grad_hidden_from_kept_tc(q, w, scale_p, rows, H, V, ghc, bwd_count, 0, bwd_count + 2, status,
                                                   stream));
    A3PO_RETURN_IF(scatter_rows_range(ghc, H, bwd_idx, bwd_count, rows, grad_hidden, stream));
    A3PO_RETURN_IF(lmhead_grad_w_from_kept_tc(q, hs, rows, H, V, grad_w, (accumulate_grad_w || i > 0) ? 1 : 0,
                                              (i == 0 && !accumulate_grad_w) ? 1 : 0, bwd_count, 0, status, stream));
  }
  A3PO_RETURN_IF(finish_batch_outputs(cb.pos, N, logp_c, logp, lse_c, lse, g_c, grad_logp, ent_c, entropy,
                                      grad_hidden, H, stream));
  return loss_finalize_partials(partials, n_chunks * loss_blocks, loss, stats, stream);
}

namespace {

// Runs [begin, end) of rows with mask != 0; two runs with fewer than min_gap rows between them are merged.
// More than max_runs runs: one run from the first to the last such row.
void mask_row_runs(const uint8_t* mask, long long n, long long min_gap, size_t max_runs,
                   std::vector<std::pair<long long, long long>>* runs) {
  runs->clear();
  long long i = 0;
  while (i < n) {
    while (i < n && mask[i] == 0) {   // skip zeros, eight at a time where possible
      if ((reinterpret_cast<uintptr_t>(mask + i) & 7u) == 0 && i + 8 <= n) {
        uint64_t word;
        std::memcpy(&word, mask + i, 8);
        if (word == 0) { i += 8; continue; }
      }
      ++i;
    }
    if (i >= n) break;
    const long long begin = i;
    const void* z = std::memchr(mask + i, 0, static_cast<size_t>(n - i));
    i = z ? static_cast<const uint8_t*>(z) - mask : n;
    if (!runs->empty() && begin - runs->back().second < min_gap) runs->back().second = i;
    else runs->emplace_back(begin, i);
  }
  if (runs->size() > max_runs) {
    const long long first = runs->front().first, last = runs->back().second;
    runs->clear();
    runs->emplace_back(first, last);
  }
}

std::atomic<long long> g_h2d_bytes{0};

}  // namespace

int64_t a3po_host_to_device_bytes(void) { return g_h2d_bytes.load(std::memory_order_relaxed); }

int a3po_train_step_host(const void* h_hidden, const int32_t* h_targets, const float* h_behav_logp,
                         const int32_t* h_versions, const float* h_adv, const uint8_t* h_mask, int64_t N, int H,
                         int V, a3po_dtype dt, int32_t current_version, float clip_eps, float inv_temperature,
                         const void* d_w, float* d_grad_w, int accumulate_grad_w, void* d_grad_hidden, void* d_stage,
                         size_t stage_bytes, void* d_ws, size_t ws_bytes, float* h_loss, a3po_stats* h_stats,
                         uint32_t* d_status, void* stream_) {
  if (N < 0 || H <= 0 || V <= 0) return A3PO_ERR_INVALID_ARG;
  if (dt != A3PO_F32 && dt != A3PO_BF16) return A3PO_ERR_UNSUPPORTED;
  if (!h_loss || !d_w || !d_grad_w || !d_stage || !d_ws) return A3PO_ERR_INVALID_ARG;
  if (N > 0 && (!h_hidden || !h_targets || !h_behav_logp || !h_versions || !h_adv || !h_mask || !d_grad_hidden))
    return A3PO_ERR_INVALID_ARG;
  if (!aligned_to(d_stage, 256)) return A3PO_ERR_WORKSPACE;
  const StageLayout s = stage_layout(N, H, dt);
  if (stage_bytes < s.total) return A3PO_ERR_WORKSPACE;
  cudaStream_t stream = as_stream(stream_);
  char* base = static_cast<char*>(d_stage);
  const size_t rows = static_cast<size_t>(N);
  auto h2d = [&](size_t off, const void* src, size_t bytes) -> bool {
    return bytes == 0 || cudaMemcpyAsync(base + off, src, bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  };
  const void* hidden = base + s.hidden;
  {
    ProfileScope scope(kKH2D, stream);   // with the per-kernel profile on, the copies show up as one entry
    bool ok = h2d(s.targets, h_targets, rows * 4) && h2d(s.behav, h_behav_logp, rows * 4) &&
              h2d(s.versions, h_versions, rows * 4) && h2d(s.adv, h_adv, rows * 4) && h2d(s.mask, h_mask, rows);
    size_t copied = rows * (4 + 4 + 4 + 4 + 1);
    // The step that keeps the softmax reads `hidden` only at rows with mask != 0 (it gathers them by index), so
    // only the runs of such rows cross the bus; runs closer together than a copy call is worth are merged.  The
    // recomputing fallback may multiply masked rows as zero rows and therefore gets every row.
    const size_t row_bytes = static_cast<size_t>(H) * elt_size(dt);
    const bool kept_path = N > 0 && use_tc(dt, hidden, d_w, N, H, V) && aligned_to(d_grad_hidden, 16) &&
                           aligned_to(d_grad_w, 16) && step_chunk_rows_for(ws_bytes, N, H, V) > 0;
    if (kept_path) {
      std::vector<std::pair<long long, long long>> runs;
      const long long min_gap = static_cast<long long>((size_t(256) << 10) / row_bytes) + 1;
      mask_row_runs(h_mask, N, min_gap, 1024, &runs);
      for (const auto& r : runs) {
        const size_t off = static_cast<size_t>(r.first) * row_bytes;
        const size_t bytes = static_cast<size_t>(r.second - r.first) * row_bytes;
        ok = ok && h2d(s.hidden + off, static_cast<const char*>(h_hidden) + off, bytes);
        copied += bytes;
      }
    } else {
      ok = ok && h2d(s.hidden, h_hidden, rows * row_bytes);
      copied += rows * row_bytes;
    }
    if (!ok) {
      cudaGetLastError();
      return A3PO_ERR_CUDA;
    }
    g_h2d_bytes.fetch_add(static_cast<long long>(copied), std::memory_order_relaxed);
  }
  const int32_t* targets = reinterpret_cast<const int32_t*>(base + s.targets);
  const float* behav = reinterpret_cast<const float*>(base + s.behav);
  const int32_t* versions = reinterpret_cast<const int32_t*>(base + s.versions);
  const float* adv = reinterpret_cast<const float*>(base + s.adv);
  const uint8_t* mask = reinterpret_cast<const uint8_t*>(base + s.mask);
  float* logp = reinterpret_cast<float*>(base + s.logp);
  float* lse = reinterpret_cast<float*>(base + s.lse);
  float* grad_logp = reinterpret_cast<float*>(base + s.grad_logp);
  float* loss = reinterpret_cast<float*>(base + s.loss);
  a3po_stats* stats = reinterpret_cast<a3po_stats*>(base + s.stats);

  A3PO_RETURN_IF(a3po_train_step(hidden, targets, behav, versions, adv, mask, N, H, V, dt, current_version, clip_eps,
                                 inv_temperature, d_w, d_grad_w, accumulate_grad_w, d_grad_hidden, logp, lse, nullptr,
                                 grad_logp, loss, stats, nullptr, d_ws, ws_bytes, d_status, stream_));
  if (cudaMemcpyAsync(h_loss, loss, sizeof(float), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      (h_stats && cudaMemcpyAsync(h_stats, stats, sizeof(a3po_stats), cudaMemcpyDeviceToHost, stream) != cudaSuccess)) {
    cudaGetLastError();
    return A3PO_ERR_CUDA;
  }
  return A3PO_OK;
}

}  // extern "C"
