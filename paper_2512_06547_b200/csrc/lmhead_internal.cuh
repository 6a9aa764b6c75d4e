// Interfaces between the LM-head dispatch (api.cu) and its two kernel families.
#pragma once

#include "a3po_common.cuh"

namespace a3po {

// Online-softmax state of one row over one vocabulary split, natural-log units:
// m = max_v z[v], s = sum_v exp(z[v] - m) over the split's columns.
struct SoftmaxPartial {
  float m;
  float s;
};

// ---- FP32-pipe kernels (lmhead_simt.cu) ----
int lmhead_fwd_simt(const void* hidden, const void* w, const int32_t* targets, long long n, int h, int v,
                    a3po_dtype dt, float inv_t, int splits, SoftmaxPartial* part, float* part_ent, float* zy,
                    cudaStream_t stream);
int lmhead_bwd_simt(const void* hidden, const void* w, const int32_t* targets, const float* lse,
                    const float* grad_logp, long long n, int h, int v, a3po_dtype dt, float inv_t, void* grad_hidden,
                    float* grad_w, int accumulate, float* ds, long long chunk_rows, cudaStream_t stream);

// ---- row compaction (compact_rows.cu), bf16 only ----
// Device buffers of one compaction; `cap` = rows of the compact space (n rounded up to 128).
struct CompactBuffers {
  long long cap;
  int* count;                    // [1]   number of kept rows (device-resident, never read by the host)
  int* block_counts;             // scan scratch
  int* block_offsets;
  int* pos;                      // [n]   original row -> compact row, or -1
  int* idx;                      // [cap] compact row -> original row
  int32_t* targets_c;            // [cap]
  float* lse_c;                  // [cap] backward only
  float* g_c;                    // [cap] backward only; zero beyond the kept rows
  __nv_bfloat16* hidden_c;       // [cap, h]; zero rows from count to the next multiple of 128
  __nv_bfloat16* grad_hidden_c;  // [cap, h] backward only
};
long long compact_capacity(long long n);
size_t compact_ws_bytes(long long n, int h, bool backward);
bool compact_carve(void* ws, size_t ws_bytes, long long n, int h, bool backward, CompactBuffers* out, size_t* used);
// Keeps row t iff (row_mask == null || row_mask[t] != 0) && (g == null || g[t] != 0).
int compact_rows(const void* hidden, int h, const int32_t* targets, const uint8_t* row_mask, const float* g,
                 const float* lse, long long n, const CompactBuffers& cb, cudaStream_t stream);
// The two halves of compact_rows: the index (count, pos, idx, compact scalars) for the whole batch, and the gather
// of hidden rows for compact rows [offset, offset + rows) into dst (zero rows up to the next multiple of 128).
int compact_index(const int32_t* targets, const uint8_t* row_mask, const float* g, const float* lse, long long n,
                  const CompactBuffers& cb, cudaStream_t stream);
int gather_rows_range(const void* hidden, int h, const int* idx, const int* count, long long offset, long long rows,
                      void* dst, cudaStream_t stream);
// dst[t, :] = src_c[pos[t], :] for kept rows, zero otherwise.
int scatter_rows(const void* src_c, int h, const int* pos, long long n, void* dst, cudaStream_t stream);

// ---- tcgen05 / TMEM / TMA kernels (lmhead_tc.cu), bf16 only ----
bool lmhead_tc_supported(const void* hidden, const void* w, long long n, int h, int v);
// Vocabulary splits the tensor-core forward wants for n rows of h, v columns: each (row tile, split) pair is one
// work item.
int lmhead_tc_fwd_splits(long long n, int h, int v);
// `dyn_rows` (device, may be null): number of rows of `hidden` that are really present (compact row space);
// partials are laid out [split][n] regardless.
int lmhead_fwd_tc(const void* hidden, const void* w, const int32_t* targets, long long n, int h, int v, float inv_t,
                  int splits, SoftmaxPartial* part, float* part_ent, float* zy, const int* dyn_rows, uint32_t* status,
                  cudaStream_t stream);
// Workspace (bytes) of the tensor-core backward for a chunk of `chunk_rows` rows.
size_t lmhead_tc_bwd_ws_bytes(long long chunk_rows, long long n, int h, int v);
// `dyn_rows` as above; when given, every per-row input is in the compact row space, rows at and beyond
// *dyn_rows carry grad_logp == 0, and hidden rows up to the next multiple of 128 are zero.
int lmhead_bwd_tc(const void* hidden, const void* w, const int32_t* targets, const float* lse,
                  const float* grad_logp, long long n, int h, int v, float inv_t, void* grad_hidden, float* grad_w,
                  int accumulate, void* ws, size_t ws_bytes, long long chunk_rows, const int* dyn_rows,
                  uint32_t* status, cudaStream_t stream);

// ---- backward without recomputation (lmhead_tc.cu, kept_rows.cu) ----
// The keeping forward works on rows [offset, offset + n) of a compact row space whose size is *dyn_rows and leaves,
// for each row, q[r, v] = exp(z[r, v] - zy[r]) in bf16 (pitch v^8, 0 at the target column) and per-split sums of q
// (the target left out).  zy is the row's target logit / T, computed beforehand by target_logits().
size_t lmhead_tc_kept_bytes(long long rows, int v);
int lmhead_fwd_keep_tc(const void* hidden, const void* w, const int32_t* targets, const float* zy, long long n, int h,
                       int v, float inv_t, int splits, float* part_s, float* part_e, void* q, const int* dyn_rows,
                       long long dyn_offset, uint32_t* status, cudaStream_t stream);
// `select`: one device int of scratch (the tile choice made from the device-resident row count).
int lmhead_grad_hidden_from_kept_tc(const void* q, const void* w, const float* row_scale, long long n, int h, int v,
                                    void* grad_hidden, const int* dyn_rows, long long dyn_offset, int* select,
                                    uint32_t* status, cudaStream_t stream);
int lmhead_grad_w_from_kept_tc(const void* q, const void* hs, long long n, int h, int v, float* grad_w, int accumulate,
                               int zero_when_empty, const int* dyn_rows, long long dyn_offset, uint32_t* status,
                               cudaStream_t stream);

// Small per-row kernels around the kept-ratio path (kept_rows.cu).  `count` is the device-resident size of the
// compact row space; every launch covers compact rows [offset, offset + rows) and arrays are indexed by compact row
// unless they say otherwise.
// hidden_c points at the launch's first row (row c of the compact space is hidden_c[c - offset, :]).
// zy[c] = dot(hidden_c[c - offset, :], W[targets_c[c], :]) / T for the rows a GEMM launch may touch (up to the next 128).
int target_logits(const void* hidden_c, const void* w, const int32_t* targets_c, const int* count, long long offset,
                  long long rows, int h, int v, float inv_t, float* zy, cudaStream_t stream);
// s = sum of the split sums; lse = zy + log1p(s), logp = -log1p(s), sprime = s,
// entropy = lse - (zy + part_e / T) / (1 + s); rows at and beyond *count get zeros.  part_* are [splits][rows].
int merge_kept(const float* part_s, const float* part_e, const float* zy, const int* count, long long offset,
               long long rows, int splits, float inv_t, float* sprime, float* logp, float* lse, float* entropy,
               uint32_t* status, cudaStream_t stream);
// Per-token inputs of the loss in the compact row space (rows beyond *count: zeros, mask 0), and *n_valid = *count.
int gather_loss_inputs(const int* idx, const int* count, long long cap, const float* behav, const int32_t* versions,
                       const float* adv, float* behav_c, int32_t* versions_c, float* adv_c, uint8_t* mask_c,
                       long long* n_valid, cudaStream_t stream);
// Chooses the backward's rows among rows [offset, offset + rows): those with g_c != 0, K of them (-> *bwd_count).
// They are made contiguous at positions 0 .. K-1 of the launch's q by moving only the rows that fill the holes
// left by rows with g_c == 0 (clipped tokens); perm[p] = row of the range now at position p.
int plan_backward_rows(const float* g_c, const int* count, long long offset, long long rows, int* bwd_count,
                       int* n_moves, int* perm, int* move_src, int* move_dst, void* q, int v, cudaStream_t stream);
// Prepares the two gradient contractions for the positions p of a launch (K = *bwd_count of them, or every row
// of [offset, offset + rows) below *count when bwd_count is null; c = offset + perm[p], or offset + p):
//   row_scale[p] = -g / (T (1 + sprime[c]))      g = g_c[c], or g_batch[idx[c]] when g_c is null
//   q[p, y_c]    = -sprime[c]                     (the target's entry: 1 - 1/p_y)
//   hs[p, :]     = row_scale[p] * hidden row      (hidden_c[c], or hidden_batch[idx[c]] when hidden_c is null)
//   bwd_idx[p]   = idx[c]                         (batch row; skipped when bwd_idx is null)
// positions from K to the next multiple of 128 get scale 0 and zero hs rows.
int prepare_kept_backward(const int* count, long long offset, long long rows, const int* bwd_count, const int* perm,
                          int h, int v, float inv_t, const float* sprime, const int32_t* targets_c, const float* g_c,
                          const float* g_batch, const int* idx, const void* hidden_c, const void* hidden_batch,
                          float* row_scale, int* bwd_idx, void* q, void* hs, cudaStream_t stream);
// dst[bwd_idx[p], :] = src[p, :] for positions p < *bwd_count.
int scatter_rows_range(const void* src, int h, const int* bwd_idx, const int* bwd_count, long long rows, void* dst,
                       cudaStream_t stream);
// Batch-space outputs from compact ones: out[t] = pos[t] >= 0 ? in_c[pos[t]] : 0 for up to four arrays (null = skip),
// and, when grad_hidden is given, zero rows of grad_hidden [n, h] for rows that were not kept or have g_c == 0.
int finish_batch_outputs(const int* pos, long long n, const float* logp_c, float* logp, const float* lse_c, float* lse,
                         const float* g_c, float* grad_logp, const float* ent_c, float* entropy, void* grad_hidden,
                         int h, cudaStream_t stream);

// ---- loss on a slice, for the row-chunked step (loss_kernels.cu) ----
// Forward + backward of the A-3PO loss on n tokens with M taken from *n_valid and the upstream gradient from
// *grad_loss (null = 1); block partials go to
// partials[0 .. blocks) (loss_partial_bytes() each), which loss_finalize_partials sums in index order.
size_t loss_partial_bytes();
int loss_max_partials();
int loss_blocks_for(long long n, int max_blocks);
int loss_fwd_bwd_slice(const float* logp, const float* behav, const int32_t* versions, const float* adv,
                       const uint8_t* mask, long long n, int32_t current_version, float clip_eps,
                       const long long* n_valid, const float* grad_loss, float* grad_logp, void* partials, int blocks,
                       cudaStream_t stream);
int loss_finalize_partials(const void* partials, int count, float* loss, a3po_stats* stats, cudaStream_t stream);

// Launches a one-warp kernel whose bounded wait must expire after timeout_ms and set the status bit.
int selftest_wait_timeout(uint32_t* status, unsigned timeout_ms, cudaStream_t stream);

}  // namespace a3po
