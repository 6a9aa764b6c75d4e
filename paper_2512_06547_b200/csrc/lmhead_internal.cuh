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
// dst[t, :] = src_c[pos[t], :] for kept rows, zero otherwise.
int scatter_rows(const void* src_c, int h, const int* pos, long long n, void* dst, cudaStream_t stream);

// ---- tcgen05 / TMEM / TMA kernels (lmhead_tc.cu), bf16 only ----
bool lmhead_tc_supported(const void* hidden, const void* w, long long n, int h, int v);
// Vocabulary splits the tensor-core forward wants for (n, v): each (row tile, split) pair is one work item.
int lmhead_tc_fwd_splits(long long n, int v);
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

// ---- backward without recomputation (lmhead_tc.cu, saved_logits.cu) ----
// The saving forward keeps, for n rows, u[n, v^8] (fp16: z log2(e)/T minus a per-(row, 256-column tile)
// reference) followed by ref[n, tiles] (fp32) in one buffer of lmhead_tc_saved_logits_bytes(n, v) bytes.
size_t lmhead_tc_saved_logits_bytes(long long n, int v);
int lmhead_fwd_save_tc(const void* hidden, const void* w, const int32_t* targets, long long n, int h, int v,
                       float inv_t, int splits, SoftmaxPartial* part, float* zy, void* saved, const int* dyn_rows,
                       uint32_t* status, cudaStream_t stream);
// dz[c, :] (bf16, pitch v^8, `bwd.cap` rows allocated) for the backward's compact rows from the kept logits;
// fwd_pos maps a batch row to its row in `saved` (null: identity).
int dz_from_saved(const void* saved, long long saved_rows, int v, const int* fwd_pos, const CompactBuffers& bwd,
                  float inv_t, void* dz, cudaStream_t stream);
int lmhead_bwd_from_dz_tc(const void* hidden, const void* w, const void* dz, long long n, int h, int v,
                          void* grad_hidden, float* grad_w, int accumulate, const int* dyn_rows, uint32_t* status,
                          cudaStream_t stream);

// Launches a one-warp kernel whose bounded wait must expire after timeout_ms and set the status bit.
int selftest_wait_timeout(uint32_t* status, unsigned timeout_ms, cudaStream_t stream);

}  // namespace a3po
