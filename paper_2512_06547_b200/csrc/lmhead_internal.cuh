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

// ---- tcgen05 / TMEM / TMA kernels (lmhead_tc.cu), bf16 only ----
bool lmhead_tc_supported(const void* hidden, const void* w, long long n, int h, int v);
// Vocabulary splits the tensor-core forward wants for (n, v): each (row tile, split) pair is one work item.
int lmhead_tc_fwd_splits(long long n, int v);
int lmhead_fwd_tc(const void* hidden, const void* w, const int32_t* targets, long long n, int h, int v, float inv_t,
                  int splits, SoftmaxPartial* part, float* part_ent, float* zy, uint32_t* status,
                  cudaStream_t stream);
// Workspace (bytes) of the tensor-core backward for a chunk of `chunk_rows` rows.
size_t lmhead_tc_bwd_ws_bytes(long long chunk_rows, long long n, int h, int v);
int lmhead_bwd_tc(const void* hidden, const void* w, const int32_t* targets, const float* lse,
                  const float* grad_logp, long long n, int h, int v, float inv_t, void* grad_hidden, float* grad_w,
                  int accumulate, void* ws, size_t ws_bytes, long long chunk_rows, uint32_t* status,
                  cudaStream_t stream);

}  // namespace a3po
