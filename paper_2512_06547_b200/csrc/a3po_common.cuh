// Shared host/device helpers of the A-3PO library (not part of the public ABI).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <stdint.h>
#include <atomic>

#include "a3po.h"

namespace a3po {

constexpr int kWarp = 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

extern std::atomic<long long> g_launches;  // defined in api.cu

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

inline bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Number of SMs of the current device (cached per device id).
int sm_count();

// Kernel identifiers for launch accounting and the optional CUDA-event profile.
enum KernelId : int {
  kKLossFwd = 0, kKLossBwd, kKLossFwdBwd, kKLossFinalize, kKMaskCount, kKMaskCountFinalize, kKExpandVersions,
  kKMergePartials, kKSimtFwd, kKSimtDz, kKSimtGemm, kKTcFwd, kKTcDz, kKTcGradHidden, kKTcGradW, kKCompact, kKGrpo,
  kKSelfTest, kKTcFwdKeep, kKKeptRows, kKH2D, kKMoveRows,
  kKernelIdCount
};

// When profiling is enabled (a3po_profile_enable), brackets one kernel launch with a pair of CUDA
// events recorded on the launch stream; otherwise does nothing.
struct ProfileScope {
  int kernel_id;
  cudaStream_t stream;
  cudaEvent_t start, stop;  // both null when profiling is off
  ProfileScope(int kernel_id, cudaStream_t s);
  ~ProfileScope();
};
#define A3PO_LAUNCH(kernel_id, stream, ...)            \
  do {                                                 \
    ::a3po::ProfileScope _a3po_scope(kernel_id, stream); \
    __VA_ARGS__;                                       \
  } while (0)

// Records one kernel launch and converts a launch error into an a3po_error.
inline int after_launch() {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  cudaError_t e = cudaPeekAtLastError();
  if (e != cudaSuccess) {
    cudaGetLastError();
    return A3PO_ERR_CUDA;
  }
  return A3PO_OK;
}

#define A3PO_RETURN_IF(expr)            \
  do {                                  \
    int _rc = (expr);                   \
    if (_rc != A3PO_OK) return _rc;     \
  } while (0)

// Bump allocator over the caller's workspace.
struct Arena {
  char* base;
  size_t size;
  size_t used = 0;
  Arena(void* p, size_t n) : base(static_cast<char*>(p)), size(n) {}
  template <typename T>
  T* take(size_t count) {
    size_t off = round_up(used, 256);
    size_t bytes = count * sizeof(T);
    if (off + bytes > size) {
      used = size + 1;
      return nullptr;
    }
    used = off + bytes;
    return reinterpret_cast<T*>(base + off);
  }
  bool ok() const { return used <= size; }
};

#ifdef __CUDACC__
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ long long warp_sum(long long v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_min(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fminf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float fast_rcp(float x) {
  float y;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float to_float(float x) { return x; }
__device__ __forceinline__ float to_float(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_float(float x);
template <> __device__ __forceinline__ float from_float<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}
#endif

}  // namespace a3po
