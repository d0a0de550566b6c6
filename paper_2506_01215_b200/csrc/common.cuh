// Shared device/host helpers of the REFORM kernels (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "reform.h"

namespace reform {

// Streaming multiprocessors of the current device (148 on a B200: 2 dies x 74); grids are sized in
// multiples of this.  Queried once per device and cached.
inline int num_sms() {
  constexpr int kMaxDevices = 64;
  static int cache[kMaxDevices] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  int n = cache[dev];
  if (n <= 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cache[dev] = n;
  }
  return n;
}

// Per-thread record of the last failing CUDA call and a process-wide launch counter.
extern thread_local int g_last_cuda_error;
extern thread_local int g_last_path;   // REFORM_PATH_* of this thread's last selection
void count_launch(int n = 1);

inline int check_launch() {
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) {
    g_last_cuda_error = (int)e;
    return REFORM_ERR_CUDA;
  }
  return REFORM_OK;
}

// Sticky per-device error word: every kernel that gives up on a bounded wait or skips a bad index
// ORs its REFORM_DEV_* bit here (and into the caller's dev_status word when one was passed), so a
// failure is never silent.  Read and cleared through reform_device_error().
__device__ int32_t g_device_error = 0;

__device__ __forceinline__ void report_device_error(int32_t* dev_status, int32_t bit) {
  atomicOr(&g_device_error, bit);
  if (dev_status) atomicOr(dev_status, bit);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

__host__ __device__ inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

template <typename T>
__device__ __forceinline__ float to_float(T x);
template <>
__device__ __forceinline__ float to_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_float(float x);
template <>
__device__ __forceinline__ float from_float<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Order-preserving map float -> uint32 (larger float <=> larger key); -0.0
// is folded onto +0.0 first so the two compare equal.
__device__ __forceinline__ uint32_t float_to_key(float f) {
  uint32_t u = __float_as_uint(f);
  if (u == 0x80000000u) u = 0u;
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

}  // namespace reform
