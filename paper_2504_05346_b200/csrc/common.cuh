// Shared host/device helpers of the Thanos sm_100a library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "thanos.h"

namespace thanos {

extern std::atomic<long long> g_launch_count;

inline void count_launch(int n = 1) { g_launch_count.fetch_add(n, std::memory_order_relaxed); }

// Launch check: cudaGetLastError right after a launch catches configuration errors only.
#define THANOS_CHECK_LAUNCH()                               \
  do {                                                      \
    ::thanos::count_launch();                               \
    if (cudaGetLastError() != cudaSuccess) return THANOS_ERR_CUDA; \
  } while (0)

#define THANOS_CUDA(call)                                   \
  do {                                                      \
    if ((call) != cudaSuccess) return THANOS_ERR_CUDA;      \
  } while (0)

#define THANOS_TRY(call)                                    \
  do {                                                      \
    thanos_status_t st__ = (call);                          \
    if (st__ != THANOS_OK) return st__;                     \
  } while (0)

// cudaFuncSetAttribute(MaxDynamicSharedMemorySize) once per device and call site instead of once
// per launch (`done` is the call site's static bit set, one bit per device).
template <typename F>
inline cudaError_t ensure_max_dyn_smem(F func, int bytes, std::atomic<unsigned long long>& done) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = 1ull << (dev & 63);
  if (done.load(std::memory_order_relaxed) & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
  if (e == cudaSuccess) done.fetch_or(bit, std::memory_order_relaxed);
  return e;
}

// Grids are sized for the 148 SMs of a B200 (this library is built for sm_100a only).
constexpr int NUM_SMS = 148;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

// Bump allocator over the caller's workspace (256-byte granules).
struct Arena {
  char* base;
  size_t size;
  size_t off;
  Arena(void* p, size_t n) : base(static_cast<char*>(p)), size(n), off(0) {}
  template <typename T>
  T* take(size_t count) {
    size_t bytes = round_up(count * sizeof(T), 256);
    if (base == nullptr || off + bytes > size) {
      off = size + 1;
      return nullptr;
    }
    T* r = reinterpret_cast<T*>(base + off);
    off += bytes;
    return r;
  }
  bool ok() const { return off <= size; }
};

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }

// x -> three bf16 planes h = bf16(x), m = bf16(x - h), l = bf16(x - h - m), `plane` elements apart
// (the operand format of the tensor-core products, see tc_gemm.cuh)
__device__ __forceinline__ void store_split3(__nv_bfloat16* __restrict__ p, int64_t plane, float d) {
#pragma unroll
  for (int pl = 0; pl < 3; ++pl) {
    const __nv_bfloat16 hb = __float2bfloat16_rn(d);
    p[(int64_t)pl * plane] = hb;
    d -= __bfloat162float(hb);
  }
}

// First device-detected error wins.
__device__ __forceinline__ void report_error(int32_t* status2, int32_t code, int32_t index) {
  if (atomicCAS(status2, 0, code) == 0) status2[1] = index;
}

}  // namespace thanos
