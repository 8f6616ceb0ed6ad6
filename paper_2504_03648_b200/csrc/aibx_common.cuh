// Shared device/host helpers of libaibx: status record, launch checks, small PTX wrappers.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <mutex>

#include <nvtx3/nvToolsExt.h>

#include "aibx.h"

namespace aibx {

// One status record per device (and per loaded copy of the library).  Kernels never trap:
// they record the most severe code seen and how many items raised one.
struct StatusRecord {
  int code;
  int pad;
  unsigned long long detail;
};

__device__ StatusRecord g_status;

__device__ __forceinline__ void raise_status(int code) {
  atomicMin(&g_status.code, code);
  atomicAdd(&g_status.detail, 1ULL);
}

__device__ __forceinline__ void raise_status_n(int code, unsigned long long items) {
  atomicMin(&g_status.code, code);
  atomicAdd(&g_status.detail, items);
}

constexpr uint64_t kKeyEmpty = 0ULL;
constexpr uint64_t kKeyTomb = ~0ULL;

__host__ __device__ __forceinline__ bool key_reserved(uint64_t k) {
  return k == kKeyEmpty || k == kKeyTomb;
}

__host__ __device__ __forceinline__ uint64_t pod_all(int P) {
  return P >= 64 ? ~0ULL : ((1ULL << P) - 1ULL);
}

// 64-bit warp shuffles (two 32-bit shuffles each).
__device__ __forceinline__ uint64_t shfl64(unsigned int mask, uint64_t v, int src_lane) {
  const unsigned int lo = __shfl_sync(mask, (unsigned int)v, src_lane);
  const unsigned int hi = __shfl_sync(mask, (unsigned int)(v >> 32), src_lane);
  return (uint64_t)lo | ((uint64_t)hi << 32);
}

__device__ __forceinline__ uint64_t shfl_xor64(unsigned int mask, uint64_t v, int lane_mask) {
  const unsigned int lo = __shfl_xor_sync(mask, (unsigned int)v, lane_mask);
  const unsigned int hi = __shfl_xor_sync(mask, (unsigned int)(v >> 32), lane_mask);
  return (uint64_t)lo | ((uint64_t)hi << 32);
}

__device__ __forceinline__ uint64_t shfl_up64(uint64_t v, int d) {
  const unsigned int lo = __shfl_up_sync(0xffffffffu, (unsigned int)v, d);
  const unsigned int hi = __shfl_up_sync(0xffffffffu, (unsigned int)(v >> 32), d);
  return (uint64_t)lo | ((uint64_t)hi << 32);
}

// Every entry point of the library shows as a named range in a timeline profiler (NVTX; a
// no-op costing a pointer test when no tool is attached).
struct CallRange {
  explicit CallRange(const char* name) { nvtxRangePushA(name); }
  ~CallRange() { nvtxRangePop(); }
  CallRange(const CallRange&) = delete;
  CallRange& operator=(const CallRange&) = delete;
};
#define AIBX_CALL_RANGE() ::aibx::CallRange aibx_call_range_(__func__)

// Result of the launches a call has just made.  cudaGetLastError, not Peek: the error is
// reported once, by the call that caused it, and does not make every later call on this thread
// fail.  (An error left behind by the caller's own earlier CUDA work is reported by the first
// aibx call that checks - and cleared with it.)
inline int32_t launch_status() {
  return cudaGetLastError() == cudaSuccess ? AIBX_OK : AIBX_ERR_CUDA;
}

// The cached per-device values below are single atomic words: two threads that race on the
// first call both compute the same value and store it.
inline int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
    cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

// Raise a kernel's dynamic shared-memory limit to `bytes` once per device (the attribute lives
// in the context); later calls with a smaller or equal size do nothing.  Under a lock, so that
// concurrent first calls cannot leave the record ahead of the attribute.
template <typename Kernel>
inline bool ensure_dynamic_smem(Kernel kernel, size_t bytes, int dev, size_t (&configured)[64],
                                std::mutex& lock) {
  std::lock_guard<std::mutex> guard(lock);
  if (bytes <= configured[dev]) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) !=
      cudaSuccess)
    return false;
  configured[dev] = bytes;
  return true;
}

}  // namespace aibx
