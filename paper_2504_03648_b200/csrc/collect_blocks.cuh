// Set of matched blocks: ascending distinct valid ids of a list, padded with AIBX_NO_BLOCK.
// A bitmap over block ids in caller-provided global scratch is marked by one thread per id,
// then one CTA turns it into the ascending list with a running popcount scan.  Short lists over
// small pools take one CTA with the bitmap in shared memory instead (one launch, no scratch).
#pragma once

#include "aibx_common.cuh"

namespace aibx {

constexpr int kCollectThreads = 1024;

// `n_dev` (nullable): the list's length read on the device instead of `n` (the grid then
// strides over it).
__global__ void collect_mark_kernel(const uint32_t* __restrict__ ids, int64_t n,
                                    const int64_t* __restrict__ n_dev, uint32_t num_blocks,
                                    unsigned int* __restrict__ bitmap) {
  if (n_dev) n = *n_dev;
  for (int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; i < n;
       i += (int64_t)gridDim.x * blockDim.x) {
    const uint32_t id = ids[i];
    if (id < num_blocks) {
      atomicOr(&bitmap[id >> 5], 1u << (id & 31u));
    } else if (id != AIBX_NO_BLOCK) {
      raise_status(AIBX_ERR_RANGE);
    }
  }
}

__global__ void __launch_bounds__(kCollectThreads)
collect_compact_kernel(const unsigned int* __restrict__ bitmap, uint32_t num_blocks, int64_t n,
                       const int64_t* __restrict__ n_dev, uint32_t* __restrict__ out,
                       uint32_t* __restrict__ count) {
  __shared__ unsigned int s_warp[32];
  __shared__ unsigned int s_base;
  if (n_dev) n = *n_dev;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const uint32_t n_words = (num_blocks + 31u) / 32u;
  if (tid == 0) s_base = 0;
  __syncthreads();
  for (uint32_t w0 = 0; w0 < n_words; w0 += kCollectThreads) {
    const uint32_t w = w0 + tid;
    unsigned int bits = (w < n_words) ? bitmap[w] : 0u;
    const unsigned int c = __popc(bits);
    // inclusive scan of c inside the warp, then across the 32 warps
    unsigned int inc = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned int o = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += o;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      unsigned int t = s_warp[lane];
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned int o = __shfl_up_sync(0xffffffffu, t, d);
        if (lane >= d) t += o;
      }
      s_warp[lane] = t;   // inclusive over warps
    }
    __syncthreads();
    const unsigned int before = s_base + (warp ? s_warp[warp - 1] : 0u) + (inc - c);
    unsigned int pos = before;
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      if ((int64_t)pos < n) out[pos] = w * 32u + (uint32_t)b;
      ++pos;
    }
    __syncthreads();
    if (tid == 0) s_base += s_warp[31];
    __syncthreads();
  }
  const unsigned int total = s_base;
  for (int64_t i = (int64_t)total + tid; i < n; i += kCollectThreads) out[i] = AIBX_NO_BLOCK;
  if (tid == 0) *count = total;
}

// The whole job in one CTA for short lists over small pools: the bitmap lives in shared memory
// (no global scratch traffic, no separate clearing and marking launches).  Same output.
constexpr uint32_t kCollectSmallWords = 8192;          // 32 KiB of shared memory: 262,144 blocks
constexpr int64_t kCollectSmallIds = 1 << 16;

__global__ void __launch_bounds__(kCollectThreads)
collect_small_kernel(const uint32_t* __restrict__ ids, int64_t n, uint32_t num_blocks,
                     uint32_t* __restrict__ out, uint32_t* __restrict__ count) {
  __shared__ unsigned int s_bits[kCollectSmallWords];
  __shared__ unsigned int s_warp[32];
  __shared__ unsigned int s_base;
  const int tid = threadIdx.x;
  const int lane = tid & 31;
  const int warp = tid >> 5;
  const uint32_t n_words = (num_blocks + 31u) / 32u;
  for (uint32_t w = tid; w < n_words; w += kCollectThreads) s_bits[w] = 0u;
  if (tid == 0) s_base = 0;
  __syncthreads();
  // eight ids per thread in flight: the list is read in a couple of memory round trips
  for (int64_t i0 = tid; i0 < n; i0 += 8 * kCollectThreads) {
    uint32_t id[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int64_t i = i0 + (int64_t)u * kCollectThreads;
      id[u] = i < n ? __ldg(ids + i) : AIBX_NO_BLOCK;
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      if (id[u] < num_blocks) {
        atomicOr(&s_bits[id[u] >> 5], 1u << (id[u] & 31u));
      } else if (id[u] != AIBX_NO_BLOCK) {
        raise_status(AIBX_ERR_RANGE);
      }
    }
  }
  __syncthreads();
  for (uint32_t w0 = 0; w0 < n_words; w0 += kCollectThreads) {
    const uint32_t w = w0 + tid;
    unsigned int bits = (w < n_words) ? s_bits[w] : 0u;
    const unsigned int c = __popc(bits);
    unsigned int inc = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned int o = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += o;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      unsigned int t = s_warp[lane];
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned int o = __shfl_up_sync(0xffffffffu, t, d);
        if (lane >= d) t += o;
      }
      s_warp[lane] = t;
    }
    __syncthreads();
    unsigned int pos = s_base + (warp ? s_warp[warp - 1] : 0u) + (inc - c);
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      if ((int64_t)pos < n) out[pos] = w * 32u + (uint32_t)b;
      ++pos;
    }
    __syncthreads();
    if (tid == 0) s_base += s_warp[31];
    __syncthreads();
  }
  const unsigned int total = s_base;
  for (int64_t i = (int64_t)total + tid; i < n; i += kCollectThreads) out[i] = AIBX_NO_BLOCK;
  if (tid == 0) *count = total;
}

}  // namespace aibx
