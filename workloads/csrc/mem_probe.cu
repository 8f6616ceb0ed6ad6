// Memory-system probes for the benchmark's rooflines: what this GPU sustains for uniformly
// random, aligned reads of 32, 64 or 128 bytes over a working set of a given size.  No part of
// the library's method is here - no keys, no table, no probing sequence: every thread draws an
// offset from a counter-based generator and reads.  The result is the measured ceiling that the
// index kernels' random-access figures are set against.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {

__device__ __forceinline__ unsigned long long mix64(unsigned long long seed,
                                                    unsigned long long counter) {
  unsigned long long z = (counter + 1ULL) * 0x9E3779B97F4A7C15ULL + seed * 0xD1B54A32D192ED03ULL;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

__device__ __forceinline__ unsigned long long load32(const unsigned long long* p) {
  unsigned long long a, b, c, d;
  asm volatile("ld.global.nc.v4.u64 {%0,%1,%2,%3}, [%4];"
               : "=l"(a), "=l"(b), "=l"(c), "=l"(d)
               : "l"(p));
  return a ^ b ^ c ^ d;
}

// SECTORS 32-byte sectors per access (1, 2 or 4), PER independent accesses per thread.
template <int SECTORS, int PER>
__global__ void random_read_kernel(const unsigned long long* __restrict__ base,
                                   unsigned long long units, unsigned long long n_reads,
                                   unsigned long long seed, unsigned long long* __restrict__ sink) {
  const unsigned long long t = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
  unsigned long long acc = 0;
  unsigned long long off[PER];
#pragma unroll
  for (int k = 0; k < PER; ++k)   // multiply-shift range reduction: any number of units
    off[k] = __umul64hi(mix64(seed, t * PER + k), units) * (4ULL * SECTORS);
#pragma unroll
  for (int k = 0; k < PER; ++k) {
    if (t * PER + k < n_reads) {
#pragma unroll
      for (int s = 0; s < SECTORS; ++s) acc ^= load32(base + off[k] + 4 * s);
    }
  }
  // one 8-byte write per warp keeps the loads alive without adding traffic of its own
  acc ^= __shfl_xor_sync(0xffffffffu, (unsigned int)acc, 16) ^
         ((unsigned long long)__shfl_xor_sync(0xffffffffu, (unsigned int)(acc >> 32), 16) << 32);
  if ((threadIdx.x & 31) == 0) sink[t >> 5] = acc;
}

}  // namespace

extern "C" {

// d_base: working set of `ws_bytes` (a multiple of 128, >= 4 KiB), 32-byte aligned; every access
// reads `gran` bytes (32, 64 or 128) at a uniformly random gran-aligned offset; `per` accesses
// per thread (1, 2 or 4) are independent; d_sink holds at least n_reads / (32 * per) + 1 words.
int32_t aibx_probe_random_reads(const void* d_base, uint64_t ws_bytes, int32_t gran, int32_t per,
                                uint64_t n_reads, uint64_t seed, void* d_sink, void* stream) {
  if (!d_base || !d_sink || ws_bytes < 4096 || (ws_bytes & 127)) return -1;
  if (gran != 32 && gran != 64 && gran != 128) return -1;
  if (per != 1 && per != 2 && per != 4) return -1;
  if (n_reads == 0) return 0;
  const unsigned long long units = ws_bytes / (unsigned long long)gran;
  const unsigned long long threads = (n_reads + per - 1) / per;
  const unsigned int grid = (unsigned int)((threads + 255) / 256);
  const unsigned long long* b = static_cast<const unsigned long long*>(d_base);
  unsigned long long* k = static_cast<unsigned long long*>(d_sink);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
#define PROBE(S, P) random_read_kernel<S, P><<<grid, 256, 0, st>>>(b, units, n_reads, seed, k)
  if (gran == 32) {
    if (per == 1) PROBE(1, 1); else if (per == 2) PROBE(1, 2); else PROBE(1, 4);
  } else if (gran == 64) {
    if (per == 1) PROBE(2, 1); else if (per == 2) PROBE(2, 2); else PROBE(2, 4);
  } else {
    if (per == 1) PROBE(4, 1); else if (per == 2) PROBE(4, 2); else PROBE(4, 4);
  }
#undef PROBE
  return cudaGetLastError() == cudaSuccess ? 0 : -4;
}

}  // extern "C"
