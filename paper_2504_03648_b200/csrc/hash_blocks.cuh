// Chained per-block prefix keys: key_i = XXH64(block i as little-endian int32, seed = key_{i-1}).
//
// The chain is serial per request (all four accumulators of block i start from key_{i-1}), so
// the kernel parallelises across requests - one warp each - and, inside a warp, takes
// everything that does not depend on the seed off the serial lane:
//   * all 32 lanes fetch the tokens with aligned 16-byte loads (1 KiB per step) into shared
//     memory, one step ahead of the chain;
//   * all 32 lanes multiply the 64-bit input lanes by PRIME64_2 (the seed-free half of a round);
//   * lane 0 walks the stripes, keeping only add/rotate/multiply per round on the critical path;
//   * the keys of a step go out with one coalesced store.
// Bound: dependent 64-bit integer latency of the longest request, not HBM.
#pragma once

#include "aibx_common.cuh"

namespace aibx {

constexpr uint64_t kP1 = 0x9E3779B185EBCA87ULL;
constexpr uint64_t kP2 = 0xC2B2AE3D27D4EB4FULL;
constexpr uint64_t kP3 = 0x165667B19E3779F9ULL;
constexpr uint64_t kP4 = 0x85EBCA77C2B2AE63ULL;

constexpr int kHashWarps = 4;          // warps (= requests) per CTA
constexpr int kStepWords = 256;        // 32-bit tokens consumed per warp step (32 stripes)
constexpr int kStepVecs = kStepWords / 4 + 1;   // +1: a request may start mid-vector

__device__ __forceinline__ uint64_t rotl64(uint64_t x, int r) {
  return (x << r) | (x >> (64 - r));
}

// Second half of a round; `pm` is the input lane already multiplied by PRIME64_2.
__device__ __forceinline__ uint64_t round_pm(uint64_t acc, uint64_t pm) {
  return rotl64(acc + pm, 31) * kP1;
}

__device__ __forceinline__ uint64_t merge_acc(uint64_t h, uint64_t v) {
  h ^= rotl64(v * kP2, 31) * kP1;
  return h * kP1 + kP4;
}

__device__ __forceinline__ uint64_t finish_block(uint64_t v1, uint64_t v2, uint64_t v3,
                                                 uint64_t v4, uint64_t len_bytes) {
  uint64_t h = rotl64(v1, 1) + rotl64(v2, 7) + rotl64(v3, 12) + rotl64(v4, 18);
  h = merge_acc(h, v1);
  h = merge_acc(h, v2);
  h = merge_acc(h, v3);
  h = merge_acc(h, v4);
  h += len_bytes;
  h ^= h >> 33;
  h *= kP2;
  h ^= h >> 29;
  h *= kP3;
  h ^= h >> 32;
  return h;
}

// One aligned 16-byte vector of tokens; words outside [0, total_words) read as 0 so that no
// load ever leaves the token array, whatever its alignment.
__device__ __forceinline__ uint4 load_token_vec(const int32_t* tokens, int64_t g0,
                                                int64_t total_words) {
  if (g0 >= 0 && g0 + 4 <= total_words) {
    return __ldg(reinterpret_cast<const uint4*>(tokens + g0));
  }
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (g0 + 0 >= 0 && g0 + 0 < total_words) v.x = (uint32_t)__ldg(tokens + g0 + 0);
  if (g0 + 1 >= 0 && g0 + 1 < total_words) v.y = (uint32_t)__ldg(tokens + g0 + 1);
  if (g0 + 2 >= 0 && g0 + 2 < total_words) v.z = (uint32_t)__ldg(tokens + g0 + 2);
  if (g0 + 3 >= 0 && g0 + 3 < total_words) v.w = (uint32_t)__ldg(tokens + g0 + 3);
  return v;
}

// SPB = stripes (32 bytes) per block when known at compile time, 0 = read it from `spb_rt`.
template <int SPB>
__global__ void __launch_bounds__(kHashWarps * 32)
hash_blocks_kernel(const int32_t* __restrict__ tokens, const int64_t* __restrict__ tok_off,
                   const int64_t* __restrict__ blk_off, int R, int spb_rt, uint64_t root_seed,
                   uint64_t* __restrict__ hashes) {
  __shared__ __align__(16) uint32_t s_raw[kHashWarps][kStepVecs * 4];
  __shared__ __align__(16) uint64_t s_pm[kHashWarps][kStepWords / 2];
  __shared__ uint64_t s_out[kHashWarps][32];

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * kHashWarps + warp;
  if (r >= R) return;

  const int spb = SPB > 0 ? SPB : spb_rt;
  const int64_t total_words = tok_off[R];
  const int64_t t0 = tok_off[r];
  const int64_t out0 = blk_off[r];
  const int64_t nblk = blk_off[r + 1] - out0;
  const int64_t n_stripes = nblk * spb;
  if (n_stripes <= 0) return;

  // tokens of this request start `mis` words into an aligned 16-byte vector
  const int mis = (int)((reinterpret_cast<uintptr_t>(tokens + t0) >> 2) & 3);
  const int64_t g_base = t0 - mis;                    // word index of that vector's start
  const int64_t need_words = n_stripes * 8 + mis;     // words [0, need_words) from g_base
  const int64_t n_steps = (n_stripes + 31) / 32;

  uint32_t* raw = s_raw[warp];
  uint64_t* pm = s_pm[warp];
  uint64_t* outk = s_out[warp];

  auto fetch = [&](int64_t step, uint4& a, uint4& b, uint4& c) {
    const int64_t w0 = step * kStepWords;             // first word of the step, from g_base
    a = b = c = make_uint4(0u, 0u, 0u, 0u);
    int64_t wa = w0 + 4 * lane;
    int64_t wb = w0 + 4 * (lane + 32);
    int64_t wc = w0 + 4 * 64;
    if (wa < need_words) a = load_token_vec(tokens, g_base + wa, total_words);
    if (wb < need_words) b = load_token_vec(tokens, g_base + wb, total_words);
    if (lane == 0 && wc < need_words) c = load_token_vec(tokens, g_base + wc, total_words);
  };

  uint4 va, vb, vc;
  fetch(0, va, vb, vc);

  // chain state, meaningful on lane 0 only
  uint64_t seed = root_seed;
  uint64_t v1 = seed + kP1 + kP2, v2 = seed + kP2, v3 = seed, v4 = seed - kP1;
  int in_block = 0;
  int64_t emitted = 0;
  const uint64_t len_bytes = (uint64_t)spb * 32ULL;

  for (int64_t step = 0; step < n_steps; ++step) {
    // 1. park the prefetched vectors
    reinterpret_cast<uint4*>(raw)[lane] = va;
    reinterpret_cast<uint4*>(raw)[lane + 32] = vb;
    if (lane == 0) reinterpret_cast<uint4*>(raw)[64] = vc;
    __syncwarp();
    // 2. seed-free half of every round: lane value * PRIME64_2 (4 lanes of 64 bits per thread)
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int t = lane + 32 * k;
      const uint64_t x = (uint64_t)raw[mis + 2 * t] | ((uint64_t)raw[mis + 2 * t + 1] << 32);
      pm[t] = x * kP2;
    }
    __syncwarp();
    // 3. next step's loads fly while lane 0 walks the chain
    if (step + 1 < n_steps) fetch(step + 1, va, vb, vc);
    // 4. the serial part
    int n_out = 0;
    if (lane == 0) {
      const int64_t s_begin = step * 32;
      const int s_count = (int)min((int64_t)32, n_stripes - s_begin);
      if constexpr (SPB > 0) {
        // whole blocks per step, fully unrolled
        const int nb = s_count / SPB;
        for (int b = 0; b < nb; ++b) {
#pragma unroll
          for (int s = 0; s < SPB; ++s) {
            const ulonglong2 p01 = reinterpret_cast<const ulonglong2*>(pm)[2 * (b * SPB + s)];
            const ulonglong2 p23 = reinterpret_cast<const ulonglong2*>(pm)[2 * (b * SPB + s) + 1];
            v1 = round_pm(v1, p01.x);
            v2 = round_pm(v2, p01.y);
            v3 = round_pm(v3, p23.x);
            v4 = round_pm(v4, p23.y);
          }
          seed = finish_block(v1, v2, v3, v4, len_bytes);
          outk[n_out++] = seed;
          v1 = seed + kP1 + kP2; v2 = seed + kP2; v3 = seed; v4 = seed - kP1;
        }
      } else {
        for (int s = 0; s < s_count; ++s) {
          const ulonglong2 p01 = reinterpret_cast<const ulonglong2*>(pm)[2 * s];
          const ulonglong2 p23 = reinterpret_cast<const ulonglong2*>(pm)[2 * s + 1];
          v1 = round_pm(v1, p01.x);
          v2 = round_pm(v2, p01.y);
          v3 = round_pm(v3, p23.x);
          v4 = round_pm(v4, p23.y);
          if (++in_block == spb) {
            in_block = 0;
            seed = finish_block(v1, v2, v3, v4, len_bytes);
            outk[n_out++] = seed;
            v1 = seed + kP1 + kP2; v2 = seed + kP2; v3 = seed; v4 = seed - kP1;
          }
        }
      }
    }
    n_out = __shfl_sync(0xffffffffu, n_out, 0);
    __syncwarp();
    // 5. one coalesced store of this step's keys
    if (lane < n_out) hashes[out0 + emitted + lane] = outk[lane];
    emitted += n_out;
    __syncwarp();
  }
}

inline int32_t launch_hash_blocks(const int32_t* d_tokens, const int64_t* d_tok_off,
                                  const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                                  uint64_t root_seed, uint64_t* d_hashes, cudaStream_t st) {
  const int spb = block_tokens / 8;
  const int grid = (R + kHashWarps - 1) / kHashWarps;
  const int threads = kHashWarps * 32;
  if (spb == 2) {
    hash_blocks_kernel<2><<<grid, threads, 0, st>>>(d_tokens, d_tok_off, d_blk_off, R, spb,
                                                    root_seed, d_hashes);
  } else if (spb == 4) {
    hash_blocks_kernel<4><<<grid, threads, 0, st>>>(d_tokens, d_tok_off, d_blk_off, R, spb,
                                                    root_seed, d_hashes);
  } else {
    hash_blocks_kernel<0><<<grid, threads, 0, st>>>(d_tokens, d_tok_off, d_blk_off, R, spb,
                                                    root_seed, d_hashes);
  }
  return launch_status();
}

}  // namespace aibx
