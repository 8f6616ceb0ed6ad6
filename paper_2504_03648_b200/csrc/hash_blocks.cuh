// Chained per-block prefix keys: key_i = XXH64(block i as little-endian int32, seed = key_{i-1}).
//
// The chain is serial per request (all four accumulators of block i start from key_{i-1}), so
// blocks of one request cannot be hashed independently; what can be spread is the work inside
// a block.  Four lanes (a quad) serve one request, one accumulator each, eight requests per warp:
//   * per 32-byte stripe every lane reads its own 8 bytes (a quad reads the stripe's 32 bytes
//     contiguously), multiplies them by PRIME64_2 and runs its accumulator's round - one
//     add/rotate/multiply on the critical path instead of four sharing one issue slot
//     (64-bit integer work issues at half rate, so a lone lane doing all four is issue-bound);
//   * tokens are fetched eight stripes ahead into registers, so memory latency never meets
//     the chain;
//   * at a block end the quad sums the rotated accumulators with two shuffle steps, exchanges
//     the four fold terms, and every lane finishes the same key, so the next seed needs no
//     further broadcast; lane 0 of the quad stores it.
// Bound: dependent 64-bit integer latency of the longest request, not HBM.
#pragma once

#include "aibx_common.cuh"

namespace aibx {

constexpr uint64_t kP1 = 0x9E3779B185EBCA87ULL;
constexpr uint64_t kP2 = 0xC2B2AE3D27D4EB4FULL;
constexpr uint64_t kP3 = 0x165667B19E3779F9ULL;
constexpr uint64_t kP4 = 0x85EBCA77C2B2AE63ULL;

constexpr int kGroupStripes = 8;                // stripes fetched ahead per lane (16 registers)

__device__ __forceinline__ uint64_t rotl64(uint64_t x, int r) {
  return (x << r) | (x >> (64 - r));
}

// End of a block: `v` is this lane's accumulator.  Returns the block's key in all four lanes.
__device__ __forceinline__ uint64_t finish_block_quad(unsigned int qmask, int quad_base, uint64_t v,
                                                      int rot, uint64_t len_bytes) {
  uint64_t h = rotl64(v, rot);
  h += shfl_xor64(qmask, h, 1);
  h += shfl_xor64(qmask, h, 2);
  const uint64_t m = rotl64(v * kP2, 31) * kP1;
  const uint64_t m0 = shfl64(qmask, m, quad_base + 0);
  const uint64_t m1 = shfl64(qmask, m, quad_base + 1);
  const uint64_t m2 = shfl64(qmask, m, quad_base + 2);
  const uint64_t m3 = shfl64(qmask, m, quad_base + 3);
  h = (h ^ m0) * kP1 + kP4;
  h = (h ^ m1) * kP1 + kP4;
  h = (h ^ m2) * kP1 + kP4;
  h = (h ^ m3) * kP1 + kP4;
  h += len_bytes;
  h ^= h >> 33;
  h *= kP2;
  h ^= h >> 29;
  h *= kP3;
  h ^= h >> 32;
  return h;
}

// SPB = stripes (32 bytes) per block when known at compile time (divides 8), 0 = `spb_rt`.
template <int SPB>
__global__ void __launch_bounds__(32)
hash_blocks_kernel(const int32_t* __restrict__ tokens, const int64_t* __restrict__ tok_off,
                   const int64_t* __restrict__ blk_off, int R, int spb_rt, uint64_t root_seed,
                   uint64_t* __restrict__ hashes, const uint32_t* __restrict__ start_blk,
                   const uint64_t* __restrict__ start_seed) {
  const int lane = threadIdx.x;
  const int k = lane & 3;                              // accumulator of this lane
  const int quad_base = lane & ~3;
  const unsigned int qmask = 0xFu << quad_base;
  const int r = blockIdx.x * 8 + (lane >> 2);
  if (r >= R) return;                                  // whole quads leave together

  const int spb = SPB > 0 ? SPB : spb_rt;
  // a resumed chain starts at block `skip` of the request, seeded with the key of block skip-1
  const int64_t skip = start_blk ? (int64_t)start_blk[r] : 0;
  const int64_t out0 = blk_off[r] + skip;
  const int64_t n_stripes = (blk_off[r + 1] - out0) * spb;
  if (n_stripes <= 0) return;
  if (start_seed) root_seed = start_seed[r];
  // this lane's 8 bytes of stripe s are words [8*s + 2*k, 8*s + 2*k + 2) of the request
  const int32_t* p = tokens + tok_off[r] + skip * spb * 8 + 2 * k;
  uint64_t* out = hashes + out0;

  // per-lane constants of the four accumulators
  const uint64_t init_add = k == 0 ? kP1 + kP2 : k == 1 ? kP2 : k == 2 ? 0ULL : 0ULL - kP1;
  const int rot = k == 0 ? 1 : k == 1 ? 7 : k == 2 ? 12 : 18;
  const uint64_t len_bytes = (uint64_t)spb * 32ULL;

  // Groups of 8 stripes: `cur` feeds the chain while `nxt` is in flight.  Whole groups run
  // without per-stripe checks; only the last, partial group of a request is guarded.
  const int n = (int)n_stripes;
  uint32_t cur_lo[kGroupStripes] = {}, cur_hi[kGroupStripes] = {};
  uint32_t nxt_lo[kGroupStripes] = {}, nxt_hi[kGroupStripes] = {};
  auto fetch = [&](const int32_t* q, int avail, uint32_t* lo, uint32_t* hi) {
    if (avail >= kGroupStripes) {
#pragma unroll
      for (int s = 0; s < kGroupStripes; ++s) {
        lo[s] = (uint32_t)__ldg(q + 8 * s);
        hi[s] = (uint32_t)__ldg(q + 8 * s + 1);
      }
    } else {
#pragma unroll
      for (int s = 0; s < kGroupStripes; ++s) {
        if (s < avail) {                               // only full blocks are ever read
          lo[s] = (uint32_t)__ldg(q + 8 * s);
          hi[s] = (uint32_t)__ldg(q + 8 * s + 1);
        }
      }
    }
  };

  uint64_t v = root_seed + init_add;
  int in_block = 0;
  auto stripe = [&](int s) {
    const uint64_t x = (uint64_t)cur_lo[s] | ((uint64_t)cur_hi[s] << 32);
    v = rotl64(v + x * kP2, 31) * kP1;
    bool block_end;
    if constexpr (SPB > 0) {
      block_end = ((s + 1) % SPB) == 0;
    } else {
      block_end = (++in_block == spb);
    }
    if (block_end) {
      in_block = 0;
      const uint64_t key = finish_block_quad(qmask, quad_base, v, rot, len_bytes);
      if (k == 0) *out = key;
      ++out;
      v = key + init_add;
    }
  };

  fetch(p, n, cur_lo, cur_hi);
  int left = n;                                        // stripes not yet consumed
  while (left >= kGroupStripes) {
    fetch(p + 8 * kGroupStripes, left - kGroupStripes, nxt_lo, nxt_hi);
#pragma unroll
    for (int s = 0; s < kGroupStripes; ++s) stripe(s);
#pragma unroll
    for (int s = 0; s < kGroupStripes; ++s) {
      cur_lo[s] = nxt_lo[s];
      cur_hi[s] = nxt_hi[s];
    }
    p += 8 * kGroupStripes;
    left -= kGroupStripes;
  }
#pragma unroll
  for (int s = 0; s < kGroupStripes; ++s) {
    if (s < left) stripe(s);                           // uniform inside the quad
  }
}

inline int32_t launch_hash_blocks(const int32_t* d_tokens, const int64_t* d_tok_off,
                                  const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                                  uint64_t root_seed, uint64_t* d_hashes, cudaStream_t st,
                                  const uint32_t* d_start_blk = nullptr,
                                  const uint64_t* d_start_seed = nullptr) {
  const int spb = block_tokens / 8;
  const int grid = (R + 7) / 8;
  if (spb == 1) {
    hash_blocks_kernel<1><<<grid, 32, 0, st>>>(d_tokens, d_tok_off, d_blk_off, R, spb, root_seed,
                                               d_hashes, d_start_blk, d_start_seed);
  } else if (spb == 2) {
    hash_blocks_kernel<2><<<grid, 32, 0, st>>>(d_tokens, d_tok_off, d_blk_off, R, spb, root_seed,
                                               d_hashes, d_start_blk, d_start_seed);
  } else if (spb == 4) {
    hash_blocks_kernel<4><<<grid, 32, 0, st>>>(d_tokens, d_tok_off, d_blk_off, R, spb, root_seed,
                                               d_hashes, d_start_blk, d_start_seed);
  } else if (spb == 8) {
    hash_blocks_kernel<8><<<grid, 32, 0, st>>>(d_tokens, d_tok_off, d_blk_off, R, spb, root_seed,
                                               d_hashes, d_start_blk, d_start_seed);
  } else {
    hash_blocks_kernel<0><<<grid, 32, 0, st>>>(d_tokens, d_tok_off, d_blk_off, R, spb, root_seed,
                                               d_hashes, d_start_blk, d_start_seed);
  }
  return launch_status();
}

}  // namespace aibx
