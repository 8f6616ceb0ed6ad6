// Scan-resistant victim choice on the GPU-resident index.
//
// Every entry has a 32-bit stamp (side array of the index): bits 0..29 the last epoch in which the entry was touched
// (0 = never), bits 30..31 the number of distinct epochs it was touched in, saturating at 3.
// priority = (touches >= 2 ? 2^30 : 0) + epoch: entries seen in fewer than two epochs - what a
// single scan leaves behind - go first, oldest first.
//
// Picking the k entries of lowest priority is a two-level radix select over the 31-bit
// priority, all on the device: histogram of the high 16 bits -> the bin holding the k-th entry
// -> histogram of the low 15 bits inside that bin -> the threshold priority T and how many
// entries equal to T are still needed -> one pass that appends every entry below T and that
// many entries equal to T.  Which of the entries AT the threshold are taken is not specified.
#pragma once

#include "aibx_common.cuh"
#include "index.cuh"

namespace aibx {

constexpr int kHist1Bins = 1 << 16;
constexpr int kHist2Bins = 1 << 15;

struct VictimState {
  unsigned long long k;          // wanted
  unsigned long long k_rem;      // still wanted inside the chosen high bin
  unsigned long long need_eq;    // entries equal to the threshold to take
  unsigned long long eq_taken;
  unsigned long long out_pos;
  unsigned int prefix;           // chosen high bin
  unsigned int threshold;        // entries with priority < threshold are all taken
};

struct VictimScratch {
  unsigned int hist1[kHist1Bins];
  unsigned int hist2[kHist2Bins];
  VictimState st;
};

__device__ __forceinline__ unsigned int stamp_priority(unsigned int stamp) {
  return ((stamp >> 30) >= 2u ? (1u << 30) : 0u) + (stamp & kEpochMask);
}

__global__ void index_touch_kernel(IndexView ix, const uint64_t* __restrict__ keys, int64_t n,
                                   unsigned int epoch) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint64_t key = keys[i];
  if (key_reserved(key)) return;
  const unsigned long long e = find_entry_rw(ix, key);
  if (e == ~0ULL) return;
  if (entry_mask_now(ix, e) == 0) return;
  touch_entry(ix, e, epoch);
}

// Reads one entry; returns whether it is live.
__device__ __forceinline__ bool live_slot(const IndexView& ix, unsigned long long i, uint64_t& key,
                                          unsigned int& prio) {
  uint64_t m;
  uint32_t id;
  const bool live = load_entry(ix, i, key, m, id);
  prio = live ? stamp_priority(__ldcg(ix.stamps + i)) : 0u;
  return live;
}

// Histogram pass.  Priorities cluster (few distinct epochs), so (1) lanes of a warp that hit the
// same bin elect one of them to add their number, and (2) a CTA collects its counts in a small
// direct-mapped table in shared memory and adds each hot bin to the global histogram once, at
// the end; only bins that collide in that table go to global memory at once.  Without (2) every
// warp of the grid queued up on the same few words of the global histogram.
constexpr int kHistCache = 256;

__global__ void __launch_bounds__(256)
victims_hist_kernel(IndexView ix, VictimScratch* sc, int level) {
  __shared__ unsigned int s_bin[kHistCache];
  __shared__ unsigned int s_cnt[kHistCache];
  const unsigned long long n = num_entries(ix);
  const unsigned int prefix = level == 2 ? sc->st.prefix : 0u;
  if (level == 2 && prefix == 0xFFFFFFFFu) return;       // everything is taken: no second level
  unsigned int* hist = level == 1 ? sc->hist1 : sc->hist2;
  for (int j = threadIdx.x; j < kHistCache; j += blockDim.x) {
    s_bin[j] = 0xFFFFFFFFu;
    s_cnt[j] = 0u;
  }
  __syncthreads();
  for (unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; i < n;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    uint64_t key;
    unsigned int p;
    if (!live_slot(ix, i, key, p)) continue;
    if (level == 2 && (p >> 15) != prefix) continue;
    const unsigned int bin = level == 1 ? p >> 15 : p & 0x7FFFu;
    const unsigned int active = __activemask();
    const unsigned int same = __match_any_sync(active, bin);
    if ((threadIdx.x & 31) == __ffs(same) - 1) {
      const unsigned int c = (unsigned int)__popc(same);
      const unsigned int slot = bin & (kHistCache - 1);
      const unsigned int seen = atomicCAS(&s_bin[slot], 0xFFFFFFFFu, bin);
      if (seen == 0xFFFFFFFFu || seen == bin) {
        atomicAdd(&s_cnt[slot], c);
      } else {
        atomicAdd(&hist[bin], c);                        // the table's slot belongs to another bin
      }
    }
  }
  __syncthreads();
  for (int j = threadIdx.x; j < kHistCache; j += blockDim.x) {
    if (s_bin[j] != 0xFFFFFFFFu && s_cnt[j]) atomicAdd(&hist[s_bin[j]], s_cnt[j]);
  }
}

// One CTA finds the bin that holds the `want`-th smallest entry of a histogram.
__global__ void __launch_bounds__(1024)
victims_select_kernel(VictimScratch* sc, int level, unsigned long long* __restrict__ d_count) {
  __shared__ unsigned long long s_warp[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned int* hist = level == 1 ? sc->hist1 : sc->hist2;
  const int nbins = level == 1 ? kHist1Bins : kHist2Bins;
  const int per = nbins / 1024;
  if (level == 2 && sc->st.prefix == 0xFFFFFFFFu) return;
  const unsigned long long want = level == 1 ? sc->st.k : sc->st.k_rem;

  // this thread's `per` consecutive bins (a multiple of 8), read as 16-byte vectors, eight
  // loads in flight at a time: one bin per dependent load made this one-CTA kernel the longest
  // of the whole selection
  unsigned long long mine = 0;
  const uint4* h4 = reinterpret_cast<const uint4*>(hist + (size_t)tid * per);
  for (int v0 = 0; v0 < per / 4; v0 += 8) {
    uint4 q[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) q[u] = __ldcg(h4 + v0 + u);
#pragma unroll
    for (int u = 0; u < 8; ++u)
      mine += (unsigned long long)q[u].x + q[u].y + q[u].z + q[u].w;
  }
  unsigned long long inc = mine;                       // inclusive scan over the CTA
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const unsigned long long o = __shfl_up_sync(0xffffffffu, inc, d);
    if (lane >= d) inc += o;
  }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    unsigned long long t = s_warp[lane];
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned long long o = __shfl_up_sync(0xffffffffu, t, d);
      if (lane >= d) t += o;
    }
    s_warp[lane] = t;
  }
  __syncthreads();
  const unsigned long long before = (warp ? s_warp[warp - 1] : 0ULL) + (inc - mine);
  const unsigned long long total = s_warp[31];

  if (level == 1 && tid == 0) {
    *d_count = want < total ? want : total;
    if (want >= total) {                                // every live entry is a victim
      sc->st.prefix = 0xFFFFFFFFu;
      sc->st.threshold = 0x80000000u;
      sc->st.need_eq = 0;
    }
  }
  if (want == 0 || (level == 1 && want >= total)) return;
  if (before < want && want <= before + mine) {
    unsigned long long c = before;
    for (int b = 0; b < per; ++b) {
      const unsigned int h = hist[tid * per + b];
      if (c < want && want <= c + h) {
        if (level == 1) {
          sc->st.prefix = (unsigned int)(tid * per + b);
          sc->st.k_rem = want - c;
        } else {
          sc->st.threshold = (sc->st.prefix << 15) | (unsigned int)(tid * per + b);
          sc->st.need_eq = want - c;
        }
        break;
      }
      c += h;
    }
  }
}

// Collect pass.  Tickets for the entries at the threshold and room in the output are reserved
// once per CTA and turn of the loop (ballots, a sum over the warps in shared memory, one atomic
// each), not once per warp: with clustered priorities nearly every warp holds threshold entries.
__global__ void __launch_bounds__(256)
victims_collect_kernel(IndexView ix, VictimScratch* sc, uint64_t* __restrict__ out_keys,
                       uint32_t* __restrict__ out_prio) {
  __shared__ unsigned int s_eq[8], s_take[8];
  __shared__ unsigned long long s_eq_base, s_out_base;
  const unsigned long long n = num_entries(ix);
  const unsigned int T = sc->st.threshold;
  const unsigned long long need_eq = sc->st.need_eq;
  const unsigned long long k = sc->st.k;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int n_warps = blockDim.x >> 5;
  for (unsigned long long cta0 = blockIdx.x * (unsigned long long)blockDim.x; cta0 < n;
       cta0 += (unsigned long long)gridDim.x * blockDim.x) {
    const unsigned long long i = cta0 + threadIdx.x;
    uint64_t key = 0;
    unsigned int p = 0;
    const bool live = i < n && live_slot(ix, i, key, p);
    bool take = live && p < T;
    // entries at the threshold are interchangeable: the first need_eq tickets win
    const bool at_thr = live && p == T && need_eq > 0;
    const unsigned int eq = __ballot_sync(0xffffffffu, at_thr);
    if (lane == 0) s_eq[warp] = __popc(eq);
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned int total = 0;
      for (int w = 0; w < n_warps; ++w) {
        const unsigned int c = s_eq[w];
        s_eq[w] = total;
        total += c;
      }
      s_eq_base = total ? atomicAdd(&sc->st.eq_taken, (unsigned long long)total) : 0ULL;
    }
    __syncthreads();
    if (at_thr) take = s_eq_base + s_eq[warp] + __popc(eq & ((1u << lane) - 1u)) < need_eq;
    const unsigned int votes = __ballot_sync(0xffffffffu, take);
    if (lane == 0) s_take[warp] = __popc(votes);
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned int total = 0;
      for (int w = 0; w < n_warps; ++w) {
        const unsigned int c = s_take[w];
        s_take[w] = total;
        total += c;
      }
      s_out_base = total ? atomicAdd(&sc->st.out_pos, (unsigned long long)total) : 0ULL;
    }
    __syncthreads();
    if (take) {
      const unsigned long long pos = s_out_base + s_take[warp] + __popc(votes & ((1u << lane) - 1u));
      if (pos < k) {
        if (out_keys) out_keys[pos] = key;
        if (out_prio) out_prio[pos] = p;
      }
    }
    __syncthreads();                                     // the shared words are reused next turn
  }
}

}  // namespace aibx
