// Integer prefix-and-load route score and its argmax: lanes over pods (two pods per lane), one
// warp per request.  The same lane code serves the stand-alone score kernel, the scoring tail of
// the fused match kernel and the sequential assignment kernel.
#pragma once

#include "aibx_common.cuh"

namespace aibx {

constexpr int kRouteWarps = 8;

struct ScoreParams {
  const int32_t* pod_load;
  uint64_t ready_mask;
  int w_prefix, w_load, thr_pct;
};

__device__ __forceinline__ long long pod_score(long long hit, long long n_r, long long load,
                                               int w_prefix, int w_load, int thr_pct) {
  const long long eff = (hit > 0 && 100LL * hit >= (long long)thr_pct * n_r) ? hit : 0LL;
  return (long long)w_prefix * eff - (long long)w_load * load;
}

// Candidate of one lane: the better of its two pods (ascending pod order, strict ">" keeps the
// lower pod on ties); pods that are not ready never become candidates.
__device__ __forceinline__ void lane_candidate(int lane, int P, uint64_t ready_mask, long long sc0,
                                               long long sc1, long long& top, int& arg) {
  top = LLONG_MIN;
  arg = AIBX_NO_POD;
  if (lane < P && ((ready_mask >> lane) & 1ULL)) {
    top = sc0;
    arg = lane;
  }
  const int p1 = lane + 32;
  if (p1 < P && ((ready_mask >> p1) & 1ULL) && (arg == AIBX_NO_POD || sc1 > top)) {
    top = sc1;
    arg = p1;
  }
}

// Warp argmax over (score, pod): higher score wins, equal scores go to the lower pod index,
// "no pod" loses to any pod.  Every lane ends with the winner.  Three warp reductions on
// 32-bit pieces (high half, low half, pod) instead of a shuffle tree on 64-bit pairs.
__device__ __forceinline__ void warp_argmax(long long& top, int& arg) {
  const bool valid = arg != AIBX_NO_POD;
  if (__ballot_sync(0xffffffffu, valid) == 0u) {
    top = LLONG_MIN;
    arg = AIBX_NO_POD;
    return;
  }
  const unsigned long long u = (unsigned long long)top ^ 0x8000000000000000ULL;   // order-preserving
  const unsigned int hi = valid ? (unsigned int)(u >> 32) : 0u;
  const unsigned int max_hi = __reduce_max_sync(0xffffffffu, hi);
  const bool c1 = valid && hi == max_hi;
  const unsigned int lo = c1 ? (unsigned int)u : 0u;
  const unsigned int max_lo = __reduce_max_sync(0xffffffffu, lo);
  const bool c2 = c1 && lo == max_lo;
  const unsigned int pod = c2 ? (unsigned int)arg : 0xFFFFFFFFu;
  const unsigned int best = __reduce_min_sync(0xffffffffu, pod);
  top = (long long)((((unsigned long long)max_hi << 32) | max_lo) ^ 0x8000000000000000ULL);
  arg = (int)best;
}

__global__ void __launch_bounds__(kRouteWarps * 32)
route_score_kernel(const uint32_t* __restrict__ match_len, const int64_t* __restrict__ blk_off,
                   int R, int P, ScoreParams sp, int32_t* __restrict__ best_pod,
                   int64_t* __restrict__ best_score, int64_t* __restrict__ scores) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * kRouteWarps + (threadIdx.x >> 5);
  if (r >= R) return;
  const long long n_r = blk_off[r + 1] - blk_off[r];
  long long sc[2] = {0, 0};
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int p = lane + 32 * half;
    if (p < P) {
      sc[half] = pod_score((long long)match_len[(int64_t)r * P + p], n_r, sp.pod_load[p],
                           sp.w_prefix, sp.w_load, sp.thr_pct);
      if (scores) scores[(int64_t)r * P + p] = sc[half];
    }
  }
  long long top;
  int arg;
  lane_candidate(lane, P, sp.ready_mask, sc[0], sc[1], top, arg);
  warp_argmax(top, arg);
  if (lane == 0) {
    best_pod[r] = arg;
    best_score[r] = top;
  }
}

// Sequential assignment: one warp walks the requests in order; the pod loads live in registers
// (two per lane) and the winner's lane bumps its own copy before the next request is scored.
// The next request's match lengths are fetched while the current one is reduced.
__global__ void __launch_bounds__(32)
route_assign_kernel(const uint32_t* __restrict__ match_len, const int64_t* __restrict__ blk_off,
                    int R, int P, int32_t* __restrict__ pod_load, uint64_t ready_mask, int w_prefix,
                    int w_load, int thr_pct, int increment, int32_t* __restrict__ best_pod,
                    int64_t* __restrict__ best_score) {
  const int lane = threadIdx.x;
  const int p0 = lane, p1 = lane + 32;
  int32_t load0 = p0 < P ? pod_load[p0] : 0;
  int32_t load1 = p1 < P ? pod_load[p1] : 0;
  uint32_t hit0 = 0, hit1 = 0;
  long long off_lo = 0, off_hi = 0;
  auto fetch = [&](int r) {
    if (p0 < P) hit0 = match_len[(int64_t)r * P + p0];
    if (p1 < P) hit1 = match_len[(int64_t)r * P + p1];
    off_lo = blk_off[r];
    off_hi = blk_off[r + 1];
  };
  if (R > 0) fetch(0);
  for (int r = 0; r < R; ++r) {
    const long long n_r = off_hi - off_lo;
    const long long sc0 = pod_score(hit0, n_r, load0, w_prefix, w_load, thr_pct);
    const long long sc1 = pod_score(hit1, n_r, load1, w_prefix, w_load, thr_pct);
    if (r + 1 < R) fetch(r + 1);
    long long top;
    int arg;
    lane_candidate(lane, P, ready_mask, sc0, sc1, top, arg);
    warp_argmax(top, arg);
    if (arg == p0) load0 = (int32_t)((uint32_t)load0 + (uint32_t)increment);
    if (arg == p1) load1 = (int32_t)((uint32_t)load1 + (uint32_t)increment);
    if (lane == 0) {
      best_pod[r] = arg;
      best_score[r] = top;
    }
  }
  if (p0 < P) pod_load[p0] = load0;
  if (p1 < P) pod_load[p1] = load1;
}

// The six per-request routing policies.  One warp per request (grid-stride), two pods per lane.
// A policy is "lowest figure over a candidate set": the candidate set is the ready pods, except
// for prefix-cache-aware, where a max-reduction over the qualifying hits first narrows it to the
// pods with the longest qualifying hit (if any).  The random policy picks the k-th ready pod
// by rank inside the ready mask.
struct PodMetrics {
  const int32_t* throughput;
  const int32_t* requests;
  const int32_t* kv_usage;
  const int32_t* queue_latency;
  const int32_t* serve_latency;
};

__global__ void __launch_bounds__(kRouteWarps * 32)
route_policy_kernel(int policy, const uint32_t* __restrict__ match_len,
                    const int64_t* __restrict__ blk_off, int R, int P, PodMetrics met,
                    const uint64_t* __restrict__ draws, uint64_t ready_mask, int thr_pct,
                    int32_t* __restrict__ best_pod) {
  const int lane = threadIdx.x & 31;
  const int p0 = lane, p1 = lane + 32;
  const int warps = gridDim.x * kRouteWarps;
  const uint64_t ready = ready_mask & pod_all(P);

  if (policy == AIBX_POLICY_RANDOM) {
    const int n = __popcll(ready);
    // rank of this lane's pods among the ready ones
    const int rank0 = __popcll(ready & ((1ULL << p0) - 1ULL));
    const int rank1 = __popcll(ready & ((1ULL << p1) - 1ULL));
    const bool in0 = (ready >> p0) & 1ULL, in1 = (ready >> p1) & 1ULL;
    for (int r = blockIdx.x * kRouteWarps + (threadIdx.x >> 5); r < R; r += warps) {
      if (n == 0) {
        if (lane == 0) best_pod[r] = AIBX_NO_POD;
        continue;
      }
      const int k = (int)(draws[r] % (unsigned long long)n);
      if (in0 && rank0 == k) best_pod[r] = p0;
      if (in1 && rank1 == k) best_pod[r] = p1;
    }
    return;
  }

  // the figure every remaining policy minimises, negated so that warp_argmax applies
  const int32_t* a = policy == AIBX_POLICY_THROUGHPUT      ? met.throughput
                     : policy == AIBX_POLICY_LEAST_KV_CACHE ? met.kv_usage
                     : policy == AIBX_POLICY_LEAST_LATENCY  ? met.queue_latency
                                                            : met.requests;
  const int32_t* b = policy == AIBX_POLICY_LEAST_LATENCY ? met.serve_latency : nullptr;
  long long sc0 = 0, sc1 = 0;
  if (p0 < P) sc0 = -((long long)a[p0] + (b ? (long long)b[p0] : 0LL));
  if (p1 < P) sc1 = -((long long)a[p1] + (b ? (long long)b[p1] : 0LL));

  if (policy != AIBX_POLICY_PREFIX_CACHE_AWARE) {
    long long top;
    int arg;
    lane_candidate(lane, P, ready, sc0, sc1, top, arg);
    warp_argmax(top, arg);
    for (int r = blockIdx.x * kRouteWarps * 32 + threadIdx.x; r < R; r += warps * 32)
      best_pod[r] = arg;                       // the same pod for every request: lanes over r
    return;
  }

  for (int r = blockIdx.x * kRouteWarps + (threadIdx.x >> 5); r < R; r += warps) {
    const long long n_r = blk_off[r + 1] - blk_off[r];
    unsigned int e0 = 0, e1 = 0;               // qualifying hit of a ready pod, else 0
    if (p0 < P && ((ready >> p0) & 1ULL)) {
      const unsigned int hit = match_len[(int64_t)r * P + p0];
      if (hit > 0 && 100LL * hit >= (long long)thr_pct * n_r) e0 = hit;
    }
    if (p1 < P && ((ready >> p1) & 1ULL)) {
      const unsigned int hit = match_len[(int64_t)r * P + p1];
      if (hit > 0 && 100LL * hit >= (long long)thr_pct * n_r) e1 = hit;
    }
    const unsigned int longest = __reduce_max_sync(0xffffffffu, e0 > e1 ? e0 : e1);
    uint64_t cand = ready;
    if (longest > 0) {
      const unsigned int c_lo = __ballot_sync(0xffffffffu, e0 == longest);
      const unsigned int c_hi = __ballot_sync(0xffffffffu, e1 == longest);
      cand = (uint64_t)c_lo | ((uint64_t)c_hi << 32);
    }
    long long top;
    int arg;
    lane_candidate(lane, P, cand, sc0, sc1, top, arg);
    warp_argmax(top, arg);
    if (lane == 0) best_pod[r] = arg;
  }
}

}  // namespace aibx
