// Integer prefix-and-load route score and its argmax: one warp per request, lanes over pods.
#pragma once

#include "aibx_common.cuh"

namespace aibx {

constexpr int kRouteWarps = 8;

__global__ void __launch_bounds__(kRouteWarps * 32)
route_score_kernel(const uint32_t* __restrict__ match_len, const int64_t* __restrict__ blk_off,
                   int R, int P, const int32_t* __restrict__ pod_load, uint64_t ready_mask,
                   int w_prefix, int w_load, int thr_pct, int32_t* __restrict__ best_pod,
                   int64_t* __restrict__ best_score, int64_t* __restrict__ scores) {
  const int lane = threadIdx.x & 31;
  const int r = blockIdx.x * kRouteWarps + (threadIdx.x >> 5);
  if (r >= R) return;
  const long long n_r = blk_off[r + 1] - blk_off[r];

  long long top = LLONG_MIN;
  int arg = AIBX_NO_POD;
#pragma unroll
  for (int half = 0; half < 2; ++half) {
    const int p = lane + 32 * half;
    if (p < P) {
      const long long hit = (long long)match_len[(int64_t)r * P + p];
      const long long eff = (hit > 0 && 100LL * hit >= (long long)thr_pct * n_r) ? hit : 0LL;
      const long long sc = (long long)w_prefix * eff - (long long)w_load * (long long)pod_load[p];
      if (scores) scores[(int64_t)r * P + p] = sc;
      // ascending p within a lane: strict ">" keeps the lower pod on ties
      if (((ready_mask >> p) & 1ULL) && (arg == AIBX_NO_POD || sc > top)) {
        top = sc;
        arg = p;
      }
    }
  }
  // warp argmax; among equal scores the lower pod index wins; "no pod" loses to any pod
#pragma unroll
  for (int d = 16; d >= 1; d >>= 1) {
    const long long o_top = __shfl_xor_sync(0xffffffffu, top, d);
    const int o_arg = __shfl_xor_sync(0xffffffffu, arg, d);
    const bool take = (o_arg != AIBX_NO_POD) &&
                      (arg == AIBX_NO_POD || o_top > top || (o_top == top && o_arg < arg));
    if (take) {
      top = o_top;
      arg = o_arg;
    }
  }
  if (lane == 0) {
    best_pod[r] = arg;
    best_score[r] = top;
  }
}

}  // namespace aibx
