// GPU-resident residency index: open addressing with linear probing over 32-byte slots, so
// that one probe touches exactly one DRAM sector holding key, pod mask and block id.
//
//   insert / evict : one thread per item, atomics only (results are order-free by construction)
//   lookup         : one thread per key
//   match_prefix   : a warp probes 32 consecutive blocks of a request at once; a ballot finds
//                    the first total miss and a prefix-AND over the lanes finds, per pod, the
//                    first block that lacks it; warps of one request combine through
//                    shared-memory minima and stop once an earlier total miss is known.
#pragma once

#include "aibx_common.cuh"
#include "route_score.cuh"

namespace aibx {

struct __align__(32) Slot {
  unsigned long long key;    // 0 = never used, ~0 = removed (reusable by insert)
  unsigned long long mask;   // pod residency bits; an entry with mask 0 is dead
  unsigned int id;           // block id, min over inserts; AIBX_NO_BLOCK = none supplied
  unsigned int stamp;        // reserved (recency stamp for eviction policies)
  unsigned long long pad;
};
static_assert(sizeof(Slot) == 32, "one slot per 32-byte sector");

struct IndexView {
  Slot* slots;
  unsigned long long cap_mask;   // capacity - 1
  int shift;                     // 64 - log2(capacity)
  int num_pods;
  unsigned long long* counters;  // [0] live entries, [1] removed slots
};

__device__ __forceinline__ unsigned long long home_slot(const IndexView& ix, uint64_t key) {
  return (key * 0x9E3779B97F4A7C15ULL) >> ix.shift;
}

// One 32-byte slot in one request: a 256-bit read-only load (slots are 32-byte aligned).
__device__ __forceinline__ void load_slot(const Slot* p, unsigned long long& k,
                                          unsigned long long& m, unsigned int& id) {
  unsigned long long w2;
  [[maybe_unused]] unsigned long long w3;       // stamp and padding: not needed by a probe
  asm volatile("ld.global.nc.v4.u64 {%0,%1,%2,%3}, [%4];"
               : "=l"(k), "=l"(m), "=l"(w2), "=l"(w3)
               : "l"(p));
  id = (unsigned int)w2;
}

// The same load with the third word (block id in its low half, stamp above) left as it arrives:
// no instruction touches the result, so issuing it never waits for the data.
__device__ __forceinline__ void load_slot_raw(const Slot* p, unsigned long long& k,
                                              unsigned long long& m, unsigned long long& id_stamp) {
  [[maybe_unused]] unsigned long long w3;
  asm volatile("ld.global.nc.v4.u64 {%0,%1,%2,%3}, [%4];"
               : "=l"(k), "=l"(m), "=l"(id_stamp), "=l"(w3)
               : "l"(p));
}

__global__ void index_clear_kernel(IndexView ix) {
  const unsigned long long n = ix.cap_mask + 1;
  for (unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; i < n;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    uint4* p = reinterpret_cast<uint4*>(ix.slots + i);
    p[0] = make_uint4(0u, 0u, 0u, 0u);                      // key, mask
    p[1] = make_uint4(AIBX_NO_BLOCK, 0u, 0u, 0u);           // id, stamp, pad
  }
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    ix.counters[0] = 0;
    ix.counters[1] = 0;
  }
}

// Read-only probe (index not modified while the kernel runs): the whole slot arrives with one
// load, so a hit costs one memory round trip.
__device__ __forceinline__ bool probe_ro(const IndexView& ix, uint64_t key, uint64_t& mask,
                                         uint32_t& id) {
  mask = 0;
  id = AIBX_NO_BLOCK;
  if (key_reserved(key)) return false;
  unsigned long long s = home_slot(ix, key);
  for (unsigned long long n = 0; n <= ix.cap_mask; ++n) {
    unsigned long long k, m;
    unsigned int sid;
    load_slot(ix.slots + s, k, m, sid);
    if (k == key) {
      if (m == 0) return false;
      mask = m;
      id = sid;
      return true;
    }
    if (k == kKeyEmpty) return false;
    s = (s + 1) & ix.cap_mask;
  }
  return false;
}

// Keys of kWalk consecutive slots of a probe run, requested together (they usually share one
// 128-byte line): a walk advances kWalk slots per memory round trip.  Volatile: other threads
// may be claiming slots meanwhile.
constexpr int kWalk = 2;
__device__ __forceinline__ void load_keys(const IndexView& ix, unsigned long long s,
                                           unsigned long long (&k)[kWalk]) {
#pragma unroll
  for (int j = 0; j < kWalk; ++j)
    k[j] = *reinterpret_cast<volatile unsigned long long*>(&ix.slots[(s + j) & ix.cap_mask].key);
}

// Probe while other threads may be claiming slots: returns the slot index or ~0.
__device__ __forceinline__ unsigned long long find_slot_rw(const IndexView& ix, uint64_t key) {
  unsigned long long s = home_slot(ix, key);
  for (unsigned long long n = 0; n <= ix.cap_mask; n += kWalk) {
    unsigned long long k[kWalk];
    load_keys(ix, s, k);
#pragma unroll
    for (int j = 0; j < kWalk; ++j) {
      if (k[j] == key) return (s + j) & ix.cap_mask;
      if (k[j] == kKeyEmpty) return ~0ULL;
    }
    s = (s + kWalk) & ix.cap_mask;
  }
  return ~0ULL;
}

// Insert or update one entry (mask already restricted to the table's pods, key not reserved).
// Returns the slot, or ~0 when the table is full.
//
// One walk from the home slot to the first never-used slot: an existing entry anywhere on the
// way wins; otherwise the first never-used or removed slot seen on the way is claimed.  An entry
// may lie BEHIND a removed slot (it was placed when that slot was taken), hence the walk to the
// end before claiming.  Every thread inserting this key walks the same path and tries the same
// slots in the same order, and no slot turns reusable while inserts run, so the loser of a race
// for a slot either finds the key there (another thread of the same key won) or starts over
// and finds the key, or the next free slot, further on.
// `added` / `reused` are raised when a slot was claimed / when that slot was a removed one: the
// caller folds them into the table's counters once per CTA (one atomic per thread on the same
// two words would serialise the whole kernel behind them).
__device__ __forceinline__ unsigned long long insert_entry(const IndexView& ix, uint64_t key,
                                                           uint64_t m, uint32_t id,
                                                           unsigned int& added,
                                                           unsigned int& reused) {
  unsigned long long slot = ~0ULL;
  // a lost race costs one more walk; each one means some slot was taken, so the table bounds them
  for (unsigned long long attempts = 0; attempts <= ix.cap_mask && slot == ~0ULL; ++attempts) {
    unsigned long long s = home_slot(ix, key);
    unsigned long long free_slot = ~0ULL, free_was = kKeyEmpty;
    bool at_end = false;
    for (unsigned long long n = 0; n <= ix.cap_mask && slot == ~0ULL && !at_end; n += kWalk) {
      unsigned long long k[kWalk];
      load_keys(ix, s, k);
#pragma unroll
      for (int j = 0; j < kWalk; ++j) {
        if (slot != ~0ULL || at_end) continue;
        const unsigned long long here = (s + j) & ix.cap_mask;
        if (k[j] == key) {
          slot = here;
        } else if (k[j] == kKeyEmpty || k[j] == kKeyTomb) {
          if (free_slot == ~0ULL) {
            free_slot = here;
            free_was = k[j];
          }
          at_end = k[j] == kKeyEmpty;
        }
      }
      s = (s + kWalk) & ix.cap_mask;
    }
    if (slot != ~0ULL) break;
    if (free_slot == ~0ULL) break;                      // no room anywhere on the path
    const unsigned long long seen =
        atomicCAS(&ix.slots[free_slot].key, free_was, (unsigned long long)key);
    if (seen == free_was) {
      added += 1u;
      if (free_was == kKeyTomb) reused += 1u;
      slot = free_slot;
    } else if (seen == key) {
      slot = free_slot;
    }
  }
  if (slot == ~0ULL) {
    raise_status(AIBX_ERR_FULL);
    return ~0ULL;
  }
  atomicOr(&ix.slots[slot].mask, (unsigned long long)m);
  atomicMin(&ix.slots[slot].id, id);
  return slot;
}

// live += added - removed, freed-slot count += removed - reused: summed over the CTA in shared
// memory, then one pair of atomics per CTA.  Every thread of the CTA must call it.
__device__ __forceinline__ void fold_counters(const IndexView& ix, unsigned int added,
                                              unsigned int reused, unsigned int removed) {
  __shared__ unsigned int s_cnt[3];
  if (threadIdx.x < 3) s_cnt[threadIdx.x] = 0u;
  __syncthreads();
  const unsigned int a = __reduce_add_sync(0xffffffffu, added);
  const unsigned int u = __reduce_add_sync(0xffffffffu, reused);
  const unsigned int d = __reduce_add_sync(0xffffffffu, removed);
  if ((threadIdx.x & 31) == 0 && (a | u | d)) {
    if (a) atomicAdd(&s_cnt[0], a);
    if (u) atomicAdd(&s_cnt[1], u);
    if (d) atomicAdd(&s_cnt[2], d);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned long long live = (unsigned long long)s_cnt[0] - (unsigned long long)s_cnt[2];
    const unsigned long long tomb = (unsigned long long)s_cnt[2] - (unsigned long long)s_cnt[1];
    if (live) atomicAdd(&ix.counters[0], live);       // two's complement: may be a decrease
    if (tomb) atomicAdd(&ix.counters[1], tomb);
  }
}

__global__ void index_insert_kernel(IndexView ix, const uint64_t* __restrict__ keys,
                                    const uint64_t* __restrict__ masks,
                                    const uint32_t* __restrict__ ids, int64_t n) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  unsigned int added = 0, reused = 0;
  if (i < n) {
    const uint64_t key = keys[i];
    const uint64_t m = masks[i] & pod_all(ix.num_pods);
    if (!key_reserved(key) && m != 0) insert_entry(ix, key, m, ids[i], added, reused);
  }
  fold_counters(ix, added, reused, 0u);
}

// Live entries of the table, in no particular order; *count ends as their number (entries
// beyond max_entries are counted but not written).  Room is reserved once per CTA and turn of
// the loop (warp ballots, a sum over the warps in shared memory, one atomic): one atomic per
// warp on the single counter was what bounded the kernel.
__global__ void index_export_kernel(IndexView ix, uint64_t* __restrict__ keys,
                                    uint64_t* __restrict__ masks, uint32_t* __restrict__ ids,
                                    unsigned long long max_entries,
                                    unsigned long long* __restrict__ count) {
  __shared__ unsigned int s_warp[32];
  __shared__ unsigned long long s_base;
  const unsigned long long n = ix.cap_mask + 1;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int n_warps = blockDim.x >> 5;
  for (unsigned long long cta0 = blockIdx.x * (unsigned long long)blockDim.x; cta0 < n;
       cta0 += (unsigned long long)gridDim.x * blockDim.x) {
    const unsigned long long i = cta0 + threadIdx.x;
    unsigned long long k = 0, m = 0;
    unsigned int id = AIBX_NO_BLOCK;
    if (i < n) {
      const uint4* p = reinterpret_cast<const uint4*>(ix.slots + i);
      const uint4 a = __ldg(p);
      const uint4 b = __ldg(p + 1);
      k = (unsigned long long)a.x | ((unsigned long long)a.y << 32);
      m = (unsigned long long)a.z | ((unsigned long long)a.w << 32);
      id = b.x;
    }
    const bool live = i < n && !key_reserved(k) && m != 0;
    const unsigned int votes = __ballot_sync(0xffffffffu, live);
    if (lane == 0) s_warp[warp] = __popc(votes);
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned int total = 0;
      for (int w = 0; w < n_warps; ++w) {
        const unsigned int c = s_warp[w];
        s_warp[w] = total;                               // exclusive prefix over the warps
        total += c;
      }
      s_base = total ? atomicAdd(count, (unsigned long long)total) : 0ULL;
    }
    __syncthreads();
    if (live) {
      const unsigned long long pos = s_base + s_warp[warp] + __popc(votes & ((1u << lane) - 1u));
      if (pos < max_entries) {
        if (keys) keys[pos] = k;
        if (masks) masks[pos] = m;
        if (ids) ids[pos] = id;
      }
    }
    __syncthreads();                                     // s_warp / s_base are reused next turn
  }
}

// Carry every live entry of one table over into another (larger or smaller) one.
__global__ void index_move_kernel(IndexView from, IndexView to) {
  const unsigned long long n = from.cap_mask + 1;
  unsigned int added = 0, reused = 0;
  for (unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; i < n;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    const uint4* p = reinterpret_cast<const uint4*>(from.slots + i);
    const uint4 a = __ldg(p);
    const uint4 b = __ldg(p + 1);
    const unsigned long long k = (unsigned long long)a.x | ((unsigned long long)a.y << 32);
    const unsigned long long m = (unsigned long long)a.z | ((unsigned long long)a.w << 32);
    if (!key_reserved(k) && m != 0) {
      const unsigned long long s = insert_entry(to, k, m, b.x, added, reused);
      if (s != ~0ULL) to.slots[s].stamp = b.y;          // the touch history moves along
    }
  }
  fold_counters(to, added, reused, 0u);
}

// evict, pass 1: clear the named pod bits
__global__ void index_evict_clear_kernel(IndexView ix, const uint64_t* __restrict__ keys,
                                         const uint64_t* __restrict__ masks, int64_t n) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint64_t key = keys[i];
  if (key_reserved(key)) return;
  const unsigned long long s = find_slot_rw(ix, key);
  if (s == ~0ULL) return;
  atomicAnd(&ix.slots[s].mask, ~(unsigned long long)masks[i]);
}

// evict, pass 2: report ids of entries left without a pod (every duplicate sees the same state)
__global__ void index_evict_report_kernel(IndexView ix, const uint64_t* __restrict__ keys,
                                          uint32_t* __restrict__ freed, int64_t n) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint64_t key = keys[i];
  uint32_t out = AIBX_NO_BLOCK;
  if (!key_reserved(key)) {
    const unsigned long long s = find_slot_rw(ix, key);
    if (s != ~0ULL) {
      const unsigned long long m = *reinterpret_cast<volatile unsigned long long*>(&ix.slots[s].mask);
      if (m == 0) out = *reinterpret_cast<volatile unsigned int*>(&ix.slots[s].id);
    }
  }
  freed[i] = out;
}

// evict, pass 3: dead entries leave the table (exactly one thread wins the removal)
__global__ void index_evict_remove_kernel(IndexView ix, const uint64_t* __restrict__ keys,
                                          int64_t n) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  unsigned int removed = 0;
  const uint64_t key = i < n ? keys[i] : kKeyEmpty;
  if (!key_reserved(key)) {
    const unsigned long long s = find_slot_rw(ix, key);
    if (s != ~0ULL &&
        *reinterpret_cast<volatile unsigned long long*>(&ix.slots[s].mask) == 0 &&
        atomicCAS(&ix.slots[s].key, (unsigned long long)key, kKeyTomb) == key) {
      ix.slots[s].id = AIBX_NO_BLOCK;      // ready for reuse by a later insert
      ix.slots[s].stamp = 0u;
      removed = 1u;
    }
  }
  fold_counters(ix, 0u, 0u, removed);     // live -= removed, freed slots += removed
}

__global__ void index_lookup_kernel(IndexView ix, const uint64_t* __restrict__ keys,
                                    uint64_t* __restrict__ out_masks,
                                    uint32_t* __restrict__ out_ids, int64_t n) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint64_t m;
  uint32_t id;
  probe_ro(ix, keys[i], m, id);
  if (out_masks) out_masks[i] = m;
  if (out_ids) out_ids[i] = id;
}

// ------------------------------------------------------------------------------------------
// Longest cached prefix, folded chunk by chunk by ONE warp that walks a request in order.
// State between chunks: the pods that hold every block so far, how many blocks are folded, and
// whether a block without any live entry has ended the request.

struct PrefixFold {
  uint64_t alive;
  unsigned int pos;
  bool ended;
};

// One chunk: lane t holds the probe result (mask, id) of block pos + t, valid for t < m.  A
// ballot finds the first block with no live entry; a prefix-AND over the lanes, seeded with
// `alive`, makes pod bits monotone, so each lane sees exactly the pods that drop out at its
// block and records them in ml[pod] (each pod at most once over the whole request).  The pods
// still there at the first total miss, or at the end of the request, are NOT recorded here:
// they all get the same value (any_len, or the request's length) from fold_finish, in parallel.
__device__ __forceinline__ void fold_chunk(PrefixFold& st, int lane, unsigned int m, uint64_t mask,
                                           uint32_t id, uint64_t all, unsigned int* ml,
                                           uint32_t* block_ids_at) {
  const bool valid = (unsigned int)lane < m;
  const unsigned int none = __ballot_sync(0xffffffffu, valid && mask == 0);
  const unsigned int f = none ? (unsigned int)__ffs(none) - 1u : 32u;   // first total miss
  uint64_t pref = valid ? mask : all;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint64_t o = shfl_up64(pref, d);
    if (lane >= d) pref &= o;
  }
  pref &= st.alive;
  const uint64_t prev = shfl_up64(pref, 1);
  const uint64_t before = lane == 0 ? st.alive : prev;
  uint64_t drops = valid ? (before & ~pref) : 0ULL;
  if ((unsigned int)lane == f) drops = 0;
  while (drops) {
    const int q = __ffsll((long long)drops) - 1;
    drops &= drops - 1;
    ml[q] = st.pos + lane;
  }
  if (valid && block_ids_at)
    block_ids_at[st.pos + lane] = (unsigned int)lane < f ? id : AIBX_NO_BLOCK;
  if (f < 32u) {
    st.ended = true;                                   // any_len = pos + f
    st.alive = shfl64(0xffffffffu, before, (int)f);    // the pods that held every block before it
    st.pos += f;
  } else {
    st.alive = shfl64(0xffffffffu, pref, (int)m - 1);
    st.pos += m;
  }
}

// After the last chunk: the pods that never dropped out, the results, the score.  `ml` is the
// warp's scratch of AIBX_MAX_PODS words (shared memory); lanes cover pods lane and lane + 32.
__device__ __forceinline__ void fold_finish(const PrefixFold& st, int lane, int P, int r,
                                            unsigned int n_r, int64_t off, unsigned int* ml,
                                            uint32_t* __restrict__ match_len,
                                            uint32_t* __restrict__ any_len,
                                            uint32_t* __restrict__ block_ids, const ScoreParams& sp,
                                            int32_t* __restrict__ best_pod,
                                            int64_t* __restrict__ best_score) {
  __syncwarp();
  const unsigned int full = st.ended ? st.pos : n_r;
  if (lane < P && ((st.alive >> lane) & 1ULL)) ml[lane] = full;
  if (lane + 32 < P && ((st.alive >> (lane + 32)) & 1ULL)) ml[lane + 32] = full;
  __syncwarp();
  const long long h0 = lane < P ? (long long)ml[lane] : 0;
  const long long h1 = lane + 32 < P ? (long long)ml[lane + 32] : 0;
  if (lane < P) match_len[(int64_t)r * P + lane] = (uint32_t)h0;
  if (lane + 32 < P) match_len[(int64_t)r * P + lane + 32] = (uint32_t)h1;
  if (lane == 0 && any_len) any_len[r] = st.pos;
  if (block_ids) {
    for (unsigned int i = st.pos + lane; i < n_r; i += 32) block_ids[off + i] = AIBX_NO_BLOCK;
  }
  if (best_pod) {
    const long long l0 = lane < P ? (long long)sp.pod_load[lane] : 0;
    const long long l1 = lane + 32 < P ? (long long)sp.pod_load[lane + 32] : 0;
    long long top;
    int arg;
    lane_candidate(lane, P, sp.ready_mask,
                   pod_score(h0, (long long)n_r, l0, sp.w_prefix, sp.w_load, sp.thr_pct),
                   pod_score(h1, (long long)n_r, l1, sp.w_prefix, sp.w_load, sp.thr_pct), top, arg);
    warp_argmax(top, arg);
    if (lane == 0) {
      best_pod[r] = arg;
      best_score[r] = top;
    }
  }
}

// One warp per request, chunks of 32 blocks in order: the shape for large batches, where there
// are warps enough without splitting a request.  No barrier, no shared-memory atomics.
constexpr int kMatchWarpKernelWarps = 4;

__global__ void __launch_bounds__(kMatchWarpKernelWarps * 32, 16)
match_prefix_warp_kernel(IndexView ix, const uint64_t* __restrict__ hashes,
                         const int64_t* __restrict__ blk_off, int R,
                         uint32_t* __restrict__ match_len, uint32_t* __restrict__ any_len,
                         uint32_t* __restrict__ block_ids, ScoreParams sp,
                         int32_t* __restrict__ best_pod, int64_t* __restrict__ best_score) {
  __shared__ unsigned int s_ml[kMatchWarpKernelWarps][AIBX_MAX_PODS];
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int r = blockIdx.x * kMatchWarpKernelWarps + warp;
  if (r >= R) return;
  const int P = ix.num_pods;
  const uint64_t all = pod_all(P);
  const int64_t off = blk_off[r];
  const unsigned int n_r = (unsigned int)(blk_off[r + 1] - off);
  PrefixFold st = {all, 0u, false};
  // the keys of the next chunk are requested before this chunk is probed: if the request goes
  // on, they are there by then (one memory round trip less per further chunk)
  uint64_t key = (unsigned int)lane < n_r ? __ldg(hashes + off + lane) : 0ULL;
  while (!st.ended && st.pos < n_r) {
    const unsigned int m = min(32u, n_r - st.pos);
    const unsigned int nxt = st.pos + 32u + (unsigned int)lane;
    const uint64_t key_next = nxt < n_r ? __ldg(hashes + off + nxt) : 0ULL;
    uint64_t mask = 0;
    uint32_t id = AIBX_NO_BLOCK;
    if ((unsigned int)lane < m) probe_ro(ix, key, mask, id);
    fold_chunk(st, lane, m, mask, id, all, s_ml[warp], block_ids ? block_ids + off : nullptr);
    key = key_next;
  }
  fold_finish(st, lane, P, r, n_r, off, s_ml[warp], match_len, any_len, block_ids, sp, best_pod,
              best_score);
}

// ------------------------------------------------------------------------------------------
// Longest cached prefix.  A group of `wpr` warps serves one request; a CTA holds kMatchWarps
// warps, i.e. kMatchWarps / wpr requests.

constexpr int kMatchWarpsMin = 4;

struct MatchShared {
  unsigned int first_miss[AIBX_MAX_PODS];   // per pod: first block whose mask lacks the pod
  unsigned int first_none;                  // first block with no entry at all
};

__global__ void match_prefix_kernel(IndexView ix, const uint64_t* __restrict__ hashes,
                                    const int64_t* __restrict__ blk_off, int R, int wpr,
                                    uint32_t* __restrict__ match_len,
                                    uint32_t* __restrict__ any_len,
                                    uint32_t* __restrict__ block_ids, ScoreParams sp,
                                    int32_t* __restrict__ best_pod,
                                    int64_t* __restrict__ best_score) {
  extern __shared__ MatchShared s_groups[];
  const int warps_per_cta = blockDim.x >> 5;
  const int groups_per_cta = warps_per_cta / wpr;
  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int group = warp / wpr;
  const int warp_in_group = warp % wpr;
  const int tid_in_group = warp_in_group * 32 + lane;
  const int group_threads = wpr * 32;
  const int P = ix.num_pods;
  const int r = blockIdx.x * groups_per_cta + group;
  const bool active = r < R;

  MatchShared& sh = s_groups[group];
  int64_t off = 0;
  unsigned int n_r = 0;
  if (active) {
    off = blk_off[r];
    n_r = (unsigned int)(blk_off[r + 1] - off);
    for (int p = tid_in_group; p < P; p += group_threads) sh.first_miss[p] = n_r;
    if (tid_in_group == 0) sh.first_none = n_r;
  }
  __syncthreads();

  if (active) {
    const uint64_t all = pod_all(P);
    for (unsigned int base = warp_in_group * 32u; base < n_r; base += wpr * 32u) {
      // blocks past a known total miss cannot change any result
      unsigned int known = 0;
      if (lane == 0) known = *reinterpret_cast<volatile unsigned int*>(&sh.first_none);
      known = __shfl_sync(0xffffffffu, known, 0);
      if (base > known) break;
      const unsigned int i = base + lane;
      const bool valid = i < n_r;
      uint64_t mask = 0;
      uint32_t id = AIBX_NO_BLOCK;
      if (valid) probe_ro(ix, __ldg(hashes + off + i), mask, id);
      if (valid && block_ids) block_ids[off + i] = id;
      const unsigned int none = __ballot_sync(0xffffffffu, valid && mask == 0);
      if (none && lane == 0) atomicMin(&sh.first_none, base + (unsigned int)__ffs(none) - 1u);
      // Per pod, the first block whose mask lacks it.  A prefix-AND over the lanes makes pod
      // bits monotone (set up to the first lacking block), so the pods that drop out exactly at
      // this lane are the bits its predecessor's prefix still had and its own has lost: every
      // pod is reported once, by one lane, instead of one ballot per pod.
      uint64_t pref = valid ? mask : all;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const unsigned int tlo = __shfl_up_sync(0xffffffffu, (unsigned int)pref, d);
        const unsigned int thi = __shfl_up_sync(0xffffffffu, (unsigned int)(pref >> 32), d);
        if (lane >= d) pref &= (uint64_t)tlo | ((uint64_t)thi << 32);
      }
      // pods already known to drop out BEFORE this chunk are not looked at again (a drop
      // recorded by a warp working on a later chunk must not hide an earlier one)
      const volatile unsigned int* fm = sh.first_miss;
      const unsigned int g_lo = __ballot_sync(0xffffffffu, lane < P && fm[lane] < base);
      const unsigned int g_hi =
          __ballot_sync(0xffffffffu, lane + 32 < P && fm[(lane + 32) & 63] < base);
      const uint64_t gone = (uint64_t)g_lo | ((uint64_t)g_hi << 32);
      const unsigned int plo = __shfl_up_sync(0xffffffffu, (unsigned int)pref, 1);
      const unsigned int phi = __shfl_up_sync(0xffffffffu, (unsigned int)(pref >> 32), 1);
      const uint64_t before = lane == 0 ? (all & ~gone) : ((uint64_t)plo | ((uint64_t)phi << 32));
      uint64_t drops = before & ~pref & all;
      // At the chunk's first block with no entry at all every pod still there drops out at
      // once: those are not recorded one by one (up to 64 atomics in one lane) - the result is
      // taken as min(first_miss, first_none) at the end instead.
      if (none && lane == __ffs(none) - 1) drops = 0;
      while (drops) {
        const int p = __ffsll((long long)drops) - 1;
        drops &= drops - 1;
        atomicMin(&sh.first_miss[p], i);
      }
    }
  }
  __syncthreads();

  if (active) {
    const unsigned int a = sh.first_none;
    for (int p = tid_in_group; p < P; p += group_threads)
      match_len[(int64_t)r * P + p] = min(sh.first_miss[p], a);
    if (any_len && tid_in_group == 0) any_len[r] = a;
    if (best_pod && warp_in_group == 0) {
      // fused scoring: the request's match lengths are still in shared memory
      const long long h0 = lane < P ? (long long)min(sh.first_miss[lane], a) : 0;
      const long long h1 = lane + 32 < P ? (long long)min(sh.first_miss[lane + 32], a) : 0;
      const long long l0 = lane < P ? (long long)sp.pod_load[lane] : 0;
      const long long l1 = lane + 32 < P ? (long long)sp.pod_load[lane + 32] : 0;
      long long top;
      int arg;
      lane_candidate(lane, P, sp.ready_mask,
                     pod_score(h0, (long long)n_r, l0, sp.w_prefix, sp.w_load, sp.thr_pct),
                     pod_score(h1, (long long)n_r, l1, sp.w_prefix, sp.w_load, sp.thr_pct), top, arg);
      warp_argmax(top, arg);
      if (lane == 0) {
        best_pod[r] = arg;
        best_score[r] = top;
      }
    }
    if (block_ids) {
      for (unsigned int i = a + tid_in_group; i < n_r; i += group_threads)
        block_ids[off + i] = AIBX_NO_BLOCK;
    }
  }
}

}  // namespace aibx
