// GPU-resident residency index: open addressing with linear probing over 32-byte SECTORS, in
// two entry widths.
//
// What the memory system gives a random probe was measured on B200 before this layout was
// chosen.  (1) An L2 miss always brings a whole 128-byte line from DRAM, whatever the load asked
// for, so the smaller the table, the more of it stays in L2 and the fewer lines a lookup costs.
// (2) Inside an SM the limit is the L1 data stage: a load whose 32 lanes go to 32 different lines
// costs 32 passes, so a lookup should be ONE 32-byte load, not two.  Hence:
//   narrow (tables of up to 32 pods): a sector holds TWO entries, {key0, key1, mask0|id0<<32,
//       mask1|id1<<32}: 16 bytes per slot of capacity, and at a load of one half nine lookups in
//       ten end with the first load;
//   wide (33 to 64 pods): a sector holds ONE entry, {key, mask, id, unused}.
// The eviction stamps, which only the touch and victim kernels need, live in a side array.
//
//   insert / evict : one thread per item, atomics only (results are order-free by construction)
//   lookup         : one thread per key
//   match_prefix   : a warp probes 32 consecutive blocks of a request at once; a ballot finds
//                    the first total miss and a prefix-AND over the lanes finds, per pod, the
//                    first block that lacks it; warps of one request combine through
//                    shared-memory minima and stop once an earlier total miss is known.
#pragma once

#include <cooperative_groups.h>

#include "aibx_common.cuh"
#include "route_score.cuh"

namespace aibx {

constexpr unsigned int kMaxWalkEntries = 4096;   // entries a probe sequence may pass

// Entry e of the table is position e % per_sector of sector e / per_sector.
struct IndexView {
  unsigned long long* words;     // nb sectors of four 64-bit words
  unsigned int* stamps;          // one recency stamp per entry (eviction policy)
  unsigned long long nb;         // sectors: capacity / 2 (narrow) or capacity (wide)
  unsigned long long capacity;   // live entries the table accepts (FULL beyond)
  unsigned int max_walk;         // sectors a probe may visit: no entry lies further from home
  int num_pods;
  int narrow;                    // 1: two 16-byte entries per sector, 0: one 32-byte entry
  unsigned long long* counters;  // [0] live entries, [1] removed entries, [2] longest insert walk
};

__device__ __forceinline__ int per_sector(const IndexView& ix) { return ix.narrow ? 2 : 1; }

__device__ __forceinline__ unsigned long long num_entries(const IndexView& ix) {
  return ix.narrow ? ix.nb * 2 : ix.nb;
}

// Multiply-shift range reduction: any sector count, no division.
__device__ __forceinline__ unsigned long long home_sector(const IndexView& ix, uint64_t key) {
  return __umul64hi(key * 0x9E3779B97F4A7C15ULL, ix.nb);
}

__device__ __forceinline__ unsigned long long next_sector(const IndexView& ix,
                                                          unsigned long long s) {
  return s + 1 == ix.nb ? 0ULL : s + 1;
}

// One whole sector in one 256-bit read-only load (the table is not modified meanwhile).
__device__ __forceinline__ void load_sector(const unsigned long long* p, unsigned long long& w0,
                                            unsigned long long& w1, unsigned long long& w2,
                                            unsigned long long& w3) {
  asm volatile("ld.global.nc.v4.u64 {%0,%1,%2,%3}, [%4];"
               : "=l"(w0), "=l"(w1), "=l"(w2), "=l"(w3)
               : "l"(p));
}

constexpr unsigned long long kNarrowEmptyValue = 0xFFFFFFFF00000000ULL;   // mask 0, id NO_BLOCK

__global__ void index_clear_kernel(IndexView ix) {
  const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
  const unsigned long long t = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x;
  // 16 bytes per thread and turn: the first half of a sector (keys, or key and mask) is zero,
  // the second half holds the "no id" patterns
  for (unsigned long long i = t; i < ix.nb * 2; i += stride) {
    uint4* p = reinterpret_cast<uint4*>(ix.words) + i;
    if ((i & 1) == 0) {
      *p = make_uint4(0u, 0u, 0u, 0u);
    } else if (ix.narrow) {
      *p = make_uint4(0u, AIBX_NO_BLOCK, 0u, AIBX_NO_BLOCK);
    } else {
      *p = make_uint4(AIBX_NO_BLOCK, 0u, 0u, 0u);
    }
  }
  for (unsigned long long i = t; i < num_entries(ix); i += stride) ix.stamps[i] = 0u;
  if (t < 3) ix.counters[t] = 0;
}

// Read-only probe: a hit in the home sector costs one memory round trip.  A sector with a
// never-used entry ends the walk: no key was ever placed beyond it.  `entry` receives the
// entry's index (for its stamp) on a hit.
template <bool NARROW>
__device__ __forceinline__ bool probe_ro_w(const IndexView& ix, uint64_t key, uint64_t& mask,
                                           uint32_t& id, unsigned long long& entry) {
  mask = 0;
  id = AIBX_NO_BLOCK;
  entry = ~0ULL;
  if (key_reserved(key)) return false;
  unsigned long long s = home_sector(ix, key);
  for (unsigned int n = 0; n < ix.max_walk; ++n) {
    unsigned long long w0, w1, w2, w3;
    load_sector(ix.words + 4 * s, w0, w1, w2, w3);
    if (NARROW) {
      unsigned long long v;
      if (w0 == key) {
        v = w2;
        entry = 2 * s;
      } else if (w1 == key) {
        v = w3;
        entry = 2 * s + 1;
      } else {
        if (w0 == kKeyEmpty || w1 == kKeyEmpty) return false;
        s = next_sector(ix, s);
        continue;
      }
      mask = (unsigned int)v;
      id = (unsigned int)(v >> 32);
    } else {
      if (w0 != key) {
        if (w0 == kKeyEmpty) return false;
        s = next_sector(ix, s);
        continue;
      }
      mask = w1;
      id = (unsigned int)w2;
      entry = s;
    }
    if (mask == 0) id = AIBX_NO_BLOCK;
    return mask != 0;
  }
  return false;
}

__device__ __forceinline__ bool probe_ro(const IndexView& ix, uint64_t key, uint64_t& mask,
                                         uint32_t& id, unsigned long long& entry) {
  return ix.narrow ? probe_ro_w<true>(ix, key, mask, id, entry)
                   : probe_ro_w<false>(ix, key, mask, id, entry);
}

__device__ __forceinline__ bool probe_ro(const IndexView& ix, uint64_t key, uint64_t& mask,
                                         uint32_t& id) {
  unsigned long long entry;
  return probe_ro(ix, key, mask, id, entry);
}

// Recency stamp of an entry: bits 0..29 the last epoch in which it was touched (0 = never), bits
// 30..31 the number of distinct epochs it was touched in, saturating at 3.  Several touches of
// one entry in one epoch count once, whoever gets there first.
constexpr unsigned int kEpochMask = (1u << 30) - 1u;

__device__ __forceinline__ void touch_entry(const IndexView& ix, unsigned long long e,
                                            unsigned int epoch) {
  unsigned int* stamp = &ix.stamps[e];
  unsigned int old = *reinterpret_cast<volatile unsigned int*>(stamp);
  for (int tries = 0; tries < 64; ++tries) {
    if ((old & kEpochMask) == epoch) return;
    const unsigned int t = old >> 30;
    const unsigned int fresh = ((t < 3u ? t + 1u : 3u) << 30) | epoch;
    const unsigned int seen = atomicCAS(stamp, old, fresh);
    if (seen == old) return;
    old = seen;
  }
}

// Where the parts of entry e live (both widths).
__device__ __forceinline__ unsigned long long* entry_key(const IndexView& ix, unsigned long long e) {
  return ix.narrow ? ix.words + 4 * (e >> 1) + (e & 1) : ix.words + 4 * e;
}
__device__ __forceinline__ unsigned int* narrow_value(const IndexView& ix, unsigned long long e) {
  return reinterpret_cast<unsigned int*>(ix.words + 4 * (e >> 1) + 2 + (e & 1));   // {mask, id}
}
__device__ __forceinline__ unsigned int* entry_id(const IndexView& ix, unsigned long long e) {
  return ix.narrow ? narrow_value(ix, e) + 1 : reinterpret_cast<unsigned int*>(ix.words + 4 * e + 2);
}
__device__ __forceinline__ unsigned long long entry_mask_now(const IndexView& ix,
                                                             unsigned long long e) {
  if (ix.narrow) return *reinterpret_cast<volatile unsigned int*>(narrow_value(ix, e));
  return *reinterpret_cast<volatile unsigned long long*>(ix.words + 4 * e + 1);
}
__device__ __forceinline__ void entry_mask_or(const IndexView& ix, unsigned long long e,
                                              unsigned long long m) {
  if (ix.narrow) atomicOr(narrow_value(ix, e), (unsigned int)m);
  else atomicOr(ix.words + 4 * e + 1, m);
}
__device__ __forceinline__ void entry_mask_clear(const IndexView& ix, unsigned long long e,
                                                 unsigned long long bits) {
  if (ix.narrow) atomicAnd(narrow_value(ix, e), ~(unsigned int)bits);
  else atomicAnd(ix.words + 4 * e + 1, ~bits);
}

// The keys of a sector while other threads may be claiming entries (k[1] only when narrow).
__device__ __forceinline__ void load_keys(const IndexView& ix, unsigned long long s,
                                          unsigned long long (&k)[2]) {
  const volatile unsigned long long* p = ix.words + 4 * s;
  k[0] = p[0];
  k[1] = ix.narrow ? p[1] : 1ULL;      // wide: a value that is neither a key's match nor free
}

// Probe while other threads may be claiming entries: returns the entry index or ~0.
__device__ __forceinline__ unsigned long long find_entry_rw(const IndexView& ix, uint64_t key) {
  const int E = per_sector(ix);
  unsigned long long s = home_sector(ix, key);
  for (unsigned int n = 0; n < ix.max_walk; ++n) {
    unsigned long long k[2];
    load_keys(ix, s, k);
    for (int j = 0; j < E; ++j) {
      if (k[j] == key) return s * E + j;
      if (k[j] == kKeyEmpty) return ~0ULL;
    }
    s = next_sector(ix, s);
  }
  return ~0ULL;
}

// Insert or update one entry (mask already restricted to the table's pods, key not reserved).
// Returns the entry, or ~0 when no room is left within max_walk sectors of the key's home.
//
// One walk from the home sector to the first sector with a never-used entry: an existing entry
// anywhere on the way wins; otherwise the first never-used or removed entry seen on the way is
// claimed.  An entry may lie BEHIND a removed one (it was placed when that one was taken), hence
// the walk to the end before claiming.  Every thread inserting this key walks the same path and
// tries the same entries in the same order, and no entry turns reusable while inserts run, so
// the loser of a race for an entry either finds the key there (another thread of the same key
// won) or starts over and finds the key, or the next free entry, further on.  Inside a sector
// a never-used entry is always the last one, which is what lets a reader stop at the first
// sector that has one.
// `added` / `reused` are raised when an entry was claimed / when it was a removed one, `walked`
// is the number of sectors visited: the caller folds them into the table's counters once per
// CTA (one atomic per thread on the same words would serialise the whole kernel behind them).
__device__ __forceinline__ unsigned long long insert_entry(const IndexView& ix, uint64_t key,
                                                           uint64_t m, uint32_t id,
                                                           unsigned int& added, unsigned int& reused,
                                                           unsigned int& walked) {
  const int E = per_sector(ix);
  unsigned long long entry = ~0ULL;
  const unsigned int max_attempts = ix.max_walk * 2u + 1u;   // each lost race fills one entry
  for (unsigned int attempts = 0; attempts < max_attempts && entry == ~0ULL; ++attempts) {
    unsigned long long s = home_sector(ix, key);
    unsigned long long free_entry = ~0ULL, free_was = kKeyEmpty;
    bool at_end = false;
    unsigned int n = 0;
    for (; n < ix.max_walk && entry == ~0ULL && !at_end; ++n) {
      unsigned long long k[2];
      load_keys(ix, s, k);
      for (int j = 0; j < E; ++j) {
        if (entry != ~0ULL || at_end) continue;
        if (k[j] == key) {
          entry = s * E + j;
        } else if (k[j] == kKeyEmpty || k[j] == kKeyTomb) {
          if (free_entry == ~0ULL) {
            free_entry = s * E + j;
            free_was = k[j];
          }
          at_end = k[j] == kKeyEmpty;
        }
      }
      s = next_sector(ix, s);
    }
    walked = max(walked, n);
    if (entry != ~0ULL) break;
    if (free_entry == ~0ULL) break;                     // no room anywhere on the path
    const unsigned long long seen =
        atomicCAS(entry_key(ix, free_entry), free_was, (unsigned long long)key);
    if (seen == free_was) {
      added += 1u;
      if (free_was == kKeyTomb) reused += 1u;
      entry = free_entry;
    } else if (seen == key) {
      entry = free_entry;
    }
  }
  if (entry == ~0ULL) {
    raise_status(AIBX_ERR_FULL);
    return ~0ULL;
  }
  entry_mask_or(ix, entry, m);
  atomicMin(entry_id(ix, entry), id);
  return entry;
}

// live += added - removed, removed-entry count += removed - reused, longest walk = max: summed
// over the CTA in shared memory, then one atomic each per CTA.  Every thread of the CTA must
// call it.  The CTA whose addition takes the live count past the table's capacity reports FULL
// for the entries beyond it (the count, not the placement, is what keeps the limit exact).
__device__ __forceinline__ void fold_counters(const IndexView& ix, unsigned int added,
                                              unsigned int reused, unsigned int removed,
                                              unsigned int walked) {
  __shared__ unsigned int s_cnt[4];
  if (threadIdx.x < 4) s_cnt[threadIdx.x] = 0u;
  __syncthreads();
  const unsigned int a = __reduce_add_sync(0xffffffffu, added);
  const unsigned int u = __reduce_add_sync(0xffffffffu, reused);
  const unsigned int d = __reduce_add_sync(0xffffffffu, removed);
  const unsigned int w = __reduce_max_sync(0xffffffffu, walked);
  if ((threadIdx.x & 31) == 0 && (a | u | d | w)) {
    if (a) atomicAdd(&s_cnt[0], a);
    if (u) atomicAdd(&s_cnt[1], u);
    if (d) atomicAdd(&s_cnt[2], d);
    if (w) atomicMax(&s_cnt[3], w);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const unsigned long long live = (unsigned long long)s_cnt[0] - (unsigned long long)s_cnt[2];
    const unsigned long long tomb = (unsigned long long)s_cnt[2] - (unsigned long long)s_cnt[1];
    if (live) {
      const unsigned long long before = atomicAdd(&ix.counters[0], live);   // may be a decrease
      if (s_cnt[0] > s_cnt[2] && before + live > ix.capacity) {
        const unsigned long long over = before + live - ix.capacity;
        raise_status_n(AIBX_ERR_FULL, over < live ? over : live);
      }
    }
    if (tomb) atomicAdd(&ix.counters[1], tomb);
    if (s_cnt[3] > 1u) atomicMax(&ix.counters[2], (unsigned long long)s_cnt[3]);
  }
}

__global__ void index_insert_kernel(IndexView ix, const uint64_t* __restrict__ keys,
                                    const uint64_t* __restrict__ masks,
                                    const uint32_t* __restrict__ ids, int64_t n) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  unsigned int added = 0, reused = 0, walked = 0;
  if (i < n) {
    const uint64_t key = keys[i];
    const uint64_t m = masks[i] & pod_all(ix.num_pods);
    if (!key_reserved(key) && m != 0) insert_entry(ix, key, m, ids[i], added, reused, walked);
  }
  fold_counters(ix, added, reused, 0u, walked);
}

// One entry as a scan sees it (entry-parallel kernels: export, move, victim choice).
__device__ __forceinline__ bool load_entry(const IndexView& ix, unsigned long long e, uint64_t& key,
                                           uint64_t& mask, uint32_t& id) {
  if (ix.narrow) {
    const unsigned long long* p = ix.words + 4 * (e >> 1);
    key = __ldg(p + (e & 1));
    const unsigned long long v = __ldg(p + 2 + (e & 1));
    mask = (unsigned int)v;
    id = (unsigned int)(v >> 32);
  } else {
    const unsigned long long* p = ix.words + 4 * e;
    key = __ldg(p);
    mask = __ldg(p + 1);
    id = (unsigned int)__ldg(p + 2);
  }
  return !key_reserved(key) && mask != 0;
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
  const unsigned long long n = num_entries(ix);
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int n_warps = blockDim.x >> 5;
  for (unsigned long long cta0 = blockIdx.x * (unsigned long long)blockDim.x; cta0 < n;
       cta0 += (unsigned long long)gridDim.x * blockDim.x) {
    const unsigned long long i = cta0 + threadIdx.x;
    uint64_t k = 0, m = 0;
    unsigned int id = AIBX_NO_BLOCK;
    const bool live = i < n && load_entry(ix, i, k, m, id);
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
  const unsigned long long n = num_entries(from);
  unsigned int added = 0, reused = 0, walked = 0;
  for (unsigned long long i = blockIdx.x * (unsigned long long)blockDim.x + threadIdx.x; i < n;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    uint64_t k, m;
    uint32_t id;
    if (load_entry(from, i, k, m, id)) {
      const unsigned long long e = insert_entry(to, k, m, id, added, reused, walked);
      if (e != ~0ULL) to.stamps[e] = from.stamps[i];    // the touch history moves along
    }
  }
  fold_counters(to, added, reused, 0u, walked);
}

// evict, pass 1: clear the named pod bits
__global__ void index_evict_clear_kernel(IndexView ix, const uint64_t* __restrict__ keys,
                                         const uint64_t* __restrict__ masks, int64_t n) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint64_t key = keys[i];
  if (key_reserved(key)) return;
  const unsigned long long e = find_entry_rw(ix, key);
  if (e == ~0ULL) return;
  entry_mask_clear(ix, e, masks[i]);
}

// evict, pass 2: report ids of entries left without a pod (every duplicate sees the same state)
__global__ void index_evict_report_kernel(IndexView ix, const uint64_t* __restrict__ keys,
                                          uint32_t* __restrict__ freed, int64_t n) {
  const int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint64_t key = keys[i];
  uint32_t out = AIBX_NO_BLOCK;
  if (!key_reserved(key)) {
    const unsigned long long e = find_entry_rw(ix, key);
    if (e != ~0ULL) {
      if (entry_mask_now(ix, e) == 0) out = *reinterpret_cast<volatile unsigned int*>(entry_id(ix, e));
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
    const unsigned long long e = find_entry_rw(ix, key);
    if (e != ~0ULL &&
        entry_mask_now(ix, e) == 0 &&
        atomicCAS(entry_key(ix, e), (unsigned long long)key, kKeyTomb) == key) {
      *entry_id(ix, e) = AIBX_NO_BLOCK;    // ready for reuse by a later insert
      ix.stamps[e] = 0u;
      removed = 1u;
    }
  }
  fold_counters(ix, 0u, 0u, removed, 0u);   // live -= removed, removed entries += removed
}

// The three passes of evict in ONE cooperative launch: every pass must see the whole batch's
// previous pass finished, which a grid-wide barrier gives without going back to the host (three
// launches cost about 10 us each for a batch that takes 3 us of work).  A thread that has a
// single item keeps the entry it found in pass 1; with more items than threads the later passes
// look their entries up again.  The launch is cooperative, so all CTAs are resident and the
// barrier cannot wait for a CTA that has not started.
__global__ void __launch_bounds__(256)
index_evict_coop_kernel(IndexView ix, const uint64_t* __restrict__ keys,
                        const uint64_t* __restrict__ masks, uint32_t* __restrict__ freed,
                        int64_t n) {
  cooperative_groups::grid_group grid = cooperative_groups::this_grid();
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t t = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
  const bool single = n <= stride;
  unsigned long long mine = ~0ULL;                       // entry of this thread's only item
  for (int64_t i = t; i < n; i += stride) {
    const uint64_t key = keys[i];
    if (key_reserved(key)) continue;
    const unsigned long long e = find_entry_rw(ix, key);
    if (e != ~0ULL) entry_mask_clear(ix, e, masks[i]);
    mine = e;
  }
  grid.sync();
  if (freed) {
    for (int64_t i = t; i < n; i += stride) {
      const uint64_t key = keys[i];
      uint32_t out = AIBX_NO_BLOCK;
      if (!key_reserved(key)) {
        const unsigned long long e = single ? mine : find_entry_rw(ix, key);
        if (e != ~0ULL && entry_mask_now(ix, e) == 0)
          out = *reinterpret_cast<volatile unsigned int*>(entry_id(ix, e));
      }
      freed[i] = out;
    }
    grid.sync();
  }
  unsigned int removed = 0;
  for (int64_t i = t; i < n; i += stride) {
    const uint64_t key = keys[i];
    if (key_reserved(key)) continue;
    // an entry another thread of the same key has already removed no longer carries the key
    const unsigned long long e = single ? mine : find_entry_rw(ix, key);
    if (e != ~0ULL &&
        entry_mask_now(ix, e) == 0 &&
        atomicCAS(entry_key(ix, e), (unsigned long long)key, kKeyTomb) == key) {
      *entry_id(ix, e) = AIBX_NO_BLOCK;
      ix.stamps[e] = 0u;
      removed += 1u;
    }
  }
  fold_counters(ix, 0u, 0u, removed, 0u);
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
// `ml` must be all zeros when the request's first chunk is folded.
__device__ __forceinline__ void fold_chunk(PrefixFold& st, int lane, unsigned int m, uint64_t mask,
                                           uint32_t id, uint64_t all, unsigned int* ml,
                                           uint32_t* block_ids_at) {
  const bool valid = (unsigned int)lane < m;
  // The common chunk changes nothing: every block of it is held by every pod still alive (so
  // none is a total miss either).  One vote instead of the scan below.
  if (st.alive != 0 &&
      __all_sync(0xffffffffu, !valid || (mask & st.alive) == st.alive)) {
    if (valid && block_ids_at) block_ids_at[st.pos + lane] = id;
    st.pos += m;
    return;
  }
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
  // The pods that lack the request's very first block - in a large fleet most of them - would
  // all be recorded by this one lane, one after the other; their length is 0, which is what the
  // caller's scratch starts as.
  if (st.pos == 0u && lane == 0) drops = 0;
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

template <bool NARROW>
__global__ void __launch_bounds__(kMatchWarpKernelWarps * 32, 16)
match_prefix_warp_kernel(IndexView ix, const uint64_t* __restrict__ hashes,
                         const int64_t* __restrict__ blk_off, int R,
                         uint32_t* __restrict__ match_len, uint32_t* __restrict__ any_len,
                         uint32_t* __restrict__ block_ids, ScoreParams sp,
                         int32_t* __restrict__ best_pod, int64_t* __restrict__ best_score,
                         unsigned int epoch) {
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
  s_ml[warp][lane] = 0u;
  s_ml[warp][lane + 32] = 0u;
  __syncwarp();
  // the keys of the next chunk are requested before this chunk is probed: if the request goes
  // on, they are there by then (one memory round trip less per further chunk)
  uint64_t key = (unsigned int)lane < n_r ? __ldg(hashes + off + lane) : 0ULL;
  while (!st.ended && st.pos < n_r) {
    const unsigned int m = min(32u, n_r - st.pos);
    const unsigned int nxt = st.pos + 32u + (unsigned int)lane;
    const uint64_t key_next = nxt < n_r ? __ldg(hashes + off + nxt) : 0ULL;
    uint64_t mask = 0;
    uint32_t id = AIBX_NO_BLOCK;
    unsigned long long entry = ~0ULL;
    if ((unsigned int)lane < m) probe_ro_w<NARROW>(ix, key, mask, id, entry);
    const unsigned int first = st.pos;
    fold_chunk(st, lane, m, mask, id, all, s_ml[warp], block_ids ? block_ids + off : nullptr);
    // the blocks of the matched prefix are marked as used, with the entry the probe just found
    if (epoch && first + (unsigned int)lane < st.pos) touch_entry(ix, entry, epoch);
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
                                    int64_t* __restrict__ best_score, unsigned int epoch) {
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
    if (epoch) {
      // Where the prefix ends is only known now that all warps of the request have met, so the
      // stamps are set in a second walk over the matched blocks; their sectors were read a
      // moment ago and are still in L2.
      for (unsigned int i = tid_in_group; i < a; i += group_threads) {
        uint64_t mask;
        uint32_t id;
        unsigned long long entry;
        if (probe_ro(ix, __ldg(hashes + off + i), mask, id, entry)) touch_entry(ix, entry, epoch);
      }
    }
  }
}

}  // namespace aibx
