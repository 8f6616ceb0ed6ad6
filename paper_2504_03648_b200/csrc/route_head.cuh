// Routing head: prefix keys and longest cached prefix in ONE kernel that stops early.
//
// Matching a request needs its keys only up to the first block that is cached nowhere; in
// shared-prompt traffic that is a small part of the chain (a 2k-token prompt in front of an 8k
// request).  The plain path hashes the whole chain first (serial, ~190 ns per block) and only
// then matches.  Here every request is hashed only until its first total miss is known; what is
// left of the chain - needed later to publish the new blocks, not to route - is hashed by
// hash_blocks_kernel from the saved (blocks done, last key) state, on whatever stream the
// caller likes, e.g. beside the KV copies.
//
// A CTA serves eight requests with nine warps:
//   hasher warp   : four lanes (a quad) per request, the XXH64 chain of hash_blocks.cuh,
//                   untouched on its critical path.  It drops every finished key into a
//                   shared-memory ring and, once per group of 8 stripes, publishes how far it
//                   is and looks at the prober's word (how far that is, and a stop bit), read a
//                   group earlier so that no load is waited for.  It touches no global memory but the tokens
//                   (the probers write the keys out), so that publishing costs no store drain.
//   prober warps  : one per request.  The warp takes whatever new keys its request has in the
//                   ring (up to 32, one per lane), probes the index for them, and folds the
//                   answers in block order exactly like match_prefix_kernel does for a chunk: a
//                   ballot finds the first block without a live entry, a prefix-AND over the
//                   lanes (seeded with the pods still alive) tells every lane which pods drop
//                   out at its block.  The first total miss ends the request and raises the
//                   stop flag; at the end the warp writes the match lengths, the score and the
//                   best pod.
// The probes must not be issued by the hashing warp itself: loads and shuffles share a warp's
// few scoreboards, so every block end would wait for the probe issued just before it (measured:
// 730 ns per block instead of 190).
// Every wait is bounded: the hasher never waits for anything but ring space, a prober gives up
// (AIBX_ERR_TIMEOUT) after a fixed number of empty polls.
#pragma once

#include "aibx_common.cuh"
#include "hash_blocks.cuh"
#include "index.cuh"
#include "route_score.cuh"

namespace aibx {

constexpr int kHeadRing = 64;            // keys per request in the shared-memory ring
constexpr unsigned int kHeadPolls = 1u << 21;   // empty polls (~0.1 us each) before giving up

struct HeadShared {
  unsigned long long ring[8][kHeadRing];
  unsigned int progress[8];              // blocks hashed (keys in the ring), per request
  unsigned int consumed[8];              // blocks the prober is done with | kHeadStopBit
  unsigned int match_len[8][AIBX_MAX_PODS];
};

// Release / acquire on a shared-memory word at CTA scope: the light way to hand data written
// before the store to whoever reads the word (a full fence would also drain unrelated traffic).
__device__ __forceinline__ void st_release_shared(unsigned int* p, unsigned int v) {
  asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned int ld_acquire_shared(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
  return v;
}

// A plain (relaxed) look at a shared-memory word another warp updates; never cached in a register
// by the compiler, yet free to be scheduled among the surrounding loads.
__device__ __forceinline__ unsigned int ld_relaxed_shared(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.relaxed.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)));
  return v;
}

constexpr unsigned int kHeadStopBit = 0x80000000u;     // in `consumed`: no more keys needed

// Polls the prober's word until it has consumed at least `need` blocks or says stop; `c` gets
// the last value seen.  False when the bounded number of polls ran out.
__device__ __noinline__ bool head_wait_for_room(const unsigned int* word, unsigned int need,
                                                unsigned int& c) {
  for (unsigned int polls = 0; polls < kHeadPolls; ++polls) {
    c = ld_relaxed_shared(word);
    if ((c & kHeadStopBit) || c >= need) return true;
  }
  return false;
}

// The set of matched blocks made by the head kernel itself (no further launch): the probers mark
// the ids of every matched prefix in a bitmap over block ids; every prober fills its own
// request's part of the output with AIBX_NO_BLOCK, counts itself in, and the warp that counts in
// last - all marks are in the bitmap by then - turns it into the ascending list.  Nobody waits:
// the last arriver does the work.  bitmap == nullptr: no set is made.
struct HeadCollect {
  unsigned int* bitmap;      // zeroed before the launch, (num_blocks + 31) / 32 words
  unsigned int* arrived;     // zeroed before the launch
  uint32_t* unique;          // [blk_off[R]] ascending distinct ids, then AIBX_NO_BLOCK
  uint32_t* count;
  uint32_t num_blocks;
};

// One warp turns the bitmap into the ascending id list (at most kCollectSmallWords words: the
// host only fuses the set into the head kernel for pools of that size).
__device__ __forceinline__ void head_compact(const HeadCollect& hc, int lane, int64_t n_total) {
  const uint32_t n_words = (hc.num_blocks + 31u) / 32u;
  unsigned int base = 0;
  for (uint32_t w0 = 0; w0 < n_words; w0 += 32) {
    const uint32_t w = w0 + lane;
    unsigned int bits = w < n_words ? __ldcg(hc.bitmap + w) : 0u;
    const unsigned int c = __popc(bits);
    unsigned int inc = c;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const unsigned int o = __shfl_up_sync(0xffffffffu, inc, d);
      if (lane >= d) inc += o;
    }
    unsigned int pos = base + inc - c;
    while (bits) {
      const int b = __ffs(bits) - 1;
      bits &= bits - 1;
      if ((int64_t)pos < n_total) hc.unique[pos] = w * 32u + (uint32_t)b;
      ++pos;
    }
    base += __shfl_sync(0xffffffffu, inc, 31);
  }
  if (lane == 0) *hc.count = base;
}

template <int SPB>   // stripes of 32 bytes per block: 1, 2, 4 or 8
__global__ void __launch_bounds__(288)
route_head_kernel(IndexView ix, const int32_t* __restrict__ tokens,
                  const int64_t* __restrict__ tok_off, const int64_t* __restrict__ blk_off, int R,
                  uint64_t root_seed, uint64_t* __restrict__ hashes, uint32_t* match_len,
                  uint32_t* __restrict__ any_len, uint32_t* __restrict__ block_ids, ScoreParams sp,
                  int32_t* __restrict__ best_pod, int64_t* __restrict__ best_score,
                  uint32_t* __restrict__ hashed_out, uint64_t* __restrict__ seed_out,
                  unsigned int epoch, HeadCollect hc) {
  constexpr int BPG = kGroupStripes / SPB;             // blocks per group of 8 stripes
  __shared__ HeadShared sh;
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int k = lane & 3;
  // request inside the CTA: by quad in the hasher warp, by warp among the probers
  const int qi = warp == 0 ? lane >> 2 : warp - 1;
  const int quad_base = lane & ~3;
  const unsigned int qmask = 0xFu << quad_base;
  const int r = blockIdx.x * 8 + qi;
  if (threadIdx.x < 8) {
    sh.progress[threadIdx.x] = 0;
    sh.consumed[threadIdx.x] = 0;
  }
  __syncthreads();
  volatile unsigned int* v_consumed = &sh.consumed[qi];
  const bool live = r < R;
  const int64_t out0 = live ? blk_off[r] : 0;
  const unsigned int n_r = live ? (unsigned int)(blk_off[r + 1] - out0) : 0u;

  if (threadIdx.x < 32) {
    // ------------------------------------------------------------------ hasher warp
    if (!live) return;                                 // whole quads leave together
    const int32_t* p = tokens + tok_off[r] + 2 * k;
    const uint64_t init_add = k == 0 ? kP1 + kP2 : k == 1 ? kP2 : k == 2 ? 0ULL : 0ULL - kP1;
    const int rot = k == 0 ? 1 : k == 1 ? 7 : k == 2 ? 12 : 18;
    const uint64_t len_bytes = (uint64_t)SPB * 32ULL;
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
          if (s < avail) {                             // only full blocks are ever read
            lo[s] = (uint32_t)__ldg(q + 8 * s);
            hi[s] = (uint32_t)__ldg(q + 8 * s + 1);
          }
        }
      }
    };
    uint64_t v = root_seed + init_add;
    unsigned int hashed = 0;
    auto stripe = [&](int s) {
      const uint64_t x = (uint64_t)cur_lo[s] | ((uint64_t)cur_hi[s] << 32);
      v = rotl64(v + x * kP2, 31) * kP1;
      if ((s + 1) % SPB == 0) {
        const uint64_t key = finish_block_quad(qmask, quad_base, v, rot, len_bytes);
        if (k == 0) sh.ring[qi][hashed % kHeadRing] = key;
        ++hashed;
        v = key + init_add;
      }
    };
    int left = (int)n_r * SPB;
    fetch(p, left, cur_lo, cur_hi);
    // What the prober says is read once per group and looked at one group LATER: a shared-memory
    // load that is consumed at once would wait together with the token loads in flight around
    // it (measured: +100 ns per block).  A stale count only errs on the safe side.
    constexpr int kPublishGroups = BPG >= 4 ? 1 : 4 / BPG;
    int groups_done = 0;
    unsigned int c = 0;
    for (;;) {
      // hot loop: runs while there is work, no stop, and room in the ring.  Room for the next
      // four groups is established every fourth group (a check in every turn of the loop cost
      // 0.16 us per group), from a count that may be stale, i.e. too small: the safe side.
      bool room = hashed + 4 * BPG <= c + kHeadRing;
      while (left > 0 && !(c & kHeadStopBit) && room) {
        const unsigned int c_next = ld_relaxed_shared(&sh.consumed[qi]);
        fetch(p + 8 * kGroupStripes, left - kGroupStripes, nxt_lo, nxt_hi);
        if (left >= kGroupStripes) {                     // whole group: no per-stripe checks
#pragma unroll
          for (int s = 0; s < kGroupStripes; ++s) stripe(s);
        } else {
#pragma unroll
          for (int s = 0; s < kGroupStripes; ++s) {
            if (s < left) stripe(s);                     // uniform inside the quad
          }
        }
#pragma unroll
        for (int s = 0; s < kGroupStripes; ++s) {
          cur_lo[s] = nxt_lo[s];
          cur_hi[s] = nxt_hi[s];
        }
        p += 8 * kGroupStripes;
        left -= kGroupStripes;
        // The keys before the count that announces them (release; the probers acquire).  The
        // release also waits for the token loads in flight, so with few blocks per group it is
        // done only every kPublishGroups groups (at least four blocks per release).
        if (++groups_done % kPublishGroups == 0 || left <= 0) {
          if (k == 0) st_release_shared(&sh.progress[qi], hashed);
        }
        c = c_next;
        // room for the next four groups is checked every fourth group
        if ((groups_done & 3) == 0) room = hashed + 4 * BPG <= c + kHeadRing;
      }
      if (left <= 0 || (c & kHeadStopBit)) break;
      // A whole ring ahead of the prober (rare; kept out of the hot loop, whose code the compiler
      // schedules much worse with a wait inside it): wait for it, bounded - it always catches up.
      if (!head_wait_for_room(&sh.consumed[qi], hashed + 4 * BPG - kHeadRing, c)) {
        if (k == 0) raise_status(AIBX_ERR_TIMEOUT);
        break;
      }
    }
    return;
  }

  // -------------------------------------------------------------------- prober warp
  if (!live) return;
  const int P = ix.num_pods;
  const uint64_t all = pod_all(P);
  PrefixFold st = {all, 0u, false};                    // see index.cuh
  sh.match_len[qi][lane] = 0u;                         // fold_chunk wants its scratch zeroed
  sh.match_len[qi][lane + 32] = 0u;
  __syncwarp();
  unsigned int idle = 0;
  unsigned int written = 0;                            // keys of this request written to `hashes`
  uint64_t last_key = root_seed;                       // the last of them: the seed to resume from
  while (!st.ended && st.pos < n_r) {
    const unsigned int avail = ld_acquire_shared(&sh.progress[qi]);   // same word for all lanes
    if (avail == st.pos) {
      if (++idle >= kHeadPolls) {                      // the hasher never delivered: give up
        if (lane == 0) {
          *v_consumed = st.pos | kHeadStopBit;
          raise_status(AIBX_ERR_TIMEOUT);
        }
        break;
      }
      __nanosleep(100);                                // a group of keys takes ~0.8 us to make
      continue;
    }
    idle = 0;
    const unsigned int m = min(32u, avail - st.pos);
    uint64_t mask = 0, key = 0;
    uint32_t id = AIBX_NO_BLOCK;
    unsigned long long entry = ~0ULL;
    if ((unsigned int)lane < m) {
      key = *reinterpret_cast<volatile unsigned long long*>(
          &sh.ring[qi][(st.pos + lane) % kHeadRing]);
      hashes[out0 + st.pos + lane] = key;              // the keys leave the CTA through the prober
      probe_ro(ix, key, mask, id, entry);
    }
    written = st.pos + m;
    last_key = shfl64(0xffffffffu, key, (int)m - 1);
    const unsigned int first = st.pos;
    fold_chunk(st, lane, m, mask, id, all, sh.match_len[qi], block_ids ? block_ids + out0 : nullptr);
    const bool matched = first + (unsigned int)lane < st.pos;
    if (epoch && matched) touch_entry(ix, entry, epoch);
    if (hc.bitmap && matched) {
      if (id < hc.num_blocks) atomicOr(&hc.bitmap[id >> 5], 1u << (id & 31u));
      else if (id != AIBX_NO_BLOCK) raise_status(AIBX_ERR_RANGE);
    }
    // Lets the hasher reuse the ring slots just read.  The keys read from them have been used
    // by now (every lane computed its probe address from its key), so the reads are complete
    // before this store is issued; a plain store is enough.
    if (lane == 0) *v_consumed = st.ended ? (st.pos | kHeadStopBit) : st.pos;
  }

  // ---- the request's results (after a time-out they are unspecified; the status says so)
  fold_finish(st, lane, P, r, n_r, out0, sh.match_len[qi], match_len, any_len, block_ids, sp,
              best_pod, best_score);
  if (lane == 0) {
    hashed_out[r] = written;                           // keys the hasher made beyond these are dropped
    seed_out[r] = last_key;
  }
  if (hc.bitmap) {
    for (unsigned int i = lane; i < n_r; i += 32) hc.unique[out0 + i] = AIBX_NO_BLOCK;
    __threadfence();                                   // marks and padding before the count
    unsigned int before = 0;
    if (lane == 0) before = atomicAdd(hc.arrived, 1u);
    before = __shfl_sync(0xffffffffu, before, 0);
    if (before == (unsigned int)R - 1u) {              // every other request has counted in
      __threadfence();
      head_compact(hc, lane, blk_off[R]);
    }
  }
}

// State for aibx_hash_blocks_resume after a path that hashed every block.
__global__ void route_head_state_full_kernel(const int64_t* __restrict__ blk_off, int R,
                                             uint64_t root_seed, const uint64_t* __restrict__ hashes,
                                             uint32_t* __restrict__ hashed_out,
                                             uint64_t* __restrict__ seed_out) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= R) return;
  const int64_t lo = blk_off[r], hi = blk_off[r + 1];
  hashed_out[r] = (uint32_t)(hi - lo);
  seed_out[r] = hi > lo ? hashes[hi - 1] : root_seed;
}

}  // namespace aibx
