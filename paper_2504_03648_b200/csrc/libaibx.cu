// libaibx: C ABI over the kernels (see include/aibx.h for the contract of every call).
// One translation unit, so the per-device status record is shared by all kernels.
#include <cuda_runtime.h>

#include <new>

#include "aibx.h"
#include "aibx_tuning.h"
#include "aibx_common.cuh"
#include "collect_blocks.cuh"
#include "hash_blocks.cuh"
#include "index.cuh"
#include "kv_copy.cuh"
#include "kv_permute.cuh"
#include "selftest.cuh"
#include "route_head.cuh"
#include "route_score.cuh"
#include "victims.cuh"

using namespace aibx;

struct aibx_index {
  IndexView view;
  uint64_t capacity;
  int device;
  VictimScratch* victim_scratch;   // allocated on first use of aibx_index_pick_victims
  // a rehash in progress (aibx_index_rehash_begin .. _finish): the table being filled, and the
  // event that says the move has finished.  Readers keep using `view` meanwhile.
  bool migrating;
  IndexView pending;
  uint64_t pending_capacity;
  cudaEvent_t moved;
};

namespace {

inline cudaStream_t as_stream(void* s) { return static_cast<cudaStream_t>(s); }

inline unsigned int blocks_for(int64_t n, int threads) {
  return (unsigned int)((n + threads - 1) / threads);
}

// The kernels that are meant to run BESIDE the KV copies (on another stream) ask for the same
// shared-memory carve-out as the copy kernel needs.  An SM cannot host kernels with different
// carve-outs at once: without this, every SM that runs one of these small kernels would keep the
// copy kernel's CTA waiting until the small kernel has drained (measured: the gather ended later
// by the whole duration of whatever ran beside it).  Once per device.
void prefer_copy_carveout() {
  static std::once_flag once[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return;
  std::call_once(once[dev], [] {
  const void* side_kernels[] = {
      (const void*)hash_blocks_kernel<0>,      (const void*)hash_blocks_kernel<1>,
      (const void*)hash_blocks_kernel<2>,      (const void*)hash_blocks_kernel<4>,
      (const void*)hash_blocks_kernel<8>,      (const void*)index_insert_kernel,
      (const void*)index_evict_clear_kernel,   (const void*)index_evict_report_kernel,
      (const void*)index_evict_remove_kernel,  (const void*)index_touch_kernel,
      (const void*)index_evict_coop_kernel,    (const void*)route_head_kernel<1>,
      (const void*)route_head_kernel<2>,       (const void*)route_head_kernel<4>,
      (const void*)route_head_kernel<8>,
  };
  for (const void* f : side_kernels)
    cudaFuncSetAttribute(f, cudaFuncAttributePreferredSharedMemoryCarveout,
                         cudaSharedmemCarveoutMaxShared);
  cudaGetLastError();   // a refused hint is not an error of the call that follows
  });
}

// Device storage of one table: sectors, stamps and counters in ONE allocation (64-byte aligned
// parts), so that creating or dropping a table is one call into the allocator.  Tables of up to
// 32 pods take the narrow entry (two per 32-byte sector), the others the wide one.
int32_t alloc_view(uint64_t capacity, int num_pods, IndexView* out) {
  const int narrow = num_pods <= 32 ? 1 : 0;
  const uint64_t nb = narrow ? capacity / 2 : capacity;
  const size_t sector_bytes = (size_t)nb * 32;
  const size_t stamp_bytes = ((size_t)capacity * sizeof(unsigned int) + 63) & ~(size_t)63;
  void* base = nullptr;
  if (cudaMalloc(&base, sector_bytes + stamp_bytes + 64) != cudaSuccess) {
    cudaGetLastError();   // an allocation failure is not sticky; leave no error behind
    return AIBX_ERR_NOMEM;
  }
  char* p = static_cast<char*>(base);
  out->words = reinterpret_cast<unsigned long long*>(p);
  out->stamps = reinterpret_cast<unsigned int*>(p + sector_bytes);
  out->counters = reinterpret_cast<unsigned long long*>(p + sector_bytes + stamp_bytes);
  out->nb = nb;
  out->capacity = capacity;
  const uint64_t walk = narrow ? kMaxWalkEntries / 2 : kMaxWalkEntries;
  out->max_walk = (unsigned int)(nb < walk ? nb : walk);
  out->num_pods = num_pods;
  out->narrow = narrow;
  return AIBX_OK;
}

void free_view(const IndexView& v) { cudaFree(v.words); }

bool capacity_ok(uint64_t c) { return c >= 8 && (c & (c - 1)) == 0 && c <= (1ULL << 40); }

// How many CTAs of the one-launch evict kernel the current device can hold at once (0: it
// cannot launch kernels cooperatively, or the query failed).
int evict_coop_ctas() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  int v = cached[dev].load(std::memory_order_relaxed);
  if (v == 0) {
    int coop = 0, per_sm = 0;
    if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, index_evict_coop_kernel, 256, 0) !=
            cudaSuccess ||
        per_sm <= 0) {
      cudaGetLastError();
      v = -1;
    } else {
      // half of what fits: the kernel usually runs beside others, and every one of its CTAs
      // must be resident before the first can pass the barrier
      v = sm_count() * (per_sm > 1 ? per_sm / 2 : 1);
    }
    cached[dev].store(v, std::memory_order_relaxed);
  }
  return v > 0 ? v : 0;
}

// Device address of the status record of the current device.
StatusRecord* status_ptr() {
  static std::atomic<StatusRecord*> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  StatusRecord* p = cached[dev].load(std::memory_order_acquire);
  if (!p) {
    void* q = nullptr;
    if (cudaGetSymbolAddress(&q, g_status) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    p = static_cast<StatusRecord*>(q);
    cached[dev].store(p, std::memory_order_release);
  }
  return p;
}

// Built-in scratch of aibx_collect_blocks_static: a bitmap over block ids that lives in the
// library image itself, so the call needs no allocation.  128 KiB per GPU that loads the
// library, held until the process exits.
constexpr uint32_t kStaticCollectMaxBlocks = 1u << 20;
static __device__ __align__(256) unsigned int g_collect_bitmap[kStaticCollectMaxBlocks / 32];

// In host code `g_collect_bitmap` is only a handle for the runtime, not a device address, so
// kernels must be given what cudaGetSymbolAddress returns.  Resolved once per device, with that
// device current; returns nullptr when the runtime refuses.
unsigned int* static_bitmap_ptr() {
  static std::atomic<unsigned int*> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  unsigned int* p = cached[dev].load(std::memory_order_acquire);
  if (!p) {
    if (cudaGetSymbolAddress((void**)&p, g_collect_bitmap) != cudaSuccess) {
      cudaGetLastError();
      return nullptr;
    }
    cached[dev].store(p, std::memory_order_release);
  }
  return p;
}

}  // namespace

extern "C" {

int32_t aibx_hash_blocks(const int32_t* d_tokens, const int64_t* d_tok_off,
                         const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                         uint64_t root_seed, uint64_t* d_hashes, void* stream) {
  AIBX_CALL_RANGE();
  if (R < 0 || block_tokens <= 0 || block_tokens % 8 != 0 || block_tokens > 1024)
    return AIBX_ERR_INVALID;
  if (R == 0) return AIBX_OK;
  if (!d_tokens || !d_tok_off || !d_blk_off || !d_hashes) return AIBX_ERR_INVALID;
  prefer_copy_carveout();
  return launch_hash_blocks(d_tokens, d_tok_off, d_blk_off, R, block_tokens, root_seed, d_hashes,
                            as_stream(stream));
}

int32_t aibx_index_create(aibx_index_t** out, uint64_t capacity_slots, int32_t num_pods) {
  AIBX_CALL_RANGE();
  if (!out) return AIBX_ERR_INVALID;
  *out = nullptr;
  if (num_pods < 1 || num_pods > AIBX_MAX_PODS) return AIBX_ERR_INVALID;
  if (!capacity_ok(capacity_slots)) return AIBX_ERR_INVALID;
  aibx_index* ix = new (std::nothrow) aibx_index();
  if (!ix) return AIBX_ERR_NOMEM;
  if (cudaGetDevice(&ix->device) != cudaSuccess) {
    delete ix;
    return AIBX_ERR_CUDA;
  }
  const int32_t rc = alloc_view(capacity_slots, num_pods, &ix->view);
  if (rc != AIBX_OK) {
    delete ix;
    return rc;
  }
  ix->capacity = capacity_slots;
  ix->migrating = false;
  ix->moved = nullptr;
  index_clear_kernel<<<sm_count() * 8, 256>>>(ix->view);
  if (cudaDeviceSynchronize() != cudaSuccess) {
    cudaGetLastError();
    free_view(ix->view);
    delete ix;
    return AIBX_ERR_CUDA;
  }
  *out = ix;
  return AIBX_OK;
}

int32_t aibx_index_destroy(aibx_index_t* ix) {
  AIBX_CALL_RANGE();
  if (!ix) return AIBX_ERR_INVALID;
  cudaDeviceSynchronize();
  if (ix->migrating) free_view(ix->pending);
  if (ix->moved) cudaEventDestroy(ix->moved);
  free_view(ix->view);
  if (ix->victim_scratch) cudaFree(ix->victim_scratch);
  delete ix;
  return AIBX_OK;
}

int32_t aibx_index_clear(aibx_index_t* ix, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || ix->migrating) return AIBX_ERR_INVALID;
  index_clear_kernel<<<sm_count() * 8, 256, 0, as_stream(stream)>>>(ix->view);
  return launch_status();
}

int32_t aibx_index_insert(aibx_index_t* ix, const uint64_t* d_keys, const uint64_t* d_pod_masks,
                          const uint32_t* d_block_ids, int64_t n, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || n < 0 || ix->migrating) return AIBX_ERR_INVALID;
  if (n == 0) return AIBX_OK;
  if (!d_keys || !d_pod_masks || !d_block_ids) return AIBX_ERR_INVALID;
  prefer_copy_carveout();
  index_insert_kernel<<<blocks_for(n, 256), 256, 0, as_stream(stream)>>>(
      ix->view, d_keys, d_pod_masks, d_block_ids, n);
  return launch_status();
}

int32_t aibx_index_evict(aibx_index_t* ix, const uint64_t* d_keys, const uint64_t* d_pod_masks,
                         uint32_t* d_freed_block_ids, int64_t n, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || n < 0 || ix->migrating) return AIBX_ERR_INVALID;
  if (n == 0) return AIBX_OK;
  if (!d_keys || !d_pod_masks) return AIBX_ERR_INVALID;
  prefer_copy_carveout();
  cudaStream_t st = as_stream(stream);
  const unsigned int grid = blocks_for(n, 256);
  const int coop = evict_coop_ctas();
  if (coop > 0) {
    IndexView view = ix->view;
    void* args[] = {&view, &d_keys, &d_pod_masks, &d_freed_block_ids, &n};
    const unsigned int g = grid < (unsigned int)coop ? grid : (unsigned int)coop;
    if (cudaLaunchCooperativeKernel((const void*)index_evict_coop_kernel, dim3(g), dim3(256), args,
                                    0, st) == cudaSuccess)
      return AIBX_OK;
    cudaGetLastError();       // fall back to the three plain launches
  }
  index_evict_clear_kernel<<<grid, 256, 0, st>>>(ix->view, d_keys, d_pod_masks, n);
  if (d_freed_block_ids)
    index_evict_report_kernel<<<grid, 256, 0, st>>>(ix->view, d_keys, d_freed_block_ids, n);
  index_evict_remove_kernel<<<grid, 256, 0, st>>>(ix->view, d_keys, n);
  return launch_status();
}

int32_t aibx_index_lookup(const aibx_index_t* ix, const uint64_t* d_keys, uint64_t* d_masks,
                          uint32_t* d_block_ids, int64_t n, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || n < 0) return AIBX_ERR_INVALID;
  if (n == 0) return AIBX_OK;
  if (!d_keys) return AIBX_ERR_INVALID;
  index_lookup_kernel<<<blocks_for(n, 256), 256, 0, as_stream(stream)>>>(ix->view, d_keys, d_masks,
                                                                         d_block_ids, n);
  return launch_status();
}

int32_t aibx_index_stats2(const aibx_index_t* ix, uint64_t* live, uint64_t* removed,
                          uint64_t* capacity, uint32_t* longest_walk, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix) return AIBX_ERR_INVALID;
  unsigned long long c[3] = {0, 0, 0};
  if (cudaMemcpyAsync(c, ix->view.counters, sizeof(c), cudaMemcpyDeviceToHost,
                      as_stream(stream)) != cudaSuccess ||
      cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) {
    cudaGetLastError();
    return AIBX_ERR_CUDA;
  }
  if (live) *live = c[0];
  if (removed) *removed = c[1];
  if (capacity) *capacity = ix->capacity;
  if (longest_walk) *longest_walk = c[2] ? (uint32_t)c[2] : 1u;   // a walk visits at least one sector
  return AIBX_OK;
}

int32_t aibx_index_stats(const aibx_index_t* ix, uint64_t* live, uint64_t* capacity,
                         void* stream) {
  AIBX_CALL_RANGE();
  return aibx_index_stats2(ix, live, nullptr, capacity, nullptr, stream);
}

int32_t aibx_index_touch(aibx_index_t* ix, const uint64_t* d_keys, int64_t n, uint32_t epoch,
                         void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || n < 0 || epoch == 0 || epoch >= (1u << 30) || ix->migrating) return AIBX_ERR_INVALID;
  if (n == 0) return AIBX_OK;
  if (!d_keys) return AIBX_ERR_INVALID;
  index_touch_kernel<<<blocks_for(n, 256), 256, 0, as_stream(stream)>>>(ix->view, d_keys, n, epoch);
  return launch_status();
}

int32_t aibx_index_pick_victims(aibx_index_t* ix, uint64_t k, uint64_t* d_keys,
                                uint32_t* d_priorities, uint64_t* d_count, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || !d_count) return AIBX_ERR_INVALID;
  cudaStream_t st = as_stream(stream);
  if (!ix->victim_scratch) {
    void* p = nullptr;
    if (cudaMalloc(&p, sizeof(VictimScratch)) != cudaSuccess) {
      cudaGetLastError();
      return AIBX_ERR_NOMEM;
    }
    ix->victim_scratch = static_cast<VictimScratch*>(p);
  }
  VictimScratch* sc = ix->victim_scratch;
  if (cudaMemsetAsync(sc, 0, sizeof(VictimScratch), st) != cudaSuccess ||
      cudaMemsetAsync(d_count, 0, sizeof(uint64_t), st) != cudaSuccess)
    return AIBX_ERR_CUDA;
  if (k == 0) return AIBX_OK;
  if (cudaMemcpyAsync(&sc->st.k, &k, sizeof(k), cudaMemcpyHostToDevice, st) != cudaSuccess)
    return AIBX_ERR_CUDA;
  const int grid = sm_count() * 8;
  unsigned long long* cnt = reinterpret_cast<unsigned long long*>(d_count);
  victims_hist_kernel<<<grid, 256, 0, st>>>(ix->view, sc, 1);
  victims_select_kernel<<<1, 1024, 0, st>>>(sc, 1, cnt);
  victims_hist_kernel<<<grid, 256, 0, st>>>(ix->view, sc, 2);
  victims_select_kernel<<<1, 1024, 0, st>>>(sc, 2, cnt);
  victims_collect_kernel<<<grid, 256, 0, st>>>(ix->view, sc, d_keys, d_priorities);
  return launch_status();
}

int32_t aibx_index_export(const aibx_index_t* ix, uint64_t* d_keys, uint64_t* d_masks,
                          uint32_t* d_block_ids, uint64_t max_entries, uint64_t* d_count,
                          void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || !d_count) return AIBX_ERR_INVALID;
  cudaStream_t st = as_stream(stream);
  if (cudaMemsetAsync(d_count, 0, sizeof(uint64_t), st) != cudaSuccess) return AIBX_ERR_CUDA;
  index_export_kernel<<<sm_count() * 8, 256, 0, st>>>(
      ix->view, d_keys, d_masks, d_block_ids, max_entries,
      reinterpret_cast<unsigned long long*>(d_count));
  return launch_status();
}

int32_t aibx_index_rehash(aibx_index_t* ix, uint64_t new_capacity) {
  AIBX_CALL_RANGE();
  if (!ix || ix->migrating) return AIBX_ERR_INVALID;
  if (!capacity_ok(new_capacity)) return AIBX_ERR_INVALID;
  if (cudaDeviceSynchronize() != cudaSuccess) return AIBX_ERR_CUDA;
  unsigned long long live = 0;
  if (cudaMemcpy(&live, ix->view.counters, sizeof(live), cudaMemcpyDeviceToHost) != cudaSuccess)
    return AIBX_ERR_CUDA;
  if (live > new_capacity) return AIBX_ERR_FULL;
  IndexView fresh;
  const int32_t rc = alloc_view(new_capacity, ix->view.num_pods, &fresh);
  if (rc != AIBX_OK) return rc;
  const IndexView old = ix->view;
  index_clear_kernel<<<sm_count() * 8, 256>>>(fresh);
  index_move_kernel<<<sm_count() * 8, 256>>>(old, fresh);      // re-counts the live entries
  if (cudaDeviceSynchronize() != cudaSuccess) {
    cudaGetLastError();
    free_view(fresh);
    return AIBX_ERR_CUDA;
  }
  free_view(old);
  ix->view = fresh;
  ix->capacity = new_capacity;
  return AIBX_OK;
}

int32_t aibx_index_rehash_begin(aibx_index_t* ix, uint64_t new_capacity, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || ix->migrating) return AIBX_ERR_INVALID;
  if (!capacity_ok(new_capacity)) return AIBX_ERR_INVALID;
  cudaStream_t st = as_stream(stream);
  // the live count as of `stream` (only this stream is waited for, not the device)
  unsigned long long live = 0;
  if (cudaMemcpyAsync(&live, ix->view.counters, sizeof(live), cudaMemcpyDeviceToHost, st) !=
          cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return AIBX_ERR_CUDA;
  if (live > new_capacity) return AIBX_ERR_FULL;
  if (!ix->moved &&
      cudaEventCreateWithFlags(&ix->moved, cudaEventDisableTiming) != cudaSuccess) {
    ix->moved = nullptr;
    return AIBX_ERR_CUDA;
  }
  IndexView fresh;                                       // its own storage: `view` stays intact
  const int32_t rc = alloc_view(new_capacity, ix->view.num_pods, &fresh);
  if (rc != AIBX_OK) return rc;
  index_clear_kernel<<<sm_count() * 8, 256, 0, st>>>(fresh);
  index_move_kernel<<<sm_count() * 8, 256, 0, st>>>(ix->view, fresh);
  if (cudaEventRecord(ix->moved, st) != cudaSuccess || launch_status() != AIBX_OK) {
    cudaStreamSynchronize(st);
    free_view(fresh);
    return AIBX_ERR_CUDA;
  }
  ix->pending = fresh;
  ix->pending_capacity = new_capacity;
  ix->migrating = true;
  return AIBX_OK;
}

int32_t aibx_index_rehash_finish(aibx_index_t* ix) {
  AIBX_CALL_RANGE();
  if (!ix || !ix->migrating) return AIBX_ERR_INVALID;
  if (cudaEventSynchronize(ix->moved) != cudaSuccess) return AIBX_ERR_CUDA;
  const IndexView old = ix->view;
  ix->view = ix->pending;
  ix->capacity = ix->pending_capacity;
  ix->migrating = false;
  // cudaFree waits for the work still using the old table (readers launched before the switch)
  free_view(old);
  return AIBX_OK;
}

namespace {

int32_t launch_match(const aibx_index_t* ix, const uint64_t* d_hashes, const int64_t* d_blk_off,
                     int32_t R, uint32_t* d_match_len, uint32_t* d_any_len, uint32_t* d_block_ids,
                     const ScoreParams& sp, int32_t* d_best_pod, int64_t* d_best_score,
                     cudaStream_t st, unsigned int epoch = 0);

}  // namespace

int32_t aibx_match_prefix(const aibx_index_t* ix, const uint64_t* d_hashes,
                          const int64_t* d_blk_off, int32_t R, uint32_t* d_match_len,
                          uint32_t* d_any_len, uint32_t* d_block_ids, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || R < 0) return AIBX_ERR_INVALID;
  if (R == 0) return AIBX_OK;
  if (!d_hashes || !d_blk_off || !d_match_len) return AIBX_ERR_INVALID;
  ScoreParams none = {nullptr, 0, 0, 0, 0};
  return launch_match(ix, d_hashes, d_blk_off, R, d_match_len, d_any_len, d_block_ids, none,
                      nullptr, nullptr, as_stream(stream));
}

int32_t aibx_match_prefix_touch(aibx_index_t* ix, const uint64_t* d_hashes,
                                const int64_t* d_blk_off, int32_t R, uint32_t epoch,
                                uint32_t* d_match_len, uint32_t* d_any_len, uint32_t* d_block_ids,
                                void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || R < 0 || epoch == 0 || epoch >= (1u << 30) || ix->migrating) return AIBX_ERR_INVALID;
  if (R == 0) return AIBX_OK;
  if (!d_hashes || !d_blk_off || !d_match_len) return AIBX_ERR_INVALID;
  ScoreParams none = {nullptr, 0, 0, 0, 0};
  return launch_match(ix, d_hashes, d_blk_off, R, d_match_len, d_any_len, d_block_ids, none,
                      nullptr, nullptr, as_stream(stream), epoch);
}

namespace {

int32_t launch_match(const aibx_index_t* ix, const uint64_t* d_hashes, const int64_t* d_blk_off,
                     int32_t R, uint32_t* d_match_len, uint32_t* d_any_len, uint32_t* d_block_ids,
                     const ScoreParams& sp, int32_t* d_best_pod, int64_t* d_best_score,
                     cudaStream_t st, unsigned int epoch) {
  // warps per request: aim at ~32 resident warps per SM; few requests get whole CTAs
  int wpr = 1;
  const long long target = (long long)sm_count() * 32;
  while (wpr < 32 && (long long)R * wpr * 2 <= target) wpr *= 2;
  if (wpr == 1) {
    // warps enough with one per request: the shape without barriers and shared-memory atomics
    const unsigned int grid = blocks_for(R, kMatchWarpKernelWarps);
    if (ix->view.narrow)
      match_prefix_warp_kernel<true><<<grid, kMatchWarpKernelWarps * 32, 0, st>>>(
          ix->view, d_hashes, d_blk_off, R, d_match_len, d_any_len, d_block_ids, sp, d_best_pod,
          d_best_score, epoch);
    else
      match_prefix_warp_kernel<false><<<grid, kMatchWarpKernelWarps * 32, 0, st>>>(
          ix->view, d_hashes, d_blk_off, R, d_match_len, d_any_len, d_block_ids, sp, d_best_pod,
          d_best_score, epoch);
    return launch_status();
  }
  const int warps_per_cta = wpr > kMatchWarpsMin ? wpr : kMatchWarpsMin;
  const int groups = warps_per_cta / wpr;
  const unsigned int grid = (unsigned int)((R + groups - 1) / groups);
  const size_t smem = (size_t)groups * sizeof(MatchShared);
  match_prefix_kernel<<<grid, warps_per_cta * 32, smem, st>>>(
      ix->view, d_hashes, d_blk_off, R, wpr, d_match_len, d_any_len, d_block_ids, sp, d_best_pod,
      d_best_score, epoch);
  return launch_status();
}

}  // namespace

int32_t aibx_route_batch(const aibx_index_t* ix, const int32_t* d_tokens, const int64_t* d_tok_off,
                         const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                         uint64_t root_seed, const int32_t* d_pod_load, uint64_t ready_mask,
                         const aibx_route_params_t* params, uint64_t* d_hashes,
                         uint32_t* d_match_len, uint32_t* d_any_len, uint32_t* d_block_ids,
                         int32_t* d_best_pod, int64_t* d_best_score, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || R < 0 || block_tokens <= 0 || block_tokens % 8 != 0 || block_tokens > 1024)
    return AIBX_ERR_INVALID;
  if (R == 0) return AIBX_OK;
  if (!d_tokens || !d_tok_off || !d_blk_off || !d_hashes || !d_match_len || !d_pod_load ||
      !d_best_pod || !d_best_score)
    return AIBX_ERR_INVALID;
  aibx_route_params_t prm = {4, 1, 50};
  if (params) prm = *params;
  cudaStream_t st = as_stream(stream);
  const int32_t rc = launch_hash_blocks(d_tokens, d_tok_off, d_blk_off, R, block_tokens, root_seed,
                                        d_hashes, st);
  if (rc != AIBX_OK) return rc;
  ScoreParams sp = {d_pod_load, ready_mask, prm.w_prefix, prm.w_load, prm.threshold_pct};
  return launch_match(ix, d_hashes, d_blk_off, R, d_match_len, d_any_len, d_block_ids, sp,
                      d_best_pod, d_best_score, st);
}

namespace {

int32_t route_head_impl(const aibx_index_t* ix, const int32_t* d_tokens, const int64_t* d_tok_off,
                        const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                        uint64_t root_seed, const int32_t* d_pod_load, uint64_t ready_mask,
                        const aibx_route_params_t* params, uint64_t* d_hashes,
                        uint32_t* d_match_len, uint32_t* d_any_len, uint32_t* d_block_ids,
                        int32_t* d_best_pod, int64_t* d_best_score, uint32_t* d_hashed,
                        uint64_t* d_next_seed, void* stream, unsigned int epoch,
                        HeadCollect hc = HeadCollect{nullptr, nullptr, nullptr, nullptr, 0u}) {
  if (!ix || R < 0 || block_tokens <= 0 || block_tokens % 8 != 0 || block_tokens > 1024)
    return AIBX_ERR_INVALID;
  if (R == 0) return AIBX_OK;
  if (!d_tokens || !d_tok_off || !d_blk_off || !d_hashes || !d_match_len || !d_hashed ||
      !d_next_seed)
    return AIBX_ERR_INVALID;
  if ((d_best_pod == nullptr) != (d_best_score == nullptr)) return AIBX_ERR_INVALID;
  if (d_best_pod && !d_pod_load) return AIBX_ERR_INVALID;
  aibx_route_params_t prm = {4, 1, 50};
  if (params) prm = *params;
  prefer_copy_carveout();      // the routing of the next batch may run beside this batch's copies
  cudaStream_t st = as_stream(stream);
  ScoreParams sp = {d_pod_load, ready_mask, prm.w_prefix, prm.w_load, prm.threshold_pct};
  const int spb = block_tokens / 8;
  const int grid = (R + 7) / 8;
#define AIBX_HEAD_LAUNCH(SPB)                                                                   \
  route_head_kernel<SPB><<<grid, 288, 0, st>>>(ix->view, d_tokens, d_tok_off, d_blk_off, R,      \
                                              root_seed, d_hashes, d_match_len, d_any_len,      \
                                              d_block_ids, sp, d_best_pod, d_best_score,        \
                                              d_hashed, d_next_seed, epoch, hc)
  if (spb == 1) {
    AIBX_HEAD_LAUNCH(1);
  } else if (spb == 2) {
    AIBX_HEAD_LAUNCH(2);
  } else if (spb == 4) {
    AIBX_HEAD_LAUNCH(4);
  } else if (spb == 8) {
    AIBX_HEAD_LAUNCH(8);
  } else {
    // other block sizes: the whole chain, then the match kernel; nothing is left to resume
    int32_t rc = launch_hash_blocks(d_tokens, d_tok_off, d_blk_off, R, block_tokens, root_seed,
                                    d_hashes, st);
    if (rc != AIBX_OK) return rc;
    rc = launch_match(ix, d_hashes, d_blk_off, R, d_match_len, d_any_len, d_block_ids, sp,
                      d_best_pod, d_best_score, st, epoch);
    if (rc != AIBX_OK) return rc;
    route_head_state_full_kernel<<<blocks_for(R, 256), 256, 0, st>>>(d_blk_off, R, root_seed,
                                                                     d_hashes, d_hashed, d_next_seed);
  }
#undef AIBX_HEAD_LAUNCH
  return launch_status();
}

}  // namespace

int32_t aibx_route_head(const aibx_index_t* ix, const int32_t* d_tokens, const int64_t* d_tok_off,
                        const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                        uint64_t root_seed, const int32_t* d_pod_load, uint64_t ready_mask,
                        const aibx_route_params_t* params, uint64_t* d_hashes,
                        uint32_t* d_match_len, uint32_t* d_any_len, uint32_t* d_block_ids,
                        int32_t* d_best_pod, int64_t* d_best_score, uint32_t* d_hashed,
                        uint64_t* d_next_seed, void* stream) {
  AIBX_CALL_RANGE();
  return route_head_impl(ix, d_tokens, d_tok_off, d_blk_off, R, block_tokens, root_seed, d_pod_load,
                         ready_mask, params, d_hashes, d_match_len, d_any_len, d_block_ids,
                         d_best_pod, d_best_score, d_hashed, d_next_seed, stream, 0u);
}

int32_t aibx_route_head_touch(aibx_index_t* ix, const int32_t* d_tokens, const int64_t* d_tok_off,
                              const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                              uint64_t root_seed, const int32_t* d_pod_load, uint64_t ready_mask,
                              const aibx_route_params_t* params, uint32_t epoch,
                              uint64_t* d_hashes, uint32_t* d_match_len, uint32_t* d_any_len,
                              uint32_t* d_block_ids, int32_t* d_best_pod, int64_t* d_best_score,
                              uint32_t* d_hashed, uint64_t* d_next_seed, void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || epoch == 0 || epoch >= (1u << 30) || ix->migrating) return AIBX_ERR_INVALID;
  return route_head_impl(ix, d_tokens, d_tok_off, d_blk_off, R, block_tokens, root_seed, d_pod_load,
                         ready_mask, params, d_hashes, d_match_len, d_any_len, d_block_ids,
                         d_best_pod, d_best_score, d_hashed, d_next_seed, stream, epoch);
}

uint64_t aibx_route_collect_scratch_bytes(uint32_t num_blocks) {
  return aibx_collect_scratch_bytes(num_blocks) + 64;    // the bitmap, then the arrival counter
}

int32_t aibx_route_head_collect(aibx_index_t* ix, const int32_t* d_tokens, const int64_t* d_tok_off,
                                const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                                uint64_t root_seed, const int32_t* d_pod_load, uint64_t ready_mask,
                                const aibx_route_params_t* params, uint32_t epoch,
                                uint64_t* d_hashes, uint32_t* d_match_len, uint32_t* d_any_len,
                                uint32_t* d_block_ids, int32_t* d_best_pod, int64_t* d_best_score,
                                uint32_t* d_hashed, uint64_t* d_next_seed, uint32_t num_blocks,
                                void* d_scratch, uint32_t* d_unique_ids, uint32_t* d_count,
                                void* stream) {
  AIBX_CALL_RANGE();
  if (!ix || epoch >= (1u << 30) || (epoch && ix->migrating)) return AIBX_ERR_INVALID;
  if (!d_count || !d_scratch || (reinterpret_cast<uintptr_t>(d_scratch) & 3)) return AIBX_ERR_INVALID;
  if (R > 0 && (!d_block_ids || !d_unique_ids)) return AIBX_ERR_INVALID;
  cudaStream_t st = as_stream(stream);
  const int spb = block_tokens / 8;
  const bool head_path = block_tokens > 0 && block_tokens % 8 == 0 &&
                         (spb == 1 || spb == 2 || spb == 4 || spb == 8);
  const uint32_t n_words = (num_blocks + 31u) / 32u;
  if (R <= 0 || !head_path || n_words > kCollectSmallWords) {
    // nothing to fuse into (no requests, another block size, a pool too large for one warp to
    // compact): the plain call, then the set from its block ids
    const int32_t rc = route_head_impl(ix, d_tokens, d_tok_off, d_blk_off, R, block_tokens,
                                       root_seed, d_pod_load, ready_mask, params, d_hashes,
                                       d_match_len, d_any_len, d_block_ids, d_best_pod,
                                       d_best_score, d_hashed, d_next_seed, stream, epoch);
    if (rc != AIBX_OK) return rc;
    if (R <= 0) return cudaMemsetAsync(d_count, 0, sizeof(uint32_t), st) == cudaSuccess
                           ? AIBX_OK : AIBX_ERR_CUDA;
    // the list's length, blk_off[R], is read on the device: no host round trip here either
    unsigned int* bitmap = static_cast<unsigned int*>(d_scratch);
    if (num_blocks > 0 &&
        cudaMemsetAsync(bitmap, 0, aibx_collect_scratch_bytes(num_blocks), st) != cudaSuccess)
      return AIBX_ERR_CUDA;
    collect_mark_kernel<<<sm_count() * 8, 256, 0, st>>>(d_block_ids, 0, d_blk_off + R, num_blocks,
                                                        bitmap);
    collect_compact_kernel<<<1, kCollectThreads, 0, st>>>(bitmap, num_blocks, 0, d_blk_off + R,
                                                          d_unique_ids, d_count);
    return launch_status();
  }
  const size_t bitmap_bytes = (size_t)aibx_collect_scratch_bytes(num_blocks);
  if (cudaMemsetAsync(d_scratch, 0, bitmap_bytes + 64, st) != cudaSuccess) return AIBX_ERR_CUDA;
  HeadCollect hc;
  hc.bitmap = static_cast<unsigned int*>(d_scratch);
  hc.arrived = reinterpret_cast<unsigned int*>(static_cast<char*>(d_scratch) + bitmap_bytes);
  hc.unique = d_unique_ids;
  hc.count = d_count;
  hc.num_blocks = num_blocks;
  return route_head_impl(ix, d_tokens, d_tok_off, d_blk_off, R, block_tokens, root_seed, d_pod_load,
                         ready_mask, params, d_hashes, d_match_len, d_any_len, d_block_ids,
                         d_best_pod, d_best_score, d_hashed, d_next_seed, stream, epoch, hc);
}

int32_t aibx_hash_blocks_resume(const int32_t* d_tokens, const int64_t* d_tok_off,
                                const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                                const uint32_t* d_hashed, const uint64_t* d_next_seed,
                                uint64_t* d_hashes, void* stream) {
  AIBX_CALL_RANGE();
  if (R < 0 || block_tokens <= 0 || block_tokens % 8 != 0 || block_tokens > 1024)
    return AIBX_ERR_INVALID;
  if (R == 0) return AIBX_OK;
  if (!d_tokens || !d_tok_off || !d_blk_off || !d_hashed || !d_next_seed || !d_hashes)
    return AIBX_ERR_INVALID;
  prefer_copy_carveout();
  return launch_hash_blocks(d_tokens, d_tok_off, d_blk_off, R, block_tokens, 0, d_hashes,
                            as_stream(stream), d_hashed, d_next_seed);
}

int32_t aibx_route_assign(const uint32_t* d_match_len, const int64_t* d_blk_off, int32_t R,
                          int32_t num_pods, int32_t* d_pod_load, uint64_t ready_mask,
                          const aibx_route_params_t* params, int32_t load_increment,
                          int32_t* d_best_pod, int64_t* d_best_score, void* stream) {
  AIBX_CALL_RANGE();
  if (R < 0 || num_pods < 1 || num_pods > AIBX_MAX_PODS) return AIBX_ERR_INVALID;
  if (R == 0) return AIBX_OK;
  if (!d_match_len || !d_blk_off || !d_pod_load || !d_best_pod || !d_best_score)
    return AIBX_ERR_INVALID;
  aibx_route_params_t prm = {4, 1, 50};
  if (params) prm = *params;
  route_assign_kernel<<<1, 32, 0, as_stream(stream)>>>(
      d_match_len, d_blk_off, R, num_pods, d_pod_load, ready_mask, prm.w_prefix, prm.w_load,
      prm.threshold_pct, load_increment, d_best_pod, d_best_score);
  return launch_status();
}

int32_t aibx_route_score(const uint32_t* d_match_len, const int64_t* d_blk_off, int32_t R,
                         int32_t num_pods, const int32_t* d_pod_load, uint64_t ready_mask,
                         const aibx_route_params_t* params, int32_t* d_best_pod,
                         int64_t* d_best_score, int64_t* d_scores, void* stream) {
  AIBX_CALL_RANGE();
  if (R < 0 || num_pods < 1 || num_pods > AIBX_MAX_PODS) return AIBX_ERR_INVALID;
  if (R == 0) return AIBX_OK;
  if (!d_match_len || !d_blk_off || !d_pod_load || !d_best_pod || !d_best_score)
    return AIBX_ERR_INVALID;
  aibx_route_params_t prm = {4, 1, 50};
  if (params) prm = *params;
  ScoreParams sp = {d_pod_load, ready_mask, prm.w_prefix, prm.w_load, prm.threshold_pct};
  route_score_kernel<<<blocks_for(R, kRouteWarps), kRouteWarps * 32, 0, as_stream(stream)>>>(
      d_match_len, d_blk_off, R, num_pods, sp, d_best_pod, d_best_score, d_scores);
  return launch_status();
}

int32_t aibx_route_policy(int32_t policy, const uint32_t* d_match_len, const int64_t* d_blk_off,
                          int32_t R, int32_t num_pods, const aibx_pod_metrics_t* metrics,
                          const uint64_t* d_draws, uint64_t ready_mask, int32_t threshold_pct,
                          int32_t* d_best_pod, void* stream) {
  AIBX_CALL_RANGE();
  if (R < 0 || num_pods < 1 || num_pods > AIBX_MAX_PODS || policy < AIBX_POLICY_RANDOM ||
      policy > AIBX_POLICY_PREFIX_CACHE_AWARE)
    return AIBX_ERR_INVALID;
  if (R == 0) return AIBX_OK;
  if (!d_best_pod) return AIBX_ERR_INVALID;
  PodMetrics met = {nullptr, nullptr, nullptr, nullptr, nullptr};
  if (policy == AIBX_POLICY_RANDOM) {
    if (!d_draws) return AIBX_ERR_INVALID;
  } else {
    if (!metrics) return AIBX_ERR_INVALID;
    met = PodMetrics{metrics->d_throughput, metrics->d_requests, metrics->d_kv_usage,
                     metrics->d_queue_latency, metrics->d_serve_latency};
    const bool have =
        policy == AIBX_POLICY_THROUGHPUT       ? met.throughput != nullptr
        : policy == AIBX_POLICY_LEAST_KV_CACHE ? met.kv_usage != nullptr
        : policy == AIBX_POLICY_LEAST_LATENCY  ? met.queue_latency && met.serve_latency
                                               : met.requests != nullptr;
    if (!have) return AIBX_ERR_INVALID;
    if (policy == AIBX_POLICY_PREFIX_CACHE_AWARE && (!d_match_len || !d_blk_off))
      return AIBX_ERR_INVALID;
  }
  // one warp per request up to a few waves of the machine, grid-stride beyond
  const int64_t want = blocks_for(R, kRouteWarps);
  const int64_t cap = (int64_t)sm_count() * 16;
  const unsigned int grid = (unsigned int)(want < cap ? want : cap);
  route_policy_kernel<<<grid, kRouteWarps * 32, 0, as_stream(stream)>>>(
      policy, d_match_len, d_blk_off, R, num_pods, met, d_draws, ready_mask, threshold_pct,
      d_best_pod);
  return launch_status();
}

uint64_t aibx_collect_scratch_bytes(uint32_t num_blocks) {
  return 4ULL * (((uint64_t)num_blocks + 31ULL) / 32ULL);
}

int32_t aibx_collect_blocks(const uint32_t* d_block_ids, int64_t n, uint32_t num_blocks,
                            void* d_scratch, uint32_t* d_unique_ids, uint32_t* d_count,
                            void* stream) {
  AIBX_CALL_RANGE();
  if (n < 0 || !d_count) return AIBX_ERR_INVALID;
  if (n > 0 && (!d_block_ids || !d_unique_ids)) return AIBX_ERR_INVALID;
  if (num_blocks > 0 && !d_scratch) return AIBX_ERR_INVALID;
  if (reinterpret_cast<uintptr_t>(d_scratch) & 3) return AIBX_ERR_INVALID;
  cudaStream_t st = as_stream(stream);
  if (n <= kCollectSmallIds && (num_blocks + 31u) / 32u <= kCollectSmallWords) {
    // a list one CTA gets through in a few microseconds: one launch, bitmap in shared memory
    collect_small_kernel<<<1, kCollectThreads, 0, st>>>(d_block_ids, n, num_blocks, d_unique_ids,
                                                        d_count);
    return launch_status();
  }
  unsigned int* bitmap = static_cast<unsigned int*>(d_scratch);
  if (num_blocks > 0 &&
      cudaMemsetAsync(bitmap, 0, aibx_collect_scratch_bytes(num_blocks), st) != cudaSuccess)
    return AIBX_ERR_CUDA;
  if (n > 0)
    collect_mark_kernel<<<blocks_for(n, 256), 256, 0, st>>>(d_block_ids, n, nullptr, num_blocks,
                                                            bitmap);
  collect_compact_kernel<<<1, kCollectThreads, 0, st>>>(bitmap, num_blocks, n, nullptr,
                                                        d_unique_ids, d_count);
  return launch_status();
}

int32_t aibx_collect_blocks_static(const uint32_t* d_block_ids, int64_t n, uint32_t num_blocks,
                                   uint32_t* d_unique_ids, uint32_t* d_count, void* stream) {
  AIBX_CALL_RANGE();
  if (n < 0 || !d_count) return AIBX_ERR_INVALID;
  if (n > 0 && (!d_block_ids || !d_unique_ids)) return AIBX_ERR_INVALID;
  if (num_blocks > kStaticCollectMaxBlocks) return AIBX_ERR_UNSUPPORTED;
  unsigned int* bitmap = static_bitmap_ptr();
  if (!bitmap) return AIBX_ERR_CUDA;
  cudaStream_t st = as_stream(stream);
  // the array still holds the previous call's marks: zero the part this call reads
  if (num_blocks > 0 &&
      cudaMemsetAsync(bitmap, 0, aibx_collect_scratch_bytes(num_blocks), st) != cudaSuccess)
    return AIBX_ERR_CUDA;
  if (n > 0)
    collect_mark_kernel<<<blocks_for(n, 256), 256, 0, st>>>(d_block_ids, n, nullptr, num_blocks,
                                                            bitmap);
  collect_compact_kernel<<<1, kCollectThreads, 0, st>>>(bitmap, num_blocks, n, nullptr,
                                                        d_unique_ids, d_count);
  return launch_status();
}

uint32_t aibx_collect_static_max_blocks(void) { return kStaticCollectMaxBlocks; }

int32_t aibx_kv_gather(const void* d_pool, const aibx_kv_layout_t* layout,
                       const uint32_t* d_block_ids, int64_t n, void* d_buf, void* stream) {
  AIBX_CALL_RANGE();
  return launch_kv_copy(d_pool, layout, d_block_ids, n, d_buf, 0, as_stream(stream));
}

int32_t aibx_kv_scatter(void* d_pool, const aibx_kv_layout_t* layout,
                        const uint32_t* d_block_ids, int64_t n, const void* d_buf,
                        void* stream) {
  AIBX_CALL_RANGE();
  return launch_kv_copy(d_pool, layout, d_block_ids, n, d_buf, 1, as_stream(stream));
}

int32_t aibx_kv_gather_to_host(const void* d_pool, const aibx_kv_layout_t* layout,
                               const uint32_t* d_block_ids, int64_t n, void* d_staging,
                               void* h_buf, void* stream) {
  AIBX_CALL_RANGE();
  if (n > 0 && !h_buf) return AIBX_ERR_INVALID;
  const int32_t rc = launch_kv_copy(d_pool, layout, d_block_ids, n, d_staging, 0, as_stream(stream));
  if (rc != AIBX_OK || n == 0) return rc;
  const size_t bytes = (size_t)n * 2u * layout->num_kv_heads * layout->block_tokens *
                       layout->head_dim * layout->elem_bytes * layout->num_layers;
  if (cudaMemcpyAsync(h_buf, d_staging, bytes, cudaMemcpyDeviceToHost, as_stream(stream)) !=
      cudaSuccess)
    return AIBX_ERR_CUDA;
  return AIBX_OK;
}

int32_t aibx_kv_scatter_from_host(void* d_pool, const aibx_kv_layout_t* layout,
                                  const uint32_t* d_block_ids, int64_t n, void* d_staging,
                                  const void* h_buf, void* stream) {
  AIBX_CALL_RANGE();
  if (!layout || n < 0) return AIBX_ERR_INVALID;
  if (n == 0) return AIBX_OK;
  if (!h_buf || !d_staging) return AIBX_ERR_INVALID;
  if (layout->num_layers <= 0 || layout->num_kv_heads <= 0 || layout->block_tokens <= 0 ||
      layout->head_dim <= 0 || layout->elem_bytes <= 0)
    return AIBX_ERR_INVALID;
  const size_t bytes = (size_t)n * 2u * layout->num_kv_heads * layout->block_tokens *
                       layout->head_dim * layout->elem_bytes * layout->num_layers;
  if (cudaMemcpyAsync(d_staging, h_buf, bytes, cudaMemcpyHostToDevice, as_stream(stream)) !=
      cudaSuccess)
    return AIBX_ERR_CUDA;
  return launch_kv_copy(d_pool, layout, d_block_ids, n, d_staging, 1, as_stream(stream));
}

int32_t aibx_kv_gather_counted(const void* d_pool, const aibx_kv_layout_t* layout,
                               const uint32_t* d_block_ids, int64_t n_max, const uint32_t* d_count,
                               void* d_buf, void* stream) {
  AIBX_CALL_RANGE();
  if (!d_count) return AIBX_ERR_INVALID;
  return launch_kv_copy(d_pool, layout, d_block_ids, n_max, d_buf, 0, as_stream(stream), d_count);
}

int32_t aibx_kv_scatter_counted(void* d_pool, const aibx_kv_layout_t* layout,
                                const uint32_t* d_block_ids, int64_t n_max,
                                const uint32_t* d_count, const void* d_buf, void* stream) {
  AIBX_CALL_RANGE();
  if (!d_count) return AIBX_ERR_INVALID;
  return launch_kv_copy(d_pool, layout, d_block_ids, n_max, d_buf, 1, as_stream(stream), d_count);
}

int32_t aibx_kv_gather_inner(const void* d_pool, const aibx_kv_layout_t* layout, int32_t pool_inner,
                             int32_t buf_inner, const uint32_t* d_block_ids, int64_t n,
                             void* d_buf, void* stream) {
  AIBX_CALL_RANGE();
  return launch_kv_permute(d_pool, layout, pool_inner, buf_inner, d_block_ids, n, d_buf, 0,
                           as_stream(stream));
}

int32_t aibx_kv_scatter_inner(void* d_pool, const aibx_kv_layout_t* layout, int32_t pool_inner,
                              int32_t buf_inner, const uint32_t* d_block_ids, int64_t n,
                              const void* d_buf, void* stream) {
  AIBX_CALL_RANGE();
  return launch_kv_permute(d_pool, layout, pool_inner, buf_inner, d_block_ids, n, d_buf, 1,
                           as_stream(stream));
}

int32_t aibx_kv_set_tuning(int32_t mode, int32_t chunk_bytes, int32_t stages,
                           int32_t ctas_per_sm) {
  std::atomic<unsigned long long>& word = tuning_word();
  unsigned long long seen = word.load(std::memory_order_acquire);
  for (;;) {
    CopyTuning t = unpack_tuning(seen);
    if (mode >= 0) t.mode = mode;
    if (chunk_bytes > 0) t.chunk_bytes = chunk_bytes;
    if (stages > 0) t.stages = stages;
    if (ctas_per_sm > 0) t.ctas_per_sm = ctas_per_sm;
    if (t.mode != 0 && t.mode != 1) return AIBX_ERR_INVALID;
    if (t.chunk_bytes % 16 != 0 || t.chunk_bytes < 1024 || t.chunk_bytes > 65536)
      return AIBX_ERR_INVALID;
    if (t.stages < 2 || t.stages > kMaxStages) return AIBX_ERR_INVALID;
    if (t.ctas_per_sm < 1 || t.ctas_per_sm > 8) return AIBX_ERR_INVALID;
    if ((long long)t.chunk_bytes * t.stages * t.ctas_per_sm > 200 * 1024) return AIBX_ERR_INVALID;
    // the arguments left at "keep" come from the word just read: swap only if it is still that
    if (word.compare_exchange_weak(seen, pack_tuning(t), std::memory_order_acq_rel)) return AIBX_OK;
  }
}

int32_t aibx_kv_get_tuning(int32_t* mode, int32_t* chunk_bytes, int32_t* stages,
                           int32_t* ctas_per_sm, int32_t* lag) {
  const CopyTuning t = copy_tuning();
  if (mode) *mode = t.mode;
  if (chunk_bytes) *chunk_bytes = t.chunk_bytes;
  if (stages) *stages = t.stages;
  if (ctas_per_sm) *ctas_per_sm = t.ctas_per_sm;
  if (lag) *lag = t.lag;
  return AIBX_OK;
}

int32_t aibx_kv_set_inner_engine(int32_t engine) {
  if (engine < 0 || engine > 2) return AIBX_ERR_INVALID;
  permute_engine().store(engine, std::memory_order_relaxed);
  return AIBX_OK;
}

int32_t aibx_kv_set_store_lag(int32_t lag) {
  if (lag < 1 || lag > 4) return AIBX_ERR_INVALID;
  std::atomic<unsigned long long>& word = tuning_word();
  unsigned long long seen = word.load(std::memory_order_acquire);
  for (;;) {
    CopyTuning t = unpack_tuning(seen);
    t.lag = lag;
    if (word.compare_exchange_weak(seen, pack_tuning(t), std::memory_order_acq_rel)) return AIBX_OK;
  }
}

int32_t aibx_selftest_bounded_wait(uint32_t spins, void* stream) {
  AIBX_CALL_RANGE();
  if (spins == 0 || spins > (1u << 20)) return AIBX_ERR_INVALID;
  bounded_wait_probe_kernel<<<1, 32, 0, as_stream(stream)>>>(spins);
  return launch_status();
}

int32_t aibx_status_fetch(void* stream, int32_t* status, int64_t* detail) {
  AIBX_CALL_RANGE();
  StatusRecord* dev = status_ptr();
  if (!dev) return AIBX_ERR_CUDA;
  cudaStream_t st = as_stream(stream);
  StatusRecord host = {0, 0, 0};
  if (cudaMemcpyAsync(&host, dev, sizeof(host), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaMemsetAsync(dev, 0, sizeof(host), st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return AIBX_ERR_CUDA;
  if (status) *status = host.code;
  if (detail) *detail = (int64_t)host.detail;
  return AIBX_OK;
}

const char* aibx_strerror(int32_t status) {
  switch (status) {
    case AIBX_OK: return "ok";
    case AIBX_ERR_INVALID: return "invalid argument";
    case AIBX_ERR_RANGE: return "block id out of range";
    case AIBX_ERR_FULL: return "index full";
    case AIBX_ERR_CUDA: return "CUDA runtime error";
    case AIBX_ERR_UNSUPPORTED: return "unsupported shape";
    case AIBX_ERR_NOMEM: return "out of device memory";
    case AIBX_ERR_TIMEOUT: return "bounded device wait gave up";
    default: return "unknown status";
  }
}

}  // extern "C"
