// Paged-KV gather / scatter: whole (item, segment) runs of bytes moved verbatim between a
// paged pool and a block-major transfer buffer.  A segment is the longest contiguous run both
// sides share: the whole block for a block-major pool, one (layer, K/V) tile for a layer-major
// pool.  Segments are cut into chunks; chunk c goes to CTA c mod grid, so at any moment the
// SMs work on neighbouring addresses.
//
// Two copy engines, same chunk schedule:
//   bulk ring (default): one thread per CTA drives a ring of shared-memory stages with
//       cp.async.bulk (global -> shared, completion on an mbarrier) and cp.async.bulk
//       (shared -> global, bulk groups).  No register or L1 traffic, ~S-1 chunks of loads in
//       flight per SM.  Every wait is bounded and reports AIBX_ERR_TIMEOUT instead of hanging.
//   ld/st loop: 16-byte streaming loads and stores, four in flight per thread.
// Bound: HBM bandwidth, 2 bytes of traffic per byte copied.
#pragma once

#include "aibx_common.cuh"

namespace aibx {

struct CopyPlan {
  const uint32_t* ids;
  char* pool;                 // paged side
  char* buf;                  // contiguous side
  long long n_items;
  long long segs_per_item;
  long long seg_bytes;
  long long pool_item_stride; // bytes between consecutive block ids in the pool
  long long pool_seg_stride;  // bytes between consecutive segments of one block in the pool
  long long chunk_bytes;
  long long chunks_per_seg;
  long long total_chunks;
  uint32_t num_blocks;
  int to_pool;                // 0 gather (pool -> buf), 1 scatter (buf -> pool)
};

struct ChunkAddr {
  const char* src;
  char* dst;
  unsigned int bytes;         // 0: nothing to copy (skipped item)
};

__device__ __forceinline__ ChunkAddr chunk_address(const CopyPlan& pl, long long c) {
  const long long per_item = pl.segs_per_item * pl.chunks_per_seg;
  const long long item = c / per_item;
  const long long rem = c - item * per_item;
  const long long seg = rem / pl.chunks_per_seg;
  const long long k = rem - seg * pl.chunks_per_seg;
  const long long off = k * pl.chunk_bytes;
  const long long len = min(pl.chunk_bytes, pl.seg_bytes - off);
  ChunkAddr a;
  a.src = nullptr;
  a.dst = nullptr;
  a.bytes = 0;
  const uint32_t id = __ldg(pl.ids + item);
  if (id >= pl.num_blocks) {
    // one report per offending item, from the thread that owns its first chunk
    if (id != AIBX_NO_BLOCK && rem == 0) raise_status(AIBX_ERR_RANGE);
    return a;
  }
  char* in_pool = pl.pool + (long long)id * pl.pool_item_stride + seg * pl.pool_seg_stride + off;
  char* in_buf = pl.buf + (item * pl.segs_per_item + seg) * pl.seg_bytes + off;
  a.src = pl.to_pool ? in_buf : in_pool;
  a.dst = pl.to_pool ? in_pool : in_buf;
  a.bytes = (unsigned int)len;
  return a;
}

// ------------------------------------------------------------------------------------------
// bulk-async ring

constexpr int kMaxStages = 16;
constexpr unsigned int kWaitSpins = 1u << 22;   // bounded mbarrier wait (~ seconds at worst)

__device__ __forceinline__ unsigned int smem_u32(const void* p) {
  return (unsigned int)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(unsigned int bar, unsigned int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned int bar, unsigned int bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned int bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned int bar, unsigned int parity) {
  unsigned int ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void bulk_load(unsigned int dst_smem, const void* src, unsigned int bytes,
                                          unsigned int bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst_smem), "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, unsigned int src_smem, unsigned int bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst),
               "r"(src_smem), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_commit() {
  asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void bulk_wait_all() {
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}

// One thread per CTA runs the whole ring.  Stage s holds chunk j with j mod S == s.
//   load(j)  : expect_tx + bulk load into stage, or a bare arrive when the chunk is skipped
//   store(j) : after the stage's barrier flips, bulk store out of it and commit a group
//   refill   : stage of chunk j-1 is loaded with chunk j-1+S once all groups but the newest
//              have finished READING shared memory
__global__ void __launch_bounds__(32, 1) kv_copy_bulk_kernel(CopyPlan pl, int stages) {
  extern __shared__ __align__(128) unsigned char s_mem[];
  __shared__ __align__(8) unsigned long long s_bar[kMaxStages];
  __shared__ char* s_dst[kMaxStages];
  __shared__ unsigned int s_len[kMaxStages];

  if (threadIdx.x != 0) return;

  const long long G = gridDim.x;
  const long long first = blockIdx.x;
  if (first >= pl.total_chunks) return;
  const long long n_my = (pl.total_chunks - first + G - 1) / G;
  const unsigned int stage_bytes = (unsigned int)pl.chunk_bytes;
  const unsigned int smem0 = smem_u32(s_mem);

  for (int s = 0; s < stages; ++s) mbar_init(smem_u32(&s_bar[s]), 1u);
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

  auto load = [&](long long j) {
    const int s = (int)(j % stages);
    const ChunkAddr a = chunk_address(pl, first + j * G);
    s_dst[s] = a.dst;
    s_len[s] = a.bytes;
    const unsigned int bar = smem_u32(&s_bar[s]);
    if (a.bytes) {
      mbar_arrive_expect_tx(bar, a.bytes);
      bulk_load(smem0 + (unsigned int)s * stage_bytes, a.src, a.bytes, bar);
    } else {
      mbar_arrive(bar);
    }
  };

  long long issued = 0;
  for (; issued < n_my && issued < stages; ++issued) load(issued);

  bool timed_out = false;
  for (long long j = 0; j < n_my; ++j) {
    const int s = (int)(j % stages);
    const unsigned int parity = (unsigned int)((j / stages) & 1);
    const unsigned int bar = smem_u32(&s_bar[s]);
    unsigned int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
      if (++spins > kWaitSpins) {
        timed_out = true;
        break;
      }
    }
    if (timed_out) break;
    if (s_len[s]) bulk_store(s_dst[s], smem0 + (unsigned int)s * stage_bytes, s_len[s]);
    bulk_commit();
    if (j >= 1 && issued < n_my) {
      bulk_wait_read<1>();        // store of chunk j-1 no longer reads its stage
      load(issued);
      ++issued;
    }
  }
  bulk_wait_all();
  if (timed_out) {
    // Loads still in flight target this CTA's shared memory: give them a bounded time to
    // land before the CTA retires, then report.
    for (long long j = 0; j < issued; ++j) {
      const int s = (int)(j % stages);
      if (j + stages < issued) continue;      // only the newest phase of each stage
      const unsigned int parity = (unsigned int)((j / stages) & 1);
      unsigned int spins = 0;
      while (!mbar_try_wait(smem_u32(&s_bar[s]), parity) && ++spins < kWaitSpins) {
      }
    }
    raise_status(AIBX_ERR_TIMEOUT);
  }
}

// ------------------------------------------------------------------------------------------
// 16-byte load/store loop

constexpr int kLdstThreads = 256;

__global__ void __launch_bounds__(kLdstThreads) kv_copy_ldst_kernel(CopyPlan pl) {
  __shared__ ChunkAddr s_addr;
  for (long long c = blockIdx.x; c < pl.total_chunks; c += gridDim.x) {
    if (threadIdx.x == 0) s_addr = chunk_address(pl, c);
    __syncthreads();
    const ChunkAddr a = s_addr;
    __syncthreads();
    if (a.bytes == 0) continue;
    const uint4* src = reinterpret_cast<const uint4*>(a.src);
    uint4* dst = reinterpret_cast<uint4*>(a.dst);
    const unsigned int nv = a.bytes >> 4;
    for (unsigned int v = threadIdx.x; v < nv; v += 4 * kLdstThreads) {
      uint4 r0, r1, r2, r3;
      const unsigned int v1 = v + kLdstThreads, v2 = v + 2 * kLdstThreads, v3 = v + 3 * kLdstThreads;
      r0 = __ldcs(src + v);
      if (v1 < nv) r1 = __ldcs(src + v1);
      if (v2 < nv) r2 = __ldcs(src + v2);
      if (v3 < nv) r3 = __ldcs(src + v3);
      __stcs(dst + v, r0);
      if (v1 < nv) __stcs(dst + v1, r1);
      if (v2 < nv) __stcs(dst + v2, r2);
      if (v3 < nv) __stcs(dst + v3, r3);
    }
  }
}

// ------------------------------------------------------------------------------------------
// host side

struct CopyTuning {
  int mode = 0;            // 0 bulk ring, 1 ld/st loop
  int chunk_bytes = 16384;
  int stages = 12;
  int ctas_per_sm = 1;
};

inline CopyTuning& copy_tuning() {
  static CopyTuning t;
  return t;
}

inline int32_t launch_kv_copy(const void* pool, const aibx_kv_layout_t* L, const uint32_t* d_ids,
                              int64_t n, const void* buf, int to_pool, cudaStream_t st) {
  if (!L || n < 0) return AIBX_ERR_INVALID;
  if ((L->layout != 0 && L->layout != 1) || L->num_layers <= 0 || L->num_kv_heads <= 0 ||
      L->block_tokens <= 0 || L->head_dim <= 0 || L->elem_bytes <= 0)
    return AIBX_ERR_INVALID;
  if (n == 0) return AIBX_OK;
  if (!pool || !buf || !d_ids) return AIBX_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(pool) & 15) || (reinterpret_cast<uintptr_t>(buf) & 15))
    return AIBX_ERR_INVALID;
  const long long tile = 2LL * L->num_kv_heads * L->block_tokens * L->head_dim * L->elem_bytes;
  if (tile % 16 != 0) return AIBX_ERR_UNSUPPORTED;
  const long long block_bytes = tile * L->num_layers;

  const CopyTuning& tn = copy_tuning();
  CopyPlan pl;
  pl.ids = d_ids;
  pl.pool = const_cast<char*>(static_cast<const char*>(pool));
  pl.buf = const_cast<char*>(static_cast<const char*>(buf));
  pl.n_items = n;
  pl.num_blocks = L->num_blocks;
  pl.to_pool = to_pool;
  if (L->layout == 0) {
    pl.segs_per_item = 1;
    pl.seg_bytes = block_bytes;
    pl.pool_item_stride = block_bytes;
    pl.pool_seg_stride = 0;
  } else {
    pl.segs_per_item = L->num_layers;
    pl.seg_bytes = tile;
    pl.pool_item_stride = tile;
    pl.pool_seg_stride = (long long)L->num_blocks * tile;
  }
  pl.chunk_bytes = tn.chunk_bytes;
  pl.chunks_per_seg = (pl.seg_bytes + pl.chunk_bytes - 1) / pl.chunk_bytes;
  pl.total_chunks = pl.n_items * pl.segs_per_item * pl.chunks_per_seg;

  long long grid = (long long)sm_count() * (tn.mode == 0 ? tn.ctas_per_sm : 8);
  if (grid > pl.total_chunks) grid = pl.total_chunks;

  if (tn.mode == 0) {
    const size_t smem = (size_t)tn.stages * tn.chunk_bytes;
    static size_t configured[64] = {0};   // per device: the attribute lives in the context
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AIBX_ERR_CUDA;
    if (smem > configured[dev]) {
      if (cudaFuncSetAttribute(kv_copy_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                               (int)smem) != cudaSuccess)
        return AIBX_ERR_CUDA;
      configured[dev] = smem;
    }
    kv_copy_bulk_kernel<<<(unsigned int)grid, 32, smem, st>>>(pl, tn.stages);
  } else {
    kv_copy_ldst_kernel<<<(unsigned int)grid, kLdstThreads, 0, st>>>(pl);
  }
  return launch_status();
}

}  // namespace aibx
