// Paged-KV gather / scatter: bytes moved verbatim between a paged pool and a block-major
// transfer buffer.
//
// The buffer side of a call is one contiguous byte stream (item 0 layer 0, item 0 layer 1, ...).
// It is cut into fixed-size chunks; chunk c goes to CTA c mod grid, so at any moment the SMs
// work on neighbouring addresses.  On the pool side a chunk is 1..4 "pieces": runs inside one
// segment, where a segment is the longest contiguous run both sides share (the whole block for
// a block-major pool, one layer's K/V tile for a layer-major pool, the K or the V half of it for
// a pool that keeps K and V of a layer as separate tensors).  Cutting the stream rather
// than the segments keeps every iteration at full size whatever the tile size is.
//
// Two copy engines, same chunk schedule:
//   bulk ring (default): a loader thread and a storer thread per CTA drive a ring of
//       shared-memory stages with cp.async.bulk (global -> shared, completion on an mbarrier)
//       and cp.async.bulk (shared -> global, bulk groups).  No register or L1 traffic.  The
//       block ids of the next chunk are requested one iteration early so the issue loop never
//       waits for them.  Every wait is bounded and reports AIBX_ERR_TIMEOUT instead of hanging.
//   ld/st loop: 16-byte streaming loads and stores, four in flight per thread.
// Bound: HBM bandwidth, 2 bytes of traffic per byte copied.
#pragma once

#include "aibx_common.cuh"

namespace aibx {

constexpr int kMaxPieces = 4;

// All sizes below are in units of 16 bytes so that they fit 32-bit arithmetic.
struct CopyPlan {
  const uint32_t* ids;
  char* pool;                    // paged side
  char* buf;                     // contiguous side
  long long pool_item_stride;    // bytes between consecutive block ids in the pool
  long long pool_seg_stride;     // bytes between consecutive segments of one block in the pool
  unsigned int segs_per_item;
  unsigned int seg_units;        // segment length
  unsigned int chunk_units;      // chunk length (a whole number of segments when shorter)
  unsigned int total_units;      // whole stream of this launch (< 2^32 - 2^22)
  unsigned int total_chunks;
  uint32_t num_blocks;
  int to_pool;                   // 0 gather (pool -> buf), 1 scatter (buf -> pool)
  const uint32_t* d_count;       // optional: number of leading items to move, read on the device
  unsigned int count_base;       // items of earlier launches of the same call
  unsigned int units_per_item;
};

// With a device-side count the stream ends after min(items of this launch, *d_count - base).
__device__ __forceinline__ void apply_device_count(CopyPlan& pl) {
  if (pl.d_count == nullptr) return;
  const unsigned int cnt = __ldg(pl.d_count);
  const unsigned int mine = cnt > pl.count_base ? cnt - pl.count_base : 0u;
  const unsigned long long units = (unsigned long long)mine * pl.units_per_item;
  if (units < pl.total_units) {
    pl.total_units = (unsigned int)units;
    pl.total_chunks = (pl.total_units + pl.chunk_units - 1) / pl.chunk_units;
  }
}

// A chunk before its block ids are known: where its pieces lie in the stream.
struct ChunkPieces {
  int np;
  unsigned int item[kMaxPieces];
  unsigned int seg[kMaxPieces];
  unsigned int off[kMaxPieces];        // offset inside the segment
  unsigned int len[kMaxPieces];
  unsigned int stream0;                // first unit of the chunk in the stream
};

__device__ __forceinline__ void chunk_pieces(const CopyPlan& pl, unsigned int c, ChunkPieces& cp) {
  unsigned int u0 = c * pl.chunk_units;
  const unsigned int u1 = min(u0 + pl.chunk_units, pl.total_units);
  unsigned int q = u0 / pl.seg_units;                 // flat segment index
  unsigned int off = u0 - q * pl.seg_units;
  cp.stream0 = u0;
  cp.np = 0;
#pragma unroll
  for (int p = 0; p < kMaxPieces; ++p) {
    cp.len[p] = 0;
    if (u0 < u1) {
      const unsigned int len = min(pl.seg_units - off, u1 - u0);
      const unsigned int item = q / pl.segs_per_item;
      cp.item[p] = item;
      cp.seg[p] = q - item * pl.segs_per_item;
      cp.off[p] = off;
      cp.len[p] = len;
      cp.np = p + 1;
      u0 += len;
      ++q;
      off = 0;
    }
  }
}

// Pool-side address of piece p, or nullptr when its block id says "skip".
__device__ __forceinline__ char* piece_pool_ptr(const CopyPlan& pl, const ChunkPieces& cp, int p,
                                                uint32_t id) {
  if (id >= pl.num_blocks) {
    // one report per offending item, from the piece that starts the item
    if (id != AIBX_NO_BLOCK && cp.seg[p] == 0 && cp.off[p] == 0) raise_status(AIBX_ERR_RANGE);
    return nullptr;
  }
  return pl.pool + (long long)id * pl.pool_item_stride +
         (long long)cp.seg[p] * pl.pool_seg_stride + (long long)cp.off[p] * 16;
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

// Two threads per CTA run the ring, one per warp, so that neither waits for the other's
// instruction latency.  Stage s holds chunk j with j mod S == s.
//   loader (warp 0): waits until the stage is free (empty barrier), then expect_tx + one bulk
//       load per piece, or a bare arrive when all pieces are skipped.  It also writes where the
//       pieces have to go; the arrive on the full barrier publishes that to the storer.
//   storer (warp 1): waits for the full barrier, issues one bulk store per piece, commits a
//       group, and once the group of `lag` iterations ago has finished READING shared memory
//       hands that stage back through its empty barrier.
// Loads in flight are bounded by the number of stages: that is the knob that keeps the bytes in
// flight near the bandwidth-delay product (more than that lowers the achieved bandwidth).
// Every wait is bounded; whoever gives up raises the abort flag so the other side stops too,
// and the storer waits (bounded) for the loads already issued before the CTA retires.
constexpr int kRoleThreads = 64;

__device__ __forceinline__ bool bounded_wait(unsigned int bar, unsigned int parity,
                                             volatile int* abort_flag) {
  unsigned int spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (++spins > kWaitSpins || ((spins & 1023u) == 0 && *abort_flag)) return false;
  }
  return true;
}

__global__ void __launch_bounds__(kRoleThreads, 1)
kv_copy_bulk_kernel(CopyPlan pl, int stages, int lag) {
  extern __shared__ __align__(128) unsigned char s_mem[];
  __shared__ __align__(8) unsigned long long s_full[kMaxStages];
  __shared__ __align__(8) unsigned long long s_empty[kMaxStages];
  __shared__ char* s_out[kMaxStages][kMaxPieces];          // store destination of each piece
  __shared__ unsigned int s_off[kMaxStages][kMaxPieces];   // its byte offset inside the stage
  __shared__ unsigned int s_len[kMaxStages][kMaxPieces];   // its bytes (0: skipped)
  __shared__ int s_abort;
  __shared__ int s_loader_done;
  __shared__ long long s_issued;

  apply_device_count(pl);
  const unsigned int G = gridDim.x;
  const unsigned int first = blockIdx.x;
  if (first >= pl.total_chunks) return;
  const long long n_my = (pl.total_chunks - first + G - 1) / G;
  const unsigned int stage_bytes = pl.chunk_units * 16u;
  const unsigned int smem0 = smem_u32(s_mem);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&s_full[s]), 1u);
      mbar_init(smem_u32(&s_empty[s]), 1u);
    }
    s_abort = 0;
    s_loader_done = 0;
    s_issued = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  volatile int* abort_flag = &s_abort;

  if (threadIdx.x < 32) {
    // ------------------------------------------------------------------ loader warp
    // A lone thread runs at a fraction of an instruction per cycle, so the address work is
    // done 32 chunks at a time, one chunk per lane; only the few instructions that arm the
    // barrier and start the copies are taken in turn, in chunk order.
    const int lane = threadIdx.x;
    bool stop = false;
    for (long long base = 0; base < n_my && !stop; base += 32) {
      const long long j = base + lane;
      const char* src[kMaxPieces];
      char* out[kMaxPieces];
      unsigned int offs[kMaxPieces], lens[kMaxPieces];
      unsigned int total = 0;
      if (j < n_my) {
        ChunkPieces cp;
        chunk_pieces(pl, first + (unsigned int)j * G, cp);
        char* buf_at = pl.buf + (long long)cp.stream0 * 16;
        unsigned int soff = 0;
#pragma unroll
        for (int p = 0; p < kMaxPieces; ++p) {
          src[p] = nullptr;
          out[p] = nullptr;
          offs[p] = soff;
          lens[p] = 0;
          if (p < cp.np) {
            char* in_pool = piece_pool_ptr(pl, cp, p, __ldg(pl.ids + cp.item[p]));
            if (in_pool) {
              lens[p] = cp.len[p] * 16u;
              src[p] = pl.to_pool ? buf_at + soff : in_pool;
              out[p] = pl.to_pool ? in_pool : buf_at + soff;
            }
            soff += cp.len[p] * 16u;
          }
          total += lens[p];
        }
      }
      const int turns = (int)min((long long)32, n_my - base);
      for (int i = 0; i < turns; ++i) {
        if (lane == i) {
          const int s = (int)(j % stages);
          bool ok = !*abort_flag;
          if (ok && j >= stages) {
            // the storer frees stage s once the store of chunk j - stages left shared memory
            ok = bounded_wait(smem_u32(&s_empty[s]), (unsigned int)(((j / stages) - 1) & 1),
                              abort_flag);
            if (!ok && !*abort_flag) raise_status(AIBX_ERR_TIMEOUT);
          }
          if (ok) {
            const unsigned int stage0 = smem0 + (unsigned int)s * stage_bytes;
            const unsigned int bar = smem_u32(&s_full[s]);
#pragma unroll
            for (int p = 0; p < kMaxPieces; ++p) {
              s_out[s][p] = out[p];
              s_off[s][p] = offs[p];
              s_len[s][p] = lens[p];
            }
            *reinterpret_cast<volatile long long*>(&s_issued) = j + 1;
            if (total) {
              mbar_arrive_expect_tx(bar, total);
#pragma unroll
              for (int p = 0; p < kMaxPieces; ++p)
                if (lens[p]) bulk_load(stage0 + offs[p], src[p], lens[p], bar);
            } else {
              mbar_arrive(bar);
            }
          } else {
            *abort_flag = 1;
          }
        }
        __syncwarp();
        if (*abort_flag) {
          stop = true;
          break;
        }
      }
    }
    if (lane == 0) *reinterpret_cast<volatile int*>(&s_loader_done) = 1;
  } else if (threadIdx.x == 32) {
    // ------------------------------------------------------------------ storer
    if (lag < 1) lag = 1;
    if (lag > stages - 1) lag = stages - 1;
    if (lag > 4) lag = 4;
    long long j = 0;
    bool gave_up = false;
    for (; j < n_my; ++j) {
      const int s = (int)(j % stages);
      if (!bounded_wait(smem_u32(&s_full[s]), (unsigned int)((j / stages) & 1), abort_flag)) {
        gave_up = true;
        break;
      }
      const unsigned int stage0 = smem0 + (unsigned int)s * stage_bytes;
#pragma unroll
      for (int p = 0; p < kMaxPieces; ++p) {
        const unsigned int bytes = s_len[s][p];
        if (bytes) bulk_store(s_out[s][p], stage0 + s_off[s][p], bytes);
      }
      bulk_commit();
      if (j >= lag) {
        // all groups but the newest `lag` have finished reading: chunk j - lag's stage is free
        if (lag >= 4) bulk_wait_read<4>();
        else if (lag == 3) bulk_wait_read<3>();
        else if (lag == 2) bulk_wait_read<2>();
        else bulk_wait_read<1>();
        mbar_arrive(smem_u32(&s_empty[(int)((j - lag) % stages)]));
      }
    }
    bulk_wait_all();
    if (gave_up) {
      if (!*abort_flag) raise_status(AIBX_ERR_TIMEOUT);
      *abort_flag = 1;
      // Loads already issued still target this CTA's shared memory: once the loader has
      // stopped, give them a bounded time to land before the CTA retires.
      for (unsigned int spins = 0;
           !*reinterpret_cast<volatile int*>(&s_loader_done) && spins < kWaitSpins; ++spins) {
      }
      const long long issued = *reinterpret_cast<volatile long long*>(&s_issued);
      for (long long i = j; i < issued; ++i) {
        unsigned int spins = 0;
        while (!mbar_try_wait(smem_u32(&s_full[(int)(i % stages)]),
                              (unsigned int)((i / stages) & 1)) &&
               ++spins < kWaitSpins) {
        }
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// 16-byte load/store loop

constexpr int kLdstThreads = 256;

__global__ void __launch_bounds__(kLdstThreads) kv_copy_ldst_kernel(CopyPlan pl) {
  __shared__ const char* s_src[kMaxPieces];
  __shared__ char* s_dst[kMaxPieces];
  __shared__ unsigned int s_units[kMaxPieces];
  apply_device_count(pl);
  for (unsigned int c = blockIdx.x; c < pl.total_chunks; c += gridDim.x) {
    if (threadIdx.x == 0) {
      ChunkPieces cp;
      chunk_pieces(pl, c, cp);
      char* buf_at = pl.buf + (long long)cp.stream0 * 16;
      unsigned int soff = 0;
      for (int p = 0; p < kMaxPieces; ++p) {
        s_units[p] = 0;
        if (p < cp.np) {
          char* in_pool = piece_pool_ptr(pl, cp, p, __ldg(pl.ids + cp.item[p]));
          if (in_pool) {
            s_units[p] = cp.len[p];
            s_src[p] = pl.to_pool ? buf_at + soff : in_pool;
            s_dst[p] = pl.to_pool ? in_pool : buf_at + soff;
          }
          soff += cp.len[p] * 16u;
        }
      }
    }
    __syncthreads();
    for (int p = 0; p < kMaxPieces; ++p) {
      const unsigned int nv = s_units[p];
      if (nv == 0) continue;
      const uint4* src = reinterpret_cast<const uint4*>(s_src[p]);
      uint4* dst = reinterpret_cast<uint4*>(s_dst[p]);
      for (unsigned int v = threadIdx.x; v < nv; v += 4 * kLdstThreads) {
        uint4 r0, r1, r2, r3;
        const unsigned int v1 = v + kLdstThreads, v2 = v + 2 * kLdstThreads,
                           v3 = v + 3 * kLdstThreads;
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
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------
// host side

struct CopyTuning {
  int mode = 0;            // 0 bulk ring, 1 ld/st loop
  int chunk_bytes = 32768;
  int stages = 3;
  int ctas_per_sm = 1;
  int lag = 1;             // store groups that may still read shared memory (1..4)
};

// The process-wide launch shape lives in ONE atomic word, so that a call on one host thread
// reads a whole setting while another thread replaces it.
//   bits 0      mode            bits 1..13  chunk_bytes / 16 (64..4096)
//   bits 14..18 stages (2..16)  bits 19..22 CTAs per SM (1..8)     bits 23..25 lag (1..4)
inline unsigned long long pack_tuning(const CopyTuning& t) {
  return (unsigned long long)(t.mode & 1) | ((unsigned long long)(t.chunk_bytes / 16) << 1) |
         ((unsigned long long)t.stages << 14) | ((unsigned long long)t.ctas_per_sm << 19) |
         ((unsigned long long)t.lag << 23);
}

inline CopyTuning unpack_tuning(unsigned long long w) {
  CopyTuning t;
  t.mode = (int)(w & 1);
  t.chunk_bytes = (int)((w >> 1) & 0x1FFF) * 16;
  t.stages = (int)((w >> 14) & 0x1F);
  t.ctas_per_sm = (int)((w >> 19) & 0xF);
  t.lag = (int)((w >> 23) & 0x7);
  return t;
}

inline std::atomic<unsigned long long>& tuning_word() {
  static std::atomic<unsigned long long> w{pack_tuning(CopyTuning())};
  return w;
}

inline CopyTuning copy_tuning() { return unpack_tuning(tuning_word().load(std::memory_order_acquire)); }

inline int32_t launch_kv_copy(const void* pool, const aibx_kv_layout_t* L, const uint32_t* d_ids,
                              int64_t n, const void* buf, int to_pool, cudaStream_t st,
                              const uint32_t* d_count = nullptr) {
  if (!L || n < 0) return AIBX_ERR_INVALID;
  if (L->layout < 0 || L->layout > 2 || L->num_layers <= 0 || L->num_kv_heads <= 0 ||
      L->block_tokens <= 0 || L->head_dim <= 0 || L->elem_bytes <= 0)
    return AIBX_ERR_INVALID;
  if (n == 0) return AIBX_OK;
  if (!pool || !buf || !d_ids) return AIBX_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(pool) & 15) || (reinterpret_cast<uintptr_t>(buf) & 15))
    return AIBX_ERR_INVALID;
  const long long tile = 2LL * L->num_kv_heads * L->block_tokens * L->head_dim * L->elem_bytes;
  const long long half = tile / 2;
  if (tile % 16 != 0 || (L->layout == 2 && half % 16 != 0)) return AIBX_ERR_UNSUPPORTED;
  const long long block_bytes = tile * L->num_layers;
  // the longest run both sides share, how many of them make an item (in buffer order), and where
  // consecutive ones lie in the pool: layout 2 keeps (layer l, K or V) at plane 2l + kv
  const long long seg_bytes = L->layout == 0 ? block_bytes : L->layout == 1 ? tile : half;
  const long long segs = L->layout == 0 ? 1 : L->layout == 1 ? L->num_layers : 2LL * L->num_layers;
  if (seg_bytes / 16 >= (1LL << 31) || block_bytes / 16 >= (1LL << 31)) return AIBX_ERR_UNSUPPORTED;

  const CopyTuning tn = copy_tuning();     // one read: the whole call uses this setting
  CopyPlan pl;
  pl.num_blocks = L->num_blocks;
  pl.to_pool = to_pool;
  pl.segs_per_item = (unsigned int)segs;
  pl.seg_units = (unsigned int)(seg_bytes / 16);
  pl.pool_item_stride = seg_bytes;
  pl.pool_seg_stride = L->layout == 0 ? 0 : (long long)L->num_blocks * seg_bytes;
  // chunk: the tuned size, or a whole number of segments when segments are shorter than that
  if (seg_bytes >= tn.chunk_bytes) {
    pl.chunk_units = (unsigned int)(tn.chunk_bytes / 16);
  } else {
    long long m = tn.chunk_bytes / seg_bytes;
    if (m > kMaxPieces) m = kMaxPieces;
    pl.chunk_units = (unsigned int)(m * pl.seg_units);
  }

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AIBX_ERR_CUDA;
  const size_t smem = (size_t)tn.stages * tn.chunk_bytes;
  if (tn.mode == 0) {
    static size_t configured[64] = {0};
    static std::mutex lock;
    if (!ensure_dynamic_smem(kv_copy_bulk_kernel, smem, dev, configured, lock)) return AIBX_ERR_CUDA;
  }

  // 32-bit stream offsets: one launch covers at most ~64 GiB; longer lists take several
  const long long units_per_item = block_bytes / 16;
  long long max_items = ((1LL << 32) - (1LL << 22)) / units_per_item;
  if (max_items < 1) max_items = 1;
  for (int64_t done = 0; done < n; done += max_items) {
    const long long items = (n - done < max_items) ? (n - done) : max_items;
    pl.ids = d_ids + done;
    pl.pool = const_cast<char*>(static_cast<const char*>(pool));
    pl.buf = const_cast<char*>(static_cast<const char*>(buf)) + done * block_bytes;
    pl.d_count = d_count;
    pl.count_base = (unsigned int)(done > 0xFFFFFFFFLL ? 0xFFFFFFFFLL : done);
    pl.units_per_item = (unsigned int)units_per_item;
    pl.total_units = (unsigned int)(items * units_per_item);
    pl.total_chunks = (pl.total_units + pl.chunk_units - 1) / pl.chunk_units;
    long long grid = (long long)sm_count() * (tn.mode == 0 ? tn.ctas_per_sm : 8);
    if (grid > pl.total_chunks) grid = pl.total_chunks;
    if (tn.mode == 0) {
      kv_copy_bulk_kernel<<<(unsigned int)grid, kRoleThreads, smem, st>>>(pl, tn.stages, tn.lag);
    } else {
      kv_copy_ldst_kernel<<<(unsigned int)grid, kLdstThreads, 0, st>>>(pl);
    }
  }
  return launch_status();
}

}  // namespace aibx
