// Paged-KV gather / scatter with a change of the order inside a tile: the pool keeps a tile as
// [K/V][head][token][dim] and the buffer wants [K/V][token][head][dim], or the other way round.
// Rows of head_dim elements move whole; what changes is where each row goes.
//
// A plane is one (item, layer, K or V): heads x tokens rows, contiguous on both sides.  Planes
// are cut into chunks of whole source rows; chunk c goes to CTA c mod grid.  Per CTA:
//   loader warp : as in the plain copy - chunk descriptors computed 32 at a time, one per lane,
//                 then in chunk order each lane arms the stage's mbarrier and starts one bulk
//                 load (cp.async.bulk) of the contiguous source rows into shared memory;
//   storer warps: wait for the stage, read it back 16 bytes per lane and write every row to its
//                 place in the destination plane with full-line coalesced streaming stores
//                 (consecutive lanes cover a row), then hand the stage back.
// The transposition happens through shared memory, so both the global reads and the global
// writes stay contiguous over at least one row.  Bound: HBM bandwidth.
#pragma once

#include "aibx_common.cuh"
#include "kv_copy.cuh"

namespace aibx {

constexpr int kPermStorerWarps = 8;
constexpr int kPermThreads = 32 + 32 * kPermStorerWarps;

struct PermPlan {
  const uint32_t* ids;
  char* pool;
  char* buf;
  long long pool_item_stride;    // bytes between consecutive block ids in the pool
  long long pool_layer_stride;   // bytes between consecutive layers of one block in the pool
  long long plane_bytes;         // heads * tokens * row_bytes
  unsigned int num_layers;
  unsigned int rows_per_plane;   // heads * tokens
  unsigned int src_inner;        // source rows are [outer][inner]: inner count
  unsigned int src_outer;        // outer count (dest row of (a, b) is b * src_outer + a)
  unsigned int vec_per_row;      // row_bytes / 16
  unsigned int rows_per_chunk;
  unsigned int chunks_per_plane;
  unsigned int total_chunks;
  uint32_t num_blocks;
  int to_pool;
};

struct PermChunk {
  const char* src;          // contiguous source rows (nullptr: skipped)
  char* dst_plane;          // base of the destination plane
  unsigned int row0;        // first source row of the chunk inside its plane
  unsigned int rows;        // 0: nothing to do
};

__device__ __forceinline__ PermChunk perm_chunk(const PermPlan& pl, unsigned int c) {
  PermChunk ch;
  ch.src = nullptr;
  ch.dst_plane = nullptr;
  ch.rows = 0;
  const unsigned int plane = c / pl.chunks_per_plane;
  const unsigned int k = c - plane * pl.chunks_per_plane;
  const unsigned int item = plane / (2u * pl.num_layers);
  const unsigned int rem = plane - item * 2u * pl.num_layers;
  const unsigned int layer = rem >> 1;
  const unsigned int kv = rem & 1u;
  ch.row0 = k * pl.rows_per_chunk;
  const unsigned int rows = min(pl.rows_per_chunk, pl.rows_per_plane - ch.row0);
  const uint32_t id = __ldg(pl.ids + item);
  if (id >= pl.num_blocks) {
    if (id != AIBX_NO_BLOCK && rem == 0 && k == 0) raise_status(AIBX_ERR_RANGE);
    return ch;
  }
  char* pool_plane = pl.pool + (long long)id * pl.pool_item_stride +
                     (long long)layer * pl.pool_layer_stride + (long long)kv * pl.plane_bytes;
  char* buf_plane = pl.buf + (long long)plane * pl.plane_bytes;
  const long long row_bytes = (long long)pl.vec_per_row * 16;
  if (pl.to_pool) {
    ch.src = buf_plane + (long long)ch.row0 * row_bytes;
    ch.dst_plane = pool_plane;
  } else {
    ch.src = pool_plane + (long long)ch.row0 * row_bytes;
    ch.dst_plane = buf_plane;
  }
  ch.rows = rows;
  return ch;
}


__global__ void __launch_bounds__(kPermThreads, 1)
kv_permute_kernel(PermPlan pl, int stages, unsigned int stage_bytes) {
  extern __shared__ __align__(128) unsigned char s_mem[];
  __shared__ __align__(8) unsigned long long s_full[kMaxStages];
  __shared__ __align__(8) unsigned long long s_empty[kMaxStages];
  __shared__ char* s_dst[kMaxStages];
  __shared__ unsigned int s_row0[kMaxStages];
  __shared__ unsigned int s_rows[kMaxStages];
  __shared__ int s_abort;

  const unsigned int G = gridDim.x;
  const unsigned int first = blockIdx.x;
  if (first >= pl.total_chunks) return;
  const long long n_my = (pl.total_chunks - first + G - 1) / G;
  const unsigned int smem0 = smem_u32(s_mem);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&s_full[s]), 1u);
      mbar_init(smem_u32(&s_empty[s]), (unsigned int)kPermStorerWarps);
    }
    s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  volatile int* abort_flag = &s_abort;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x < 32) {
    // ------------------------------------------------------------------ loader warp
    long long issued = 0;
    bool stop = false;
    for (long long base = 0; base < n_my && !stop; base += 32) {
      const long long j = base + lane;
      PermChunk ch;
      ch.src = nullptr;
      ch.dst_plane = nullptr;
      ch.row0 = 0;
      ch.rows = 0;
      if (j < n_my) ch = perm_chunk(pl, first + (unsigned int)j * G);
      const int turns = (int)min((long long)32, n_my - base);
      for (int i = 0; i < turns; ++i) {
        if (lane == i) {
          const int s = (int)(j % stages);
          bool ok = !*abort_flag;
          if (ok && j >= stages) {
            ok = bounded_wait(smem_u32(&s_empty[s]), (unsigned int)(((j / stages) - 1) & 1),
                              abort_flag);
            if (!ok && !*abort_flag) raise_status(AIBX_ERR_TIMEOUT);
          }
          if (ok) {
            s_dst[s] = ch.dst_plane;
            s_row0[s] = ch.row0;
            s_rows[s] = ch.rows;
            const unsigned int bar = smem_u32(&s_full[s]);
            if (ch.rows) {
              const unsigned int bytes = ch.rows * pl.vec_per_row * 16u;
              mbar_arrive_expect_tx(bar, bytes);
              bulk_load(smem0 + (unsigned int)s * stage_bytes, ch.src, bytes, bar);
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
        ++issued;
      }
    }
    if (stop && lane == 0) {
      // loads already started still target this CTA's shared memory: bounded wait for them
      for (long long i = issued > stages ? issued - stages : 0; i < issued; ++i) {
        unsigned int spins = 0;
        while (!mbar_try_wait(smem_u32(&s_full[(int)(i % stages)]),
                              (unsigned int)((i / stages) & 1)) &&
               ++spins < kWaitSpins) {
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ storer warps
    const unsigned int tid = threadIdx.x - 32;
    const unsigned int nthreads = 32 * kPermStorerWarps;
    const unsigned int vpr = pl.vec_per_row;
    for (long long j = 0; j < n_my; ++j) {
      const int s = (int)(j % stages);
      if (!bounded_wait(smem_u32(&s_full[s]), (unsigned int)((j / stages) & 1), abort_flag)) {
        if (!*abort_flag) raise_status(AIBX_ERR_TIMEOUT);
        *abort_flag = 1;
        break;
      }
      const unsigned int rows = s_rows[s];
      if (rows) {
        const uint4* stage = reinterpret_cast<const uint4*>(s_mem + (size_t)s * stage_bytes);
        uint4* dst = reinterpret_cast<uint4*>(s_dst[s]);
        const unsigned int row0 = s_row0[s];
        const unsigned int nvec = rows * vpr;
        if (rows == pl.rows_per_plane) {
          // the whole plane is on chip: walk the DESTINATION in order, so that the CTA's
          // stores of one pass form one contiguous run
          for (unsigned int v = tid; v < nvec; v += nthreads) {
            const unsigned int rd = v / vpr;                     // destination row [b][a]
            const unsigned int col = v - rd * vpr;
            const unsigned int b = rd / pl.src_outer;
            const unsigned int a = rd - b * pl.src_outer;
            const unsigned int rs = a * pl.src_inner + b;        // source row [a][b]
            __stcs(dst + v, stage[(size_t)rs * vpr + col]);
          }
        } else {
          for (unsigned int v = tid; v < nvec; v += nthreads) {
            const unsigned int r_local = v / vpr;
            const unsigned int col = v - r_local * vpr;
            const unsigned int rs = row0 + r_local;              // source row [a][b]
            const unsigned int a = rs / pl.src_inner;
            const unsigned int b = rs - a * pl.src_inner;
            const unsigned int rd = b * pl.src_outer + a;        // destination row [b][a]
            __stcs(dst + (size_t)rd * vpr + col, stage[v]);
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&s_empty[s]));
    }
  }
}

inline int32_t launch_kv_permute(const void* pool, const aibx_kv_layout_t* L, int32_t pool_inner,
                                 int32_t buf_inner, const uint32_t* d_ids, int64_t n,
                                 const void* buf, int to_pool, cudaStream_t st) {
  if (!L || n < 0) return AIBX_ERR_INVALID;
  if ((L->layout != 0 && L->layout != 1) || L->num_layers <= 0 || L->num_kv_heads <= 0 ||
      L->block_tokens <= 0 || L->head_dim <= 0 || L->elem_bytes <= 0)
    return AIBX_ERR_INVALID;
  if ((pool_inner != 0 && pool_inner != 1) || (buf_inner != 0 && buf_inner != 1))
    return AIBX_ERR_INVALID;
  if (pool_inner == buf_inner) return launch_kv_copy(pool, L, d_ids, n, buf, to_pool, st);
  if (n == 0) return AIBX_OK;
  if (!pool || !buf || !d_ids) return AIBX_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(pool) & 15) || (reinterpret_cast<uintptr_t>(buf) & 15))
    return AIBX_ERR_INVALID;
  const long long row_bytes = (long long)L->head_dim * L->elem_bytes;
  if (row_bytes % 16 != 0) return AIBX_ERR_UNSUPPORTED;
  const long long rows = (long long)L->num_kv_heads * L->block_tokens;
  const long long plane = rows * row_bytes;
  const long long tile = 2 * plane;

  constexpr long long kStageBytes = 32768;
  constexpr int kStages = 3;
  if (row_bytes > kStageBytes) return AIBX_ERR_UNSUPPORTED;
  PermPlan pl;
  pl.ids = d_ids;
  pl.pool = const_cast<char*>(static_cast<const char*>(pool));
  pl.buf = const_cast<char*>(static_cast<const char*>(buf));
  pl.pool_item_stride = L->layout == 0 ? tile * L->num_layers : tile;
  pl.pool_layer_stride = L->layout == 0 ? tile : (long long)L->num_blocks * tile;
  pl.plane_bytes = plane;
  pl.num_layers = (unsigned int)L->num_layers;
  pl.rows_per_plane = (unsigned int)rows;
  const int src_order = to_pool ? buf_inner : pool_inner;     // 0: [head][token], 1: [token][head]
  pl.src_inner = (unsigned int)(src_order == 0 ? L->block_tokens : L->num_kv_heads);
  pl.src_outer = (unsigned int)(src_order == 0 ? L->num_kv_heads : L->block_tokens);
  pl.vec_per_row = (unsigned int)(row_bytes / 16);
  long long rpc = kStageBytes / row_bytes;
  if (rpc > rows) rpc = rows;
  pl.rows_per_chunk = (unsigned int)rpc;
  pl.chunks_per_plane = (unsigned int)((rows + rpc - 1) / rpc);
  const long long total = n * 2 * L->num_layers * pl.chunks_per_plane;
  if (total >= (1LL << 31)) return AIBX_ERR_UNSUPPORTED;
  pl.total_chunks = (unsigned int)total;
  pl.num_blocks = L->num_blocks;
  pl.to_pool = to_pool;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AIBX_ERR_CUDA;
  const size_t smem = (size_t)kStages * kStageBytes;
  static bool configured[64] = {false};
  if (!configured[dev]) {
    if (cudaFuncSetAttribute(kv_permute_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
      return AIBX_ERR_CUDA;
    configured[dev] = true;
  }
  long long grid = sm_count();
  if (grid > total) grid = total;
  kv_permute_kernel<<<(unsigned int)grid, kPermThreads, smem, st>>>(pl, kStages,
                                                                    (unsigned int)kStageBytes);
  return launch_status();
}

}  // namespace aibx
