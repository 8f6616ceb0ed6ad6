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
//
// Two engines write the destination:
//   tensor store (default): the destination side is described by a 4-D tensor map
//       (row, source-inner index, source-outer index, plane) whose strides are those of the
//       DESTINATION order, so one cp.async.bulk.tensor store of a box that lies in shared memory
//       in source order lands every row in its transposed place.  No thread touches the data:
//       a loader warp and a storer thread, as in the plain copy.
//   storer warps (fallback for rows over 2 KiB or when no tensor map can be made): the stage is
//       read back 16 bytes per lane and written with coalesced streaming stores.
#pragma once

#include <cuda.h>

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
  long long pool_kv_stride;      // bytes from the K plane of a tile to its V plane in the pool
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
                     (long long)layer * pl.pool_layer_stride + (long long)kv * pl.pool_kv_stride;
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

// ------------------------------------------------------------------------------------------
// tensor-store engine

// A source plane is [outer a][inner b][row].  A chunk is a box of `box_a` outer x `box_b` inner
// indices (box_b = all of them unless one outer index alone overflows a stage) times `box_w`
// planes (2 = the K and the V plane of one tile, adjacent on both sides, when both fit a stage).
struct TmaPermPlan {
  const uint32_t* ids;
  const char* pool;
  const char* buf;
  long long pool_item_stride;    // bytes between consecutive block ids in the pool
  long long pool_layer_stride;   // bytes between consecutive layers of one block in the pool
  long long pool_kv_stride;      // bytes from the K plane of a tile to its V plane in the pool
  long long pool_item_planes;    // the same three strides in planes (tensor-map coordinate w)
  long long pool_layer_planes;
  long long pool_kv_planes;
  long long plane_bytes;
  unsigned int row_bytes;
  unsigned int num_layers;
  unsigned int inner, outer;     // source order
  unsigned int box_a, box_b, box_w;
  unsigned int chunks_b;         // chunks along the inner index (1 when box_b == inner)
  unsigned int chunks_a;         // chunks along the outer index
  unsigned int total_chunks;
  uint32_t num_blocks;
  int to_pool;
};

struct TmaChunk {
  const char* src0;              // first contiguous run to load (nullptr: skipped)
  const char* src1;              // second plane's run when box_w == 2
  unsigned int bytes;            // per run
  unsigned int plane_stride_smem;  // where the second plane's box starts in the stage
  int y, z, w;                   // destination coordinates (inner index, outer index, plane)
};

__device__ __forceinline__ TmaChunk tma_chunk(const TmaPermPlan& pl, unsigned int c) {
  TmaChunk ch;
  ch.src0 = ch.src1 = nullptr;
  ch.bytes = 0;
  ch.plane_stride_smem = pl.box_a * pl.box_b * pl.row_bytes;
  ch.y = ch.z = ch.w = 0;
  const unsigned int per_group = pl.chunks_a * pl.chunks_b;      // chunks per plane group
  const unsigned int group = c / per_group;                      // plane group: box_w planes
  const unsigned int k = c - group * per_group;
  const unsigned int ka = k / pl.chunks_b;
  const unsigned int kb = k - ka * pl.chunks_b;
  const unsigned int plane = group * pl.box_w;                   // first plane, buffer numbering
  const unsigned int item = plane / (2u * pl.num_layers);
  const unsigned int rem = plane - item * 2u * pl.num_layers;
  const unsigned int layer = rem >> 1;
  const unsigned int kv = rem & 1u;
  const uint32_t id = __ldg(pl.ids + item);
  if (id >= pl.num_blocks) {
    if (id != AIBX_NO_BLOCK && rem == 0 && k == 0) raise_status(AIBX_ERR_RANGE);
    return ch;
  }
  const unsigned int a0 = ka * pl.box_a, b0 = kb * pl.box_b;
  // contiguous source rows of the chunk inside a plane
  const unsigned int rows = pl.box_b == pl.inner ? min(pl.box_a, pl.outer - a0) * pl.inner
                                                 : min(pl.box_b, pl.inner - b0);
  const long long row_off = ((long long)a0 * pl.inner + b0) * pl.row_bytes;
  const long long pool_plane = (long long)id * pl.pool_item_stride +
                               (long long)layer * pl.pool_layer_stride + (long long)kv * pl.pool_kv_stride;
  const long long buf_plane = (long long)plane * pl.plane_bytes;
  const char* src = pl.to_pool ? pl.buf + buf_plane : pl.pool + pool_plane;
  ch.src0 = src + row_off;
  // the second plane of a two-plane box is the V plane of the same tile
  if (pl.box_w == 2) ch.src1 = ch.src0 + (pl.to_pool ? pl.plane_bytes : pl.pool_kv_stride);
  ch.bytes = rows * pl.row_bytes;
  ch.y = (int)b0;
  ch.z = (int)a0;
  ch.w = pl.to_pool ? (int)((long long)id * pl.pool_item_planes +
                            (long long)layer * pl.pool_layer_planes + kv * pl.pool_kv_planes)
                    : (int)plane;
  return ch;
}

__device__ __forceinline__ void tensor_store_4d(const CUtensorMap* map, unsigned int src_smem, int x,
                                                int y, int z, int w) {
  asm volatile(
      "cp.async.bulk.tensor.4d.global.shared::cta.bulk_group [%0, {%1, %2, %3, %4}], [%5];"
      ::"l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(src_smem)
      : "memory");
}

// Roles as in kv_copy_bulk_kernel: warp 0 loads (chunk descriptors 32 at a time, one per lane),
// thread 32 stores.  Every wait is bounded.
__global__ void __launch_bounds__(kRoleThreads, 1)
kv_permute_tma_kernel(const __grid_constant__ CUtensorMap dst_map, TmaPermPlan pl, int stages,
                      unsigned int stage_bytes) {
  extern __shared__ __align__(128) unsigned char s_mem[];
  __shared__ __align__(8) unsigned long long s_full[kMaxStages];
  __shared__ __align__(8) unsigned long long s_empty[kMaxStages];
  __shared__ int s_y[kMaxStages], s_z[kMaxStages], s_w[kMaxStages];
  __shared__ unsigned int s_bytes[kMaxStages];
  __shared__ int s_abort;
  __shared__ int s_loader_done;
  __shared__ long long s_issued;

  const unsigned int G = gridDim.x;
  const unsigned int first = blockIdx.x;
  if (first >= pl.total_chunks) return;
  const long long n_my = (pl.total_chunks - first + G - 1) / G;
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
    const int lane = threadIdx.x;
    bool stop = false;
    for (long long base = 0; base < n_my && !stop; base += 32) {
      const long long j = base + lane;
      TmaChunk ch;
      ch.src0 = ch.src1 = nullptr;
      ch.bytes = 0;
      ch.plane_stride_smem = 0;
      ch.y = ch.z = ch.w = 0;
      if (j < n_my) ch = tma_chunk(pl, first + (unsigned int)j * G);
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
            const unsigned int stage0 = smem0 + (unsigned int)s * stage_bytes;
            const unsigned int bar = smem_u32(&s_full[s]);
            s_y[s] = ch.y;
            s_z[s] = ch.z;
            s_w[s] = ch.w;
            s_bytes[s] = ch.src0 ? ch.bytes : 0u;
            *reinterpret_cast<volatile long long*>(&s_issued) = j + 1;
            if (ch.src0) {
              mbar_arrive_expect_tx(bar, ch.src1 ? 2u * ch.bytes : ch.bytes);
              bulk_load(stage0, ch.src0, ch.bytes, bar);
              if (ch.src1) bulk_load(stage0 + ch.plane_stride_smem, ch.src1, ch.bytes, bar);
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
    long long j = 0;
    bool gave_up = false;
    for (; j < n_my; ++j) {
      const int s = (int)(j % stages);
      if (!bounded_wait(smem_u32(&s_full[s]), (unsigned int)((j / stages) & 1), abort_flag)) {
        gave_up = true;
        break;
      }
      // rows of a partial box that were not loaded lie beyond the tensor's extent in their
      // dimension, where a tensor store writes nothing
      if (s_bytes[s])
        tensor_store_4d(&dst_map, smem0 + (unsigned int)s * stage_bytes, 0, s_y[s], s_z[s], s_w[s]);
      bulk_commit();
      if (j >= 1) {
        bulk_wait_read<1>();
        mbar_arrive(smem_u32(&s_empty[(int)((j - 1) % stages)]));
      }
    }
    bulk_wait_all();
    if (gave_up) {
      if (!*abort_flag) raise_status(AIBX_ERR_TIMEOUT);
      *abort_flag = 1;
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

// cuTensorMapEncodeTiled through the runtime's entry-point lookup (no link against libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
    else
      cudaGetLastError();
  });
  return fn;
}

// Byte strides of a pool: from block to block, from layer to layer, from the K plane of a tile
// to its V plane.
inline void pool_strides(const aibx_kv_layout_t* L, long long tile, long long plane,
                         long long& item, long long& layer, long long& kv) {
  if (L->layout == 0) {            // [block][layer][K/V]...
    item = tile * L->num_layers;
    layer = tile;
    kv = plane;
  } else if (L->layout == 1) {     // [layer][block][K/V]...
    item = tile;
    layer = (long long)L->num_blocks * tile;
    kv = plane;
  } else {                         // [layer][K/V][block]...
    item = plane;
    layer = 2LL * L->num_blocks * plane;
    kv = (long long)L->num_blocks * plane;
  }
}

inline std::atomic<int>& permute_engine() {
  static std::atomic<int> engine{0};   // 0 tensor store where the shape allows it, 1 storer
                                       // warps, 2 tensor store or UNSUPPORTED
  return engine;
}

// Returns AIBX_ERR_UNSUPPORTED when this engine cannot take the shape (the caller then uses the
// storer-warp kernel), another code on a real error.
inline int32_t launch_kv_permute_tma(const void* pool, const aibx_kv_layout_t* L, int src_order,
                                     const uint32_t* d_ids, int64_t n, const void* buf, int to_pool,
                                     cudaStream_t st) {
  constexpr long long kStageBytes = 32768;
  constexpr int kStages = 3;
  const long long row_bytes = (long long)L->head_dim * L->elem_bytes;
  const long long inner = src_order == 0 ? L->block_tokens : L->num_kv_heads;
  const long long outer = src_order == 0 ? L->num_kv_heads : L->block_tokens;
  const long long plane = inner * outer * row_bytes;
  const long long tile = 2 * plane;
  if (row_bytes % 16 != 0 || row_bytes > 2048) return AIBX_ERR_UNSUPPORTED;   // box row <= 256 x 8 B
  EncodeTiledFn encode = encode_tiled_fn();
  if (!encode) return AIBX_ERR_UNSUPPORTED;

  TmaPermPlan pl;
  const long long stage_rows = kStageBytes / row_bytes;
  long long box_b = inner < stage_rows ? inner : stage_rows;
  if (box_b > 256) box_b = 256;
  long long box_a = 1;
  if (box_b == inner) {
    box_a = stage_rows / inner;
    if (box_a > outer) box_a = outer;
    if (box_a > 256) box_a = 256;
    if (box_a < 1) box_a = 1;
  }
  // two planes per box (K and V of a tile) only where the DESTINATION keeps them adjacent: the
  // buffer always does, a pool with separate K and V tensors does not
  const bool dst_kv_adjacent = !(to_pool && L->layout == 2);
  const long long box_w =
      (box_a == outer && box_b == inner && 2 * plane <= kStageBytes && dst_kv_adjacent) ? 2 : 1;
  pl.ids = d_ids;
  pl.pool = static_cast<const char*>(pool);
  pl.buf = static_cast<const char*>(buf);
  pool_strides(L, tile, plane, pl.pool_item_stride, pl.pool_layer_stride, pl.pool_kv_stride);
  pl.pool_item_planes = pl.pool_item_stride / plane;
  pl.pool_layer_planes = pl.pool_layer_stride / plane;
  pl.pool_kv_planes = pl.pool_kv_stride / plane;
  pl.plane_bytes = plane;
  pl.row_bytes = (unsigned int)row_bytes;
  pl.num_layers = (unsigned int)L->num_layers;
  pl.inner = (unsigned int)inner;
  pl.outer = (unsigned int)outer;
  pl.box_a = (unsigned int)box_a;
  pl.box_b = (unsigned int)box_b;
  pl.box_w = (unsigned int)box_w;
  pl.chunks_b = (unsigned int)((inner + box_b - 1) / box_b);
  pl.chunks_a = (unsigned int)((outer + box_a - 1) / box_a);
  const long long groups = n * 2 * L->num_layers / box_w;
  const long long total = groups * pl.chunks_a * pl.chunks_b;
  const long long dst_planes = to_pool ? 2LL * L->num_layers * L->num_blocks : 2LL * L->num_layers * n;
  if (total >= (1LL << 31) || dst_planes >= (1LL << 31)) return AIBX_ERR_UNSUPPORTED;
  pl.total_chunks = (unsigned int)total;
  pl.num_blocks = L->num_blocks;
  pl.to_pool = to_pool;

  // Destination as (row in 8-byte words, source-inner b, source-outer a, plane): the destination
  // keeps a plane as [b][a][row], so b strides over `outer` rows and a over one.
  alignas(64) CUtensorMap map;
  const cuuint64_t dims[4] = {(cuuint64_t)(row_bytes / 8), (cuuint64_t)inner, (cuuint64_t)outer,
                              (cuuint64_t)dst_planes};
  const cuuint64_t strides[3] = {(cuuint64_t)(outer * row_bytes), (cuuint64_t)row_bytes,
                                 (cuuint64_t)plane};
  const cuuint32_t box[4] = {(cuuint32_t)(row_bytes / 8), (cuuint32_t)box_b, (cuuint32_t)box_a,
                             (cuuint32_t)box_w};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  void* dst_base = const_cast<void*>(to_pool ? pool : buf);
  if (encode(&map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 4, dst_base, dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE,
             CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return AIBX_ERR_UNSUPPORTED;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AIBX_ERR_CUDA;
  const size_t smem = (size_t)kStages * kStageBytes;
  static size_t configured[64] = {0};
  static std::mutex lock;
  if (!ensure_dynamic_smem(kv_permute_tma_kernel, smem, dev, configured, lock)) return AIBX_ERR_CUDA;
  long long grid = sm_count();
  if (grid > total) grid = total;
  kv_permute_tma_kernel<<<(unsigned int)grid, kRoleThreads, smem, st>>>(map, pl, kStages,
                                                                        (unsigned int)kStageBytes);
  return launch_status();
}

inline int32_t launch_kv_permute(const void* pool, const aibx_kv_layout_t* L, int32_t pool_inner,
                                 int32_t buf_inner, const uint32_t* d_ids, int64_t n,
                                 const void* buf, int to_pool, cudaStream_t st) {
  if (!L || n < 0) return AIBX_ERR_INVALID;
  if (L->layout < 0 || L->layout > 2 || L->num_layers <= 0 || L->num_kv_heads <= 0 ||
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

  const int src_order = to_pool ? buf_inner : pool_inner;     // 0: [head][token], 1: [token][head]
  const int engine = permute_engine().load(std::memory_order_relaxed);   // one read per call
  if (engine != 1) {
    const int32_t rc = launch_kv_permute_tma(pool, L, src_order, d_ids, n, buf, to_pool, st);
    if (rc != AIBX_ERR_UNSUPPORTED || engine == 2) return rc;
  }

  constexpr long long kStageBytes = 32768;
  constexpr int kStages = 3;
  if (row_bytes > kStageBytes) return AIBX_ERR_UNSUPPORTED;
  PermPlan pl;
  pl.ids = d_ids;
  pl.pool = const_cast<char*>(static_cast<const char*>(pool));
  pl.buf = const_cast<char*>(static_cast<const char*>(buf));
  pool_strides(L, tile, plane, pl.pool_item_stride, pl.pool_layer_stride, pl.pool_kv_stride);
  pl.plane_bytes = plane;
  pl.num_layers = (unsigned int)L->num_layers;
  pl.rows_per_plane = (unsigned int)rows;
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
  static size_t configured[64] = {0};
  static std::mutex lock;
  if (!ensure_dynamic_smem(kv_permute_kernel, smem, dev, configured, lock)) return AIBX_ERR_CUDA;
  long long grid = sm_count();
  if (grid > total) grid = total;
  kv_permute_kernel<<<(unsigned int)grid, kPermThreads, smem, st>>>(pl, kStages,
                                                                    (unsigned int)kStageBytes);
  return launch_status();
}

}  // namespace aibx
