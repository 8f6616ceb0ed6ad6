/*
 * aibxo.h - CPU oracle for the KV-reuse hot path (prefix keys, residency index, longest
 * cached prefix, route score, paged-KV gather/scatter).
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, single-threaded C program that writes
 * out the definitions the GPU library must reproduce bit for bit.  It shares no source,
 * header, table or helper with the CUDA path and must never be reached from the product
 * path: only the tests, the smoke check and the benchmark's CPU-baseline leg call it.
 *
 * The paper (AIBrix, arXiv 2504.03648) gives these operations in prose only (Section 3.2.2
 * routing policies; Section 3.2.5 distributed KV cache pool) and prints no worked value for
 * any of them, so none of the functions below is pinned by the paper itself.  They are
 * pinned instead by: published XXH64 test values and an independent XXH64 library, brute
 * force over tiny inputs, hand-worked examples, algebraic invariants, and special cases that
 * reduce to a library routine (a dict, an index_select).  See tests/test_oracle_*.py.
 *
 * All pointers are HOST memory.  Status codes have the same numeric values as the GPU
 * library's, restated here because the two share no header.
 */
#ifndef AIBXO_H_
#define AIBXO_H_

#include <stddef.h>
#include <stdint.h>

#define AIBXO_OK               0
#define AIBXO_ERR_INVALID     (-1)
#define AIBXO_ERR_RANGE       (-2)
#define AIBXO_ERR_FULL        (-3)
#define AIBXO_ERR_UNSUPPORTED (-5)
#define AIBXO_ERR_NOMEM       (-6)

#define AIBXO_NO_BLOCK 0xFFFFFFFFu
#define AIBXO_NO_POD   (-1)

typedef struct aibxo_index aibxo_index_t;

/* XXH64 of `len` bytes with `seed`, all input lengths (xxHash specification, 64-bit variant). */
uint64_t aibxo_xxh64(const void* data, size_t len, uint64_t seed);

/* Chained per-block prefix keys (Section 3.2.2; hash and block size are this library's
 * reading since the paper fixes neither). */
int32_t aibxo_hash_blocks(const int32_t* tokens, const int64_t* tok_off, const int64_t* blk_off,
                          int32_t R, int32_t block_tokens, uint64_t root_seed, uint64_t* hashes);

/* Residency metadata: key -> (pod mask, block id)  (Sections 3.2.2 / 3.2.5). */
int32_t aibxo_index_create(aibxo_index_t** out, uint64_t capacity, int32_t num_pods);
int32_t aibxo_index_destroy(aibxo_index_t* ix);
int32_t aibxo_index_clear(aibxo_index_t* ix);
int32_t aibxo_index_insert(aibxo_index_t* ix, const uint64_t* keys, const uint64_t* masks,
                           const uint32_t* ids, int64_t n);
int32_t aibxo_index_evict(aibxo_index_t* ix, const uint64_t* keys, const uint64_t* masks,
                          uint32_t* freed, int64_t n);
int32_t aibxo_index_lookup(const aibxo_index_t* ix, const uint64_t* keys, uint64_t* masks,
                           uint32_t* ids, int64_t n);
int32_t aibxo_index_stats(const aibxo_index_t* ix, uint64_t* live, uint64_t* capacity);

/* Operational calls (Section 3.2.5 speaks of metadata that is published and kept up to date;
 * a table that fills up has to be carried over into a larger one).
 * export: all live entries, ascending by key; *count = number of live entries, of which at most
 *         max_entries are written.
 * rehash: change the capacity, keeping every live entry; FULL (and no change) if the live
 *         entries do not fit, INVALID for a capacity that is not a power of two >= 8. */
/* Scan-resistant victim choice (Section 3.2.5 names a scan-resistant eviction policy without
 * giving it; the reading here: an entry touched in fewer than two epochs is "scan-like" and goes
 * before any entry touched in two or more, oldest last touch first).  See aibxo.c. */
int32_t aibxo_index_touch(aibxo_index_t* ix, const uint64_t* keys, int64_t n, uint32_t epoch);
int32_t aibxo_index_pick_victims(const aibxo_index_t* ix, uint64_t k, uint64_t* keys,
                                 uint32_t* priorities, uint64_t* count);
int32_t aibxo_index_export(const aibxo_index_t* ix, uint64_t* keys, uint64_t* masks, uint32_t* ids,
                           uint64_t max_entries, uint64_t* count);
int32_t aibxo_index_rehash(aibxo_index_t* ix, uint64_t new_capacity);

/* Longest cached prefix per request per pod (Section 3.2.2, prefix-cache-aware). */
int32_t aibxo_match_prefix(const aibxo_index_t* ix, const uint64_t* hashes,
                           const int64_t* blk_off, int32_t R, uint32_t* match_len,
                           uint32_t* any_len, uint32_t* block_ids);

/* Integer prefix-and-load score and its argmax (Section 3.2.2, prefix-cache-aware with a
 * hit threshold combined with least-request). */
typedef struct {
  int32_t w_prefix;
  int32_t w_load;
  int32_t threshold_pct;
} aibxo_route_params_t;

int32_t aibxo_route_score(const uint32_t* match_len, const int64_t* blk_off, int32_t R,
                          int32_t num_pods, const int32_t* pod_load, uint64_t ready_mask,
                          const aibxo_route_params_t* params, int32_t* best_pod,
                          int64_t* best_score, int64_t* scores);

/* Sequential assignment (Section 3.2.2, least-request read over a batch: every admitted request
 * raises the chosen instance's count before the next one is routed).  Requests are taken in
 * order; request r is scored against the CURRENT pod_load, and load[best] += load_increment
 * before request r+1.  pod_load is updated in place.  increment 0 equals aibxo_route_score. */
int32_t aibxo_route_assign(const uint32_t* match_len, const int64_t* blk_off, int32_t R,
                           int32_t num_pods, int32_t* pod_load, uint64_t ready_mask,
                           const aibxo_route_params_t* params, int32_t load_increment,
                           int32_t* best_pod, int64_t* best_score);

/* The six per-request routing policies of Section 3.2.2, one pod per request, all requests of a
 * call seeing the same snapshot of the per-pod figures.  Only ready pods (ready_mask bit set,
 * pod < num_pods) can be chosen; with none ready the answer is NO_POD.  Ties go to the lowest
 * pod index.  Readings fixed here:
 *   0 random            : the (draws[r] mod n)-th ready pod in ascending order, n = ready pods;
 *                         the random numbers are an input (draws[R])
 *   1 throughput        : lowest throughput[p]
 *   2 least-request     : lowest requests[p]
 *   3 least-kv-cache    : lowest kv_usage[p]
 *   4 least-latency     : lowest queue_latency[p] + serve_latency[p] (sum taken in int64)
 *   5 prefix-cache-aware: among pods whose hit = match_len[r][p] is > 0 and has
 *                         100*hit >= threshold_pct*n_r, the largest hit, ties to the lowest
 *                         requests[p]; if no pod qualifies, policy 2.
 * Arrays a policy does not read may be NULL. */
typedef struct {
  const int32_t* throughput;
  const int32_t* requests;
  const int32_t* kv_usage;
  const int32_t* queue_latency;
  const int32_t* serve_latency;
} aibxo_pod_metrics_t;

int32_t aibxo_route_policy(int32_t policy, const uint32_t* match_len, const int64_t* blk_off,
                           int32_t R, int32_t num_pods, const aibxo_pod_metrics_t* metrics,
                           const uint64_t* draws, uint64_t ready_mask, int32_t threshold_pct,
                           int32_t* best_pod);

/* Ascending distinct valid block ids, padded with NO_BLOCK; returns RANGE if any id other
 * than NO_BLOCK is >= num_blocks (those are dropped). */
int32_t aibxo_collect_blocks(const uint32_t* block_ids, int64_t n, uint32_t num_blocks,
                             uint32_t* unique_ids, uint32_t* count);

/* Paged-KV gather / scatter (Section 3.2.5 put/get data movement). */
typedef struct {
  int32_t layout; /* 0 [block][layer][K/V]..., 1 [layer][block][K/V]..., 2 [layer][K/V][block]...
                     (K and V of a layer as separate tensors) */
  int32_t num_layers;
  int32_t num_kv_heads;
  int32_t block_tokens;
  int32_t head_dim;
  int32_t elem_bytes;
  uint32_t num_blocks;
} aibxo_kv_layout_t;

/* *bad (nullable) receives the number of skipped out-of-range items. */
int32_t aibxo_kv_gather(const void* pool, const aibxo_kv_layout_t* lay, const uint32_t* ids,
                        int64_t n, void* buf, int64_t* bad);
int32_t aibxo_kv_scatter(void* pool, const aibxo_kv_layout_t* lay, const uint32_t* ids,
                         int64_t n, const void* buf, int64_t* bad);

/* Gather / scatter with a change of the order inside a tile (Section 3.2.5: engines differ in
 * how they store a block, so the exchange buffer may need another order than the pool).
 * inner order 0 = [K/V][head][token][dim], 1 = [K/V][token][head][dim]; rows of head_dim elements
 * move whole.  Equal orders reduce to aibxo_kv_gather / aibxo_kv_scatter. */
int32_t aibxo_kv_gather_inner(const void* pool, const aibxo_kv_layout_t* lay, int32_t pool_inner,
                              int32_t buf_inner, const uint32_t* ids, int64_t n, void* buf,
                              int64_t* bad);
int32_t aibxo_kv_scatter_inner(void* pool, const aibxo_kv_layout_t* lay, int32_t pool_inner,
                               int32_t buf_inner, const uint32_t* ids, int64_t n, const void* buf,
                               int64_t* bad);

#endif /* AIBXO_H_ */
