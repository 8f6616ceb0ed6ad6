/*
 * aibx.h - C ABI of libaibx: the data-parallel hot path behind KV-cache reuse in a
 * prefix-aware LLM gateway with a distributed KV cache (AIBrix, arXiv 2504.03648).
 *
 * The paper describes the system in prose only (Section 3.2.2, routing policies, and
 * Section 3.2.5, distributed KV cache pool); it prints no algorithm, hash function, block
 * size or formula.  Each call below cites the passage whose operation it implements and
 * states the concrete reading this library fixes.
 *
 * Conventions
 *   - Every pointer named d_* is DEVICE memory owned by the caller, naturally aligned for its
 *     element type.  KV pool and transfer buffer must be 16-byte aligned.  Pointers named
 *     h_* / plain out-parameters are HOST memory.  No call keeps a caller pointer after it
 *     returns; the only memory the library owns is the index behind aibx_index_t and one
 *     small per-device status record.
 *   - Every call that takes a stream only ENQUEUES work on that stream and returns without
 *     synchronising, except where noted ("syncs").  `stream` is a cudaStream_t passed as
 *     void* so that this header needs no CUDA include (0 = the legacy default stream).
 *   - Return value: an aibx status (0 = AIBX_OK, negative = error) for errors the host can
 *     see (null pointer, negative size, bad layout).  Errors only the device can see (a block
 *     id out of range, a full table) are accumulated in the per-device status record and read
 *     with aibx_status_fetch.  Nothing aborts, throws or traps.
 *   - All arithmetic is integer; results are defined bit-exactly.
 *   - Threads: calls on different indexes, pools and streams may come from different host
 *     threads at any time (the few one-time per-device settings - kernel attributes, the address
 *     of the status record - are made under a lock or as single atomic words).  Calls on one
 *     index are ordered by the caller.
 */
#ifndef AIBX_H_
#define AIBX_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define AIBX_OK               0
#define AIBX_ERR_INVALID     (-1)  /* null pointer, negative count, bad parameter          */
#define AIBX_ERR_RANGE       (-2)  /* a block id >= num_blocks (item skipped)               */
#define AIBX_ERR_FULL        (-3)  /* more live entries than capacity, or no room near home */
#define AIBX_ERR_CUDA        (-4)  /* a CUDA runtime call failed                            */
#define AIBX_ERR_UNSUPPORTED (-5)  /* shape outside what the kernels handle                 */
#define AIBX_ERR_NOMEM       (-6)  /* device allocation failed                              */
#define AIBX_ERR_TIMEOUT     (-7)  /* a bounded in-kernel wait gave up                      */

#define AIBX_NO_BLOCK 0xFFFFFFFFu   /* "no block id": skipped silently by gather/scatter    */
#define AIBX_NO_POD   (-1)
#define AIBX_MAX_PODS 64

typedef struct aibx_index aibx_index_t;   /* opaque; host handle of a device-resident index */

/* ---------------------------------------------------------------------------------------
 * Prefix keys (Section 3.2.2: the gateway analyses the token pattern of each request to find
 * reusable prefix cache).  Reading fixed here: request r with tokens t[0..len_r) has
 * n_r = floor(len_r / block_tokens) keys; key i = XXH64(message, seed) where message is the
 * 4*block_tokens bytes of t[i*B .. (i+1)*B) written as little-endian int32 and seed is key
 * i-1 (root_seed for i = 0).  A trailing partial block has no key.
 *
 *   d_tokens   [tok_off[R]]      int32 token ids of all requests, concatenated
 *   d_tok_off  [R+1]             int64 start of each request in d_tokens (tok_off[0] = 0)
 *   d_blk_off  [R+1]             int64 prefix sum of n_r (blk_off[r+1]-blk_off[r] = n_r)
 *   d_hashes   [blk_off[R]]      out: uint64 keys, request r at [blk_off[r], blk_off[r+1])
 *   block_tokens                 positive multiple of 8 (whole 32-byte stripes), at most 1024
 * Errors: INVALID for null pointers (when R > 0), R < 0 or a bad block_tokens.  R = 0 is a
 * no-op.  The offsets are trusted (they are the caller's own prefix sums).
 */
int32_t aibx_hash_blocks(const int32_t* d_tokens, const int64_t* d_tok_off,
                         const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                         uint64_t root_seed, uint64_t* d_hashes, void* stream);

/* ---------------------------------------------------------------------------------------
 * Prefix/KV-locality metadata (Sections 3.2.2 and 3.2.5: the gateway knows which instance
 * caches which prefix, and the cache publishes metadata updates).  Reading fixed here: a map  key -> (pod_mask != 0, block_id),
 * where bit p of pod_mask says pod p holds the block and block_id names its slot in the KV
 * pool.  Keys 0 and ~0 are reserved: inserting them is a no-op, looking them up misses.
 *
 * create:  allocates a table for up to capacity_slots entries (power of two, >= 8) on the
 *          current device; num_pods in 1..64.  The table is an array of 32-byte sectors probed
 *          linearly: with up to 32 pods a sector holds two entries (key, 32-bit pod mask, block
 *          id: 16 bytes per slot), with more pods one entry (32 bytes per slot); 4 more bytes
 *          per slot hold the eviction stamps.  Syncs.  NOMEM if the allocation fails.  Size it
 *          for a load of about one half (capacity_slots = twice the entries expected).
 * destroy: frees it (syncs the device).     clear: empties it (async on stream).
 */
int32_t aibx_index_create(aibx_index_t** out, uint64_t capacity_slots, int32_t num_pods);
int32_t aibx_index_destroy(aibx_index_t* index);
int32_t aibx_index_clear(aibx_index_t* index, void* stream);

/* insert: for every i < n (order-free): skip if key reserved or (mask & podmask(P)) == 0;
 *         absent key -> create (mask & podmask, id); present -> mask |= ..., id = min(id, new).
 *         AIBX_NO_BLOCK as id means "no id supplied" (identity of min).
 *         Device status FULL (detail = number of entries refused or in excess) when the live
 *         entries would exceed capacity_slots, or when a new key finds no free entry within
 *         4,096 entries of its home sector - no entry is ever placed further away, which bounds
 *         every later probe; tables up to a load of 0.9 stay far below that.  After FULL the index content is unspecified until aibx_index_clear or
 *         aibx_index_rehash.  Entries removed by evict are reused by later inserts that pass
 *         them, but a probe for an absent key only stops at a NEVER-used entry: under steady
 *         publish/expire churn those run out, probes grow towards the 4,096-entry bound, and
 *         the table wants a rehash - aibx_index_stats2 says when.
 * evict:  batch-atomic.  First mask &= ~masks[i] for all present keys; then
 *         freed[i] = id if key i was present and its mask is now 0, else AIBX_NO_BLOCK
 *         (duplicates of a key all report the same value); then entries with mask 0 vanish.
 *         d_freed_block_ids may be null.
 * lookup: d_masks[i], d_block_ids[i] = entry of key i, or (0, AIBX_NO_BLOCK).  Either output
 *         may be null.
 * stats:  live entries and capacity.  Syncs the stream.
 * stats2: the same plus what tells when aibx_index_rehash is due: `removed` = entries freed by
 *         evict and not yet reused (live + removed, not live alone, is what the probe length
 *         follows: rehash once it passes three quarters of capacity_slots), `longest_walk` = the
 *         most sectors any insert has had to visit since the table was created, cleared or
 *         rehashed (1 = every key so far went into its home sector; a healthy table at a load
 *         of one half stays below 20).  Any out-pointer may be null.  Syncs the stream.
 */
int32_t aibx_index_insert(aibx_index_t* index, const uint64_t* d_keys,
                          const uint64_t* d_pod_masks, const uint32_t* d_block_ids,
                          int64_t n, void* stream);
int32_t aibx_index_evict(aibx_index_t* index, const uint64_t* d_keys,
                         const uint64_t* d_pod_masks, uint32_t* d_freed_block_ids,
                         int64_t n, void* stream);
int32_t aibx_index_lookup(const aibx_index_t* index, const uint64_t* d_keys,
                          uint64_t* d_masks, uint32_t* d_block_ids, int64_t n, void* stream);
int32_t aibx_index_stats(const aibx_index_t* index, uint64_t* live, uint64_t* capacity,
                         void* stream);
int32_t aibx_index_stats2(const aibx_index_t* index, uint64_t* live, uint64_t* removed,
                          uint64_t* capacity, uint32_t* longest_walk, void* stream);

/* Scan-resistant victim choice (Section 3.2.5 names a scan-resistant eviction policy without
 * describing it; the reading fixed here).  Every entry remembers the last epoch it was touched in
 * and in how many distinct epochs (saturating at 3); epochs are caller-defined integers in
 * 1..2^30-1, normally increasing (one per routed batch, say).
 * touch: marks the present keys among d_keys as used in `epoch`; several touches of a key in
 *        one epoch count once, so one scan over many blocks leaves each at a single touch.
 *        New entries start untouched; re-inserting an existing key keeps its history.
 * pick_victims: the k live entries of lowest priority, priority = (touched in >= 2 epochs ?
 *        2^30 : 0) + last epoch - entries seen in fewer than two epochs go first, oldest first.
 *        d_keys [k] and d_priorities [k] (either may be null) receive them in no particular order;
 *        *d_count (uint64, device) = min(k, live entries).  Every entry below the threshold
 *        priority is returned; among entries AT the threshold the choice is unspecified.
 *        The caller removes them with aibx_index_evict (mask of all ones).  The first call
 *        allocates 384 KiB of scratch that belongs to the index (NOMEM if that fails).
 */
int32_t aibx_index_touch(aibx_index_t* index, const uint64_t* d_keys, int64_t n, uint32_t epoch,
                         void* stream);
int32_t aibx_index_pick_victims(aibx_index_t* index, uint64_t k, uint64_t* d_keys,
                                uint32_t* d_priorities, uint64_t* d_count, void* stream);

/* export: every live entry (key, pod mask, block id) into caller arrays of max_entries
 *         elements, in no particular order; *d_count (uint64, device) = number of live entries,
 *         which may exceed max_entries (the surplus is counted, not written).  Arrays may be
 *         null to only count.  Async on stream.
 * rehash: move the index into a fresh table of new_capacity slots (power of two >= 8; the same
 *         size is fine), dropping the entries freed by evict on the way, so that probes are
 *         short again; also the way out of a FULL table.  FULL (and no change) if
 *         the live entries do not fit, NOMEM if the new table cannot be allocated.  Syncs the
 *         device; the handle stays valid.
 */
int32_t aibx_index_export(const aibx_index_t* index, uint64_t* d_keys, uint64_t* d_masks,
                          uint32_t* d_block_ids, uint64_t max_entries, uint64_t* d_count,
                          void* stream);
int32_t aibx_index_rehash(aibx_index_t* index, uint64_t new_capacity);

/* The same move without stopping the readers (Section 3.2.5: metadata is updated beside the
 * traffic, not in its way).  _begin allocates the new table and enqueues the move on `stream`,
 * waiting only for that stream (to read the live count), then returns; until _finish the handle
 * keeps answering from the old table, so aibx_index_lookup / aibx_match_prefix / aibx_route_* /
 * aibx_index_export / aibx_index_stats calls on any stream run beside the move and see the
 * content as it was.  Calls that would change the index (insert, evict, clear, touch, rehash)
 * return INVALID between _begin and _finish: nothing is lost, the caller holds them back.
 * _finish waits for the move, switches the handle to the new table and frees the old one (which
 * waits for readers still using it).  Updates enqueued before _begin must be ordered before
 * `stream` by the caller.  Codes of _begin as aibx_index_rehash; INVALID if a move is already
 * under way, for _finish if none is.
 */
int32_t aibx_index_rehash_begin(aibx_index_t* index, uint64_t new_capacity, void* stream);
int32_t aibx_index_rehash_finish(aibx_index_t* index);

/* ---------------------------------------------------------------------------------------
 * Longest cached prefix (Section 3.2.2, policy prefix-cache-aware: how much of a request's
 * prefix each instance can reuse).  For request r and pod p:
 *   match_len[r][p] = max k <= n_r such that every key i < k is in the index with bit p set;
 *   any_len[r]      = max k <= n_r such that every key i < k is in the index at all;
 *   block_ids[j]    = id of key j for blk_off[r] <= j < blk_off[r] + any_len[r],
 *                     AIBX_NO_BLOCK for the rest of the request.
 * Lengths are in blocks.  A prefix is contiguous from block 0: residency after a hole does
 * not count.
 *   d_match_len [R * num_pods] row-major uint32;  d_any_len [R] nullable;
 *   d_block_ids [blk_off[R]] nullable.
 */
int32_t aibx_match_prefix(const aibx_index_t* index, const uint64_t* d_hashes,
                          const int64_t* d_blk_off, int32_t R, uint32_t* d_match_len,
                          uint32_t* d_any_len, uint32_t* d_block_ids, void* stream);

/* The same, and every entry of the matched prefix of every request (blocks below any_len[r])
 * is marked as used in `epoch`, exactly as aibx_index_touch of those keys would (Section 3.2.5,
 * scan-resistant eviction: what routing hits is what is hot).  The stamp is written while the
 * probe still has the entry in hand, so matching and touching cost one pass over the index
 * instead of two.  epoch in 1..2^30-1; INVALID otherwise and while a rehash is under way.
 */
int32_t aibx_match_prefix_touch(aibx_index_t* index, const uint64_t* d_hashes,
                                const int64_t* d_blk_off, int32_t R, uint32_t epoch,
                                uint32_t* d_match_len, uint32_t* d_any_len, uint32_t* d_block_ids,
                                void* stream);

/* ---------------------------------------------------------------------------------------
 * Prefix-and-load route score (Section 3.2.2: prefix-cache-aware prefers instances whose
 * cache hit exceeds a threshold; least-request prefers the lowest number of admitted
 * requests).  Integer reading fixed here, with hit = match_len[r][p], n_r from blk_off:
 *   eff   = hit  if hit > 0 and 100*hit >= threshold_pct*n_r, else 0
 *   score = w_prefix*eff - w_load*load[p]                      (int64)
 *   best_pod[r] = argmax of score over pods with their ready_mask bit set, ties to the lowest
 *   pod; AIBX_NO_POD and INT64_MIN if none is ready.  All requests see the same load snapshot.
 *   d_scores [R * num_pods] nullable (pods that are not ready still get their score there).
 * params == NULL means {4, 1, 50}.
 */
typedef struct {
  int32_t w_prefix;
  int32_t w_load;
  int32_t threshold_pct;
} aibx_route_params_t;

int32_t aibx_route_score(const uint32_t* d_match_len, const int64_t* d_blk_off, int32_t R,
                         int32_t num_pods, const int32_t* d_pod_load, uint64_t ready_mask,
                         const aibx_route_params_t* params, int32_t* d_best_pod,
                         int64_t* d_best_score, int64_t* d_scores, void* stream);

/* ---------------------------------------------------------------------------------------
 * Routing in one call (Section 3.2.2: what the gateway does per pending request - token pattern,
 * cache availability, load - taken for a whole batch).  Same results as aibx_hash_blocks, then
 * aibx_match_prefix, then aibx_route_score with d_scores = NULL, written to the same outputs;
 * two launches instead of three (the score is computed by the match kernel while the request's
 * match lengths are still on chip) and one crossing of this boundary.
 *   d_hashes [blk_off[R]] out; d_match_len [R * num_pods] out; d_any_len, d_block_ids nullable.
 */
int32_t aibx_route_batch(const aibx_index_t* index, const int32_t* d_tokens,
                         const int64_t* d_tok_off, const int64_t* d_blk_off, int32_t R,
                         int32_t block_tokens, uint64_t root_seed, const int32_t* d_pod_load,
                         uint64_t ready_mask, const aibx_route_params_t* params,
                         uint64_t* d_hashes, uint32_t* d_match_len, uint32_t* d_any_len,
                         uint32_t* d_block_ids, int32_t* d_best_pod, int64_t* d_best_score,
                         void* stream);

/* ---------------------------------------------------------------------------------------
 * Routing with the critical path cut short (Section 3.2.2: the routing decision depends on the
 * reusable prefix only; nothing past the first block that no instance caches can change it,
 * while hashing a chain is serial in its length).  aibx_route_head hashes every request only as
 * far as matching needs - it probes the index for each key as it is produced and stops soon
 * after the first block without a live entry - and leaves the rest of the chain to
 * aibx_hash_blocks_resume, which may run on another stream, e.g. beside the KV copies.
 *
 * After aibx_route_head: d_match_len, d_any_len, d_block_ids, d_best_pod, d_best_score hold what
 * aibx_route_batch would have written (same definitions, bit for bit); d_hashes holds the first
 * d_hashed[r] keys of every request, with any_len[r] + 1 <= d_hashed[r] <= n_r (or = n_r);
 * d_next_seed[r] is the key of block d_hashed[r] - 1 (root_seed when d_hashed[r] = 0).  How far
 * past any_len a request was hashed is not specified.
 * After aibx_hash_blocks_resume with that state: d_hashes is complete, as from aibx_hash_blocks.
 *   d_hashed [R] uint32, d_next_seed [R] uint64: out of the first call, in of the second.
 *   d_any_len, d_block_ids nullable; d_best_pod and d_best_score both given (then d_pod_load is
 *   required) or both NULL.  Block sizes other than 8, 16, 32, 64 tokens are hashed in full by
 *   the first call (d_hashed[r] = n_r).
 * Worth it when the cached prefix is a small part of a request (a shared prompt in front of a
 * long unique tail); a batch whose requests are cached almost to the end gains nothing (the
 * hashing inside this call is a little slower per block than aibx_hash_blocks).
 */
int32_t aibx_route_head(const aibx_index_t* index, const int32_t* d_tokens,
                        const int64_t* d_tok_off, const int64_t* d_blk_off, int32_t R,
                        int32_t block_tokens, uint64_t root_seed, const int32_t* d_pod_load,
                        uint64_t ready_mask, const aibx_route_params_t* params,
                        uint64_t* d_hashes, uint32_t* d_match_len, uint32_t* d_any_len,
                        uint32_t* d_block_ids, int32_t* d_best_pod, int64_t* d_best_score,
                        uint32_t* d_hashed, uint64_t* d_next_seed, void* stream);

/* aibx_route_head that also marks the entries of every request's matched prefix as used in
 * `epoch` (see aibx_match_prefix_touch): the prober that has just found an entry stamps it.
 */
int32_t aibx_route_head_touch(aibx_index_t* index, const int32_t* d_tokens,
                              const int64_t* d_tok_off, const int64_t* d_blk_off, int32_t R,
                              int32_t block_tokens, uint64_t root_seed, const int32_t* d_pod_load,
                              uint64_t ready_mask, const aibx_route_params_t* params,
                              uint32_t epoch, uint64_t* d_hashes, uint32_t* d_match_len,
                              uint32_t* d_any_len, uint32_t* d_block_ids, int32_t* d_best_pod,
                              int64_t* d_best_score, uint32_t* d_hashed, uint64_t* d_next_seed,
                              void* stream);
/* aibx_route_head that also makes the set of matched blocks (what aibx_collect_blocks gives for
 * d_block_ids: ascending distinct valid ids of all matched prefixes in d_unique_ids [blk_off[R]],
 * padded with AIBX_NO_BLOCK, their number in *d_count) without a further launch: the probers
 * mark the ids in a bitmap and the last one to finish turns it into the list, so the copies can
 * follow the routing kernel directly (Section 3.2.5: a block shared by several requests moves
 * once).  epoch = 0: no stamping; otherwise as aibx_route_head_touch.  d_scratch: device memory
 * of aibx_route_collect_scratch_bytes(num_blocks) bytes, 4-byte aligned, contents irrelevant
 * (cleared by the call).  d_block_ids is required.  Pools of more than 262,144 blocks and block
 * sizes other than 8, 16, 32, 64 tokens take the routing call followed by the collect kernels
 * (same results; the list length is read on the device, so there is still no host round trip).
 * Ids >= num_blocks other than AIBX_NO_BLOCK raise device status RANGE and are left out.
 */
uint64_t aibx_route_collect_scratch_bytes(uint32_t num_blocks);
int32_t aibx_route_head_collect(aibx_index_t* index, const int32_t* d_tokens,
                                const int64_t* d_tok_off, const int64_t* d_blk_off, int32_t R,
                                int32_t block_tokens, uint64_t root_seed,
                                const int32_t* d_pod_load, uint64_t ready_mask,
                                const aibx_route_params_t* params, uint32_t epoch,
                                uint64_t* d_hashes, uint32_t* d_match_len, uint32_t* d_any_len,
                                uint32_t* d_block_ids, int32_t* d_best_pod, int64_t* d_best_score,
                                uint32_t* d_hashed, uint64_t* d_next_seed, uint32_t num_blocks,
                                void* d_scratch, uint32_t* d_unique_ids, uint32_t* d_count,
                                void* stream);
int32_t aibx_hash_blocks_resume(const int32_t* d_tokens, const int64_t* d_tok_off,
                                const int64_t* d_blk_off, int32_t R, int32_t block_tokens,
                                const uint32_t* d_hashed, const uint64_t* d_next_seed,
                                uint64_t* d_hashes, void* stream);

/* ---------------------------------------------------------------------------------------
 * The routing policies the gateway offers per pending request (Section 3.2.2 lists six: random,
 * throughput, least-request, least-kv-cache, least-latency, prefix-cache-aware), taken for a
 * batch: one pod per request, every request of the call seeing the same snapshot of the per-pod
 * figures.  Only ready pods (ready_mask bit set, pod < num_pods) can be chosen; if none is
 * ready the answer is AIBX_NO_POD.  Ties go to the lowest pod index.  Readings fixed here (the
 * paper gives one sentence per policy and no units; the figures are the caller's integers):
 *   RANDOM             the (d_draws[r] mod n)-th ready pod in ascending order, n = ready pods.
 *                      The random numbers are an input: d_draws [R] uint64.
 *   THROUGHPUT         lowest d_throughput[p]            (tokens per second being served)
 *   LEAST_REQUEST      lowest d_requests[p]              (admitted requests)
 *   LEAST_KV_CACHE     lowest d_kv_usage[p]              (average KV-cache usage)
 *   LEAST_LATENCY      lowest d_queue_latency[p] + d_serve_latency[p], summed in int64
 *   PREFIX_CACHE_AWARE among pods with hit = d_match_len[r][p] > 0 and
 *                      100*hit >= threshold_pct*n_r: the largest hit, ties to the lowest
 *                      d_requests[p]; if no pod qualifies, LEAST_REQUEST.
 * Arrays a policy does not read may be NULL (metrics itself may be NULL for RANDOM;
 * d_match_len / d_blk_off / threshold_pct are read by PREFIX_CACHE_AWARE only).  Each metrics
 * array is [num_pods] int32 in device memory; the struct itself is host memory, read during
 * the call.  d_best_pod [R] out.  INVALID for an unknown policy or a missing array.
 */
#define AIBX_POLICY_RANDOM             0
#define AIBX_POLICY_THROUGHPUT         1
#define AIBX_POLICY_LEAST_REQUEST      2
#define AIBX_POLICY_LEAST_KV_CACHE     3
#define AIBX_POLICY_LEAST_LATENCY      4
#define AIBX_POLICY_PREFIX_CACHE_AWARE 5

typedef struct {
  const int32_t* d_throughput;
  const int32_t* d_requests;
  const int32_t* d_kv_usage;
  const int32_t* d_queue_latency;
  const int32_t* d_serve_latency;
} aibx_pod_metrics_t;

int32_t aibx_route_policy(int32_t policy, const uint32_t* d_match_len, const int64_t* d_blk_off,
                          int32_t R, int32_t num_pods, const aibx_pod_metrics_t* metrics,
                          const uint64_t* d_draws, uint64_t ready_mask, int32_t threshold_pct,
                          int32_t* d_best_pod, void* stream);

/* Sequential assignment of a batch (Section 3.2.2, least-request: the count of admitted
 * requests of an instance grows with every request routed to it).  Requests are taken in
 * order r = 0..R-1; request r is scored as in aibx_route_score against the CURRENT d_pod_load,
 * then d_pod_load[best_pod[r]] += load_increment before request r+1 is scored.  d_pod_load is
 * updated in place (num_pods int32).  load_increment = 0 gives aibx_route_score's results.
 * One warp walks the batch: the dependence between requests is inherent.
 */
int32_t aibx_route_assign(const uint32_t* d_match_len, const int64_t* d_blk_off, int32_t R,
                          int32_t num_pods, int32_t* d_pod_load, uint64_t ready_mask,
                          const aibx_route_params_t* params, int32_t load_increment,
                          int32_t* d_best_pod, int64_t* d_best_score, void* stream);

/* ---------------------------------------------------------------------------------------
 * Set of matched blocks (supporting call between match and gather: Section 3.2.5 speaks of
 * reducing redundant transfers, so a block shared by several requests moves once).
 *   d_unique_ids [n] = the distinct values of d_block_ids[0..n) that are < num_blocks, in
 *   ascending order, padded with AIBX_NO_BLOCK;  *d_count (uint32) = how many.
 *   Values >= num_blocks other than AIBX_NO_BLOCK are dropped and raise device status RANGE.
 *   d_scratch: caller-owned device scratch of aibx_collect_scratch_bytes(num_blocks) bytes,
 *   4-byte aligned; contents on entry are irrelevant, contents on exit unspecified.
 */
uint64_t aibx_collect_scratch_bytes(uint32_t num_blocks);
int32_t aibx_collect_blocks(const uint32_t* d_block_ids, int64_t n, uint32_t num_blocks,
                            void* d_scratch, uint32_t* d_unique_ids, uint32_t* d_count,
                            void* stream);

/* ---------------------------------------------------------------------------------------
 * aibx_collect_blocks without any allocation (the paper has no counterpart: this is a
 * packaging variant of the call above, not an operation of the method).
 *
 * For callers that cannot obtain device memory at the moment they need the call: a routing
 * plug-in living inside an inference engine whose KV pool has already claimed nearly all of
 * HBM (a cudaMalloc there can fail, or stall the engine because it synchronises the device),
 * or code running in a callback or latency-critical loop where allocating is forbidden.  Such a
 * caller still passes its inputs and outputs; only the scratch bitmap comes from the library: a
 * fixed array of 128 KiB in the library's device image, present on every GPU that loads the
 * library until the process exits.
 *
 *   Same results as aibx_collect_blocks (ascending distinct valid ids, NO_BLOCK padding,
 *   *d_count, RANGE status for bad ids).  The call itself never calls cudaMalloc, cudaFree
 *   or any allocating routine.
 *   num_blocks > aibx_collect_static_max_blocks() (1,048,576)  ->  AIBX_ERR_UNSUPPORTED, nothing
 *   is enqueued.  Use aibx_collect_blocks with your own scratch for larger pools.
 *   The first call on each device looks up the array's device address (once, with that device
 *   current; AIBX_ERR_CUDA if the runtime refuses).  Make that first call before starting any
 *   stream capture.
 *   All calls on a device share the one array, which keeps the marks of the previous call; each
 *   call zeroes the part it uses first.  Two calls whose work overlaps on the GPU (different
 *   streams, no ordering between them) race on the array and give wrong results: order them.
 */
int32_t aibx_collect_blocks_static(const uint32_t* d_block_ids, int64_t n, uint32_t num_blocks,
                                   uint32_t* d_unique_ids, uint32_t* d_count, void* stream);
uint32_t aibx_collect_static_max_blocks(void);

/* ---------------------------------------------------------------------------------------
 * Paged-KV data movement (Section 3.2.5: put/get between the engine's paged KV pool and the
 * cache, with exchange through a contiguous buffer when cache and engine are colocated).
 *   tile        = 2 (K,V) * num_kv_heads * block_tokens * head_dim * elem_bytes   bytes
 *   block_bytes = num_layers * tile
 *   pool offset of (block b, layer l) = (b*num_layers + l)*tile      layout 0, block-major
 *                                     = (l*num_blocks + b)*tile      layout 1, layer-major
 *   layout 2, [layer][K/V][block][head][token][dim]: K and V of a layer are separate tensors (the
 *   shape of a per-layer paged cache); the K (kv = 0) or V (kv = 1) half of (block b, layer l)
 *   starts at ((l*2 + kv)*num_blocks + b) * tile/2, and tile/2 must be a multiple of 16 bytes
 *   buffer offset of (item i, layer l) = (i*num_layers + l)*tile     always block-major, K then V
 * gather:  buffer item i <- pool block ids[i]   (ids may repeat)
 * scatter: pool block ids[i] <- buffer item i   (ids must be distinct; pool != buffer)
 * Bytes move verbatim.  An id equal to AIBX_NO_BLOCK is skipped silently; any other id
 * >= num_blocks is skipped and raises device status RANGE (detail counts such items).
 * tile must be a multiple of 16 bytes (UNSUPPORTED otherwise); pool and buffer 16-byte
 * aligned (INVALID otherwise).  n = 0 is a no-op.
 */
typedef struct {
  int32_t layout;        /* 0 block-major, 1 layer-major, 2 layer-major with split K and V */
  int32_t num_layers;
  int32_t num_kv_heads;
  int32_t block_tokens;
  int32_t head_dim;
  int32_t elem_bytes;    /* 1 (fp8) or 2 (bf16/fp16) or 4 */
  uint32_t num_blocks;
} aibx_kv_layout_t;

int32_t aibx_kv_gather(const void* d_pool, const aibx_kv_layout_t* layout,
                       const uint32_t* d_block_ids, int64_t n, void* d_buf, void* stream);
int32_t aibx_kv_scatter(void* d_pool, const aibx_kv_layout_t* layout,
                        const uint32_t* d_block_ids, int64_t n, const void* d_buf,
                        void* stream);

/* The same two movements with the far end in HOST memory (Section 3.2.5: the cache pool lives in
 * host DRAM; put = engine pool -> cache, get = cache -> engine pool).  d_staging is a device
 * buffer of n * block_bytes owned by the caller; h_buf is host memory of the same size (pinned
 * memory makes the copy asynchronous; pageable memory works but blocks the calling thread).
 *   gather_to_host   : aibx_kv_gather into d_staging, then d_staging -> h_buf, both on `stream`.
 *                      Items the gather skips leave their part of h_buf as d_staging had it.
 *   scatter_from_host: h_buf -> d_staging, then aibx_kv_scatter from d_staging, both on `stream`.
 * Both only enqueue.  To keep both directions of the link busy, cut a list into pieces and give
 * consecutive pieces to different streams: the copy of one piece then runs beside the kernel of
 * the next.  Arguments and codes as aibx_kv_gather / aibx_kv_scatter; CUDA if a copy cannot be
 * enqueued.
 */
int32_t aibx_kv_gather_to_host(const void* d_pool, const aibx_kv_layout_t* layout,
                               const uint32_t* d_block_ids, int64_t n, void* d_staging,
                               void* h_buf, void* stream);
int32_t aibx_kv_scatter_from_host(void* d_pool, const aibx_kv_layout_t* layout,
                                  const uint32_t* d_block_ids, int64_t n, void* d_staging,
                                  const void* h_buf, void* stream);

/* The same with the item count on the device: moves the first min(n_max, *d_count) items of the
 * list (d_count: one uint32 in device memory, read when the kernel starts).  Lets the output
 * of aibx_collect_blocks (ids + count) flow into the copy without a host round trip; the buffer
 * must have room for n_max items only if that many can be valid.  INVALID if d_count is null.
 */
int32_t aibx_kv_gather_counted(const void* d_pool, const aibx_kv_layout_t* layout,
                               const uint32_t* d_block_ids, int64_t n_max, const uint32_t* d_count,
                               void* d_buf, void* stream);
int32_t aibx_kv_scatter_counted(void* d_pool, const aibx_kv_layout_t* layout,
                                const uint32_t* d_block_ids, int64_t n_max,
                                const uint32_t* d_count, const void* d_buf, void* stream);

/* Gather / scatter with a change of the order inside a tile (Section 3.2.5: the cache serves
 * different engines, and engines differ in how they lay a block out).  Inner order
 * AIBX_INNER_HEAD_TOKEN (0) = [K/V][head][token][dim], AIBX_INNER_TOKEN_HEAD (1) =
 * [K/V][token][head][dim]; pool_inner describes the pool's tiles, buf_inner the buffer's.  Rows
 * of head_dim elements move whole (head_dim * elem_bytes must be a multiple of 16 and at most
 * 32 KiB: UNSUPPORTED otherwise); everything else - layouts, ids, skipping, errors - is as in
 * aibx_kv_gather / aibx_kv_scatter, to which equal orders reduce.  The transposition goes
 * through shared memory so that global reads and writes both stay whole rows (aibx_tuning.h
 * describes the two engines that write the destination).
 */
#define AIBX_INNER_HEAD_TOKEN 0
#define AIBX_INNER_TOKEN_HEAD 1
int32_t aibx_kv_gather_inner(const void* d_pool, const aibx_kv_layout_t* layout, int32_t pool_inner,
                             int32_t buf_inner, const uint32_t* d_block_ids, int64_t n,
                             void* d_buf, void* stream);
int32_t aibx_kv_scatter_inner(void* d_pool, const aibx_kv_layout_t* layout, int32_t pool_inner,
                              int32_t buf_inner, const uint32_t* d_block_ids, int64_t n,
                              const void* d_buf, void* stream);


/* ---------------------------------------------------------------------------------------
 * Device status of the current device: the most severe (most negative) code recorded by any
 * kernel since the last fetch, and how many items raised one.  Syncs `stream`, then resets
 * the record.  One record per device, shared by all streams.
 */
int32_t aibx_status_fetch(void* stream, int32_t* status, int64_t* detail);

/* Self-test of the bounded waits used by the copy kernels: enqueues one thread that waits on a
 * barrier nobody completes, gives up after `spins` polls (1..2^20) and records AIBX_ERR_TIMEOUT
 * in the device status, exactly as a copy kernel would.  Nothing faults or hangs; the device
 * stays usable.  For health checks and tests of the error path.
 */
int32_t aibx_selftest_bounded_wait(uint32_t spins, void* stream);

const char* aibx_strerror(int32_t status);

#ifdef __cplusplus
}
#endif
#endif /* AIBX_H_ */
