/*
 * aibxo.c - CPU oracle (test infrastructure only; see aibxo.h).
 *
 * Plain C99, single-threaded, libc only.  Every function writes out its definition without
 * blocking, fusion or reordering so that it can be checked against the text by eye.  The
 * index is a sorted array searched by bsearch() - on purpose nothing like a hash table.
 *
 * Parity pins (none comes from the paper, which prints no value for these operations):
 *   aibxo_xxh64 / aibxo_hash_blocks : published XXH64 values, independent library, suffix
 *                                     invariance, hand-built chains
 *   aibxo_index_*                   : Python dict model, operation-log brute force
 *   aibxo_match_prefix              : brute-force rescan, hand example, monotonicity
 *   aibxo_route_score               : hand example, least-request special case, recompute
 *   aibxo_route_policy              : numpy argmin, list indexing, sorted tuples, hand example,
 *                                     equality with aibxo_route_score under a dominating weight
 *   aibxo_collect_blocks            : sorted(set(...))
 *   aibxo_kv_gather / scatter       : index_select, direct indexing, round trips
 */
#include "aibxo.h"

#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ XXH64 ------------- */
/* 64-bit xxHash as published in the xxHash algorithm specification: five odd 64-bit primes,
 * four accumulators over 32-byte stripes, convergence, length, tail lanes, avalanche. */

static const uint64_t PRIME64_1 = 0x9E3779B185EBCA87ULL;
static const uint64_t PRIME64_2 = 0xC2B2AE3D27D4EB4FULL;
static const uint64_t PRIME64_3 = 0x165667B19E3779F9ULL;
static const uint64_t PRIME64_4 = 0x85EBCA77C2B2AE63ULL;
static const uint64_t PRIME64_5 = 0x27D4EB2F165667C5ULL;

static uint64_t rotl64(uint64_t x, int r) { return (x << r) | (x >> (64 - r)); }

/* little-endian reads, byte by byte, so the host's own endianness never matters */
static uint64_t read_le64(const uint8_t* p) {
  uint64_t v = 0;
  for (int i = 7; i >= 0; --i) v = (v << 8) | p[i];
  return v;
}
static uint32_t read_le32(const uint8_t* p) {
  uint32_t v = 0;
  for (int i = 3; i >= 0; --i) v = (v << 8) | p[i];
  return v;
}

/* one accumulator round: acc = rotl(acc + lane*P2, 31) * P1 */
static uint64_t xxh_round(uint64_t acc, uint64_t lane) {
  acc += lane * PRIME64_2;
  acc = rotl64(acc, 31);
  acc *= PRIME64_1;
  return acc;
}

/* fold one accumulator into the converged value */
static uint64_t xxh_merge(uint64_t acc, uint64_t val) {
  acc ^= xxh_round(0, val);
  acc = acc * PRIME64_1 + PRIME64_4;
  return acc;
}

uint64_t aibxo_xxh64(const void* data, size_t len, uint64_t seed) {
  const uint8_t* p = (const uint8_t*)data;
  size_t remaining = len;
  uint64_t acc;

  if (len >= 32) {
    uint64_t a1 = seed + PRIME64_1 + PRIME64_2;
    uint64_t a2 = seed + PRIME64_2;
    uint64_t a3 = seed;
    uint64_t a4 = seed - PRIME64_1;
    while (remaining >= 32) {
      a1 = xxh_round(a1, read_le64(p));
      a2 = xxh_round(a2, read_le64(p + 8));
      a3 = xxh_round(a3, read_le64(p + 16));
      a4 = xxh_round(a4, read_le64(p + 24));
      p += 32;
      remaining -= 32;
    }
    acc = rotl64(a1, 1) + rotl64(a2, 7) + rotl64(a3, 12) + rotl64(a4, 18);
    acc = xxh_merge(acc, a1);
    acc = xxh_merge(acc, a2);
    acc = xxh_merge(acc, a3);
    acc = xxh_merge(acc, a4);
  } else {
    acc = seed + PRIME64_5;
  }

  acc += (uint64_t)len;

  while (remaining >= 8) {
    acc ^= xxh_round(0, read_le64(p));
    acc = rotl64(acc, 27) * PRIME64_1 + PRIME64_4;
    p += 8;
    remaining -= 8;
  }
  if (remaining >= 4) {
    acc ^= (uint64_t)read_le32(p) * PRIME64_1;
    acc = rotl64(acc, 23) * PRIME64_2 + PRIME64_3;
    p += 4;
    remaining -= 4;
  }
  while (remaining > 0) {
    acc ^= (uint64_t)(*p) * PRIME64_5;
    acc = rotl64(acc, 11) * PRIME64_1;
    p += 1;
    remaining -= 1;
  }

  acc ^= acc >> 33;
  acc *= PRIME64_2;
  acc ^= acc >> 29;
  acc *= PRIME64_3;
  acc ^= acc >> 32;
  return acc;
}

/* ------------------------------------------------------------------ hash chain -------- */
/* key_i = XXH64(little-endian int32 bytes of block i, seed = key_{i-1}), key_{-1} = root. */

int32_t aibxo_hash_blocks(const int32_t* tokens, const int64_t* tok_off, const int64_t* blk_off,
                          int32_t R, int32_t block_tokens, uint64_t root_seed,
                          uint64_t* hashes) {
  if (R < 0 || block_tokens <= 0) return AIBXO_ERR_INVALID;
  if (R == 0) return AIBXO_OK;
  if (!tok_off || !blk_off) return AIBXO_ERR_INVALID;
  uint8_t* msg = (uint8_t*)malloc((size_t)block_tokens * 4);
  if (!msg) return AIBXO_ERR_NOMEM;
  for (int32_t r = 0; r < R; ++r) {
    int64_t len = tok_off[r + 1] - tok_off[r];
    int64_t nblk = len / block_tokens;
    const int32_t* t = tokens + tok_off[r];
    uint64_t* out = hashes + blk_off[r];
    uint64_t parent = root_seed;
    for (int64_t i = 0; i < nblk; ++i) {
      for (int32_t j = 0; j < block_tokens; ++j) {
        uint32_t v = (uint32_t)t[i * block_tokens + j];
        msg[4 * j + 0] = (uint8_t)(v);
        msg[4 * j + 1] = (uint8_t)(v >> 8);
        msg[4 * j + 2] = (uint8_t)(v >> 16);
        msg[4 * j + 3] = (uint8_t)(v >> 24);
      }
      parent = aibxo_xxh64(msg, (size_t)block_tokens * 4, parent);
      out[i] = parent;
    }
  }
  free(msg);
  return AIBXO_OK;
}

/* ------------------------------------------------------------------ index ------------- */
/* State: entries sorted by key, keys unique, every mask != 0. */

typedef struct {
  uint64_t key;
  uint64_t mask;
  uint32_t id;
  uint32_t present; /* scratch for evict: 1 if the key existed when the call began */
  uint32_t touches; /* epochs in which the entry was touched, saturating at 3 */
  uint32_t epoch;   /* last epoch it was touched in; 0 = never */
} entry_t;

struct aibxo_index {
  entry_t* e;
  uint64_t live;
  uint64_t alloc;
  uint64_t capacity;
  int32_t num_pods;
};

static uint64_t pod_all(int32_t P) { return P >= 64 ? ~0ULL : ((1ULL << P) - 1ULL); }
static int key_reserved(uint64_t k) { return k == 0ULL || k == ~0ULL; }

static int cmp_entry_key(const void* a, const void* b) {
  uint64_t ka = ((const entry_t*)a)->key, kb = ((const entry_t*)b)->key;
  return (ka > kb) - (ka < kb);
}

static entry_t* find_entry(const aibxo_index_t* ix, uint64_t key) {
  entry_t probe;
  probe.key = key;
  if (ix->live == 0) return NULL;
  return (entry_t*)bsearch(&probe, ix->e, (size_t)ix->live, sizeof(entry_t), cmp_entry_key);
}

int32_t aibxo_index_create(aibxo_index_t** out, uint64_t capacity, int32_t num_pods) {
  if (!out || num_pods < 1 || num_pods > 64) return AIBXO_ERR_INVALID;
  if (capacity < 8 || (capacity & (capacity - 1)) != 0) return AIBXO_ERR_INVALID;
  aibxo_index_t* ix = (aibxo_index_t*)calloc(1, sizeof(*ix));
  if (!ix) return AIBXO_ERR_NOMEM;
  ix->capacity = capacity;
  ix->num_pods = num_pods;
  *out = ix;
  return AIBXO_OK;
}

int32_t aibxo_index_destroy(aibxo_index_t* ix) {
  if (!ix) return AIBXO_ERR_INVALID;
  free(ix->e);
  free(ix);
  return AIBXO_OK;
}

int32_t aibxo_index_clear(aibxo_index_t* ix) {
  if (!ix) return AIBXO_ERR_INVALID;
  ix->live = 0;
  return AIBXO_OK;
}

int32_t aibxo_index_insert(aibxo_index_t* ix, const uint64_t* keys, const uint64_t* masks,
                           const uint32_t* ids, int64_t n) {
  if (!ix || n < 0) return AIBXO_ERR_INVALID;
  if (n == 0) return AIBXO_OK;
  if (!keys || !masks || !ids) return AIBXO_ERR_INVALID;
  /* append the batch behind the current entries, sort everything by key, fold equal keys */
  uint64_t need = ix->live + (uint64_t)n;
  if (need > ix->alloc) {
    entry_t* ne = (entry_t*)realloc(ix->e, (size_t)need * sizeof(entry_t));
    if (!ne) return AIBXO_ERR_NOMEM;
    ix->e = ne;
    ix->alloc = need;
  }
  uint64_t m = ix->live;
  uint64_t all = pod_all(ix->num_pods);
  for (int64_t i = 0; i < n; ++i) {
    if (key_reserved(keys[i])) continue;
    if ((masks[i] & all) == 0) continue;
    ix->e[m].key = keys[i];
    ix->e[m].mask = masks[i] & all;
    ix->e[m].id = ids[i];
    ix->e[m].present = 0;
    ix->e[m].touches = 0;
    ix->e[m].epoch = 0;
    ++m;
  }
  qsort(ix->e, (size_t)m, sizeof(entry_t), cmp_entry_key);
  uint64_t w = 0;
  for (uint64_t i = 0; i < m; ++i) {
    if (w > 0 && ix->e[w - 1].key == ix->e[i].key) {
      ix->e[w - 1].mask |= ix->e[i].mask;
      if (ix->e[i].id < ix->e[w - 1].id) ix->e[w - 1].id = ix->e[i].id;
      /* an insert never touches: the entry that already existed keeps its history */
      if (ix->e[i].epoch > ix->e[w - 1].epoch) ix->e[w - 1].epoch = ix->e[i].epoch;
      if (ix->e[i].touches > ix->e[w - 1].touches) ix->e[w - 1].touches = ix->e[i].touches;
    } else {
      ix->e[w++] = ix->e[i];
    }
  }
  ix->live = w;
  if (ix->live > ix->capacity) return AIBXO_ERR_FULL;
  return AIBXO_OK;
}

int32_t aibxo_index_evict(aibxo_index_t* ix, const uint64_t* keys, const uint64_t* masks,
                          uint32_t* freed, int64_t n) {
  if (!ix || n < 0) return AIBXO_ERR_INVALID;
  if (n == 0) return AIBXO_OK;
  if (!keys || !masks) return AIBXO_ERR_INVALID;
  /* step 1: clear the named pod bits of every present key */
  for (int64_t i = 0; i < n; ++i) {
    entry_t* e = key_reserved(keys[i]) ? NULL : find_entry(ix, keys[i]);
    if (e) e->mask &= ~masks[i];
  }
  /* step 2: report the ids of entries that ended with no pod */
  if (freed) {
    for (int64_t i = 0; i < n; ++i) {
      entry_t* e = key_reserved(keys[i]) ? NULL : find_entry(ix, keys[i]);
      freed[i] = (e && e->mask == 0) ? e->id : AIBXO_NO_BLOCK;
    }
  }
  /* step 3: entries with no pod left vanish (order of the survivors is kept) */
  uint64_t w = 0;
  for (uint64_t i = 0; i < ix->live; ++i) {
    if (ix->e[i].mask != 0) ix->e[w++] = ix->e[i];
  }
  ix->live = w;
  return AIBXO_OK;
}

int32_t aibxo_index_lookup(const aibxo_index_t* ix, const uint64_t* keys, uint64_t* masks,
                           uint32_t* ids, int64_t n) {
  if (!ix || n < 0) return AIBXO_ERR_INVALID;
  if (n == 0) return AIBXO_OK;
  if (!keys) return AIBXO_ERR_INVALID;
  for (int64_t i = 0; i < n; ++i) {
    const entry_t* e = key_reserved(keys[i]) ? NULL : find_entry(ix, keys[i]);
    if (masks) masks[i] = e ? e->mask : 0;
    if (ids) ids[i] = e ? e->id : AIBXO_NO_BLOCK;
  }
  return AIBXO_OK;
}

int32_t aibxo_index_stats(const aibxo_index_t* ix, uint64_t* live, uint64_t* capacity) {
  if (!ix) return AIBXO_ERR_INVALID;
  if (live) *live = ix->live;
  if (capacity) *capacity = ix->capacity;
  return AIBXO_OK;
}

/* ---- scan-resistant victim choice -------------------------------------------------------
 * touch: a present key that was not yet touched in `epoch` counts one more touch (at most 3)
 *        and remembers the epoch.  Several touches in one epoch count once, so a single scan
 *        over many blocks leaves every one of them at one touch.
 * priority of an entry = (touches >= 2 ? 2^30 : 0) + epoch: entries seen in fewer than two
 *        epochs go first, oldest first.  pick_victims returns the k entries of lowest priority
 *        in ascending (priority, key) order. */

int32_t aibxo_index_touch(aibxo_index_t* ix, const uint64_t* keys, int64_t n, uint32_t epoch) {
  if (!ix || n < 0 || epoch == 0 || epoch >= (1u << 30)) return AIBXO_ERR_INVALID;
  if (n == 0) return AIBXO_OK;
  if (!keys) return AIBXO_ERR_INVALID;
  for (int64_t i = 0; i < n; ++i) {
    entry_t* e = key_reserved(keys[i]) ? NULL : find_entry(ix, keys[i]);
    if (!e || e->epoch == epoch) continue;
    if (e->touches < 3) e->touches += 1;
    e->epoch = epoch;
  }
  return AIBXO_OK;
}

static uint32_t entry_priority(const entry_t* e) {
  return (e->touches >= 2 ? (1u << 30) : 0u) + e->epoch;
}

static int cmp_entry_priority(const void* a, const void* b) {
  const entry_t* x = *(const entry_t* const*)a;
  const entry_t* y = *(const entry_t* const*)b;
  uint32_t px = entry_priority(x), py = entry_priority(y);
  if (px != py) return (px > py) - (px < py);
  return (x->key > y->key) - (x->key < y->key);
}

int32_t aibxo_index_pick_victims(const aibxo_index_t* ix, uint64_t k, uint64_t* keys,
                                 uint32_t* priorities, uint64_t* count) {
  if (!ix || !count) return AIBXO_ERR_INVALID;
  uint64_t m = ix->live < k ? ix->live : k;
  *count = m;
  if (m == 0) return AIBXO_OK;
  const entry_t** order = (const entry_t**)malloc((size_t)ix->live * sizeof(*order));
  if (!order) return AIBXO_ERR_NOMEM;
  for (uint64_t i = 0; i < ix->live; ++i) order[i] = &ix->e[i];
  qsort(order, (size_t)ix->live, sizeof(*order), cmp_entry_priority);
  for (uint64_t i = 0; i < m; ++i) {
    if (keys) keys[i] = order[i]->key;
    if (priorities) priorities[i] = entry_priority(order[i]);
  }
  free(order);
  return AIBXO_OK;
}

int32_t aibxo_index_export(const aibxo_index_t* ix, uint64_t* keys, uint64_t* masks, uint32_t* ids,
                           uint64_t max_entries, uint64_t* count) {
  if (!ix || !count) return AIBXO_ERR_INVALID;
  *count = ix->live;
  for (uint64_t i = 0; i < ix->live && i < max_entries; ++i) {
    if (keys) keys[i] = ix->e[i].key;
    if (masks) masks[i] = ix->e[i].mask;
    if (ids) ids[i] = ix->e[i].id;
  }
  return AIBXO_OK;
}

int32_t aibxo_index_rehash(aibxo_index_t* ix, uint64_t new_capacity) {
  if (!ix) return AIBXO_ERR_INVALID;
  if (new_capacity < 8 || (new_capacity & (new_capacity - 1)) != 0) return AIBXO_ERR_INVALID;
  if (ix->live > new_capacity) return AIBXO_ERR_FULL;
  ix->capacity = new_capacity;   /* the content of the map does not depend on its capacity */
  return AIBXO_OK;
}

/* ------------------------------------------------------------------ longest prefix ---- */
/* match_len[r][p] = largest k <= n_r with every key i < k present and holding bit p;
 * any_len[r] the same with "present at all".  Written per pod, straight from that sentence. */

int32_t aibxo_match_prefix(const aibxo_index_t* ix, const uint64_t* hashes,
                           const int64_t* blk_off, int32_t R, uint32_t* match_len,
                           uint32_t* any_len, uint32_t* block_ids) {
  if (!ix || R < 0) return AIBXO_ERR_INVALID;
  if (R == 0) return AIBXO_OK;
  if (!blk_off || !match_len) return AIBXO_ERR_INVALID;
  int32_t P = ix->num_pods;
  for (int32_t r = 0; r < R; ++r) {
    const uint64_t* h = hashes + blk_off[r];
    int64_t n_r = blk_off[r + 1] - blk_off[r];
    for (int32_t p = 0; p < P; ++p) {
      int64_t k = 0;
      while (k < n_r) {
        const entry_t* e = key_reserved(h[k]) ? NULL : find_entry(ix, h[k]);
        if (!e || ((e->mask >> p) & 1ULL) == 0) break;
        ++k;
      }
      match_len[(int64_t)r * P + p] = (uint32_t)k;
    }
    int64_t a = 0;
    while (a < n_r) {
      const entry_t* e = key_reserved(h[a]) ? NULL : find_entry(ix, h[a]);
      if (!e) break;
      ++a;
    }
    if (any_len) any_len[r] = (uint32_t)a;
    if (block_ids) {
      for (int64_t i = 0; i < n_r; ++i) {
        if (i < a) {
          block_ids[blk_off[r] + i] = find_entry(ix, h[i])->id;
        } else {
          block_ids[blk_off[r] + i] = AIBXO_NO_BLOCK;
        }
      }
    }
  }
  return AIBXO_OK;
}

/* ------------------------------------------------------------------ route score ------- */

int32_t aibxo_route_score(const uint32_t* match_len, const int64_t* blk_off, int32_t R,
                          int32_t num_pods, const int32_t* pod_load, uint64_t ready_mask,
                          const aibxo_route_params_t* params, int32_t* best_pod,
                          int64_t* best_score, int64_t* scores) {
  if (R < 0 || num_pods < 1 || num_pods > 64) return AIBXO_ERR_INVALID;
  if (R == 0) return AIBXO_OK;
  if (!match_len || !blk_off || !pod_load || !best_pod || !best_score) return AIBXO_ERR_INVALID;
  aibxo_route_params_t prm = {4, 1, 50};
  if (params) prm = *params;
  for (int32_t r = 0; r < R; ++r) {
    int64_t n_r = blk_off[r + 1] - blk_off[r];
    int32_t arg = AIBXO_NO_POD;
    int64_t top = INT64_MIN;
    for (int32_t p = 0; p < num_pods; ++p) {
      int64_t hit = (int64_t)match_len[(int64_t)r * num_pods + p];
      int64_t eff = 0;
      if (hit > 0 && 100 * hit >= (int64_t)prm.threshold_pct * n_r) eff = hit;
      int64_t score = (int64_t)prm.w_prefix * eff - (int64_t)prm.w_load * (int64_t)pod_load[p];
      if (scores) scores[(int64_t)r * num_pods + p] = score;
      if (((ready_mask >> p) & 1ULL) == 0) continue;
      if (arg == AIBXO_NO_POD || score > top) { /* strict ">" keeps the lowest pod on ties */
        arg = p;
        top = score;
      }
    }
    best_pod[r] = arg;
    best_score[r] = top;
  }
  return AIBXO_OK;
}

int32_t aibxo_route_assign(const uint32_t* match_len, const int64_t* blk_off, int32_t R,
                           int32_t num_pods, int32_t* pod_load, uint64_t ready_mask,
                           const aibxo_route_params_t* params, int32_t load_increment,
                           int32_t* best_pod, int64_t* best_score) {
  if (R < 0 || num_pods < 1 || num_pods > 64) return AIBXO_ERR_INVALID;
  if (R == 0) return AIBXO_OK;
  if (!match_len || !blk_off || !pod_load || !best_pod || !best_score) return AIBXO_ERR_INVALID;
  /* one request at a time, each seeing the loads its predecessors left behind */
  for (int32_t r = 0; r < R; ++r) {
    int32_t rc = aibxo_route_score(match_len + (int64_t)r * num_pods, blk_off + r, 1, num_pods,
                                   pod_load, ready_mask, params, best_pod + r, best_score + r,
                                   NULL);
    if (rc != AIBXO_OK) return rc;
    if (best_pod[r] != AIBXO_NO_POD)
      pod_load[best_pod[r]] = (int32_t)((uint32_t)pod_load[best_pod[r]] + (uint32_t)load_increment);
  }
  return AIBXO_OK;
}

/* ------------------------------------------------------------------ routing policies -- */

/* lowest value[p] over the ready pods, first one on ties; NO_POD if none is ready */
static int32_t lowest_ready(const int64_t* value, int32_t num_pods, uint64_t ready_mask) {
  int32_t arg = AIBXO_NO_POD;
  for (int32_t p = 0; p < num_pods; ++p) {
    if (((ready_mask >> p) & 1ULL) == 0) continue;
    if (arg == AIBXO_NO_POD || value[p] < value[arg]) arg = p;
  }
  return arg;
}

int32_t aibxo_route_policy(int32_t policy, const uint32_t* match_len, const int64_t* blk_off,
                           int32_t R, int32_t num_pods, const aibxo_pod_metrics_t* metrics,
                           const uint64_t* draws, uint64_t ready_mask, int32_t threshold_pct,
                           int32_t* best_pod) {
  if (R < 0 || num_pods < 1 || num_pods > 64 || policy < 0 || policy > 5) return AIBXO_ERR_INVALID;
  if (R == 0) return AIBXO_OK;
  if (!best_pod) return AIBXO_ERR_INVALID;
  const int32_t P = num_pods;
  int64_t value[64];

  if (policy == 0) { /* random */
    if (!draws) return AIBXO_ERR_INVALID;
    int32_t ready[64];
    int32_t n = 0;
    for (int32_t p = 0; p < P; ++p)
      if ((ready_mask >> p) & 1ULL) ready[n++] = p;
    for (int32_t r = 0; r < R; ++r)
      best_pod[r] = n == 0 ? AIBXO_NO_POD : ready[draws[r] % (uint64_t)n];
    return AIBXO_OK;
  }

  if (!metrics) return AIBXO_ERR_INVALID;
  if (policy >= 1 && policy <= 4) { /* lowest figure, the same pod for every request */
    const int32_t* a = policy == 1 ? metrics->throughput
                     : policy == 2 ? metrics->requests
                     : policy == 3 ? metrics->kv_usage
                                   : metrics->queue_latency;
    const int32_t* b = policy == 4 ? metrics->serve_latency : NULL;
    if (!a || (policy == 4 && !b)) return AIBXO_ERR_INVALID;
    for (int32_t p = 0; p < P; ++p) value[p] = (int64_t)a[p] + (b ? (int64_t)b[p] : 0);
    const int32_t arg = lowest_ready(value, P, ready_mask);
    for (int32_t r = 0; r < R; ++r) best_pod[r] = arg;
    return AIBXO_OK;
  }

  /* prefix-cache-aware */
  if (!match_len || !blk_off || !metrics->requests) return AIBXO_ERR_INVALID;
  for (int32_t p = 0; p < P; ++p) value[p] = (int64_t)metrics->requests[p];
  for (int32_t r = 0; r < R; ++r) {
    const int64_t n_r = blk_off[r + 1] - blk_off[r];
    int32_t arg = AIBXO_NO_POD;
    int64_t arg_hit = 0;
    for (int32_t p = 0; p < P; ++p) {
      if (((ready_mask >> p) & 1ULL) == 0) continue;
      const int64_t hit = (int64_t)match_len[(int64_t)r * P + p];
      if (!(hit > 0 && 100 * hit >= (int64_t)threshold_pct * n_r)) continue;
      if (arg == AIBXO_NO_POD || hit > arg_hit || (hit == arg_hit && value[p] < value[arg])) {
        arg = p;
        arg_hit = hit;
      }
    }
    if (arg == AIBXO_NO_POD) arg = lowest_ready(value, P, ready_mask);
    best_pod[r] = arg;
  }
  return AIBXO_OK;
}

/* ------------------------------------------------------------------ matched-block set - */

static int cmp_u32(const void* a, const void* b) {
  uint32_t x = *(const uint32_t*)a, y = *(const uint32_t*)b;
  return (x > y) - (x < y);
}

int32_t aibxo_collect_blocks(const uint32_t* block_ids, int64_t n, uint32_t num_blocks,
                             uint32_t* unique_ids, uint32_t* count) {
  if (n < 0) return AIBXO_ERR_INVALID;
  if (!count) return AIBXO_ERR_INVALID;
  *count = 0;
  if (n == 0) return AIBXO_OK;
  if (!block_ids || !unique_ids) return AIBXO_ERR_INVALID;
  int32_t rc = AIBXO_OK;
  int64_t m = 0;
  for (int64_t i = 0; i < n; ++i) {
    if (block_ids[i] < num_blocks) {
      unique_ids[m++] = block_ids[i];
    } else if (block_ids[i] != AIBXO_NO_BLOCK) {
      rc = AIBXO_ERR_RANGE;
    }
  }
  qsort(unique_ids, (size_t)m, sizeof(uint32_t), cmp_u32);
  int64_t w = 0;
  for (int64_t i = 0; i < m; ++i) {
    if (w == 0 || unique_ids[w - 1] != unique_ids[i]) unique_ids[w++] = unique_ids[i];
  }
  for (int64_t i = w; i < n; ++i) unique_ids[i] = AIBXO_NO_BLOCK;
  *count = (uint32_t)w;
  return rc;
}

/* ------------------------------------------------------------------ gather / scatter -- */

static int64_t tile_bytes(const aibxo_kv_layout_t* L) {
  return 2LL * L->num_kv_heads * L->block_tokens * L->head_dim * L->elem_bytes;
}

static int layout_ok(const aibxo_kv_layout_t* L) {
  return L && L->layout >= 0 && L->layout <= 2 && L->num_layers > 0 && L->num_kv_heads > 0 &&
         L->block_tokens > 0 && L->head_dim > 0 && L->elem_bytes > 0;
}

/* Where the K (kv = 0) or V (kv = 1) half of the tile of (block b, layer l) starts in the pool.
 *   layout 0  [block][layer][K/V][head][token][dim]
 *   layout 1  [layer][block][K/V][head][token][dim]
 *   layout 2  [layer][K/V][block][head][token][dim]   (K and V of a layer are separate tensors) */
static int64_t pool_offset(const aibxo_kv_layout_t* L, uint32_t b, int32_t l, int32_t kv) {
  int64_t half = tile_bytes(L) / 2;
  if (L->layout == 0) return (((int64_t)b * L->num_layers + l) * 2 + kv) * half;
  if (L->layout == 1) return (((int64_t)l * L->num_blocks + b) * 2 + kv) * half;
  return (((int64_t)l * 2 + kv) * L->num_blocks + b) * half;
}

/* The buffer is always [item][layer][K/V][head][token][dim]. */
static int64_t buf_offset(const aibxo_kv_layout_t* L, int64_t i, int32_t l, int32_t kv) {
  return ((i * L->num_layers + l) * 2 + kv) * (tile_bytes(L) / 2);
}

int32_t aibxo_kv_gather(const void* pool, const aibxo_kv_layout_t* L, const uint32_t* ids,
                        int64_t n, void* buf, int64_t* bad) {
  if (bad) *bad = 0;
  if (!layout_ok(L) || n < 0) return AIBXO_ERR_INVALID;
  if (n == 0) return AIBXO_OK;
  if (!pool || !ids || !buf) return AIBXO_ERR_INVALID;
  int64_t half = tile_bytes(L) / 2;
  int64_t nbad = 0;
  for (int64_t i = 0; i < n; ++i) {
    if (ids[i] == AIBXO_NO_BLOCK) continue;
    if (ids[i] >= L->num_blocks) { ++nbad; continue; }
    for (int32_t l = 0; l < L->num_layers; ++l)
      for (int32_t kv = 0; kv < 2; ++kv)
        memcpy((uint8_t*)buf + buf_offset(L, i, l, kv),
               (const uint8_t*)pool + pool_offset(L, ids[i], l, kv), (size_t)half);
  }
  if (bad) *bad = nbad;
  return nbad ? AIBXO_ERR_RANGE : AIBXO_OK;
}

int32_t aibxo_kv_scatter(void* pool, const aibxo_kv_layout_t* L, const uint32_t* ids,
                         int64_t n, const void* buf, int64_t* bad) {
  if (bad) *bad = 0;
  if (!layout_ok(L) || n < 0) return AIBXO_ERR_INVALID;
  if (n == 0) return AIBXO_OK;
  if (!pool || !ids || !buf) return AIBXO_ERR_INVALID;
  int64_t half = tile_bytes(L) / 2;
  int64_t nbad = 0;
  for (int64_t i = 0; i < n; ++i) {
    if (ids[i] == AIBXO_NO_BLOCK) continue;
    if (ids[i] >= L->num_blocks) { ++nbad; continue; }
    for (int32_t l = 0; l < L->num_layers; ++l)
      for (int32_t kv = 0; kv < 2; ++kv)
        memcpy((uint8_t*)pool + pool_offset(L, ids[i], l, kv),
               (const uint8_t*)buf + buf_offset(L, i, l, kv), (size_t)half);
  }
  if (bad) *bad = nbad;
  return nbad ? AIBXO_ERR_RANGE : AIBXO_OK;
}

/* ------------------------------------------------------------------ inner-order change - */
/* Offset of row (head, token) inside the K or V half of a tile stored in the given inner order. */

static int64_t row_offset(const aibxo_kv_layout_t* L, int32_t inner, int32_t head, int32_t token) {
  int64_t row = (int64_t)L->head_dim * L->elem_bytes;
  int64_t H = L->num_kv_heads, T = L->block_tokens;
  if (inner == 0) return ((int64_t)head * T + token) * row;
  return ((int64_t)token * H + head) * row;
}

static int32_t copy_inner(uint8_t* pool, const aibxo_kv_layout_t* L, int32_t pool_inner,
                          int32_t buf_inner, const uint32_t* ids, int64_t n, uint8_t* buf,
                          int to_pool, int64_t* bad) {
  if (bad) *bad = 0;
  if (!layout_ok(L) || n < 0) return AIBXO_ERR_INVALID;
  if ((pool_inner != 0 && pool_inner != 1) || (buf_inner != 0 && buf_inner != 1))
    return AIBXO_ERR_INVALID;
  if (n == 0) return AIBXO_OK;
  if (!pool || !ids || !buf) return AIBXO_ERR_INVALID;
  int64_t row = (int64_t)L->head_dim * L->elem_bytes;
  int64_t nbad = 0;
  for (int64_t i = 0; i < n; ++i) {
    if (ids[i] == AIBXO_NO_BLOCK) continue;
    if (ids[i] >= L->num_blocks) { ++nbad; continue; }
    for (int32_t l = 0; l < L->num_layers; ++l)
      for (int32_t kv = 0; kv < 2; ++kv) {
        uint8_t* phalf = pool + pool_offset(L, ids[i], l, kv);
        uint8_t* bhalf = buf + buf_offset(L, i, l, kv);
        for (int32_t h = 0; h < L->num_kv_heads; ++h)
          for (int32_t tok = 0; tok < L->block_tokens; ++tok) {
            uint8_t* prow = phalf + row_offset(L, pool_inner, h, tok);
            uint8_t* brow = bhalf + row_offset(L, buf_inner, h, tok);
            if (to_pool) memcpy(prow, brow, (size_t)row);
            else memcpy(brow, prow, (size_t)row);
          }
      }
  }
  if (bad) *bad = nbad;
  return nbad ? AIBXO_ERR_RANGE : AIBXO_OK;
}

int32_t aibxo_kv_gather_inner(const void* pool, const aibxo_kv_layout_t* L, int32_t pool_inner,
                              int32_t buf_inner, const uint32_t* ids, int64_t n, void* buf,
                              int64_t* bad) {
  return copy_inner((uint8_t*)pool, L, pool_inner, buf_inner, ids, n, (uint8_t*)buf, 0, bad);
}

int32_t aibxo_kv_scatter_inner(void* pool, const aibxo_kv_layout_t* L, int32_t pool_inner,
                               int32_t buf_inner, const uint32_t* ids, int64_t n, const void* buf,
                               int64_t* bad) {
  return copy_inner((uint8_t*)pool, L, pool_inner, buf_inner, ids, n, (uint8_t*)buf, 1, bad);
}
