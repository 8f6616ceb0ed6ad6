/*
 * aibx_tuning.h - measurement knobs of libaibx.  Not part of the product boundary (aibx.h does
 * not include this file): these calls exist so that benchmarks and tests can sweep the launch
 * shape of the KV copies and pick the engine of the inner-order conversion.  The paper has no
 * counterpart for any of them.
 *
 * All settings are process-wide.  Each is kept in ONE atomic word: a setter replaces the whole
 * word, and every gather/scatter call reads it once when it starts, so a call running on
 * another host thread sees either the old or the new setting in full, never a mixture.
 */
#ifndef AIBX_TUNING_H_
#define AIBX_TUNING_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Launch shape of gather/scatter; for measurement sweeps.  mode 0 = bulk-async
 * (TMA) ring through shared memory, 1 = 16-byte load/store loop.  chunk_bytes (multiple of 16,
 * 1 KiB..64 KiB) and stages (2..16) size the ring (chunk*stages <= 200 KiB; the stage count
 * bounds the loads in flight per CTA); ctas_per_sm 1..8.
 * Any argument <= 0 keeps its current value.  INVALID on an out-of-range value.
 */
int32_t aibx_kv_set_tuning(int32_t mode, int32_t chunk_bytes, int32_t stages,
                           int32_t ctas_per_sm);
/* Which engine writes the destination of the _inner calls, process-wide; for measurement and
 * tests.  0 (default) = a tensor-map store (cp.async.bulk.tensor) whose strides are those of the
 * destination order, falling back to 1 for shapes it cannot take (rows of head_dim*elem_bytes
 * over 2 KiB); 1 = storer warps (shared memory read back, coalesced streaming stores);
 * 2 = the tensor-map store or AIBX_ERR_UNSUPPORTED, never the fallback.  INVALID otherwise.
 */
int32_t aibx_kv_set_inner_engine(int32_t engine);


/* Bulk ring only, process-wide: how many store groups may still be reading shared memory
 * before their stage is handed back to the loader (1..4; default 1).  INVALID otherwise.
 */
int32_t aibx_kv_set_store_lag(int32_t lag);

/* The launch shape as a gather/scatter call starting now would read it (any pointer may be
 * null).  Always AIBX_OK.
 */
int32_t aibx_kv_get_tuning(int32_t* mode, int32_t* chunk_bytes, int32_t* stages,
                           int32_t* ctas_per_sm, int32_t* lag);

#ifdef __cplusplus
}
#endif

#endif /* AIBX_TUNING_H_ */
