"""Thin ctypes binding of libaibx: one Python function per C entry point, same names without
the ``aibx_`` prefix.  Argument marshalling only - every step of the path runs in the CUDA
kernels behind the C ABI (include/aibx.h).  There is no CPU fallback: if the library has not
been built, loading fails with an error.

Tensors are torch CUDA tensors used purely as device memory; the current torch stream is
passed to every call.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libaibx.so")

OK = 0
ERR_INVALID, ERR_RANGE, ERR_FULL, ERR_CUDA, ERR_UNSUPPORTED, ERR_NOMEM, ERR_TIMEOUT = (
    -1, -2, -3, -4, -5, -6, -7)
NO_BLOCK = 0xFFFFFFFF
NO_POD = -1


class AibxError(RuntimeError):
    def __init__(self, call: str, code: int):
        self.code = code
        super().__init__("%s failed: %d (%s)" % (call, code, strerror(code)))


class RouteParams(C.Structure):
    _fields_ = [("w_prefix", C.c_int32), ("w_load", C.c_int32), ("threshold_pct", C.c_int32)]


class KVLayout(C.Structure):
    _fields_ = [
        ("layout", C.c_int32),
        ("num_layers", C.c_int32),
        ("num_kv_heads", C.c_int32),
        ("block_tokens", C.c_int32),
        ("head_dim", C.c_int32),
        ("elem_bytes", C.c_int32),
        ("num_blocks", C.c_uint32),
    ]

    @property
    def tile_bytes(self) -> int:
        return 2 * self.num_kv_heads * self.block_tokens * self.head_dim * self.elem_bytes

    @property
    def block_bytes(self) -> int:
        return self.num_layers * self.tile_bytes


class PodMetrics(C.Structure):
    _fields_ = [(f, C.c_void_p) for f in ("d_throughput", "d_requests", "d_kv_usage",
                                          "d_queue_latency", "d_serve_latency")]


POLICY_RANDOM, POLICY_THROUGHPUT, POLICY_LEAST_REQUEST, POLICY_LEAST_KV_CACHE, \
    POLICY_LEAST_LATENCY, POLICY_PREFIX_CACHE_AWARE = range(6)

_lib = None


def lib():
    """The loaded C library.  Raises if it was never built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                "libaibx.so is missing at %s: build it with "
                "`python -m paper_2504_03648_b200.build` (needs nvcc, sm_100a)" % LIB_PATH)
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u32, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64
        sig = {
            "aibx_hash_blocks": [vp, vp, vp, i32, i32, u64, vp, vp],
            "aibx_index_create": [C.POINTER(vp), u64, i32],
            "aibx_index_destroy": [vp],
            "aibx_index_clear": [vp, vp],
            "aibx_index_insert": [vp, vp, vp, vp, i64, vp],
            "aibx_index_evict": [vp, vp, vp, vp, i64, vp],
            "aibx_index_lookup": [vp, vp, vp, vp, i64, vp],
            "aibx_index_stats": [vp, C.POINTER(u64), C.POINTER(u64), vp],
            "aibx_index_stats2": [vp, C.POINTER(u64), C.POINTER(u64), C.POINTER(u64),
                                  C.POINTER(u32), vp],
            "aibx_index_touch": [vp, vp, i64, u32, vp],
            "aibx_index_pick_victims": [vp, u64, vp, vp, vp, vp],
            "aibx_index_export": [vp, vp, vp, vp, u64, vp, vp],
            "aibx_index_rehash": [vp, u64],
            "aibx_index_rehash_begin": [vp, u64, vp],
            "aibx_index_rehash_finish": [vp],
            "aibx_match_prefix": [vp, vp, vp, i32, vp, vp, vp, vp],
            "aibx_route_score": [vp, vp, i32, i32, vp, u64, C.POINTER(RouteParams), vp, vp, vp, vp],
            "aibx_route_batch": [vp, vp, vp, vp, i32, i32, u64, vp, u64, C.POINTER(RouteParams),
                                 vp, vp, vp, vp, vp, vp, vp],
            "aibx_route_assign": [vp, vp, i32, i32, vp, u64, C.POINTER(RouteParams), i32, vp, vp, vp],
            "aibx_route_head": [vp, vp, vp, vp, i32, i32, u64, vp, u64, C.POINTER(RouteParams),
                                vp, vp, vp, vp, vp, vp, vp, vp, vp],
            "aibx_route_head_touch": [vp, vp, vp, vp, i32, i32, u64, vp, u64, C.POINTER(RouteParams),
                                      u32, vp, vp, vp, vp, vp, vp, vp, vp, vp],
            "aibx_route_head_collect": [vp, vp, vp, vp, i32, i32, u64, vp, u64, C.POINTER(RouteParams),
                                        u32, vp, vp, vp, vp, vp, vp, vp, vp, u32, vp, vp, vp, vp],
            "aibx_match_prefix_touch": [vp, vp, vp, i32, u32, vp, vp, vp, vp],
            "aibx_hash_blocks_resume": [vp, vp, vp, i32, i32, vp, vp, vp, vp],
            "aibx_route_policy": [i32, vp, vp, i32, i32, C.POINTER(PodMetrics), vp, u64, i32, vp, vp],
            "aibx_collect_blocks": [vp, i64, u32, vp, vp, vp, vp],
            "aibx_collect_blocks_static": [vp, i64, u32, vp, vp, vp],
            "aibx_kv_gather": [vp, C.POINTER(KVLayout), vp, i64, vp, vp],
            "aibx_kv_scatter": [vp, C.POINTER(KVLayout), vp, i64, vp, vp],
            "aibx_kv_gather_to_host": [vp, C.POINTER(KVLayout), vp, i64, vp, vp, vp],
            "aibx_kv_scatter_from_host": [vp, C.POINTER(KVLayout), vp, i64, vp, vp, vp],
            "aibx_kv_gather_counted": [vp, C.POINTER(KVLayout), vp, i64, vp, vp, vp],
            "aibx_kv_scatter_counted": [vp, C.POINTER(KVLayout), vp, i64, vp, vp, vp],
            "aibx_kv_gather_inner": [vp, C.POINTER(KVLayout), i32, i32, vp, i64, vp, vp],
            "aibx_kv_scatter_inner": [vp, C.POINTER(KVLayout), i32, i32, vp, i64, vp, vp],
            "aibx_kv_set_tuning": [i32, i32, i32, i32],
            "aibx_kv_set_store_lag": [i32],
            "aibx_kv_get_tuning": [vp, vp, vp, vp, vp],
            "aibx_kv_set_inner_engine": [i32],
            "aibx_selftest_bounded_wait": [u32, vp],
            "aibx_status_fetch": [vp, C.POINTER(i32), C.POINTER(i64)],
        }
        for name, args in sig.items():
            fn = getattr(L, name)
            fn.argtypes = args
            fn.restype = i32
        L.aibx_collect_scratch_bytes.argtypes = [u32]
        L.aibx_collect_scratch_bytes.restype = u64
        L.aibx_route_collect_scratch_bytes.argtypes = [u32]
        L.aibx_route_collect_scratch_bytes.restype = u64
        L.aibx_collect_static_max_blocks.argtypes = []
        L.aibx_collect_static_max_blocks.restype = u32
        L.aibx_strerror.argtypes = [i32]
        L.aibx_strerror.restype = C.c_char_p
        _lib = L
    return _lib


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t, dtype=None):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensor expected"
    if dtype is not None:
        assert t.dtype == dtype, (t.dtype, dtype)
    return t.data_ptr()


def _check(call: str, rc: int) -> int:
    if rc != OK:
        raise AibxError(call, rc)
    return rc


def strerror(code: int) -> str:
    return lib().aibx_strerror(code).decode()


def hash_blocks(tokens, tok_off, blk_off, block_tokens: int, root_seed: int, hashes) -> None:
    R = tok_off.numel() - 1
    _check("aibx_hash_blocks", lib().aibx_hash_blocks(
        _ptr(tokens, torch.int32), _ptr(tok_off, torch.int64), _ptr(blk_off, torch.int64), R,
        block_tokens, root_seed & (2**64 - 1), _ptr(hashes, torch.uint64), _stream()))


class Index:
    """Host handle of a device-resident index (aibx_index_t)."""

    def __init__(self, capacity_slots: int, num_pods: int):
        h = C.c_void_p()
        self._h = None
        _check("aibx_index_create", lib().aibx_index_create(C.byref(h), capacity_slots, num_pods))
        self._h = h
        self.capacity = capacity_slots
        self.num_pods = num_pods

    def destroy(self) -> None:
        if self._h is not None:
            lib().aibx_index_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def clear(self) -> None:
        _check("aibx_index_clear", lib().aibx_index_clear(self._h, _stream()))

    def insert(self, keys, pod_masks, block_ids) -> None:
        n = keys.numel()
        _check("aibx_index_insert", lib().aibx_index_insert(
            self._h, _ptr(keys, torch.uint64), _ptr(pod_masks, torch.uint64),
            _ptr(block_ids, torch.uint32), n, _stream()))

    def evict(self, keys, pod_masks, freed_block_ids=None) -> None:
        n = keys.numel()
        _check("aibx_index_evict", lib().aibx_index_evict(
            self._h, _ptr(keys, torch.uint64), _ptr(pod_masks, torch.uint64),
            _ptr(freed_block_ids, torch.uint32), n, _stream()))

    def lookup(self, keys, masks=None, block_ids=None) -> None:
        n = keys.numel()
        _check("aibx_index_lookup", lib().aibx_index_lookup(
            self._h, _ptr(keys, torch.uint64), _ptr(masks, torch.uint64),
            _ptr(block_ids, torch.uint32), n, _stream()))

    def stats(self):
        live, cap = C.c_uint64(), C.c_uint64()
        _check("aibx_index_stats",
               lib().aibx_index_stats(self._h, C.byref(live), C.byref(cap), _stream()))
        return live.value, cap.value

    def stats2(self):
        """(live, removed, capacity, longest_walk)."""
        live, removed, cap, walk = C.c_uint64(), C.c_uint64(), C.c_uint64(), C.c_uint32()
        _check("aibx_index_stats2", lib().aibx_index_stats2(
            self._h, C.byref(live), C.byref(removed), C.byref(cap), C.byref(walk), _stream()))
        return live.value, removed.value, cap.value, walk.value

    def touch(self, keys, epoch: int) -> None:
        _check("aibx_index_touch", lib().aibx_index_touch(
            self._h, _ptr(keys, torch.uint64), keys.numel(), epoch, _stream()))

    def pick_victims(self, k: int, keys, priorities, count) -> None:
        _check("aibx_index_pick_victims", lib().aibx_index_pick_victims(
            self._h, k, _ptr(keys, torch.uint64), _ptr(priorities, torch.uint32),
            _ptr(count, torch.uint64), _stream()))

    def export(self, keys, masks, block_ids, count) -> None:
        """Live entries into the given arrays (any of them may be None); count: uint64[1]."""
        cap = min(t.numel() for t in (keys, masks, block_ids) if t is not None) \
            if any(t is not None for t in (keys, masks, block_ids)) else 0
        _check("aibx_index_export", lib().aibx_index_export(
            self._h, _ptr(keys, torch.uint64), _ptr(masks, torch.uint64),
            _ptr(block_ids, torch.uint32), cap, _ptr(count, torch.uint64), _stream()))

    def rehash(self, new_capacity: int) -> None:
        _check("aibx_index_rehash", lib().aibx_index_rehash(self._h, new_capacity))
        self.capacity = new_capacity

    def rehash_begin(self, new_capacity: int) -> None:
        """Start moving the index into a table of another size on the current stream; readers
        keep working on the old table until rehash_finish()."""
        _check("aibx_index_rehash_begin",
               lib().aibx_index_rehash_begin(self._h, new_capacity, _stream()))
        self._pending_capacity = new_capacity

    def rehash_finish(self) -> None:
        _check("aibx_index_rehash_finish", lib().aibx_index_rehash_finish(self._h))
        self.capacity = self._pending_capacity

    def match_prefix(self, hashes, blk_off, match_len, any_len=None, block_ids=None) -> None:
        R = blk_off.numel() - 1
        _check("aibx_match_prefix", lib().aibx_match_prefix(
            self._h, _ptr(hashes, torch.uint64), _ptr(blk_off, torch.int64), R,
            _ptr(match_len, torch.uint32), _ptr(any_len, torch.uint32),
            _ptr(block_ids, torch.uint32), _stream()))

    def match_prefix_touch(self, hashes, blk_off, epoch: int, match_len, any_len=None,
                           block_ids=None) -> None:
        """match_prefix that also marks the entries of every matched prefix as used in `epoch`."""
        R = blk_off.numel() - 1
        _check("aibx_match_prefix_touch", lib().aibx_match_prefix_touch(
            self._h, _ptr(hashes, torch.uint64), _ptr(blk_off, torch.int64), R, epoch,
            _ptr(match_len, torch.uint32), _ptr(any_len, torch.uint32),
            _ptr(block_ids, torch.uint32), _stream()))


def route_score(match_len, blk_off, num_pods: int, pod_load, ready_mask: int, params,
                best_pod, best_score, scores=None) -> None:
    R = blk_off.numel() - 1
    prm = None if params is None else C.byref(RouteParams(*params))
    _check("aibx_route_score", lib().aibx_route_score(
        _ptr(match_len, torch.uint32), _ptr(blk_off, torch.int64), R, num_pods,
        _ptr(pod_load, torch.int32), ready_mask & (2**64 - 1), prm, _ptr(best_pod, torch.int32),
        _ptr(best_score, torch.int64), _ptr(scores, torch.int64), _stream()))


def route_batch(index: Index, tokens, tok_off, blk_off, block_tokens: int, root_seed: int,
                pod_load, ready_mask: int, params, hashes, match_len, any_len, block_ids,
                best_pod, best_score) -> None:
    R = tok_off.numel() - 1
    prm = None if params is None else C.byref(RouteParams(*params))
    _check("aibx_route_batch", lib().aibx_route_batch(
        index._h, _ptr(tokens, torch.int32), _ptr(tok_off, torch.int64), _ptr(blk_off, torch.int64),
        R, block_tokens, root_seed & (2**64 - 1), _ptr(pod_load, torch.int32),
        ready_mask & (2**64 - 1), prm, _ptr(hashes, torch.uint64), _ptr(match_len, torch.uint32),
        _ptr(any_len, torch.uint32), _ptr(block_ids, torch.uint32), _ptr(best_pod, torch.int32),
        _ptr(best_score, torch.int64), _stream()))


def route_head(index: Index, tokens, tok_off, blk_off, block_tokens: int, root_seed: int,
               pod_load, ready_mask: int, params, hashes, match_len, any_len, block_ids,
               best_pod, best_score, hashed, next_seed) -> None:
    """Hash only as far as matching needs, match and score; `hashed`/`next_seed` receive the
    state hash_blocks_resume continues from."""
    R = tok_off.numel() - 1
    prm = None if params is None else C.byref(RouteParams(*params))
    _check("aibx_route_head", lib().aibx_route_head(
        index._h, _ptr(tokens, torch.int32), _ptr(tok_off, torch.int64), _ptr(blk_off, torch.int64),
        R, block_tokens, root_seed & (2**64 - 1), _ptr(pod_load, torch.int32),
        ready_mask & (2**64 - 1), prm, _ptr(hashes, torch.uint64), _ptr(match_len, torch.uint32),
        _ptr(any_len, torch.uint32), _ptr(block_ids, torch.uint32), _ptr(best_pod, torch.int32),
        _ptr(best_score, torch.int64), _ptr(hashed, torch.uint32), _ptr(next_seed, torch.uint64),
        _stream()))


def route_head_touch(index: Index, tokens, tok_off, blk_off, block_tokens: int, root_seed: int,
                     pod_load, ready_mask: int, params, epoch: int, hashes, match_len, any_len,
                     block_ids, best_pod, best_score, hashed, next_seed) -> None:
    """route_head that also marks the entries of every matched prefix as used in `epoch`."""
    R = tok_off.numel() - 1
    prm = None if params is None else C.byref(RouteParams(*params))
    _check("aibx_route_head_touch", lib().aibx_route_head_touch(
        index._h, _ptr(tokens, torch.int32), _ptr(tok_off, torch.int64), _ptr(blk_off, torch.int64),
        R, block_tokens, root_seed & (2**64 - 1), _ptr(pod_load, torch.int32),
        ready_mask & (2**64 - 1), prm, epoch, _ptr(hashes, torch.uint64),
        _ptr(match_len, torch.uint32), _ptr(any_len, torch.uint32), _ptr(block_ids, torch.uint32),
        _ptr(best_pod, torch.int32), _ptr(best_score, torch.int64), _ptr(hashed, torch.uint32),
        _ptr(next_seed, torch.uint64), _stream()))


def route_collect_scratch_bytes(num_blocks: int) -> int:
    return int(lib().aibx_route_collect_scratch_bytes(num_blocks))


def route_head_collect(index: Index, tokens, tok_off, blk_off, block_tokens: int, root_seed: int,
                       pod_load, ready_mask: int, params, epoch: int, hashes, match_len, any_len,
                       block_ids, best_pod, best_score, hashed, next_seed, num_blocks: int,
                       scratch, unique_ids, count) -> None:
    """route_head (+ stamping when epoch > 0) that also leaves the set of matched blocks in
    unique_ids / count, without a further launch."""
    R = tok_off.numel() - 1
    prm = None if params is None else C.byref(RouteParams(*params))
    _check("aibx_route_head_collect", lib().aibx_route_head_collect(
        index._h, _ptr(tokens, torch.int32), _ptr(tok_off, torch.int64), _ptr(blk_off, torch.int64),
        R, block_tokens, root_seed & (2**64 - 1), _ptr(pod_load, torch.int32),
        ready_mask & (2**64 - 1), prm, epoch, _ptr(hashes, torch.uint64),
        _ptr(match_len, torch.uint32), _ptr(any_len, torch.uint32), _ptr(block_ids, torch.uint32),
        _ptr(best_pod, torch.int32), _ptr(best_score, torch.int64), _ptr(hashed, torch.uint32),
        _ptr(next_seed, torch.uint64), num_blocks, _ptr(scratch), _ptr(unique_ids, torch.uint32),
        _ptr(count, torch.uint32), _stream()))


def hash_blocks_resume(tokens, tok_off, blk_off, block_tokens: int, hashed, next_seed,
                       hashes) -> None:
    R = tok_off.numel() - 1
    _check("aibx_hash_blocks_resume", lib().aibx_hash_blocks_resume(
        _ptr(tokens, torch.int32), _ptr(tok_off, torch.int64), _ptr(blk_off, torch.int64), R,
        block_tokens, _ptr(hashed, torch.uint32), _ptr(next_seed, torch.uint64),
        _ptr(hashes, torch.uint64), _stream()))


def route_assign(match_len, blk_off, num_pods: int, pod_load, ready_mask: int, params,
                 load_increment: int, best_pod, best_score) -> None:
    R = blk_off.numel() - 1
    prm = None if params is None else C.byref(RouteParams(*params))
    _check("aibx_route_assign", lib().aibx_route_assign(
        _ptr(match_len, torch.uint32), _ptr(blk_off, torch.int64), R, num_pods,
        _ptr(pod_load, torch.int32), ready_mask & (2**64 - 1), prm, load_increment,
        _ptr(best_pod, torch.int32), _ptr(best_score, torch.int64), _stream()))


def route_policy(policy: int, num_pods: int, R: int, ready_mask: int, best_pod, throughput=None,
                 requests=None, kv_usage=None, queue_latency=None, serve_latency=None,
                 match_len=None, blk_off=None, draws=None, threshold_pct: int = 50) -> None:
    """One pod per request under one of the six policies (POLICY_* numbers); the per-pod
    figures are int32 device tensors, only those the policy reads are needed."""
    figs = (throughput, requests, kv_usage, queue_latency, serve_latency)
    met = None
    if any(t is not None for t in figs):
        met = C.byref(PodMetrics(*[_ptr(t, torch.int32) for t in figs]))
    _check("aibx_route_policy", lib().aibx_route_policy(
        policy, _ptr(match_len, torch.uint32), _ptr(blk_off, torch.int64), R, num_pods, met,
        _ptr(draws, torch.uint64), ready_mask & (2**64 - 1), threshold_pct,
        _ptr(best_pod, torch.int32), _stream()))


def collect_scratch_bytes(num_blocks: int) -> int:
    return int(lib().aibx_collect_scratch_bytes(num_blocks))


def collect_blocks(block_ids, num_blocks: int, scratch, unique_ids, count) -> None:
    n = block_ids.numel()
    assert scratch.numel() * scratch.element_size() >= collect_scratch_bytes(num_blocks)
    assert unique_ids.numel() >= n
    _check("aibx_collect_blocks", lib().aibx_collect_blocks(
        _ptr(block_ids, torch.uint32), n, num_blocks, _ptr(scratch), _ptr(unique_ids, torch.uint32),
        _ptr(count, torch.uint32), _stream()))


def collect_static_max_blocks() -> int:
    return int(lib().aibx_collect_static_max_blocks())


def collect_blocks_static(block_ids, num_blocks: int, unique_ids, count) -> None:
    """collect_blocks for callers that must not allocate: the bitmap is the library's own fixed
    array (pools up to collect_static_max_blocks() blocks).  Calls on one device share that
    array, so they must not overlap on the GPU."""
    n = block_ids.numel()
    assert unique_ids.numel() >= n
    _check("aibx_collect_blocks_static", lib().aibx_collect_blocks_static(
        _ptr(block_ids, torch.uint32), n, num_blocks, _ptr(unique_ids, torch.uint32),
        _ptr(count, torch.uint32), _stream()))


def kv_gather(pool, layout: KVLayout, block_ids, n: int, buf) -> None:
    _check("aibx_kv_gather", lib().aibx_kv_gather(
        _ptr(pool), C.byref(layout), _ptr(block_ids, torch.uint32), n, _ptr(buf), _stream()))


def kv_scatter(pool, layout: KVLayout, block_ids, n: int, buf) -> None:
    _check("aibx_kv_scatter", lib().aibx_kv_scatter(
        _ptr(pool), C.byref(layout), _ptr(block_ids, torch.uint32), n, _ptr(buf), _stream()))


def kv_gather_to_host(pool, layout: KVLayout, block_ids, n: int, staging, host_buf) -> None:
    """Gather into the device staging buffer, then on to `host_buf` (a CPU tensor, pinned for an
    asynchronous copy), all on the current stream."""
    assert not host_buf.is_cuda and host_buf.is_contiguous()
    _check("aibx_kv_gather_to_host", lib().aibx_kv_gather_to_host(
        _ptr(pool), C.byref(layout), _ptr(block_ids, torch.uint32), n, _ptr(staging),
        host_buf.data_ptr(), _stream()))


def kv_scatter_from_host(pool, layout: KVLayout, block_ids, n: int, staging, host_buf) -> None:
    """`host_buf` (CPU tensor) into the device staging buffer, then scatter, on the current stream."""
    assert not host_buf.is_cuda and host_buf.is_contiguous()
    _check("aibx_kv_scatter_from_host", lib().aibx_kv_scatter_from_host(
        _ptr(pool), C.byref(layout), _ptr(block_ids, torch.uint32), n, _ptr(staging),
        host_buf.data_ptr(), _stream()))


def kv_gather_counted(pool, layout: KVLayout, block_ids, n_max: int, count, buf) -> None:
    _check("aibx_kv_gather_counted", lib().aibx_kv_gather_counted(
        _ptr(pool), C.byref(layout), _ptr(block_ids, torch.uint32), n_max,
        _ptr(count, torch.uint32), _ptr(buf), _stream()))


def kv_scatter_counted(pool, layout: KVLayout, block_ids, n_max: int, count, buf) -> None:
    _check("aibx_kv_scatter_counted", lib().aibx_kv_scatter_counted(
        _ptr(pool), C.byref(layout), _ptr(block_ids, torch.uint32), n_max,
        _ptr(count, torch.uint32), _ptr(buf), _stream()))


def kv_gather_inner(pool, layout: KVLayout, pool_inner: int, buf_inner: int, block_ids, n: int,
                    buf) -> None:
    _check("aibx_kv_gather_inner", lib().aibx_kv_gather_inner(
        _ptr(pool), C.byref(layout), pool_inner, buf_inner, _ptr(block_ids, torch.uint32), n,
        _ptr(buf), _stream()))


def kv_scatter_inner(pool, layout: KVLayout, pool_inner: int, buf_inner: int, block_ids, n: int,
                     buf) -> None:
    _check("aibx_kv_scatter_inner", lib().aibx_kv_scatter_inner(
        _ptr(pool), C.byref(layout), pool_inner, buf_inner, _ptr(block_ids, torch.uint32), n,
        _ptr(buf), _stream()))


def kv_set_tuning(mode: int = -1, chunk_bytes: int = 0, stages: int = 0,
                  ctas_per_sm: int = 0) -> None:
    _check("aibx_kv_set_tuning", lib().aibx_kv_set_tuning(mode, chunk_bytes, stages, ctas_per_sm))


def kv_get_tuning():
    """(mode, chunk_bytes, stages, ctas_per_sm, lag) as a copy call starting now would read them."""
    v = [C.c_int32() for _ in range(5)]
    _check("aibx_kv_get_tuning", lib().aibx_kv_get_tuning(*[C.addressof(x) for x in v]))
    return tuple(x.value for x in v)


def kv_set_inner_engine(engine: int = 0) -> None:
    """0 tensor-map store with fallback, 1 storer warps, 2 tensor-map store or UNSUPPORTED."""
    _check("aibx_kv_set_inner_engine", lib().aibx_kv_set_inner_engine(engine))


def kv_set_store_lag(lag: int = 1) -> None:
    _check("aibx_kv_set_store_lag", lib().aibx_kv_set_store_lag(lag))


def selftest_bounded_wait(spins: int = 1000) -> None:
    _check("aibx_selftest_bounded_wait", lib().aibx_selftest_bounded_wait(spins, _stream()))


def status_fetch():
    """(status, detail) of the current device since the last fetch; synchronises the stream."""
    st, det = C.c_int32(), C.c_int64()
    _check("aibx_status_fetch", lib().aibx_status_fetch(_stream(), C.byref(st), C.byref(det)))
    return st.value, det.value
