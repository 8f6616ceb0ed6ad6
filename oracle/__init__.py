"""CPU oracle for the KV-reuse hot path: numpy-facing wrapper around ``aibxo.c``.

TEST INFRASTRUCTURE ONLY.  Nothing in the product package imports this module; only the
tests, the smoke check and the benchmark's CPU-baseline leg do.  The C source is compiled
with gcc on first use (``build()``), and every function here only marshals numpy arrays into
the plain-C oracle and back - the arithmetic lives in ``aibxo.c``.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aibxo.c")
_HDR = os.path.join(_HERE, "aibxo.h")
_LIB = os.path.join(_HERE, "libaibxo.so")

OK, ERR_INVALID, ERR_RANGE, ERR_FULL = 0, -1, -2, -3
NO_BLOCK = 0xFFFFFFFF
NO_POD = -1

_lib = None


def build(force: bool = False) -> str:
    """Compile ``aibxo.c`` into ``libaibxo.so`` next to it (no-op when up to date).

    ``AIBXO_LIB_OVERRIDE`` names another build of the same source to load instead; the tests
    use it to show that the pins reject deliberately broken copies of the oracle."""
    override = os.environ.get("AIBXO_LIB_OVERRIDE")
    if override:
        return override
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < newest:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-std=c99", "-O2", "-Wall", "-Wextra", "-fPIC", "-shared", _SRC, "-o", tmp]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Params(C.Structure):
    _fields_ = [("w_prefix", C.c_int32), ("w_load", C.c_int32), ("threshold_pct", C.c_int32)]


class _Layout(C.Structure):
    _fields_ = [
        ("layout", C.c_int32),
        ("num_layers", C.c_int32),
        ("num_kv_heads", C.c_int32),
        ("block_tokens", C.c_int32),
        ("head_dim", C.c_int32),
        ("elem_bytes", C.c_int32),
        ("num_blocks", C.c_uint32),
    ]


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        vp, i32, i64, u32, u64 = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64
        L.aibxo_xxh64.restype = u64
        L.aibxo_xxh64.argtypes = [vp, C.c_size_t, u64]
        L.aibxo_hash_blocks.argtypes = [vp, vp, vp, i32, i32, u64, vp]
        L.aibxo_index_create.argtypes = [C.POINTER(vp), u64, i32]
        L.aibxo_index_destroy.argtypes = [vp]
        L.aibxo_index_clear.argtypes = [vp]
        L.aibxo_index_insert.argtypes = [vp, vp, vp, vp, i64]
        L.aibxo_index_evict.argtypes = [vp, vp, vp, vp, i64]
        L.aibxo_index_lookup.argtypes = [vp, vp, vp, vp, i64]
        L.aibxo_index_stats.argtypes = [vp, C.POINTER(u64), C.POINTER(u64)]
        L.aibxo_index_touch.argtypes = [vp, vp, i64, u32]
        L.aibxo_index_pick_victims.argtypes = [vp, u64, vp, vp, C.POINTER(u64)]
        L.aibxo_index_export.argtypes = [vp, vp, vp, vp, u64, C.POINTER(u64)]
        L.aibxo_index_rehash.argtypes = [vp, u64]
        L.aibxo_match_prefix.argtypes = [vp, vp, vp, i32, vp, vp, vp]
        L.aibxo_route_score.argtypes = [vp, vp, i32, i32, vp, u64, C.POINTER(_Params), vp, vp, vp]
        L.aibxo_route_assign.argtypes = [vp, vp, i32, i32, vp, u64, C.POINTER(_Params), i32, vp, vp]
        L.aibxo_route_policy.argtypes = [i32, vp, vp, i32, i32, C.POINTER(_Metrics), vp, u64, i32, vp]
        L.aibxo_collect_blocks.argtypes = [vp, i64, u32, vp, C.POINTER(u32)]
        L.aibxo_kv_gather.argtypes = [vp, C.POINTER(_Layout), vp, i64, vp, C.POINTER(i64)]
        L.aibxo_kv_scatter.argtypes = [vp, C.POINTER(_Layout), vp, i64, vp, C.POINTER(i64)]
        L.aibxo_kv_gather_inner.argtypes = [vp, C.POINTER(_Layout), i32, i32, vp, i64, vp,
                                            C.POINTER(i64)]
        L.aibxo_kv_scatter_inner.argtypes = [vp, C.POINTER(_Layout), i32, i32, vp, i64, vp,
                                             C.POINTER(i64)]
        for name in (
            "aibxo_hash_blocks aibxo_index_create aibxo_index_destroy aibxo_index_clear "
            "aibxo_index_insert aibxo_index_evict aibxo_index_lookup aibxo_index_stats "
            "aibxo_index_export aibxo_index_rehash aibxo_index_touch aibxo_index_pick_victims "
            "aibxo_match_prefix aibxo_route_score aibxo_route_assign aibxo_route_policy "
            "aibxo_collect_blocks aibxo_kv_gather "
            "aibxo_kv_scatter aibxo_kv_gather_inner aibxo_kv_scatter_inner"
        ).split():
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _p(a):
    return None if a is None else a.ctypes.data


def xxh64(data: bytes, seed: int = 0) -> int:
    buf = np.frombuffer(bytes(data), dtype=np.uint8)
    return int(lib().aibxo_xxh64(_p(buf) if len(buf) else None, len(buf), seed & (2**64 - 1)))


def block_offsets(tok_off, block_tokens: int) -> np.ndarray:
    """Prefix sum of floor(len_r / block_tokens): argument marshalling, not method arithmetic."""
    tok_off = np.asarray(tok_off, dtype=np.int64)
    n = (tok_off[1:] - tok_off[:-1]) // block_tokens
    out = np.zeros(len(tok_off), dtype=np.int64)
    np.cumsum(n, out=out[1:])
    return out


def hash_blocks(tokens, tok_off, block_tokens: int, root_seed: int = 0):
    tokens = _arr(tokens, np.int32)
    tok_off = _arr(tok_off, np.int64)
    blk_off = block_offsets(tok_off, block_tokens)
    R = len(tok_off) - 1
    hashes = np.zeros(int(blk_off[-1]), dtype=np.uint64)
    rc = lib().aibxo_hash_blocks(_p(tokens), _p(tok_off), _p(blk_off), R, block_tokens,
                                 root_seed & (2**64 - 1), _p(hashes))
    if rc != OK:
        raise RuntimeError("aibxo_hash_blocks -> %d" % rc)
    return hashes, blk_off


class Index:
    """key -> (pod mask, block id) with the batch semantics of the GPU index."""

    def __init__(self, capacity: int, num_pods: int):
        h = C.c_void_p()
        rc = lib().aibxo_index_create(C.byref(h), capacity, num_pods)
        if rc != OK:
            raise ValueError("aibxo_index_create -> %d" % rc)
        self._h = h
        self.num_pods = num_pods
        self.capacity = capacity

    def __del__(self):
        # at interpreter shutdown the module globals may already be gone: then leave it
        if getattr(self, "_h", None) and _lib is not None:
            _lib.aibxo_index_destroy(self._h)
            self._h = None

    def clear(self):
        return lib().aibxo_index_clear(self._h)

    def insert(self, keys, masks, ids) -> int:
        keys, masks, ids = _arr(keys, np.uint64), _arr(masks, np.uint64), _arr(ids, np.uint32)
        assert len(keys) == len(masks) == len(ids)
        return lib().aibxo_index_insert(self._h, _p(keys), _p(masks), _p(ids), len(keys))

    def evict(self, keys, masks):
        keys, masks = _arr(keys, np.uint64), _arr(masks, np.uint64)
        freed = np.zeros(len(keys), dtype=np.uint32)
        rc = lib().aibxo_index_evict(self._h, _p(keys), _p(masks), _p(freed), len(keys))
        return rc, freed

    def lookup(self, keys):
        keys = _arr(keys, np.uint64)
        masks = np.zeros(len(keys), dtype=np.uint64)
        ids = np.zeros(len(keys), dtype=np.uint32)
        rc = lib().aibxo_index_lookup(self._h, _p(keys), _p(masks), _p(ids), len(keys))
        assert rc == OK
        return masks, ids

    def stats(self):
        live, cap = C.c_uint64(), C.c_uint64()
        lib().aibxo_index_stats(self._h, C.byref(live), C.byref(cap))
        return live.value, cap.value

    def touch(self, keys, epoch: int) -> int:
        keys = _arr(keys, np.uint64)
        return lib().aibxo_index_touch(self._h, _p(keys), len(keys), epoch)

    def pick_victims(self, k: int):
        """(keys, priorities) of the k entries of lowest priority, ascending (priority, key)."""
        m = min(k, self.stats()[0])
        keys = np.zeros(m, dtype=np.uint64)
        prio = np.zeros(m, dtype=np.uint32)
        cnt = C.c_uint64()
        rc = lib().aibxo_index_pick_victims(self._h, k, _p(keys), _p(prio), C.byref(cnt))
        assert rc == OK and cnt.value == m
        return keys, prio

    def export(self, max_entries=None):
        """(keys, masks, ids) of all live entries, ascending by key, and the live count."""
        live = self.stats()[0]
        m = live if max_entries is None else max_entries
        keys = np.zeros(m, dtype=np.uint64)
        masks = np.zeros(m, dtype=np.uint64)
        ids = np.zeros(m, dtype=np.uint32)
        cnt = C.c_uint64()
        rc = lib().aibxo_index_export(self._h, _p(keys), _p(masks), _p(ids), m, C.byref(cnt))
        assert rc == OK
        return keys, masks, ids, cnt.value

    def rehash(self, new_capacity: int) -> int:
        rc = lib().aibxo_index_rehash(self._h, new_capacity)
        if rc == OK:
            self.capacity = new_capacity
        return rc

    def match_prefix(self, hashes, blk_off):
        hashes, blk_off = _arr(hashes, np.uint64), _arr(blk_off, np.int64)
        R = len(blk_off) - 1
        match_len = np.zeros((R, self.num_pods), dtype=np.uint32)
        any_len = np.zeros(R, dtype=np.uint32)
        block_ids = np.zeros(len(hashes), dtype=np.uint32)
        rc = lib().aibxo_match_prefix(self._h, _p(hashes), _p(blk_off), R, _p(match_len),
                                      _p(any_len), _p(block_ids))
        assert rc == OK
        return match_len, any_len, block_ids


def route_score(match_len, blk_off, pod_load, ready_mask, params=None):
    match_len = _arr(match_len, np.uint32)
    R, P = match_len.shape
    blk_off, pod_load = _arr(blk_off, np.int64), _arr(pod_load, np.int32)
    best_pod = np.zeros(R, dtype=np.int32)
    best_score = np.zeros(R, dtype=np.int64)
    scores = np.zeros((R, P), dtype=np.int64)
    prm = None if params is None else C.byref(_Params(*params))
    rc = lib().aibxo_route_score(_p(match_len), _p(blk_off), R, P, _p(pod_load),
                                 ready_mask & (2**64 - 1), prm, _p(best_pod), _p(best_score),
                                 _p(scores))
    assert rc == OK, rc
    return best_pod, best_score, scores


def route_assign(match_len, blk_off, pod_load, ready_mask, params=None, load_increment=1):
    """Sequential assignment; returns (best_pod, best_score, loads after the batch)."""
    match_len = _arr(match_len, np.uint32)
    R, P = match_len.shape
    blk_off = _arr(blk_off, np.int64)
    load = np.array(pod_load, dtype=np.int32, copy=True)
    best_pod = np.zeros(R, dtype=np.int32)
    best_score = np.zeros(R, dtype=np.int64)
    prm = None if params is None else C.byref(_Params(*params))
    rc = lib().aibxo_route_assign(_p(match_len), _p(blk_off), R, P, _p(load),
                                  ready_mask & (2**64 - 1), prm, load_increment, _p(best_pod),
                                  _p(best_score))
    assert rc == OK, rc
    return best_pod, best_score, load


POLICIES = ("random", "throughput", "least-request", "least-kv-cache", "least-latency",
            "prefix-cache-aware")
_METRIC_FIELDS = ("throughput", "requests", "kv_usage", "queue_latency", "serve_latency")


class _Metrics(C.Structure):
    _fields_ = [(f, C.c_void_p) for f in _METRIC_FIELDS]


def route_policy(policy, num_pods, R, ready_mask, metrics=None, match_len=None, blk_off=None,
                 draws=None, threshold_pct=50, expect=OK):
    """One pod per request under one of the six policies (name or number).  `metrics` maps
    field names (throughput, requests, kv_usage, queue_latency, serve_latency) to per-pod
    int32 arrays.  Returns best_pod, or the error code when `expect` is not OK."""
    pol = POLICIES.index(policy) if isinstance(policy, str) else int(policy)
    keep = []
    m = _Metrics()
    for f in _METRIC_FIELDS:
        a = None if metrics is None or metrics.get(f) is None else _arr(metrics[f], np.int32)
        keep.append(a)
        setattr(m, f, _p(a))
    match_len = None if match_len is None else _arr(match_len, np.uint32)
    blk_off = None if blk_off is None else _arr(blk_off, np.int64)
    draws = None if draws is None else _arr(draws, np.uint64)
    best_pod = np.full(R, -7, dtype=np.int32)
    rc = lib().aibxo_route_policy(pol, _p(match_len), _p(blk_off), R, num_pods,
                                  None if metrics is None else C.byref(m), _p(draws),
                                  ready_mask & (2**64 - 1), threshold_pct, _p(best_pod))
    assert rc == expect, rc
    return best_pod if expect == OK else rc


def collect_blocks(block_ids, num_blocks: int):
    block_ids = _arr(block_ids, np.uint32)
    out = np.zeros(len(block_ids), dtype=np.uint32)
    cnt = C.c_uint32()
    rc = lib().aibxo_collect_blocks(_p(block_ids), len(block_ids), num_blocks, _p(out),
                                    C.byref(cnt))
    return rc, out, cnt.value


def kv_layout(layout, num_layers, num_kv_heads, block_tokens, head_dim, elem_bytes, num_blocks):
    return _Layout(layout, num_layers, num_kv_heads, block_tokens, head_dim, elem_bytes,
                   num_blocks)


def kv_gather(pool: np.ndarray, lay: _Layout, ids, buf: np.ndarray):
    """pool, buf: flat uint8 arrays.  Returns (status, number of skipped out-of-range ids)."""
    ids = _arr(ids, np.uint32)
    assert pool.dtype == np.uint8 and buf.dtype == np.uint8
    assert pool.flags.c_contiguous and buf.flags.c_contiguous
    bad = C.c_int64()
    rc = lib().aibxo_kv_gather(_p(pool), C.byref(lay), _p(ids), len(ids), _p(buf), C.byref(bad))
    return rc, bad.value


def kv_scatter(pool: np.ndarray, lay: _Layout, ids, buf: np.ndarray):
    ids = _arr(ids, np.uint32)
    assert pool.dtype == np.uint8 and buf.dtype == np.uint8
    assert pool.flags.c_contiguous and buf.flags.c_contiguous
    bad = C.c_int64()
    rc = lib().aibxo_kv_scatter(_p(pool), C.byref(lay), _p(ids), len(ids), _p(buf), C.byref(bad))
    return rc, bad.value


def kv_gather_inner(pool: np.ndarray, lay: _Layout, pool_inner: int, buf_inner: int, ids,
                    buf: np.ndarray):
    ids = _arr(ids, np.uint32)
    assert pool.dtype == np.uint8 and buf.dtype == np.uint8
    assert pool.flags.c_contiguous and buf.flags.c_contiguous
    bad = C.c_int64()
    rc = lib().aibxo_kv_gather_inner(_p(pool), C.byref(lay), pool_inner, buf_inner, _p(ids),
                                     len(ids), _p(buf), C.byref(bad))
    return rc, bad.value


def kv_scatter_inner(pool: np.ndarray, lay: _Layout, pool_inner: int, buf_inner: int, ids,
                     buf: np.ndarray):
    ids = _arr(ids, np.uint32)
    assert pool.dtype == np.uint8 and buf.dtype == np.uint8
    assert pool.flags.c_contiguous and buf.flags.c_contiguous
    bad = C.c_int64()
    rc = lib().aibxo_kv_scatter_inner(_p(pool), C.byref(lay), pool_inner, buf_inner, _p(ids),
                                      len(ids), _p(buf), C.byref(bad))
    return rc, bad.value
