"""Native synthetic KV content (ctypes binding of libaibx_synth.so): the GPU twin of
``workloads.pool_bytes`` for pools too large to generate on the host, and a native host twin
for tests that regenerate such pools chunk by chunk.  Input generation only."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libaibx_synth.so")
_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libaibx_synth.so is missing: run `python -m workloads.build`")
        L = C.CDLL(LIB_PATH)
        L.aibx_synth_fill_linear.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_void_p]
        L.aibx_synth_fill_linear.restype = C.c_int32
        L.aibx_synth_fill_pool.argtypes = [C.c_void_p, C.c_uint64, C.c_int32, C.c_uint64, C.c_uint64,
                                           C.c_uint64, C.c_void_p]
        L.aibx_synth_fill_pool.restype = C.c_int32
        L.aibx_synth_fill_host.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64]
        L.aibx_synth_fill_host.restype = C.c_int32
        L.aibx_probe_random_reads.argtypes = [C.c_void_p, C.c_uint64, C.c_int32, C.c_int32,
                                              C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
        L.aibx_probe_random_reads.restype = C.c_int32
        _lib = L
    return _lib


def fill_host(out: np.ndarray, seed: int, first_byte: int = 0) -> None:
    """out (contiguous uint8 host array) <- bytes [first_byte, first_byte + out.size) of stream
    `seed`: what ``workloads.pool_bytes`` returns, about fifty times faster.  The call releases
    the interpreter lock, so several threads can fill disjoint arrays at once."""
    assert out.dtype == np.uint8 and out.flags.c_contiguous and out.flags.writeable
    rc = lib().aibx_synth_fill_host(out.ctypes.data, out.size, seed, first_byte)
    if rc != 0:
        raise RuntimeError("aibx_synth_fill_host -> %d" % rc)


def fill_linear(t, seed: int, first_byte: int = 0) -> None:
    """t (any dtype, contiguous, CUDA) <- bytes [first_byte, first_byte + nbytes) of stream `seed`."""
    import torch

    assert t.is_cuda and t.is_contiguous()
    rc = lib().aibx_synth_fill_linear(t.data_ptr(), t.numel() * t.element_size(), seed, first_byte,
                                      torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise RuntimeError("aibx_synth_fill_linear -> %d" % rc)


def fill_pool(pool, kv) -> None:
    """Fill a whole pool (KVSpec `kv`) with its logical content in its physical layout."""
    import torch

    assert pool.is_cuda and pool.is_contiguous()
    assert pool.numel() * pool.element_size() == kv.pool_bytes
    rc = lib().aibx_synth_fill_pool(pool.data_ptr(), kv.seed, kv.layout, kv.num_layers,
                                    kv.num_blocks, kv.tile_bytes,
                                    torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise RuntimeError("aibx_synth_fill_pool -> %d" % rc)


def probe_random_reads(base, ws_bytes: int, gran: int, per: int, n_reads: int, seed, sink) -> None:
    """Memory-system probe (no method code): n_reads uniformly random, aligned reads of `gran`
    bytes (32 / 64 / 128) over the first ws_bytes (a multiple of 128) of the CUDA tensor `base`,
    `per` independent reads per thread; `sink` (uint64, n_reads / (32 * per) + 1 words) keeps the
    loads alive.  Enqueued on the current stream."""
    import torch

    assert base.is_cuda and sink.is_cuda and base.numel() * base.element_size() >= ws_bytes
    assert sink.numel() * sink.element_size() >= 8 * (n_reads // (32 * per) + 1)
    rc = lib().aibx_probe_random_reads(base.data_ptr(), ws_bytes, gran, per, n_reads, seed,
                                       sink.data_ptr(), torch.cuda.current_stream().cuda_stream)
    if rc != 0:
        raise RuntimeError("aibx_probe_random_reads -> %d" % rc)
