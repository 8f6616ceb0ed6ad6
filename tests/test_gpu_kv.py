"""GPU parity, data-movement half of the path: paged-KV gather and scatter against the CPU
oracle, byte for byte, through the C ABI - small pools in full, and the large configurations at
full size: every byte of a gathered buffer and of the whole pool (regenerated on the host chunk
by chunk and passed through the oracle), plus sampled blocks after every other call."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import (NO_BLOCK, PoolModel, check_gather_full, check_pool_full, dev, empty, host,
                      kv_layout_gpu, kv_layout_oracle, read_block)
from paper_2504_03648_b200 import binding as aibx
from workloads import synth
import workloads as W

pytestmark = pytest.mark.gpu

GUARD = 4096


@pytest.fixture(autouse=True)
def _default_tuning():
    aibx.kv_set_tuning(0, 32768, 3, 1)
    aibx.kv_set_store_lag(1)
    yield
    aibx.kv_set_tuning(0, 32768, 3, 1)
    aibx.kv_set_store_lag(1)


def guarded(n_bytes, fill):
    """Device byte buffer with guard bands on both sides; returns (whole, payload view)."""
    whole = torch.full((n_bytes + 2 * GUARD,), fill, dtype=torch.uint8, device="cuda")
    return whole, whole[GUARD: GUARD + n_bytes]


def guards_intact(whole, n_bytes, fill):
    h = host(whole)
    return (h[:GUARD] == fill).all() and (h[GUARD + n_bytes:] == fill).all()


def check_gather_scatter(kv, ids_g, ids_s, mode_args):
    aibx.kv_set_tuning(*mode_args[:4])
    aibx.kv_set_store_lag(mode_args[4])
    pool_h = W.host_pool(kv)
    lay_g, lay_o = kv_layout_gpu(kv), kv_layout_oracle(kv)
    n = len(ids_g)
    buf_bytes = n * kv.block_bytes
    # gather
    pool_w, pool_d = guarded(kv.pool_bytes, 0xA5)
    pool_d.copy_(torch.from_numpy(pool_h))
    buf_w, buf_d = guarded(buf_bytes, 0xEE)
    aibx.kv_gather(pool_d, lay_g, dev(ids_g), n, buf_d)
    want = np.full(buf_bytes, 0xEE, dtype=np.uint8)
    rc, bad = oracle.kv_gather(pool_h, lay_o, ids_g, want)
    assert np.array_equal(host(buf_d), want)
    st, detail = aibx.status_fetch()
    assert (st, detail) == ((aibx.ERR_RANGE, bad) if bad else (0, 0))
    assert np.array_equal(host(pool_d), pool_h)                    # source untouched
    assert guards_intact(buf_w, buf_bytes, 0xEE) and guards_intact(pool_w, kv.pool_bytes, 0xA5)
    # scatter the gathered buffer to another id list
    ns = len(ids_s)
    aibx.kv_scatter(pool_d, lay_g, dev(ids_s), ns, buf_d)
    pool_want = pool_h.copy()
    rc, bad = oracle.kv_scatter(pool_want, lay_o, ids_s, want)
    assert np.array_equal(host(pool_d), pool_want)
    assert np.array_equal(host(buf_d), want)                       # source untouched
    st, detail = aibx.status_fetch()
    assert (st, detail) == ((aibx.ERR_RANGE, bad) if bad else (0, 0))
    assert guards_intact(buf_w, buf_bytes, 0xEE) and guards_intact(pool_w, kv.pool_bytes, 0xA5)


# (mode, chunk bytes, stages, CTAs per SM, store lag)
MODES = [(0, 32768, 3, 1, 1), (0, 16384, 12, 1, 1), (0, 4096, 3, 2, 2), (0, 1024, 16, 1, 4), (1, 16384, 2, 1, 1),
         (0, 49152, 4, 1, 2), (0, 14848, 5, 1, 1), (0, 2048, 2, 1, 1)]


@pytest.mark.parametrize("mode_args", MODES)
def test_cfg1_tiny(mode_args):
    kv = W.cfg1_kv()
    ids_g = W.distinct_ids(0, kv.num_blocks, 64)
    ids_s = W.distinct_ids(100, kv.num_blocks, 64)
    assert not np.array_equal(ids_g, ids_s)
    check_gather_scatter(kv, ids_g, ids_s, mode_args)


@pytest.mark.parametrize("mode_args", MODES)
@pytest.mark.parametrize("layout", [0, 1, 2])
def test_shapes_with_ragged_chunks(layout, mode_args):
    # tile = 2*3*5*24*1 = 720 bytes (not a multiple of any chunk size), 7 layers; with K and V
    # apart a half tile must be a multiple of 16 bytes: 2*3*5*32*1 = 960-byte tiles there
    kv = W.KVSpec("ragged", 5, layout, 7, 3, 5, 24 if layout < 2 else 32, 1, 61)
    rng = np.random.default_rng(layout)
    ids_g = rng.integers(0, 61, 200).astype(np.uint32)               # repeats allowed
    ids_g[[3, 50]] = NO_BLOCK
    ids_g[[7, 120, 199]] = [61, 1 << 31, 0xFFFFFFFE]                 # out of range
    ids_s = np.concatenate([rng.permutation(61)[:40], [NO_BLOCK, 77]]).astype(np.uint32)
    check_gather_scatter(kv, ids_g, ids_s, mode_args)
    # bigger tiles: 2*2*16*64*2 = 8 KiB and 40 KiB blocks
    kv = W.KVSpec("mid", 6, layout, 5, 2, 16, 64, 2, 300)
    ids_g = W.distinct_ids(1, 300, 257)
    ids_s = W.distinct_ids(2, 300, 257)
    check_gather_scatter(kv, ids_g, ids_s, mode_args)
    # 12,800-byte tiles, 38,400-byte blocks: chunks straddle segments and items, with skipped
    # and out-of-range ids in the middle of straddling chunks
    kv = W.KVSpec("straddle", 7, layout, 3, 5, 16, 40, 2, 97)
    ids_g = rng.integers(0, 97, 333).astype(np.uint32)
    ids_g[rng.random(333) < 0.15] = NO_BLOCK
    ids_g[[1, 100, 332]] = [97, 5000, 0xFFFFFFFE]
    ids_s = np.concatenate([rng.permutation(97)[:90], [NO_BLOCK, 97, NO_BLOCK]]).astype(np.uint32)
    rng.shuffle(ids_s)
    check_gather_scatter(kv, ids_g, ids_s, mode_args)


def test_round_trips_and_single_item():
    kv = W.KVSpec("rt", 8, 1, 3, 2, 16, 128, 2, 40)                 # 16 KiB tiles, layer-major
    lay = kv_layout_gpu(kv)
    pool_h = W.host_pool(kv)
    pool_d = dev(pool_h)
    ids = W.distinct_ids(3, 40, 17)
    buf = empty(17 * kv.block_bytes, torch.uint8)
    aibx.kv_gather(pool_d, lay, dev(ids), 17, buf)
    snapshot = host(buf).copy()
    aibx.kv_scatter(pool_d, lay, dev(ids), 17, buf)                 # scatter after gather: identity
    assert np.array_equal(host(pool_d), pool_h)
    buf2 = empty(17 * kv.block_bytes, torch.uint8)
    aibx.kv_gather(pool_d, lay, dev(ids), 17, buf2)                 # gather after scatter: the buffer
    assert np.array_equal(host(buf2), snapshot)
    one = empty(kv.block_bytes, torch.uint8)
    aibx.kv_gather(pool_d, lay, dev(ids[5:6]), 1, one)
    assert np.array_equal(host(one), snapshot[5 * kv.block_bytes: 6 * kv.block_bytes])
    assert aibx.status_fetch() == (0, 0)


def test_invalid_arguments():
    kv = W.cfg1_kv()
    lay = kv_layout_gpu(kv)
    pool, buf, ids = empty(kv.pool_bytes, torch.uint8), empty(kv.block_bytes, torch.uint8), dev(np.zeros(1, np.uint32))
    lib = aibx.lib()
    import ctypes as C
    assert lib.aibx_kv_gather(pool.data_ptr(), C.byref(lay), ids.data_ptr(), 0, buf.data_ptr(), None) == 0
    assert lib.aibx_kv_gather(None, C.byref(lay), ids.data_ptr(), 1, buf.data_ptr(), None) == -1
    assert lib.aibx_kv_gather(pool.data_ptr(), None, ids.data_ptr(), 1, buf.data_ptr(), None) == -1
    assert lib.aibx_kv_gather(pool.data_ptr(), C.byref(lay), ids.data_ptr(), -1, buf.data_ptr(), None) == -1
    assert lib.aibx_kv_gather(pool.data_ptr() + 8, C.byref(lay), ids.data_ptr(), 1, buf.data_ptr(), None) == -1
    bad = aibx.KVLayout(-1, 2, 4, 16, 64, 2, 256)
    assert lib.aibx_kv_scatter(pool.data_ptr(), C.byref(bad), ids.data_ptr(), 1, buf.data_ptr(), None) == -1
    odd = aibx.KVLayout(0, 2, 1, 1, 3, 1, 256)                      # 6-byte tiles
    assert lib.aibx_kv_gather(pool.data_ptr(), C.byref(odd), ids.data_ptr(), 1, buf.data_ptr(), None) == -5
    split = aibx.KVLayout(2, 2, 1, 1, 24, 1, 256)                   # 48-byte tiles, 24-byte halves
    assert lib.aibx_kv_gather(pool.data_ptr(), C.byref(split), ids.data_ptr(), 1, buf.data_ptr(), None) == -5
    assert lib.aibx_kv_gather(pool.data_ptr(), C.byref(aibx.KVLayout(3, 2, 4, 16, 64, 2, 256)),
                              ids.data_ptr(), 1, buf.data_ptr(), None) == -1


# ------------------------------------------------------------------ large configurations

def _fit_blocks(kv, extra_bytes):
    """Shrink the pool (never the batch) if the device cannot hold the full configuration."""
    import gc

    gc.collect()
    torch.cuda.empty_cache()                       # earlier tests' pools go back to the driver
    free, _ = torch.cuda.mem_get_info()
    room = free - extra_bytes - (6 << 30)
    if kv.pool_bytes <= room:
        return kv, False
    nb = int(room // kv.block_bytes)
    return W.scaled(kv, num_blocks=nb), True


def _sample_gather_check(kv, pool_seed_kv, ids, buf_d, sample):
    """Sampled items of a gathered buffer against the oracle run on a mini pool of those blocks."""
    lay1 = kv_layout_oracle(kv, layout=0, num_blocks=len(sample))
    mini = W.logical_blocks(pool_seed_kv, ids[sample])
    want = np.zeros(len(sample) * kv.block_bytes, dtype=np.uint8)
    rc, bad = oracle.kv_gather(mini, lay1, np.arange(len(sample), dtype=np.uint32), want)
    assert rc == oracle.OK
    want = want.reshape(len(sample), kv.block_bytes)
    bview = buf_d.view(-1, kv.block_bytes)
    for j, i in enumerate(sample):
        assert np.array_equal(host(bview[int(i)]), want[j]), int(i)


def test_cfg2_full_size():
    kv = W.cfg2_kv()
    n = 1660
    kv, shrunk = _fit_blocks(kv, n * kv.block_bytes)
    assert not shrunk, "8 GiB pool must fit"
    pool = empty(kv.pool_bytes, torch.uint8)
    synth.fill_pool(pool, kv)
    ids = np.sort(W.distinct_ids(7, kv.num_blocks, n))            # ascending, like the matched set
    buf = empty(n * kv.block_bytes, torch.uint8)
    lay = kv_layout_gpu(kv)
    aibx.kv_gather(pool, lay, dev(ids), n, buf)
    assert aibx.status_fetch() == (0, 0)
    sample = np.concatenate([[0, 1, n - 1], W.Stream(7, 9).randint(0, n, 9)])
    _sample_gather_check(kv, kv, ids, buf, sample)
    model = PoolModel(kv)
    assert check_gather_full(model, ids, buf) == []                # every byte, against the oracle
    # and the same property on the device: the buffer rows equal the pool rows they name
    got = buf.view(n, kv.block_bytes)
    src = pool.view(kv.num_blocks, kv.block_bytes)
    idx = dev(ids.astype(np.int64))
    for lo in range(0, n, 256):
        assert torch.equal(got[lo: lo + 256], src[idx[lo: lo + 256]])
    # scatter back to the same ids leaves the pool as generated (sampled) ...
    aibx.kv_scatter(pool, lay, dev(ids), n, buf)
    for b in ids[sample]:
        assert np.array_equal(read_block(pool, kv, int(b)), W.logical_blocks(kv, [b]))
    # ... and scattering fresh content lands where the oracle puts it
    synth.fill_linear(buf, 1234)
    aibx.kv_scatter(pool, lay, dev(ids), n, buf)
    assert aibx.status_fetch() == (0, 0)
    model.scattered(ids, 1234)
    assert check_pool_full(model, pool) == []                      # all 8 GiB
    for i in sample[:6]:
        mini = np.zeros(kv.block_bytes, dtype=np.uint8)
        item = W.pool_bytes(1234, int(i) * kv.block_bytes, kv.block_bytes)
        rc, _ = oracle.kv_scatter(mini, kv_layout_oracle(kv, layout=0, num_blocks=1),
                                  np.zeros(1, np.uint32), item)
        assert np.array_equal(read_block(pool, kv, int(ids[int(i)])), mini)


def test_cfg4_full_size_layer_major():
    kv0 = W.cfg4_kv()
    n = 2048
    kv, shrunk = _fit_blocks(kv0, n * kv0.block_bytes)
    pool = empty(kv.pool_bytes, torch.uint8)
    synth.fill_pool(pool, kv)
    buf = empty(n * kv.block_bytes, torch.uint8)
    lay = kv_layout_gpu(kv)
    model = PoolModel(kv)                                          # generated content + scatters

    for it in range(4):                                            # put, get, put, get
        ids = W.distinct_ids(1000 + it, kv.num_blocks, n)
        sample = np.concatenate([[0, n - 1], W.Stream(it, 11).randint(0, n, 4)])
        if it % 2 == 0:
            aibx.kv_gather(pool, lay, dev(ids), n, buf)
            # every byte of the buffer (from the second put on, a tenth of the ids name blocks
            # that hold scattered content)
            assert check_gather_full(model, ids, buf) == []
        else:
            synth.fill_linear(buf, 5000 + it)
            aibx.kv_scatter(pool, lay, dev(ids), n, buf)
            model.scattered(ids, 5000 + it)
            for i in sample:
                b = int(ids[int(i)])
                mini, _ = model.mini_pool(np.array([b]))           # one block: layouts coincide
                assert np.array_equal(read_block(pool, kv, b), mini)
        assert aibx.status_fetch() == (0, 0)
    # every byte of the pool: scattered blocks hold what the oracle's scatter puts there, all
    # others their generated content
    assert check_pool_full(model, pool) == []
    print("cfg4 pool blocks used:", kv.num_blocks, "(shrunk)" if shrunk else "(full)")


@pytest.mark.parametrize("which", ["cfg2", "cfg4"])
def test_split_kv_pools_at_full_size(which):
    """The Llama-3-8B and Llama-3-70B pools with K and V of every layer as separate tensors
    ([layer][K/V][block]...): a put, a get of fresh content into other blocks, a put of those -
    every byte of both buffers and of the whole pool against the oracle."""
    kv0 = W.scaled(W.cfg2_kv() if which == "cfg2" else W.cfg4_kv(), layout=2)
    n = 1660 if which == "cfg2" else 2048
    kv, shrunk = _fit_blocks(kv0, n * kv0.block_bytes)
    pool = empty(kv.pool_bytes, torch.uint8)
    synth.fill_pool(pool, kv)
    buf = empty(n * kv.block_bytes, torch.uint8)
    lay = kv_layout_gpu(kv)
    model = PoolModel(kv)
    ids = W.distinct_ids(2000, kv.num_blocks, n)
    aibx.kv_gather(pool, lay, dev(ids), n, buf)
    assert aibx.status_fetch() == (0, 0)
    assert check_gather_full(model, ids, buf) == []
    ids2 = W.distinct_ids(2001, kv.num_blocks, n)
    synth.fill_linear(buf, 6000)
    aibx.kv_scatter(pool, lay, dev(ids2), n, buf)
    model.scattered(ids2, 6000)
    ids3 = np.concatenate([ids2[: n // 2], ids[: n - n // 2]])        # half of them just written
    aibx.kv_gather(pool, lay, dev(ids3), n, buf)
    assert aibx.status_fetch() == (0, 0)
    assert check_gather_full(model, ids3, buf) == []
    assert check_pool_full(model, pool) == []
    print(which, "split-K/V pool blocks used:", kv.num_blocks, "(shrunk)" if shrunk else "(full)")


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("layout", [0, 1, 2])
def test_host_side_put_and_get(layout, pinned):
    """gather_to_host / scatter_from_host: the far end of the transfer in host memory (pinned or
    pageable), byte for byte against the oracle's gather and scatter."""
    kv = W.KVSpec("host", 31, layout, 3, 4, 16, 64, 2, 90)
    lay_g, lay_o = kv_layout_gpu(kv), kv_layout_oracle(kv)
    pool_h = W.host_pool(kv)
    rng = np.random.default_rng(layout + 5)
    n = 57
    ids_g = rng.integers(0, kv.num_blocks, n).astype(np.uint32)
    ids_g[[4, 30]] = NO_BLOCK
    ids_g[9] = kv.num_blocks + 3                                  # out of range: skipped, RANGE
    pool_d = dev(pool_h)
    staging = torch.full((n * kv.block_bytes,), 0x5A, dtype=torch.uint8, device="cuda")
    h_buf = torch.zeros(n * kv.block_bytes, dtype=torch.uint8)
    if pinned:
        h_buf = h_buf.pin_memory()
    aibx.kv_gather_to_host(pool_d, lay_g, dev(ids_g), n, staging, h_buf)
    assert aibx.status_fetch() == (aibx.ERR_RANGE, 1)             # syncs the stream
    want = np.full(n * kv.block_bytes, 0x5A, dtype=np.uint8)      # skipped items: staging as it was
    oracle.kv_gather(pool_h, lay_o, ids_g, want)
    assert np.array_equal(h_buf.numpy(), want) and np.array_equal(host(staging), want)
    assert np.array_equal(host(pool_d), pool_h)
    # get: other content from the host into a distinct set of blocks
    ids_s = rng.permutation(kv.num_blocks)[:n].astype(np.uint32)
    ids_s[3] = NO_BLOCK
    src = torch.from_numpy(rng.integers(0, 256, n * kv.block_bytes, dtype=np.uint8))
    if pinned:
        src = src.pin_memory()
    aibx.kv_scatter_from_host(pool_d, lay_g, dev(ids_s), n, staging, src)
    assert aibx.status_fetch() == (0, 0)
    pool_want = pool_h.copy()
    oracle.kv_scatter(pool_want, lay_o, ids_s, src.numpy().copy())
    assert np.array_equal(host(pool_d), pool_want)
    # nothing to do, and what the host can refuse
    aibx.kv_gather_to_host(pool_d, lay_g, dev(ids_g), 0, staging, h_buf)
    aibx.kv_scatter_from_host(pool_d, lay_g, dev(ids_s), 0, staging, src)
    lib = aibx.lib()
    import ctypes as C
    assert lib.aibx_kv_gather_to_host(pool_d.data_ptr(), C.byref(lay_g), dev(ids_g).data_ptr(), n,
                                      staging.data_ptr(), None, None) == aibx.ERR_INVALID
    assert lib.aibx_kv_scatter_from_host(pool_d.data_ptr(), C.byref(lay_g), dev(ids_s).data_ptr(), n,
                                         None, src.data_ptr(), None) == aibx.ERR_INVALID
    assert aibx.status_fetch() == (0, 0)


def test_list_longer_than_one_launch_covers():
    """A launch addresses its transfer buffer with 32-bit offsets in 16-byte units, i.e. about
    64 GiB; a longer list is cut into several launches.  13,500 items of the 5 MiB Llama-3-70B
    block shape (65.9 GiB of buffer, ids repeating over a 64-block layer-major pool) cross that
    line after item 13,093: items on both sides of it, and the last one, are checked against the
    oracle, and so is the counted variant, whose device-side count ends inside the second launch."""
    import gc

    gc.collect()
    torch.cuda.empty_cache()                       # earlier tests' pools go back to the driver
    free, _ = torch.cuda.mem_get_info()
    kv = W.scaled(W.cfg4_kv(), num_blocks=64)
    n = 13500
    if free < n * kv.block_bytes + kv.pool_bytes + (8 << 30):
        pytest.skip("needs 75 GiB of free device memory")
    first_launch = ((1 << 32) - (1 << 22)) // (kv.block_bytes // 16)
    assert first_launch == 13094 and n > first_launch
    pool = empty(kv.pool_bytes, torch.uint8)
    synth.fill_pool(pool, kv)
    ids = W.Stream(77, 3).randint(0, kv.num_blocks, n).astype(np.uint32)
    ids[first_launch + 5] = NO_BLOCK                                # a skipped item past the line
    lay, lay1 = kv_layout_gpu(kv), kv_layout_oracle(kv, layout=0, num_blocks=1)
    buf = empty(n * kv.block_bytes, torch.uint8)
    d_ids = dev(ids)

    def check(upto):
        view = buf.view(n, kv.block_bytes)
        for i in (0, 1, first_launch - 1, first_launch, first_launch + 1, first_launch + 5,
                  first_launch + 6, n - 2, n - 1):
            want = np.full(kv.block_bytes, 0xAB, dtype=np.uint8)
            if i < upto and ids[i] != NO_BLOCK:
                oracle.kv_gather(W.logical_blocks(kv, [int(ids[i])]), lay1, np.zeros(1, np.uint32), want)
            assert np.array_equal(host(view[i]), want), i

    buf.fill_(0xAB)
    aibx.kv_gather(pool, lay, d_ids, n, buf)
    assert aibx.status_fetch() == (0, 0)
    check(n)
    buf.fill_(0xAB)
    cnt = first_launch + 3                                          # ends inside the second launch
    aibx.kv_gather_counted(pool, lay, d_ids, n, dev(np.array([cnt], np.uint32)), buf)
    assert aibx.status_fetch() == (0, 0)
    check(cnt)


def test_cfg5_full_size_fp8_mixed():
    kv0 = W.cfg5_kv()
    kv, shrunk = _fit_blocks(kv0, 3000 * kv0.block_bytes + 1000 * kv0.block_bytes)
    per = 4000 if not shrunk else (kv.num_blocks // 32) // 4 * 4
    n_get, n_put = per * 3 // 4, per // 4
    pool = empty(kv.pool_bytes, torch.uint8)
    synth.fill_pool(pool, kv)
    lay = kv_layout_gpu(kv)
    get_buf = empty(n_get * kv.block_bytes, torch.uint8)
    put_buf = empty(n_put * kv.block_bytes, torch.uint8)
    model = PoolModel(kv)
    for r in (0, 13, 31):
        table = (r * per + W.Stream(4, 100 + r).permutation(per)).astype(np.uint32)
        ids_get, ids_put = table[:n_get], table[n_get:]
        aibx.kv_gather(pool, lay, dev(ids_get), n_get, get_buf)
        synth.fill_linear(put_buf, 900 + r)
        aibx.kv_scatter(pool, lay, dev(ids_put), n_put, put_buf)
        assert aibx.status_fetch() == (0, 0)
        assert check_gather_full(model, ids_get, get_buf) == []          # every byte
        model.scattered(ids_put, 900 + r)
        for i in (0, n_put - 1):
            b = int(ids_put[i])
            assert np.array_equal(read_block(pool, kv, b), model.mini_pool(np.array([b]))[0])
    assert check_pool_full(model, pool) == []                            # every byte of the pool
    print("cfg5 pool blocks used:", kv.num_blocks, "(shrunk)" if shrunk else "(full)")


@pytest.mark.parametrize("mode", [0, 1])
@pytest.mark.parametrize("layout", [0, 1, 2])
def test_counted_variants_stop_at_the_device_count(layout, mode):
    aibx.kv_set_tuning(mode, 16384, 4, 1)
    kv = W.KVSpec("counted", 9, layout, 3, 5, 16, 40, 2, 97)          # 38,400-byte blocks
    lay_g, lay_o = kv_layout_gpu(kv), kv_layout_oracle(kv)
    pool_h = W.host_pool(kv)
    ids = W.distinct_ids(4, 97, 60)
    ids[7] = NO_BLOCK
    for cnt in (0, 1, 33, 60, 1000):
        m = min(cnt, 60)
        pool_d = dev(pool_h)
        buf_w, buf_d = guarded(60 * kv.block_bytes, 0xEE)
        d_cnt = dev(np.array([cnt], np.uint32))
        aibx.kv_gather_counted(pool_d, lay_g, dev(ids), 60, d_cnt, buf_d)
        want = np.full(60 * kv.block_bytes, 0xEE, dtype=np.uint8)
        oracle.kv_gather(pool_h, lay_o, ids[:m], want[: m * kv.block_bytes])
        assert np.array_equal(host(buf_d), want), cnt
        assert guards_intact(buf_w, 60 * kv.block_bytes, 0xEE)
        # scatter the first `cnt` items of a fresh buffer into a shuffled id list
        ids_s = W.distinct_ids(5, 97, 60)
        fresh = W.pool_bytes(77, 0, 60 * kv.block_bytes)
        aibx.kv_scatter_counted(pool_d, lay_g, dev(ids_s), 60, d_cnt, dev(fresh))
        pool_want = pool_h.copy()
        oracle.kv_scatter(pool_want, lay_o, ids_s[:m], fresh[: m * kv.block_bytes].copy())
        assert np.array_equal(host(pool_d), pool_want), cnt
        assert aibx.status_fetch() == (0, 0)


def test_latent_single_stream_shape():
    """An MLA-style pool keeps one latent vector per token (no separate K and V).  The bytes are
    opaque to gather/scatter, so such a pool is described by any layout with the same tile size:
    576 latent dims x 16 tokens x 2 bytes = 18,432 bytes = 2 x 1 head x 16 tokens x 288 dims."""
    for layout in (0, 1):
        kv = W.KVSpec("latent", 13, layout, 6, 1, 16, 288, 2, 120)
        assert kv.tile_bytes == 16 * 576 * 2
        ids_g = W.distinct_ids(6, 120, 77)
        ids_s = W.distinct_ids(8, 120, 77)
        check_gather_scatter(kv, ids_g, ids_s, (0, 32768, 3, 1, 1))


def test_a_wait_that_runs_out_becomes_a_status_not_a_hang():
    """The error path of the bounded waits, exercised without any fault: a probe thread waits
    on a barrier nobody completes, gives up after 1,000 polls, and the host reads TIMEOUT; the
    device keeps working."""
    assert aibx.status_fetch() == (0, 0)
    aibx.selftest_bounded_wait(1000)
    st, detail = aibx.status_fetch()
    assert st == aibx.ERR_TIMEOUT and detail == 1
    assert aibx.strerror(st) == "bounded device wait gave up"
    assert aibx.status_fetch() == (0, 0)
    kv = W.cfg1_kv()
    check_gather_scatter(kv, W.distinct_ids(0, 256, 64), W.distinct_ids(100, 256, 64), (0, 32768, 3, 1, 1))
    with pytest.raises(aibx.AibxError):
        aibx.selftest_bounded_wait(0)


def test_calls_from_several_host_threads_while_the_launch_shape_changes():
    """Two host threads gather and scatter on their own streams and pools while a third keeps
    switching the process-wide launch shape: every call reads one whole setting, so every result
    is the oracle's whatever shape each launch happened to get."""
    import threading

    kv = W.KVSpec("mt", 41, 1, 4, 2, 16, 64, 2, 200)                  # 8 KiB tiles, layer-major
    lay_g, lay_o = kv_layout_gpu(kv), kv_layout_oracle(kv)
    pool_h = W.host_pool(kv)
    stop = threading.Event()
    errors = []

    def switcher():
        shapes = [(0, 32768, 3, 1), (0, 4096, 12, 2), (1, 16384, 2, 1), (0, 16384, 6, 1)]
        i = 0
        while not stop.is_set():
            aibx.kv_set_tuning(*shapes[i % len(shapes)])
            aibx.kv_set_store_lag(1 + i % 3)
            i += 1

    def worker(seed):
        try:
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                pool_d = dev(pool_h)
                want_pool = pool_h.copy()
                for it in range(12):
                    ids = W.distinct_ids(seed * 100 + it, kv.num_blocks, 50)
                    buf = torch.zeros(50 * kv.block_bytes, dtype=torch.uint8, device="cuda")
                    aibx.kv_gather(pool_d, lay_g, dev(ids), 50, buf)
                    want = np.zeros(50 * kv.block_bytes, dtype=np.uint8)
                    oracle.kv_gather(want_pool, lay_o, ids, want)
                    stream.synchronize()
                    if not np.array_equal(host(buf), want):
                        errors.append(("gather", seed, it))
                    dst = W.distinct_ids(seed * 100 + it + 50, kv.num_blocks, 50)
                    aibx.kv_scatter(pool_d, lay_g, dev(dst), 50, buf)
                    oracle.kv_scatter(want_pool, lay_o, dst, want)
                stream.synchronize()
                if not np.array_equal(host(pool_d), want_pool):
                    errors.append(("pool", seed))
        except Exception as e:                                        # pragma: no cover
            errors.append(("exception", seed, repr(e)))

    threads = [threading.Thread(target=worker, args=(s,)) for s in (1, 2)]
    sw = threading.Thread(target=switcher)
    sw.start()
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    stop.set()
    sw.join()
    torch.cuda.synchronize()
    assert errors == []
    assert aibx.status_fetch() == (0, 0)


def test_plain_copy_random_shapes_all_layouts():
    """Ninety random shapes (element size, head dim, heads, tokens, layers, pool size; tiles from
    32 bytes to 200 KiB) on the three pool layouts and two launch shapes: gather with repeats,
    skips and out-of-range ids, scatter to distinct ids, every byte against the oracle."""
    done = 0
    for seed in range(90):
        rng = np.random.default_rng(7000 + seed)
        layout = seed % 3
        E = int(rng.choice([1, 2, 4]))
        D = int(rng.choice([16, 32, 64, 128, 256]))
        H = int(rng.integers(1, 9))
        T = int(rng.integers(1, 65))
        L = int(rng.integers(1, 6))
        nb = int(rng.integers(3, 40))
        kv = W.KVSpec("rnd", 300 + seed, layout, L, H, T, D, E, nb)
        half = kv.tile_bytes // 2
        if kv.pool_bytes > (64 << 20) or (layout == 2 and half % 16) or kv.tile_bytes % 16:
            continue
        n = int(rng.integers(1, 3 * nb))
        ids_g = rng.integers(0, nb, n).astype(np.uint32)
        if n > 4:
            ids_g[int(rng.integers(0, n))] = NO_BLOCK
            ids_g[int(rng.integers(0, n))] = nb + int(rng.integers(0, 5))
        m = int(rng.integers(1, nb + 1))
        ids_s = rng.permutation(nb)[:m].astype(np.uint32)
        mode_args = (0, 32768, 3, 1, 1) if seed % 2 == 0 else (0, int(rng.choice([1024, 4096, 16384])),
                                                              int(rng.integers(2, 9)), 1, 1)
        aibx.kv_set_tuning(*mode_args[:4])
        lay_g, lay_o = kv_layout_gpu(kv), kv_layout_oracle(kv)
        pool_h = W.host_pool(kv)
        pool_d = dev(pool_h)
        buf_w, buf_d = guarded(n * kv.block_bytes, 0xEE)
        aibx.kv_gather(pool_d, lay_g, dev(ids_g), n, buf_d)
        want = np.full(n * kv.block_bytes, 0xEE, dtype=np.uint8)
        rc, bad = oracle.kv_gather(pool_h, lay_o, ids_g, want)
        assert np.array_equal(host(buf_d), want), (seed, "gather")
        assert aibx.status_fetch() == ((aibx.ERR_RANGE, bad) if bad else (0, 0)), seed
        assert guards_intact(buf_w, n * kv.block_bytes, 0xEE)
        src = dev(W.pool_bytes(900 + seed, 0, (m * kv.block_bytes + 7) // 8 * 8)[: m * kv.block_bytes])
        aibx.kv_scatter(pool_d, lay_g, dev(ids_s), m, src)
        pool_want = pool_h.copy()
        oracle.kv_scatter(pool_want, lay_o, ids_s, host(src).copy())
        assert np.array_equal(host(pool_d), pool_want), (seed, "scatter")
        assert aibx.status_fetch() == (0, 0)
        done += 1
    assert done >= 60
