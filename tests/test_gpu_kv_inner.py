"""GPU parity for gather/scatter with a change of the order inside a tile (head/token
transposition staged through shared memory), byte for byte against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import NO_BLOCK, dev, empty, host, kv_layout_gpu, kv_layout_oracle
from paper_2504_03648_b200 import binding as aibx
from workloads import synth
import workloads as W

pytestmark = pytest.mark.gpu

SHAPES = [
    # layers, heads, tokens, dim, elem bytes, blocks
    (2, 4, 16, 64, 2, 50),      # 128-byte rows, 8 KiB planes
    (3, 8, 16, 128, 2, 40),     # Llama-class: 256-byte rows, 32 KiB planes (one chunk each)
    (2, 8, 32, 128, 2, 30),     # 64 KiB planes: two chunks per plane
    (2, 5, 7, 24, 2, 33),       # odd counts, 48-byte rows
    (1, 4, 32, 128, 1, 64),     # fp8: 128-byte rows
    (1, 3, 5, 520, 4, 9),       # 2,080-byte rows, 15 rows per chunk of a 15-row plane
    (1, 6, 48, 128, 2, 12),     # boxes of 2 heads x 48 tokens / of 21 tokens x 6 heads (ragged: 21, 21, 6)
    (1, 2, 200, 128, 2, 6),     # one head's 200 rows overflow a stage: boxes of 128 and 72 rows
]

ENGINES = [1, 2]                # storer warps; tensor-map store (no fallback)


@pytest.fixture(autouse=True)
def _default_engine_afterwards():
    yield
    aibx.kv_set_inner_engine(0)


@pytest.mark.parametrize("engine", ENGINES)
@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("layout", [0, 1, 2])
def test_inner_order_gather_and_scatter(layout, shape, engine):
    L, H, T, D, E, nb = shape
    if engine == 2 and D * E > 2048:
        # rows too long for one box: the tensor-map engine says so, the default falls back
        aibx.kv_set_inner_engine(2)
        kv0 = W.KVSpec("inner", 21, layout, L, H, T, D, E, nb)
        with pytest.raises(aibx.AibxError) as e:
            aibx.kv_gather_inner(empty(kv0.pool_bytes, torch.uint8), kv_layout_gpu(kv0), 0, 1,
                                 dev(np.zeros(1, np.uint32)), 1, empty(kv0.block_bytes, torch.uint8))
        assert e.value.code == aibx.ERR_UNSUPPORTED
        engine = 0
    aibx.kv_set_inner_engine(engine)
    kv = W.KVSpec("inner", 21, layout, L, H, T, D, E, nb)
    lay_g, lay_o = kv_layout_gpu(kv), kv_layout_oracle(kv)
    pool_h = W.host_pool(kv)
    rng = np.random.default_rng(L * 100 + H)
    n = 70
    ids_g = rng.integers(0, nb, n).astype(np.uint32)
    ids_g[[2, 40]] = NO_BLOCK
    ids_g[[5, 69]] = [nb, 0xFFFFFFFE]
    ids_s = rng.permutation(nb)[: min(nb, n)].astype(np.uint32)
    ids_s[1] = NO_BLOCK
    for pi, bi in ((0, 1), (1, 0), (0, 0), (1, 1)):
        pool_d = dev(pool_h)
        buf_d = torch.full((n * kv.block_bytes,), 0xEE, dtype=torch.uint8, device="cuda")
        aibx.kv_gather_inner(pool_d, lay_g, pi, bi, dev(ids_g), n, buf_d)
        want = np.full(n * kv.block_bytes, 0xEE, dtype=np.uint8)
        rc, bad = oracle.kv_gather_inner(pool_h, lay_o, pi, bi, ids_g, want)
        assert np.array_equal(host(buf_d), want), (pi, bi)
        assert aibx.status_fetch() == (aibx.ERR_RANGE, bad) and bad == 2
        assert np.array_equal(host(pool_d), pool_h)
        m = len(ids_s)
        aibx.kv_scatter_inner(pool_d, lay_g, pi, bi, dev(ids_s), m, buf_d)
        pool_want = pool_h.copy()
        oracle.kv_scatter_inner(pool_want, lay_o, pi, bi, ids_s, want[: m * kv.block_bytes].copy())
        assert np.array_equal(host(pool_d), pool_want), (pi, bi)
        assert np.array_equal(host(buf_d), want)
        assert aibx.status_fetch() == (0, 0)


def test_inner_order_round_trip_and_invalid():
    kv = W.KVSpec("rt", 22, 1, 2, 8, 16, 128, 2, 64)
    lay = kv_layout_gpu(kv)
    pool_h = W.host_pool(kv)
    pool_d = dev(pool_h)
    ids = W.distinct_ids(9, 64, 48)
    buf = empty(48 * kv.block_bytes, torch.uint8)
    aibx.kv_gather_inner(pool_d, lay, 0, 1, dev(ids), 48, buf)
    plain = empty(48 * kv.block_bytes, torch.uint8)
    aibx.kv_gather(pool_d, lay, dev(ids), 48, plain)
    # the transposed buffer is the plain one with head and token axes swapped
    p = host(plain).reshape(48, 2, 2, 8, 16, 256)
    assert np.array_equal(host(buf).reshape(48, 2, 2, 16, 8, 256), p.transpose(0, 1, 2, 4, 3, 5))
    pool_d.zero_()
    aibx.kv_scatter_inner(pool_d, lay, 0, 1, dev(ids), 48, buf)
    back = empty(48 * kv.block_bytes, torch.uint8)
    aibx.kv_gather(pool_d, lay, dev(ids), 48, back)
    assert torch.equal(back, plain)
    for pi, bi in ((2, 0), (0, -1)):
        with pytest.raises(aibx.AibxError) as e:
            aibx.kv_gather_inner(pool_d, lay, pi, bi, dev(ids), 48, buf)
        assert e.value.code == aibx.ERR_INVALID
    for bad_engine in (-1, 3):
        with pytest.raises(aibx.AibxError) as e:
            aibx.kv_set_inner_engine(bad_engine)
        assert e.value.code == aibx.ERR_INVALID
    odd = aibx.KVLayout(0, 1, 2, 4, 12, 2, 8)                 # 24-byte rows, 384-byte tiles
    with pytest.raises(aibx.AibxError) as e:
        aibx.kv_gather_inner(pool_d, odd, 0, 1, dev(ids[:2]), 2, buf)
    assert e.value.code == aibx.ERR_UNSUPPORTED
    assert aibx.status_fetch() == (0, 0)


@pytest.mark.parametrize("layout", [0, 2])
def test_inner_order_large_launch_bandwidth_shape(layout):
    """cfg2 block shape, 600 blocks out of a 2 GiB pool (block-major, and with K and V of a layer
    as separate tensors): sampled against the oracle, engine against engine in full."""
    kv = W.scaled(W.cfg2_kv(), num_blocks=1000, layout=layout)
    pool = empty(kv.pool_bytes, torch.uint8)
    synth.fill_pool(pool, kv)
    n = 600
    ids = W.distinct_ids(3, kv.num_blocks, n)
    lay = kv_layout_gpu(kv)
    lay1 = kv_layout_oracle(kv, layout=0, num_blocks=1)
    bufs = []
    for engine in (2, 1):
        aibx.kv_set_inner_engine(engine)
        buf = empty(n * kv.block_bytes, torch.uint8)
        aibx.kv_gather_inner(pool, lay, 0, 1, dev(ids), n, buf)
        assert aibx.status_fetch() == (0, 0)
        for i in (0, 1, 299, n - 1):
            mini = W.logical_blocks(kv, [ids[i]])
            want = np.zeros(kv.block_bytes, dtype=np.uint8)
            oracle.kv_gather_inner(mini, lay1, 0, 1, np.zeros(1, np.uint32), want)
            assert np.array_equal(host(buf.view(n, kv.block_bytes)[i]), want)
        bufs.append(buf)
    assert torch.equal(bufs[0], bufs[1])                   # every byte, engine against engine


def test_inner_order_on_the_full_cfg4_pool():
    """The 97.7 GiB layer-major pool of the Llama-3-70B configuration: the tensor map of a
    scatter spans all 3.2 million planes of the pool, and the blocks picked include the last
    ones, so the largest plane coordinates are exercised.  Gathered items and scattered blocks
    are checked against the oracle."""
    import gc

    gc.collect()
    torch.cuda.empty_cache()
    kv = W.cfg4_kv()
    n = 48
    free, _ = torch.cuda.mem_get_info()
    if free < kv.pool_bytes + n * kv.block_bytes + (6 << 30):
        kv = W.scaled(kv, num_blocks=int((free - n * kv.block_bytes - (6 << 30)) // kv.block_bytes))
    nb = kv.num_blocks
    pool = empty(kv.pool_bytes, torch.uint8)
    synth.fill_pool(pool, kv)
    middle = W.distinct_ids(5, nb - 3, n - 3) + 1             # distinct ids in [1, nb - 3]
    ids = np.concatenate([[nb - 1, nb - 2, 0], middle]).astype(np.uint32)
    lay = kv_layout_gpu(kv)
    lay1 = kv_layout_oracle(kv, layout=0, num_blocks=1)
    for engine in (2, 1):
        aibx.kv_set_inner_engine(engine)
        buf = torch.full((n * kv.block_bytes,), 0xCD, dtype=torch.uint8, device="cuda")
        aibx.kv_gather_inner(pool, lay, 0, 1, dev(ids), n, buf)
        assert aibx.status_fetch() == (0, 0)
        for i in (0, 1, 2, n // 2, n - 1):
            want = np.zeros(kv.block_bytes, dtype=np.uint8)
            oracle.kv_gather_inner(W.logical_blocks(kv, [int(ids[i])]), lay1, 0, 1,
                                   np.zeros(1, np.uint32), want)
            assert np.array_equal(host(buf.view(n, kv.block_bytes)[i]), want), (engine, i)
        # scatter other content into the same blocks, converting back on the way
        synth.fill_linear(buf, 900 + engine)
        aibx.kv_scatter_inner(pool, lay, 0, 1, dev(ids), n, buf)
        assert aibx.status_fetch() == (0, 0)
        for i in (0, 1, n - 1):
            item = W.pool_bytes(900 + engine, i * kv.block_bytes, kv.block_bytes)
            want = np.zeros(kv.block_bytes, dtype=np.uint8)
            oracle.kv_scatter_inner(want, lay1, 0, 1, np.zeros(1, np.uint32), item)
            got = host(pool.view(kv.num_layers, nb, kv.tile_bytes)[:, int(ids[i])].contiguous()).reshape(-1)
            assert np.array_equal(got, want), (engine, i)
        synth.fill_pool(pool, kv)                             # generated content again


def test_inner_order_random_shapes():
    """Sixty random shapes (element size, row length, heads, tokens, layers, layout; planes from
    a few rows to several stages, ragged boxes): the tensor-map engine against the oracle, and
    against the storer-warp engine byte for byte, gather and scatter, both directions of the swap."""
    done = 0
    for seed in range(60):
        rng = np.random.default_rng(900 + seed)
        E = int(rng.choice([1, 2, 4]))
        D = int(rng.choice([16, 32, 64, 128, 256]))
        H = int(rng.integers(1, 20))
        T = int(rng.integers(1, 300 if rng.random() < 0.2 else 40))
        L, layout = int(rng.integers(1, 4)), int(rng.integers(0, 3))
        nb = int(rng.integers(2, 10))
        kv = W.KVSpec("rnd", seed, layout, L, H, T, D, E, nb)
        if kv.pool_bytes > (256 << 20):
            continue
        lay_g, lay_o = kv_layout_gpu(kv), kv_layout_oracle(kv)
        pool_h = W.host_pool(kv)
        n = int(rng.integers(1, 2 * nb))
        ids = rng.integers(0, nb, n).astype(np.uint32)
        ids_s = rng.permutation(nb)[: min(nb, n)].astype(np.uint32)
        for pi, bi in ((0, 1), (1, 0)):
            want = np.zeros(n * kv.block_bytes, dtype=np.uint8)
            oracle.kv_gather_inner(pool_h, lay_o, pi, bi, ids, want)
            bufs = []
            for engine in (2, 1):
                aibx.kv_set_inner_engine(engine)
                buf = empty(n * kv.block_bytes, torch.uint8)
                aibx.kv_gather_inner(dev(pool_h), lay_g, pi, bi, dev(ids), n, buf)
                bufs.append(buf)
            assert np.array_equal(host(bufs[0]), want), (seed, pi, bi)
            assert torch.equal(bufs[0], bufs[1]), (seed, pi, bi)
            m = len(ids_s)
            pool_want = pool_h.copy()
            oracle.kv_scatter_inner(pool_want, lay_o, pi, bi, ids_s, want[: m * kv.block_bytes].copy())
            for engine in (2, 1):
                aibx.kv_set_inner_engine(engine)
                pool_d = dev(pool_h)
                aibx.kv_scatter_inner(pool_d, lay_g, pi, bi, dev(ids_s), m, bufs[0])
                assert np.array_equal(host(pool_d), pool_want), (seed, pi, bi, engine)
            done += 1
    assert done >= 100 and aibx.status_fetch() == (0, 0)
