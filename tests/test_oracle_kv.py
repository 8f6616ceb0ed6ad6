"""Pins for paged-KV gather/scatter (CPU only): library index_select, direct indexing,
round trips, untouched bytes."""
import numpy as np
import pytest
import torch

import oracle

NO_BLOCK = 0xFFFFFFFF


def _pool(rng, layout, L, nb, tile):
    shape = (nb, L, tile) if layout == 0 else (L, nb, tile)
    return rng.integers(0, 256, shape, dtype=np.uint8)


def _split_pool(rng, L, nb, half):
    """Layout 2: K and V of a layer are separate tensors, [layer][K/V][block][half tile]."""
    return rng.integers(0, 256, (L, 2, nb, half), dtype=np.uint8)


def test_split_kv_gather_is_index_select_per_plane():
    rng = np.random.default_rng(77)
    L, H, Bt, D, E, nb = 3, 2, 4, 8, 2, 19
    half = H * Bt * D * E
    pool = _split_pool(rng, L, nb, half)
    ids = rng.integers(0, nb, 13).astype(np.uint32)
    lay = oracle.kv_layout(2, L, H, Bt, D, E, nb)
    buf = np.zeros(13 * L * 2 * half, dtype=np.uint8)
    before = pool.copy()
    rc, bad = oracle.kv_gather(pool.reshape(-1), lay, ids, buf)
    assert rc == oracle.OK and bad == 0 and np.array_equal(pool, before)
    # library form: select the blocks on the block axis, then bring the item axis to the front
    tp = torch.from_numpy(pool)
    want = torch.index_select(tp, 2, torch.from_numpy(ids.astype(np.int64)))    # [L][2][n][half]
    want = want.permute(2, 0, 1, 3).contiguous()                                # [n][L][2][half]
    assert np.array_equal(buf, want.numpy().reshape(-1))
    # the same content held layer-major gathers to the same buffer
    lm = np.ascontiguousarray(pool.transpose(0, 2, 1, 3))                       # [L][nb][2][half]
    buf1 = np.zeros_like(buf)
    oracle.kv_gather(lm.reshape(-1), oracle.kv_layout(1, L, H, Bt, D, E, nb), ids, buf1)
    assert np.array_equal(buf, buf1)


def test_split_kv_hand_example_and_scatter():
    # 2 layers, 3 blocks, half tile of 1 byte... a row must hold 1 head x 1 token x 1 dim x 1 byte
    lay = oracle.kv_layout(2, 2, 1, 1, 1, 1, 3)
    # pool bytes [layer][K/V][block]: K of layer 0 = 0,1,2  V of layer 0 = 3,4,5  K1 = 6,7,8  V1 = 9,10,11
    pool = np.arange(12, dtype=np.uint8)
    buf = np.zeros(8, dtype=np.uint8)
    rc, _ = oracle.kv_gather(pool, lay, np.array([2, 0], np.uint32), buf)
    assert rc == oracle.OK
    # item 0 = block 2: (l0 K, l0 V, l1 K, l1 V) = 2, 5, 8, 11; item 1 = block 0: 0, 3, 6, 9
    assert buf.tolist() == [2, 5, 8, 11, 0, 3, 6, 9]
    out = np.full(12, 0xEE, dtype=np.uint8)
    rc, _ = oracle.kv_scatter(out, lay, np.array([1, NO_BLOCK, 0], np.uint32),
                              np.arange(100, 112, dtype=np.uint8))
    # item 0 (100..103) -> block 1, item 2 (108..111) -> block 0, block 2 untouched
    assert out.tolist() == [108, 100, 0xEE, 109, 101, 0xEE, 110, 102, 0xEE, 111, 103, 0xEE]


def test_split_kv_round_trips_and_inner_order():
    rng = np.random.default_rng(78)
    L, H, Bt, D, E, nb = 2, 3, 4, 8, 1, 11
    row = D * E
    half = H * Bt * row
    pool = _split_pool(rng, L, nb, half)
    lay = oracle.kv_layout(2, L, H, Bt, D, E, nb)
    ids = rng.permutation(nb)[:7].astype(np.uint32)
    buf = np.zeros(7 * L * 2 * half, dtype=np.uint8)
    oracle.kv_gather(pool.reshape(-1), lay, ids, buf)
    fresh = np.zeros_like(pool)
    oracle.kv_scatter(fresh.reshape(-1), lay, ids, buf)
    assert np.array_equal(fresh[:, :, ids], pool[:, :, ids])
    rest = np.setdiff1d(np.arange(nb), ids)
    assert not fresh[:, :, rest].any()
    # inner-order change: [head][token] rows of every plane become [token][head]
    got = np.zeros_like(buf)
    rc, _ = oracle.kv_gather_inner(pool.reshape(-1), lay, 0, 1, ids, got)
    assert rc == oracle.OK
    want = buf.reshape(7, L, 2, H, Bt, row).transpose(0, 1, 2, 4, 3, 5)
    assert np.array_equal(got, np.ascontiguousarray(want).reshape(-1))
    back = np.zeros_like(pool)
    oracle.kv_scatter_inner(back.reshape(-1), lay, 0, 1, ids, got)
    assert np.array_equal(back[:, :, ids], pool[:, :, ids])


@pytest.mark.parametrize("layout", [0, 1])
def test_gather_is_index_select(layout):
    rng = np.random.default_rng(layout)
    L, H, Bt, D, E, nb = 3, 2, 4, 8, 2, 17
    tile = 2 * H * Bt * D * E
    pool = _pool(rng, layout, L, nb, tile)
    ids = rng.integers(0, nb, 11).astype(np.uint32)          # repeats allowed
    lay = oracle.kv_layout(layout, L, H, Bt, D, E, nb)
    buf = np.zeros(11 * L * tile, dtype=np.uint8)
    pool_before = pool.copy()
    rc, bad = oracle.kv_gather(pool.reshape(-1), lay, ids, buf)
    assert rc == oracle.OK and bad == 0
    assert np.array_equal(pool, pool_before)                # the source side is only read
    tp = torch.from_numpy(pool)
    ti = torch.from_numpy(ids.astype(np.int64))
    if layout == 0:
        want = torch.index_select(tp, 0, ti)
    else:
        want = tp[:, ti].transpose(0, 1).contiguous()
    assert np.array_equal(buf, want.numpy().reshape(-1))


@pytest.mark.parametrize("layout", [0, 1])
def test_scatter_direct_indexing_and_round_trips(layout):
    rng = np.random.default_rng(10 + layout)
    L, H, Bt, D, E, nb = 4, 1, 2, 4, 1, 23
    tile = 2 * H * Bt * D * E
    pool = _pool(rng, layout, L, nb, tile)
    lay = oracle.kv_layout(layout, L, H, Bt, D, E, nb)
    ids = rng.permutation(nb)[:9].astype(np.uint32)
    buf = rng.integers(0, 256, 9 * L * tile, dtype=np.uint8)
    before = pool.copy()
    buf_before = buf.copy()
    flat = pool.reshape(-1)
    rc, bad = oracle.kv_scatter(flat, lay, ids, buf)
    assert rc == oracle.OK
    assert np.array_equal(buf, buf_before)                  # the source side is only read
    b3 = buf_before.reshape(9, L, tile)
    touched = np.zeros(nb, dtype=bool)
    for i, b in enumerate(ids):
        got = pool[b] if layout == 0 else pool[:, b]
        assert np.array_equal(got, b3[i])
        touched[b] = True
    rest = ~touched
    if layout == 0:
        assert np.array_equal(pool[rest], before[rest])
    else:
        assert np.array_equal(pool[:, rest], before[:, rest])
    # gather after scatter returns the buffer; scatter after gather leaves the pool alone
    back = np.zeros_like(buf)
    oracle.kv_gather(flat, lay, ids, back)
    assert np.array_equal(back, buf)
    snap = pool.copy()
    oracle.kv_scatter(flat, lay, ids, back)
    assert np.array_equal(pool, snap)


def test_skips_and_range_errors():
    L, H, Bt, D, E, nb = 2, 1, 1, 8, 1, 5
    tile = 2 * H * Bt * D * E
    pool = np.arange(nb * L * tile, dtype=np.uint8)
    lay = oracle.kv_layout(0, L, H, Bt, D, E, nb)
    ids = np.array([1, NO_BLOCK, 7, 4], dtype=np.uint32)
    buf = np.full(4 * L * tile, 0xEE, dtype=np.uint8)
    rc, bad = oracle.kv_gather(pool, lay, ids, buf)
    assert rc == oracle.ERR_RANGE and bad == 1
    bb = buf.reshape(4, L * tile)
    pp = pool.reshape(nb, L * tile)
    assert np.array_equal(bb[0], pp[1]) and np.array_equal(bb[3], pp[4])
    assert (bb[1] == 0xEE).all() and (bb[2] == 0xEE).all()
    snap = pool.copy()
    rc, bad = oracle.kv_scatter(pool, lay, np.array([NO_BLOCK, 9], dtype=np.uint32),
                                buf[:2 * L * tile].copy())
    assert rc == oracle.ERR_RANGE and bad == 1 and np.array_equal(pool, snap)
    rc, bad = oracle.kv_gather(pool, lay, np.zeros(0, dtype=np.uint32), buf)
    assert rc == oracle.OK


@pytest.mark.parametrize("layout", [0, 1])
def test_inner_order_change_is_a_numpy_transpose(layout):
    rng = np.random.default_rng(40 + layout)
    L, H, Bt, D, E, nb = 3, 4, 6, 8, 2, 13
    row = D * E
    tile = 2 * H * Bt * row
    pool = _pool(rng, layout, L, nb, tile)
    lay = oracle.kv_layout(layout, L, H, Bt, D, E, nb)
    ids = rng.integers(0, nb, 9).astype(np.uint32)
    ids[4] = NO_BLOCK
    plain = np.full(9 * L * tile, 0xEE, dtype=np.uint8)
    oracle.kv_gather(pool.reshape(-1), lay, ids, plain)
    for pi in (0, 1):
        for bi in (0, 1):
            got = np.full(9 * L * tile, 0xEE, dtype=np.uint8)
            rc, bad = oracle.kv_gather_inner(pool.reshape(-1), lay, pi, bi, ids, got)
            assert rc == oracle.OK
            # view the plainly gathered tiles in the pool's inner order, reorder with numpy
            shape_p = (9, L, 2, H, Bt, row) if pi == 0 else (9, L, 2, Bt, H, row)
            v = plain.reshape(shape_p)
            want = v if pi == bi else v.transpose(0, 1, 2, 4, 3, 5)
            want = np.ascontiguousarray(want).reshape(-1)
            assert np.array_equal(got, want), (pi, bi)
            # scatter with the same orders brings every named block back
            pool2 = np.zeros_like(pool)
            keep = ids != NO_BLOCK
            oracle.kv_scatter_inner(pool2.reshape(-1), lay, pi, bi, ids, got)
            for b in set(ids[keep].tolist()):
                a = pool[b] if layout == 0 else pool[:, b]
                c = pool2[b] if layout == 0 else pool2[:, b]
                assert np.array_equal(a, c)


def test_inner_order_hand_example():
    # one block, one layer, 2 heads x 3 tokens, rows of 1 byte: K rows 0..5, V rows 6..11
    lay = oracle.kv_layout(0, 1, 2, 3, 1, 1, 1)
    pool = np.arange(12, dtype=np.uint8)                 # [kv][head][token]
    buf = np.zeros(12, dtype=np.uint8)
    oracle.kv_gather_inner(pool, lay, 0, 1, np.zeros(1, np.uint32), buf)
    assert buf.tolist() == [0, 3, 1, 4, 2, 5, 6, 9, 7, 10, 8, 11]   # [kv][token][head]
    back = np.zeros(12, dtype=np.uint8)
    oracle.kv_scatter_inner(back, lay, 0, 1, np.zeros(1, np.uint32), buf)
    assert back.tolist() == list(range(12))
    rc, _ = oracle.kv_gather_inner(pool, lay, 2, 0, np.zeros(1, np.uint32), buf)
    assert rc == oracle.ERR_INVALID
