"""GPU parity, routing half of the path: prefix keys, index, longest cached prefix, route
score, matched-block set.  Every comparison is bit-exact against the CPU oracle on the same
seeded inputs; all calls go through the C ABI."""
import os

import numpy as np
import pytest
import torch

import oracle
from gpu_util import (NO_BLOCK, assert_routing_equal, dev, empty, gpu_hash, host, routing_gpu,
                      routing_oracle)
from paper_2504_03648_b200 import binding as aibx
import workloads as W

pytestmark = pytest.mark.gpu
ALL = (1 << 64) - 1


# ------------------------------------------------------------------ prefix keys

def test_hash_stored_chains():
    path = os.path.join(os.path.dirname(__file__), "golden", "hash_chains.txt")
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        head, vals = line.split(":")
        name, B, root, rule, n = head.split()
        B, root, n = int(B), int(root), int(n)
        j = np.arange(n, dtype=np.int64)
        toks = j.astype(np.int32) if rule == "iota" else ((1000003 * j + 7) % 128256).astype(np.int32)
        h, _ = gpu_hash(toks, np.array([0, n]), B, root)
        assert [int(x) for x in h] == [int(v, 16) for v in vals.split()], name


@pytest.mark.parametrize("B", [8, 16, 32, 40, 64, 256, 1024])
def test_hash_ragged_batch(B):
    rng = np.random.default_rng(B)
    # lengths around step boundaries (a warp step is 256 tokens), empty and sub-block requests,
    # odd starts so that requests begin at every alignment inside a 16-byte vector
    lens = [0, 1, B - 1, B, B + 1, 255, 256, 257, 511, 513, 1027, 2 * B + 3, 4099, 0, 7, 3000]
    toks = rng.integers(-2**31, 2**31 - 1, sum(lens), dtype=np.int64).astype(np.int32)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    for root in (0, 0xDEADBEEFCAFEF00D):
        want, _ = oracle.hash_blocks(toks, off, B, root)
        got, _ = gpu_hash(toks, off, B, root)
        assert np.array_equal(got, want)


def test_hash_unaligned_token_base():
    rng = np.random.default_rng(1)
    toks = rng.integers(0, 32000, 1000).astype(np.int32)
    big = dev(np.concatenate([np.full(3, -1, np.int32), toks]))
    for shift in (1, 2, 3):                       # token array starting 4, 8, 12 bytes off
        view = big[shift:]
        n = view.numel()
        sub = host(view)
        off = np.array([0, 100, 100, 517, n], dtype=np.int64)
        bo = oracle.block_offsets(off, 16)
        d_h = empty(int(bo[-1]), torch.uint64)
        aibx.hash_blocks(view, dev(off), dev(bo), 16, 5, d_h)
        want, _ = oracle.hash_blocks(sub, off, 16, 5)
        assert np.array_equal(host(d_h), want)


def test_hash_invalid_arguments():
    t = empty(64, torch.int32)
    off = dev(np.array([0, 64], dtype=np.int64))
    bo = dev(np.array([0, 4], dtype=np.int64))
    h = empty(4, torch.uint64)
    for B in (0, 12, -16, 2048):
        with pytest.raises(aibx.AibxError) as e:
            aibx.hash_blocks(t, off, bo, B, 0, h)
        assert e.value.code == aibx.ERR_INVALID
    lib = aibx.lib()
    assert lib.aibx_hash_blocks(None, None, None, 0, 16, 0, None, None) == 0      # R = 0: no-op
    assert lib.aibx_hash_blocks(None, off.data_ptr(), bo.data_ptr(), 1, 16, 0, h.data_ptr(), None) == -1


# ------------------------------------------------------------------ index

def _rand_ops(rng, universe, P, n_ops, max_batch):
    ops = []
    for _ in range(n_ops):
        kind = "insert" if rng.random() < 0.6 else "evict"
        n = int(rng.integers(0, max_batch + 1))
        keys = rng.choice(universe, n).astype(np.uint64)
        masks = rng.integers(0, 1 << min(P + 1, 63), n).astype(np.uint64)
        if kind == "evict" and n:
            masks[rng.random(n) < 0.3] = np.uint64(ALL)
        ids = rng.integers(0, 1000, n).astype(np.uint32)
        if n:
            ids[rng.random(n) < 0.1] = NO_BLOCK
        ops.append((kind, keys, masks, ids))
    return ops


@pytest.mark.parametrize("capacity,P,n_keys", [(8, 1, 4), (16, 3, 8), (64, 6, 30), (64, 64, 32),
                                                (4096, 16, 2000)])
def test_index_random_ops(capacity, P, n_keys):
    rng = np.random.default_rng(capacity + P)
    universe = np.concatenate([rng.integers(1, 1 << 63, n_keys).astype(np.uint64),
                               np.array([0, ALL], dtype=np.uint64)])
    probe = np.concatenate([universe, rng.integers(1, 1 << 63, 16).astype(np.uint64)])
    g, o = aibx.Index(capacity, P), oracle.Index(capacity, P)
    for kind, keys, masks, ids in _rand_ops(rng, universe, P, 25, n_keys):
        if kind == "insert":
            assert o.insert(keys, masks, ids) == oracle.OK
            g.insert(dev(keys), dev(masks), dev(ids)) if len(keys) else None
        else:
            rc, want_freed = o.evict(keys, masks)
            if len(keys):
                d_f = empty(len(keys), torch.uint32)
                g.evict(dev(keys), dev(masks), d_f)
                assert np.array_equal(host(d_f), want_freed)
        assert aibx.status_fetch() == (0, 0)   # removed slots are reused: never FULL here
        d_m, d_i = empty(len(probe), torch.uint64), empty(len(probe), torch.uint32)
        g.lookup(dev(probe), d_m, d_i)
        wm, wi = o.lookup(probe)
        assert np.array_equal(host(d_m), wm) and np.array_equal(host(d_i), wi)
        assert g.stats() == (o.stats()[0], capacity)


def test_index_colliding_keys_wrap_around():
    # brute-force search for keys sharing the last home slot of a 16-slot table is not needed:
    # with 14 of 16 slots taken every probe sequence wraps
    rng = np.random.default_rng(0)
    keys = rng.integers(1, 1 << 63, 14).astype(np.uint64)
    masks = rng.integers(1, 8, 14).astype(np.uint64)
    ids = np.arange(14, dtype=np.uint32)
    g, o = aibx.Index(16, 3), oracle.Index(16, 3)
    g.insert(dev(keys), dev(masks), dev(ids)); o.insert(keys, masks, ids)
    probe = np.concatenate([keys, rng.integers(1, 1 << 63, 50).astype(np.uint64)])
    d_m, d_i = empty(len(probe), torch.uint64), empty(len(probe), torch.uint32)
    g.lookup(dev(probe), d_m, d_i)
    wm, wi = o.lookup(probe)
    assert np.array_equal(host(d_m), wm) and np.array_equal(host(d_i), wi)
    assert aibx.status_fetch() == (0, 0)


def test_index_full_is_reported_not_hung():
    g, o = aibx.Index(8, 1), oracle.Index(8, 1)
    keys = np.arange(1, 10, dtype=np.uint64)
    ones, zeros = np.ones(9, dtype=np.uint64), np.zeros(9, dtype=np.uint32)
    assert o.insert(keys, ones, zeros) == oracle.ERR_FULL
    g.insert(dev(keys), dev(ones), dev(zeros))
    st, detail = aibx.status_fetch()
    assert st == aibx.ERR_FULL and detail == 1
    assert aibx.status_fetch() == (0, 0)            # fetch resets the record
    g.clear()
    assert g.stats() == (0, 8)


def test_index_invalid_arguments():
    for cap, P in [(12, 4), (4, 4), (16, 0), (16, 65)]:
        with pytest.raises(aibx.AibxError) as e:
            aibx.Index(cap, P)
        assert e.value.code == aibx.ERR_INVALID
    g = aibx.Index(16, 2)
    lib = aibx.lib()
    assert lib.aibx_index_insert(g._h, None, None, None, 0, None) == 0
    assert lib.aibx_index_insert(g._h, None, None, None, 3, None) == -1
    assert lib.aibx_index_insert(g._h, None, None, None, -1, None) == -1
    assert lib.aibx_index_evict(None, None, None, None, 0, None) == -1


def test_duplicate_keys_in_one_batch_are_order_free():
    rng = np.random.default_rng(12)
    base = rng.integers(1, 1 << 63, 50).astype(np.uint64)
    keys = np.repeat(base, 40)                      # 40 threads racing on each key
    masks = rng.integers(0, 1 << 10, len(keys)).astype(np.uint64)
    ids = rng.integers(0, 1 << 20, len(keys)).astype(np.uint32)
    perm = rng.permutation(len(keys))
    g, o = aibx.Index(256, 10), oracle.Index(256, 10)
    g.insert(dev(keys[perm]), dev(masks[perm]), dev(ids[perm])); o.insert(keys, masks, ids)
    d_m, d_i = empty(50, torch.uint64), empty(50, torch.uint32)
    g.lookup(dev(base), d_m, d_i)
    wm, wi = o.lookup(base)
    assert np.array_equal(host(d_m), wm) and np.array_equal(host(d_i), wi)
    assert g.stats()[0] == o.stats()[0]
    # evict the same key many times in one batch: every duplicate reports the same id
    ek = np.repeat(base[:5], 7)
    em = np.full(len(ek), ALL, dtype=np.uint64)
    d_f = empty(len(ek), torch.uint32)
    g.evict(dev(ek), dev(em), d_f)
    rc, wf = o.evict(ek, em)
    assert np.array_equal(host(d_f), wf) and g.stats()[0] == o.stats()[0]


# ------------------------------------------------------------------ whole routing path

def test_routing_cfg1_tiny():
    w = W.build_routing(W.cfg1_routing())
    g, o = routing_gpu(w), routing_oracle(w)
    assert_routing_equal(g, o)
    assert o["any_len"].max() == 8                  # the shared 128-token prefixes are found


def test_match_hand_example():
    A, B, C, D = 0xA1, 0xB2, 0xC3, 0xD4
    g = aibx.Index(16, 3)
    g.insert(dev(np.array([A, B, C], np.uint64)), dev(np.array([3, 1, 6], np.uint64)),
             dev(np.array([5, 9, 2], np.uint32)))
    ml, al, ids = empty(3, torch.uint32), empty(1, torch.uint32), empty(4, torch.uint32)
    g.match_prefix(dev(np.array([A, B, C, D], np.uint64)), dev(np.array([0, 4], np.int64)), ml, al, ids)
    assert host(ml).tolist() == [2, 1, 0] and host(al).tolist() == [3]
    assert host(ids).tolist() == [5, 9, 2, NO_BLOCK]
    bp, bs, sc = empty(1, torch.int32), empty(1, torch.int64), empty(3, torch.int64)
    aibx.route_score(ml, dev(np.array([0, 4], np.int64)), 3, dev(np.array([10, 3, 0], np.int32)), 7,
                     (4, 1, 50), bp, bs, sc)
    assert host(sc).tolist() == [-2, -3, 0] and host(bp).tolist() == [2] and host(bs).tolist() == [0]
    aibx.route_score(ml, dev(np.array([0, 4], np.int64)), 3, dev(np.array([5, 3, 9], np.int32)), 0,
                     None, bp, bs, None)
    assert host(bp).tolist() == [aibx.NO_POD] and host(bs).tolist() == [-(1 << 63)]


@pytest.mark.parametrize("wide", [False, True])
@pytest.mark.parametrize("R", [1, 3, 40, 200, 700, 1500, 5000])
def test_match_group_shapes_and_holes(R, wide):
    """Every warps-per-request choice (R picks it) on both entry widths of the index (up to 32
    pods / more), requests of 0..600 blocks, random holes."""
    rng = np.random.default_rng(R + 100 * wide)
    P = int(rng.integers(33, 65)) if wide else int(rng.integers(1, 33))
    lens = rng.integers(0, 600 if R < 100 else 80, R)
    lens[rng.random(R) < 0.1] = 0
    bo = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    hashes = rng.integers(1, 1 << 63, int(bo[-1])).astype(np.uint64)
    allm = ALL if P == 64 else (1 << P) - 1
    masks = np.full(len(hashes), allm, dtype=np.uint64)
    # pods drop out at random places; some blocks are absent altogether; a few reserved keys
    drop = rng.random(len(hashes)) < 0.02
    masks[drop] &= rng.integers(0, 1 << 62, int(drop.sum())).astype(np.uint64)
    present = rng.random(len(hashes)) > 0.004
    hashes[rng.random(len(hashes)) < 0.0005] = 0
    ids = rng.integers(0, 1 << 20, len(hashes)).astype(np.uint32)
    cap = 1 << int(np.ceil(np.log2(max(2 * len(hashes), 8))))
    g, o = aibx.Index(cap, P), oracle.Index(cap, P)
    sel = present & (masks != 0)
    o.insert(hashes[sel], masks[sel], ids[sel])
    if sel.any():
        g.insert(dev(hashes[sel]), dev(masks[sel]), dev(ids[sel]))
    nb = max(len(hashes), 1)
    d_ml, d_al, d_ids = empty(R * P, torch.uint32), empty(R, torch.uint32), empty(nb, torch.uint32)
    g.match_prefix(dev(hashes) if len(hashes) else empty(1, torch.uint64), dev(bo), d_ml, d_al, d_ids)
    wml, wal, wids = o.match_prefix(hashes, bo)
    assert np.array_equal(host(d_ml).reshape(R, P), wml)
    assert np.array_equal(host(d_al), wal)
    assert np.array_equal(host(d_ids)[: len(hashes)], wids)
    # nullable outputs
    d_ml2 = empty(R * P, torch.uint32)
    g.match_prefix(dev(hashes) if len(hashes) else empty(1, torch.uint64), dev(bo), d_ml2, None, None)
    assert np.array_equal(host(d_ml2), host(d_ml))
    assert aibx.status_fetch() == (0, 0)


def test_route_score_parameters_and_ready_masks():
    rng = np.random.default_rng(77)
    for P in (1, 7, 32, 33, 64):
        R = 300
        n = rng.integers(0, 60, R)
        bo = np.concatenate([[0], np.cumsum(n)]).astype(np.int64)
        ml = (rng.random((R, P)) * (n[:, None] + 1)).astype(np.uint32)
        load = rng.integers(0, 5, P).astype(np.int32)
        for ready in (ALL, 0, 1 << (P - 1), int(rng.integers(0, 1 << 62)) & ((1 << P) - 1)):
            for prm in (None, (4, 1, 50), (0, 1, 50), (1, 0, 0), (-3, -2, 120), (2**31 - 1, 2**31 - 1, 100)):
                d_bp, d_bs, d_sc = empty(R, torch.int32), empty(R, torch.int64), empty(R * P, torch.int64)
                aibx.route_score(dev(ml.reshape(-1)), dev(bo), P, dev(load), ready, prm, d_bp, d_bs, d_sc)
                wbp, wbs, wsc = oracle.route_score(ml, bo, load, ready, prm)
                assert np.array_equal(host(d_bp), wbp), (P, ready, prm)
                assert np.array_equal(host(d_bs), wbs)
                assert np.array_equal(host(d_sc).reshape(R, P), wsc)


def test_collect_blocks():
    rng = np.random.default_rng(6)
    for num_blocks, n in [(1, 5), (31, 100), (32, 100), (33, 1000), (4096, 14000), (100000, 3000),
                          (1 << 20, 70000)]:
        ids = rng.integers(0, num_blocks + num_blocks // 8 + 1, n).astype(np.uint32)
        ids[rng.random(n) < 0.2] = NO_BLOCK
        scratch = torch.full((aibx.collect_scratch_bytes(num_blocks) // 4 + 1,), 0x5A5A5A5A,
                             dtype=torch.int32, device="cuda")     # dirty scratch on entry
        d_un, d_cnt = empty(n, torch.uint32), empty(1, torch.uint32)
        aibx.collect_blocks(dev(ids), num_blocks, scratch, d_un, d_cnt)
        rc, wun, wcnt = oracle.collect_blocks(ids, num_blocks)
        assert int(host(d_cnt)[0]) == wcnt and np.array_equal(host(d_un), wun)
        st, detail = aibx.status_fetch()
        n_bad = int(((ids >= num_blocks) & (ids != NO_BLOCK)).sum())
        assert (st == aibx.ERR_RANGE) == (rc == oracle.ERR_RANGE) and detail == n_bad
    d_cnt = torch.full((1,), 9, dtype=torch.int32, device="cuda").view(torch.uint32)
    aibx.collect_blocks(empty(0, torch.uint32), 64, empty(2, torch.uint32), empty(0, torch.uint32), d_cnt)
    assert int(host(d_cnt)[0]) == 0


# ------------------------------------------------------------------ configurations at full size

def test_routing_cfg2_full():
    w = W.build_routing(W.cfg2_routing())
    g, o = routing_gpu(w), routing_oracle(w)
    assert_routing_equal(g, o)
    assert o["count"] > 1000                        # thousands of distinct matched blocks


def test_routing_cfg3_full():
    w = W.build_routing(W.cfg3_routing())
    g, o = routing_gpu(w), routing_oracle(w)
    assert_routing_equal(g, o)
    for prm in ((4, 1, 0), (4, 1, 25)):
        P, R = w.spec.num_pods, w.spec.R
        d_bp, d_bs = empty(R, torch.int32), empty(R, torch.int64)
        aibx.route_score(dev(o["match_len"].reshape(-1)), dev(o["blk_off"]), P, dev(w.pod_load),
                         w.ready_mask, prm, d_bp, d_bs, None)
        wbp, wbs, _ = oracle.route_score(o["match_len"], o["blk_off"], w.pod_load, w.ready_mask, prm)
        assert np.array_equal(host(d_bp), wbp) and np.array_equal(host(d_bs), wbs)


def test_routing_cfg5_full():
    w = W.build_routing(W.cfg5_routing())
    g, o = routing_gpu(w), routing_oracle(w)
    assert_routing_equal(g, o)
    assert (o["any_len"] == 3000).all()
    for r in range(w.spec.R):                       # matched ids are the request's block table
        seg = o["block_ids"][o["blk_off"][r]: o["blk_off"][r] + 3000]
        assert np.array_equal(seg, w.block_table[r, :3000])


# ------------------------------------------------------------------ fused call, sequential assignment

@pytest.mark.parametrize("mk", [W.cfg1_routing, W.cfg2_routing, W.cfg3_routing])
def test_route_batch_equals_the_three_calls(mk):
    w = W.build_routing(mk())
    s = w.spec
    B, P, R = s.block_tokens, s.num_pods, s.R
    o = routing_oracle(w)
    sh, _ = gpu_hash(w.src_tokens, w.src_tok_off, B)
    from gpu_util import fill_entries
    keys, masks, ids = fill_entries(w, sh)
    ix = aibx.Index(s.capacity, P)
    ix.insert(dev(keys), dev(masks), dev(ids))
    bo = o["blk_off"]
    nb = max(int(bo[-1]), 1)
    d_h = empty(nb, torch.uint64)
    d_ml, d_al, d_ids = empty(R * P, torch.uint32), empty(R, torch.uint32), empty(nb, torch.uint32)
    d_bp, d_bs = empty(R, torch.int32), empty(R, torch.int64)
    for prm, ready in ((None, w.ready_mask), ((7, 3, 25), w.ready_mask & 0xF0F0F0F0F0F0F0F5)):
        aibx.route_batch(ix, dev(w.tokens), dev(w.tok_off), dev(bo), B, 0, dev(w.pod_load), ready,
                         prm, d_h, d_ml, d_al, d_ids, d_bp, d_bs)
        wbp, wbs, _ = oracle.route_score(o["match_len"], bo, w.pod_load, ready, prm)
        n = int(bo[-1])
        assert np.array_equal(host(d_h)[:n], o["hashes"])
        assert np.array_equal(host(d_ml).reshape(R, P), o["match_len"])
        assert np.array_equal(host(d_al), o["any_len"])
        assert np.array_equal(host(d_ids)[:n], o["block_ids"])
        assert np.array_equal(host(d_bp), wbp) and np.array_equal(host(d_bs), wbs)
    # nullable outputs
    aibx.route_batch(ix, dev(w.tokens), dev(w.tok_off), dev(bo), B, 0, dev(w.pod_load),
                     w.ready_mask, None, d_h, d_ml, None, None, d_bp, d_bs)
    assert np.array_equal(host(d_bp), o["best_pod"])
    assert aibx.status_fetch() == (0, 0)


def test_route_assign_sequential():
    rng = np.random.default_rng(55)
    for P in (1, 5, 32, 33, 64):
        R = 700
        n = rng.integers(0, 50, R)
        bo = np.concatenate([[0], np.cumsum(n)]).astype(np.int64)
        ml = (rng.random((R, P)) * (n[:, None] + 1)).astype(np.uint32)
        load0 = rng.integers(0, 9, P).astype(np.int32)
        for ready in ((1 << 64) - 1, 0, int(rng.integers(1, 1 << 62)) & ((1 << P) - 1)):
            for prm, inc in ((None, 1), ((4, 1, 50), 0), ((2, 5, 10), 3), ((0, 1, 50), 1),
                             ((1, 1, 0), 2**31 - 1)):
                d_load = dev(load0.copy())
                d_bp, d_bs = empty(R, torch.int32), empty(R, torch.int64)
                aibx.route_assign(dev(ml.reshape(-1)), dev(bo), P, d_load, ready, prm, inc, d_bp, d_bs)
                wbp, wbs, wload = oracle.route_assign(ml, bo, load0, ready, prm, inc)
                assert np.array_equal(host(d_bp), wbp), (P, ready, prm, inc)
                assert np.array_equal(host(d_bs), wbs)
                assert np.array_equal(host(d_load), wload)
    # the three-request hand example: pods 1, 2, then 0
    d_load = dev(np.array([1, 0, 0], np.int32))
    d_bp, d_bs = empty(3, torch.int32), empty(3, torch.int64)
    aibx.route_assign(dev(np.zeros(9, np.uint32)), dev(np.array([0, 4, 8, 12], np.int64)), 3, d_load,
                      7, (4, 1, 50), 1, d_bp, d_bs)
    assert host(d_bp).tolist() == [1, 2, 0] and host(d_load).tolist() == [2, 1, 1]


# ------------------------------------------------------------------ the six routing policies

def test_route_policies():
    rng = np.random.default_rng(91)
    fields = ("throughput", "requests", "kv_usage", "queue_latency", "serve_latency")
    for P in (1, 6, 32, 33, 64):
        R = 2500 if P == 33 else 400                  # 2,500 requests: several requests per warp slot
        n = rng.integers(0, 50, R)
        bo = np.concatenate([[0], np.cumsum(n)]).astype(np.int64)
        ml = (rng.random((R, P)) * (n[:, None] + 1)).astype(np.uint32)
        ml[rng.random((R, P)) < 0.3] = 0
        draws = np.frombuffer(rng.bytes(8 * R), dtype=np.uint64).copy()
        for wide in (False, True):
            if wide:                                  # whole int32 range, latency sums past 2^31
                met = {f: rng.integers(-2**31, 2**31, P).astype(np.int32) for f in fields}
                met["queue_latency"][: P // 2] = 2**31 - 1
                met["serve_latency"][: P // 2] = 2**31 - 1 - rng.integers(0, 3, P // 2)
            else:
                met = {f: rng.integers(0, 4, P).astype(np.int32) for f in fields}   # many ties
            d_met = {f: dev(a) for f, a in met.items()}
            for ready in (ALL, 0, 1 << (P - 1), int(rng.integers(0, 1 << 62)) & ((1 << P) - 1)):
                for pol, name in enumerate(oracle.POLICIES):
                    for thr in ((0, 50, 100) if name == "prefix-cache-aware" else (50,)):
                        d_bp = torch.full((R,), -9, dtype=torch.int32, device="cuda")
                        aibx.route_policy(pol, P, R, ready, d_bp, match_len=dev(ml.reshape(-1)),
                                          blk_off=dev(bo), draws=dev(draws), threshold_pct=thr,
                                          **d_met)
                        want = oracle.route_policy(name, P, R, ready, met, ml, bo, draws, thr)
                        assert np.array_equal(host(d_bp), want), (P, wide, ready, name, thr)
    # the hand example of the oracle's pins
    met = {"throughput": [900, 400, 650], "requests": [3, 5, 2], "kv_usage": [70, 10, 40],
           "queue_latency": [5, 50, 20], "serve_latency": [100, 40, 90]}
    d_met = {f: dev(np.array(a, np.int32)) for f, a in met.items()}
    ml = np.array([[2, 3, 0], [2, 2, 0], [1, 0, 0], [0, 0, 0]], dtype=np.uint32)
    bo = np.array([0, 4, 8, 12, 16], np.int64)
    d_bp = empty(4, torch.int32)
    aibx.route_policy(aibx.POLICY_PREFIX_CACHE_AWARE, 3, 4, 7, d_bp, match_len=dev(ml.reshape(-1)),
                      blk_off=dev(bo), **d_met)
    assert host(d_bp).tolist() == [1, 0, 2, 2]
    aibx.route_policy(aibx.POLICY_LEAST_LATENCY, 3, 4, 7, d_bp, **d_met)
    assert host(d_bp).tolist() == [1, 1, 1, 1]
    # only the arrays a policy reads are needed; a missing one is refused on the host
    aibx.route_policy(aibx.POLICY_LEAST_KV_CACHE, 3, 4, 0b101, d_bp, kv_usage=d_met["kv_usage"])
    assert host(d_bp).tolist() == [2] * 4
    for bad in (dict(policy=6), dict(policy=-1), dict(policy=1, requests=d_met["requests"]),
                dict(policy=0), dict(policy=5, requests=d_met["requests"]),
                dict(policy=4, queue_latency=d_met["queue_latency"])):
        pol = bad.pop("policy")
        with pytest.raises(aibx.AibxError) as e:
            aibx.route_policy(pol, 3, 4, 7, d_bp, **bad)
        assert e.value.code == aibx.ERR_INVALID
    aibx.route_policy(2, 3, 0, 7, None, requests=d_met["requests"])          # R = 0: no-op
    assert aibx.status_fetch() == (0, 0)


# ------------------------------------------------------------------ export and rehash

def test_index_export_and_rehash():
    rng = np.random.default_rng(88)
    P = 12
    keys = rng.integers(1, 1 << 62, 3000).astype(np.uint64)
    masks = rng.integers(0, 1 << P, 3000).astype(np.uint64)
    ids = rng.integers(0, 1 << 20, 3000).astype(np.uint32)
    g, o = aibx.Index(4096, P), oracle.Index(4096, P)
    g.insert(dev(keys), dev(masks), dev(ids)); o.insert(keys, masks, ids)
    ev = np.full(500, ALL, dtype=np.uint64)
    g.evict(dev(keys[:500]), dev(ev)); o.evict(keys[:500], ev)
    wk, wm, wi, wcnt = o.export()

    def export_sorted(ix, room):
        d_k, d_m, d_i = empty(room, torch.uint64), empty(room, torch.uint64), empty(room, torch.uint32)
        d_c = empty(1, torch.uint64)
        ix.export(d_k, d_m, d_i, d_c)
        cnt = int(host(d_c)[0])
        m = min(cnt, room)
        k, mm, ii = host(d_k)[:m], host(d_m)[:m], host(d_i)[:m]
        order = np.argsort(k, kind="stable")
        return k[order], mm[order], ii[order], cnt

    k, m, i, cnt = export_sorted(g, 4096)
    assert cnt == wcnt and np.array_equal(k, wk) and np.array_equal(m, wm) and np.array_equal(i, wi)
    # too little room: the count is still the number of live entries, what is written is valid
    k2, m2, i2, cnt2 = export_sorted(g, 100)
    assert cnt2 == wcnt and len(k2) == 100 and np.isin(k2, wk).all()
    d_c = empty(1, torch.uint64)
    g.export(None, None, None, d_c)                       # count only
    assert int(host(d_c)[0]) == wcnt
    # rehash up and down keeps every lookup and drops the freed slots
    probe = np.concatenate([keys, rng.integers(1, 1 << 62, 200).astype(np.uint64)])
    want_m, want_i = o.lookup(probe)
    for cap in (16384, 4096):
        g.rehash(cap)
        assert o.rehash(cap) == oracle.OK
        d_m, d_i = empty(len(probe), torch.uint64), empty(len(probe), torch.uint32)
        g.lookup(dev(probe), d_m, d_i)
        assert np.array_equal(host(d_m), want_m) and np.array_equal(host(d_i), want_i)
        assert g.stats() == (wcnt, cap)
    with pytest.raises(aibx.AibxError) as e:
        g.rehash(1024)                                    # 2,5xx live entries do not fit
    assert e.value.code == aibx.ERR_FULL and o.rehash(1024) == oracle.ERR_FULL
    with pytest.raises(aibx.AibxError) as e:
        g.rehash(5000)
    assert e.value.code == aibx.ERR_INVALID
    assert g.stats() == (wcnt, 4096)
    # a table filled to the brim recovers by growing: FULL before, none after
    small_g, small_o = aibx.Index(8, 1), oracle.Index(8, 1)
    k8 = np.arange(1, 9, dtype=np.uint64)
    small_g.insert(dev(k8), dev(np.ones(8, np.uint64)), dev(np.arange(8, dtype=np.uint32)))
    small_g.rehash(32)
    extra = np.arange(100, 110, dtype=np.uint64)
    small_g.insert(dev(extra), dev(np.ones(10, np.uint64)), dev(np.zeros(10, np.uint32)))
    assert aibx.status_fetch() == (0, 0) and small_g.stats() == (18, 32)


def test_rehash_beside_the_readers():
    """rehash_begin .. rehash_finish: lookups and matches issued on another stream while the move
    runs answer from the old table (same results as before and after), calls that would change
    the index are refused meanwhile, and afterwards the larger table holds the same content."""
    rng = np.random.default_rng(99)
    P, n = 20, 300000
    keys = np.unique(rng.integers(1, 1 << 62, n).astype(np.uint64))
    n = len(keys)
    masks = (rng.integers(0, 1 << P, n) | 1).astype(np.uint64)
    ids = rng.integers(0, 1 << 20, n).astype(np.uint32)
    g, o = aibx.Index(1 << 19, P), oracle.Index(1 << 19, P)
    g.insert(dev(keys), dev(masks), dev(ids)); assert o.insert(keys, masks, ids) == oracle.OK
    gone = keys[::7]
    g.evict(dev(gone), dev(np.full(len(gone), ALL, np.uint64))); o.evict(gone, np.full(len(gone), ALL, np.uint64))
    live = o.stats()[0]
    probe = np.concatenate([keys[:50000], rng.integers(1, 1 << 62, 5000).astype(np.uint64)])
    want_m, want_i = o.lookup(probe)
    # requests made of resident keys, with holes where keys were evicted
    bo = np.arange(0, 50001, 50, dtype=np.int64)
    wml, wal, wids = o.match_prefix(keys[:50000], bo)
    d_probe, d_req, d_bo = dev(probe), dev(keys[:50000]), dev(bo)
    R = len(bo) - 1

    def read_all():
        d_m, d_i = empty(len(probe), torch.uint64), empty(len(probe), torch.uint32)
        g.lookup(d_probe, d_m, d_i)
        d_ml, d_al, d_ids = empty(R * P, torch.uint32), empty(R, torch.uint32), empty(50000, torch.uint32)
        g.match_prefix(d_req, d_bo, d_ml, d_al, d_ids)
        return d_m, d_i, d_ml, d_al, d_ids

    def check(res):
        d_m, d_i, d_ml, d_al, d_ids = res
        assert np.array_equal(host(d_m), want_m) and np.array_equal(host(d_i), want_i)
        assert np.array_equal(host(d_ml).reshape(R, P), wml) and np.array_equal(host(d_al), wal)
        assert np.array_equal(host(d_ids), wids)

    check(read_all())
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        g.rehash_begin(1 << 21)                          # the move runs on the side stream
    during = [read_all() for _ in range(4)]              # readers on the main stream, beside it
    for call in (lambda: g.insert(dev(keys[:4]), dev(masks[:4]), dev(ids[:4])),
                 lambda: g.evict(dev(keys[:4]), dev(masks[:4])),
                 lambda: g.clear(), lambda: g.rehash(1 << 20),
                 lambda: g.rehash_begin(1 << 20)):
        with pytest.raises(aibx.AibxError) as e:
            call()
        assert e.value.code == aibx.ERR_INVALID
    assert g.stats() == (live, 1 << 19)                  # still the old table
    g.rehash_finish()
    for res in during:
        check(res)
    check(read_all())
    assert g.stats() == (live, 1 << 21)
    with pytest.raises(aibx.AibxError) as e:
        g.rehash_finish()                                # nothing under way
    assert e.value.code == aibx.ERR_INVALID
    # the index takes updates again, in step with the oracle
    more = rng.integers(1, 1 << 62, 1000).astype(np.uint64)
    g.insert(dev(more), dev(np.ones(1000, np.uint64)), dev(np.zeros(1000, np.uint32)))
    o.rehash(1 << 21); o.insert(more, np.ones(1000, np.uint64), np.zeros(1000, np.uint32))
    assert g.stats() == (o.stats()[0], 1 << 21)
    with pytest.raises(aibx.AibxError) as e:
        g.rehash_begin(1 << 17)                          # the live entries do not fit
    assert e.value.code == aibx.ERR_FULL
    assert aibx.status_fetch() == (0, 0)


def test_index_duplicate_heavy_random_batches():
    """Many short op sequences on small and mid-sized tables, every batch drawing its keys with
    heavy repetition from a small universe (so that threads race for the same slots), checked
    after every call against the oracle: evict's freed ids, every lookup, the live count."""
    checked = 0
    for seed in range(120):
        rng = np.random.default_rng(5000 + seed)
        cap = int(rng.choice([8, 16, 64, 1024, 65536]))
        P = int(rng.integers(1, 65))
        universe = rng.integers(1, 1 << 62, max(4, int(cap * rng.choice([0.3, 0.6, 0.9])))).astype(np.uint64)
        g, o = aibx.Index(cap, P), oracle.Index(cap, P)
        for step in range(8):
            n = int(rng.integers(1, 4 * len(universe)))
            ks = universe[rng.integers(0, len(universe), n)]
            if rng.random() < 0.1:
                ks[rng.integers(0, n)] = 0                       # a reserved key in the batch
            ms = (rng.integers(0, 1 << 63, n).astype(np.uint64) * 2
                  + rng.integers(0, 2, n).astype(np.uint64))
            if rng.random() < 0.6:
                ids = rng.integers(0, 1 << 20, n).astype(np.uint32)
                assert o.insert(ks, ms, ids) == oracle.OK
                g.insert(dev(ks), dev(ms), dev(ids))
            else:
                if rng.random() < 0.5:
                    ms[:] = ALL
                _, wf = o.evict(ks, ms)
                d_f = empty(n, torch.uint32)
                g.evict(dev(ks), dev(ms), d_f)
                assert np.array_equal(host(d_f), wf), (seed, step)
            assert aibx.status_fetch() == (0, 0), (seed, step)
            probe = np.concatenate([universe, rng.integers(1, 1 << 62, 8).astype(np.uint64)])
            wm, wi = o.lookup(probe)
            d_m, d_i = empty(len(probe), torch.uint64), empty(len(probe), torch.uint32)
            g.lookup(dev(probe), d_m, d_i)
            assert np.array_equal(host(d_m), wm) and np.array_equal(host(d_i), wi), (seed, step)
            assert g.stats()[0] == o.stats()[0], (seed, step)
            checked += 1
        g.destroy()
    assert checked == 960


def test_churn_fills_the_table_with_removed_entries_and_rehash_clears_them():
    """Publish/expire churn in a 64-slot table: every batch inserts fresh keys and evicts them
    again.  Live entries stay few, but never-used entries run out, so a probe for an absent key
    has to walk further and further; stats2 shows it (removed count, longest insert walk), the
    walk stays bounded, results stay those of the oracle, and a rehash to the same size brings
    the probes back to one sector."""
    rng = np.random.default_rng(64)
    g, o = aibx.Index(64, 4), oracle.Index(64, 4)
    keep = rng.integers(1, 1 << 62, 10).astype(np.uint64)            # entries that stay
    km, ki = np.full(10, 5, np.uint64), np.arange(10, dtype=np.uint32)
    g.insert(dev(keep), dev(km), dev(ki)); o.insert(keep, km, ki)
    probe = np.concatenate([keep, rng.integers(1, 1 << 62, 200).astype(np.uint64)])
    ones = np.full(16, ALL, np.uint64)
    for batch in range(12):
        fresh = rng.integers(1, 1 << 62, 16).astype(np.uint64)
        m, i = np.full(16, 3, np.uint64), rng.integers(0, 100, 16).astype(np.uint32)
        g.insert(dev(fresh), dev(m), dev(i)); assert o.insert(fresh, m, i) == oracle.OK
        d_f = empty(16, torch.uint32)
        g.evict(dev(fresh), dev(ones), d_f)
        rc, want = o.evict(fresh, ones)
        assert np.array_equal(host(d_f), want)
        d_m, d_i = empty(len(probe), torch.uint64), empty(len(probe), torch.uint32)
        g.lookup(dev(probe), d_m, d_i)
        wm, wi = o.lookup(probe)
        assert np.array_equal(host(d_m), wm) and np.array_equal(host(d_i), wi)
        assert aibx.status_fetch() == (0, 0)
    live, removed, cap, walk = g.stats2()
    assert (live, cap) == (10, 64) == (o.stats()[0], 64)
    # 64 entries of room, 10 live, 192 publish/expire pairs
    assert 16 <= removed <= 54 and live + removed <= 64
    assert 1 <= walk <= 32                                            # 32 sectors = the whole table
    g.rehash(64)
    live, removed, cap, walk = g.stats2()
    assert (live, removed, cap) == (10, 0, 64) and walk <= 3
    d_m, d_i = empty(len(probe), torch.uint64), empty(len(probe), torch.uint32)
    g.lookup(dev(probe), d_m, d_i)
    wm, wi = o.lookup(probe)
    assert np.array_equal(host(d_m), wm) and np.array_equal(host(d_i), wi)
    assert aibx.status_fetch() == (0, 0)


def test_full_counts_the_entries_in_excess_of_capacity():
    """capacity is a limit on live entries, kept by counting: 70 distinct keys into a 64-slot
    table report FULL with detail 6, as the oracle does for the 65th key on."""
    g, o = aibx.Index(64, 2), oracle.Index(64, 2)
    keys = np.arange(1, 71, dtype=np.uint64) * np.uint64(0x9E3779B97F4A7C15)
    m, i = np.ones(70, np.uint64), np.zeros(70, np.uint32)
    assert o.insert(keys[:64], m[:64], i[:64]) == oracle.OK
    g.insert(dev(keys[:64]), dev(m[:64]), dev(i[:64]))
    assert aibx.status_fetch() == (0, 0) and g.stats() == (64, 64)
    assert o.insert(keys[64:], m[64:], i[64:]) == oracle.ERR_FULL
    g.insert(dev(keys[64:]), dev(m[64:]), dev(i[64:]))
    st, detail = aibx.status_fetch()
    assert st == aibx.ERR_FULL and detail == 6
