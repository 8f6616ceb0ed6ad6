"""GPU parity of the routing head (hash only as far as matching needs, probe while hashing) and
of the resumed chain: every result that is defined must equal the CPU oracle's hash_blocks +
match_prefix + route_score bit for bit; how far past the first miss a request was hashed is
free, so it is checked for validity (bounds, and that the saved seed is the right key)."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import NO_BLOCK, dev, empty, fill_entries, gpu_hash, host, routing_oracle
from paper_2504_03648_b200 import binding as aibx
import workloads as W

pytestmark = pytest.mark.gpu
ALL = (1 << 64) - 1


def _run_head(ix, tokens, tok_off, bo, B, P, pod_load, ready, prm, root=0, score=True):
    R = len(tok_off) - 1
    nb = max(int(bo[-1]), 1)
    d_tok = dev(tokens, np.int32) if len(tokens) else empty(4, torch.int32)
    d_toff, d_bo = dev(tok_off, np.int64), dev(bo, np.int64)
    d_h = torch.full((nb,), 0x5151515151515151, dtype=torch.uint64, device="cuda")
    d_ml, d_al = empty(R * P, torch.uint32), empty(R, torch.uint32)
    d_ids = torch.full((nb,), 0x77, dtype=torch.uint32, device="cuda")
    d_bp = empty(R, torch.int32) if score else None
    d_bs = empty(R, torch.int64) if score else None
    d_done, d_seed = empty(R, torch.uint32), empty(R, torch.uint64)
    aibx.route_head(ix, d_tok, d_toff, d_bo, B, root, dev(pod_load, np.int32), ready, prm, d_h,
                    d_ml, d_al, d_ids, d_bp, d_bs, d_done, d_seed)
    head = dict(hashes=host(d_h).copy(), match_len=host(d_ml).reshape(R, P), any_len=host(d_al),
                block_ids=host(d_ids)[: int(bo[-1])], done=host(d_done).astype(np.int64),
                seed=host(d_seed), best_pod=None if not score else host(d_bp),
                best_score=None if not score else host(d_bs))
    aibx.hash_blocks_resume(d_tok, d_toff, d_bo, B, d_done, d_seed, d_h)
    head["all_hashes"] = host(d_h)[: int(bo[-1])]
    return head


def _check(head, want_h, bo, wml, wal, wids, wbp, wbs, root=0):
    n = np.diff(bo)
    assert np.array_equal(head["match_len"], wml)
    assert np.array_equal(head["any_len"], wal)
    assert np.array_equal(head["block_ids"], wids)
    if wbp is not None:
        assert np.array_equal(head["best_pod"], wbp) and np.array_equal(head["best_score"], wbs)
    done = head["done"]
    assert (done <= n).all() and (done >= np.minimum(wal.astype(np.int64) + 1, n)).all()
    for r in range(len(n)):
        lo = int(bo[r])
        assert np.array_equal(head["hashes"][lo: lo + done[r]], want_h[lo: lo + done[r]]), r
        # nothing past the hashed part was written by the head
        assert (head["hashes"][lo + done[r]: int(bo[r + 1])] == 0x5151515151515151).all(), r
        assert head["seed"][r] == (want_h[lo + done[r] - 1] if done[r] else root), r
    assert np.array_equal(head["all_hashes"], want_h)


@pytest.mark.parametrize("mk", [W.cfg1_routing, W.cfg2_routing, W.cfg3_routing, W.cfg5_routing])
def test_route_head_on_the_configurations(mk):
    w = W.build_routing(mk())
    s = w.spec
    B, P = s.block_tokens, s.num_pods
    o = routing_oracle(w)
    sh, _ = gpu_hash(w.src_tokens, w.src_tok_off, B)
    keys, masks, ids = fill_entries(w, sh)
    ix = aibx.Index(s.capacity, P)
    ix.insert(dev(keys), dev(masks), dev(ids))
    for prm, ready in ((None, w.ready_mask), ((7, 3, 25), w.ready_mask & 0xF0F0F0F0F0F0F0F5)):
        head = _run_head(ix, w.tokens, w.tok_off, o["blk_off"], B, P, w.pod_load, ready, prm)
        wbp, wbs, _ = oracle.route_score(o["match_len"], o["blk_off"], w.pod_load, ready, prm)
        _check(head, o["hashes"], o["blk_off"], o["match_len"], o["any_len"], o["block_ids"], wbp, wbs)
    if mk is W.cfg2_routing:
        # the point of the call: requests of up to 512 blocks are hashed little past their
        # prompt (at most the 64 keys the hasher may run ahead, plus the group in progress)
        n = np.diff(o["blk_off"])
        assert (head["done"] <= o["any_len"].astype(np.int64) + 64 + 2 * (64 // B)).all()
        assert n.max() > 400 and head["done"].max() < 260
    assert aibx.status_fetch() == (0, 0)


@pytest.mark.parametrize("B", [8, 16, 32, 64, 24])
@pytest.mark.parametrize("case", ["sparse", "crowded", "tombstones"])
def test_route_head_random_indexes(B, case):
    """Requests of 0..300 blocks with cached prefixes of random length, pods dropping out at
    random places, holes; tables from half empty to nearly full (probe runs far longer than the
    four slots one round trip covers) and with removed entries left in the runs."""
    rng = np.random.default_rng(B * 7 + len(case))
    R = 45
    P = int(rng.integers(1, 65))
    root = int(rng.integers(0, 1 << 62))
    nblk = rng.integers(0, 300 if B <= 16 else 120, R)
    nblk[:3] = [0, 1, 2]
    lens = nblk * B + rng.integers(0, B, R)                     # ragged tails are not hashed
    tok_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    tokens = rng.integers(0, 128256, int(tok_off[-1])).astype(np.int32)
    tokens[tok_off[5]: tok_off[5] + 40 * B] = tokens[tok_off[6]: tok_off[6] + 40 * B]   # shared prefix
    want_h, bo = oracle.hash_blocks(tokens, tok_off, B, root)
    allm = ALL if P == 64 else (1 << P) - 1
    keys, masks = [], []
    for r in range(R):
        c = int(rng.integers(0, nblk[r] + 1)) if rng.random() < 0.8 else int(nblk[r])
        h = want_h[bo[r]: bo[r] + c]
        m = np.full(c, allm, dtype=np.uint64)
        drop = rng.random(c) < 0.05
        m[drop] &= rng.integers(0, 1 << 62, int(drop.sum())).astype(np.uint64) | np.uint64(1)
        if c > 3 and rng.random() < 0.3:
            h = np.delete(h, c // 2)                             # a hole in the middle
            m = np.delete(m, c // 2)
        keys.append(h)
        masks.append(m)
    keys, masks = np.concatenate(keys), np.concatenate(masks)
    ids = rng.integers(0, 1 << 20, len(keys)).astype(np.uint32)
    n_keys = len(np.unique(keys))
    if case == "sparse":
        cap = 1 << int(np.ceil(np.log2(max(2 * n_keys, 8))))
        filler = np.zeros(0, dtype=np.uint64)
    else:
        cap = 1 << int(np.ceil(np.log2(max(n_keys * 1.15, 8))))
        room = cap - n_keys
        filler = rng.integers(1, 1 << 63, max(int(room * 0.9), 0)).astype(np.uint64)
    g, o = aibx.Index(cap, P), oracle.Index(cap, P)
    fm = np.full(len(filler), 1, dtype=np.uint64)
    fi = np.zeros(len(filler), dtype=np.uint32)
    if case == "tombstones" and len(filler):
        # the fillers go in first and most of them leave again: their slots stay in the runs
        g.insert(dev(filler), dev(fm), dev(fi))
        o.insert(filler, fm, fi)
        gone = filler[: len(filler) * 3 // 4]
        g.evict(dev(gone), dev(np.full(len(gone), ALL, dtype=np.uint64)), None)
        o.evict(gone, np.full(len(gone), ALL, dtype=np.uint64))
        filler = np.zeros(0, dtype=np.uint64)
    allk = np.concatenate([keys, filler])
    allmask = np.concatenate([masks, np.full(len(filler), 1, dtype=np.uint64)])
    allid = np.concatenate([ids, np.zeros(len(filler), dtype=np.uint32)])
    if len(allk):
        assert o.insert(allk, allmask, allid) == oracle.OK
        g.insert(dev(allk), dev(allmask), dev(allid))
    wml, wal, wids = o.match_prefix(want_h, bo)
    load = rng.integers(0, 40, P).astype(np.int32)
    ready = int(rng.integers(1, 1 << 62)) | 1
    wbp, wbs, _ = oracle.route_score(wml, bo, load, ready, (4, 1, 50))
    head = _run_head(g, tokens, tok_off, bo, B, P, load, ready, (4, 1, 50), root)
    _check(head, want_h, bo, wml, wal, wids, wbp, wbs, root)
    # without the score, and again (the index is not changed by the call)
    head = _run_head(g, tokens, tok_off, bo, B, P, load, ready, None, root, score=False)
    _check(head, want_h, bo, wml, wal, wids, None, None, root)
    assert aibx.status_fetch() == (0, 0)


def test_route_head_invalid_arguments_and_empty_batch():
    ix = aibx.Index(64, 4)
    t, o2 = dev(np.zeros(32, np.int32)), dev(np.array([0, 32], np.int64))
    bo = dev(np.array([0, 2], np.int64))
    h, ml, al, ids = empty(2, torch.uint64), empty(4, torch.uint32), empty(1, torch.uint32), empty(2, torch.uint32)
    bp, bs, dn, sd = empty(1, torch.int32), empty(1, torch.int64), empty(1, torch.uint32), empty(1, torch.uint64)
    load = dev(np.zeros(4, np.int32))
    for kw in (dict(B=12), dict(B=0), dict(hashes=None), dict(hashed=None), dict(best_score=None),
               dict(pod_load=None)):
        a = dict(B=16, hashes=h, hashed=dn, best_score=bs, pod_load=load)
        a.update(kw)
        with pytest.raises(aibx.AibxError) as e:
            aibx.route_head(ix, t, o2, bo, a["B"], 0, a["pod_load"], 15, None, a["hashes"], ml, al, ids,
                            bp, a["best_score"], a["hashed"], sd)
        assert e.value.code == aibx.ERR_INVALID
    with pytest.raises(aibx.AibxError) as e:
        aibx.hash_blocks_resume(t, o2, bo, 16, dn, None, h)
    assert e.value.code == aibx.ERR_INVALID
    # an empty index: nothing matches, one block is enough to know it
    aibx.route_head(ix, t, o2, bo, 16, 0, load, 15, None, h, ml, al, ids, bp, bs, dn, sd)
    assert host(al).tolist() == [0] and host(ml).tolist() == [0] * 4
    assert host(ids).tolist() == [NO_BLOCK, NO_BLOCK] and 1 <= int(host(dn)[0]) <= 2
    assert aibx.status_fetch() == (0, 0)


@pytest.mark.parametrize("B", [8, 16, 32, 40, 1024])
def test_resume_from_any_block(B):
    """aibx_hash_blocks_resume on its own: every request resumed at a random block (0, the last
    one and past-the-end included) with the key before it as seed gives the oracle's keys from
    there on and leaves the earlier part of the output alone."""
    rng = np.random.default_rng(B)
    R = 37
    nblk = rng.integers(0, 60 if B < 1024 else 5, R)
    lens = nblk * B + rng.integers(0, B, R)
    tok_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    tokens = rng.integers(-5, 128256, int(tok_off[-1])).astype(np.int32)
    root = 0x1234ABCD
    want, bo = oracle.hash_blocks(tokens, tok_off, B, root)
    start = np.array([rng.integers(0, n + 1) for n in nblk], dtype=np.uint32)
    start[:3] = [0, nblk[1], nblk[2]]
    seed = np.array([want[bo[r] + start[r] - 1] if start[r] else root for r in range(R)], dtype=np.uint64)
    nb = max(int(bo[-1]), 1)
    d_h = torch.full((nb,), 0x7E7E7E7E7E7E7E7E, dtype=torch.uint64, device="cuda")
    aibx.hash_blocks_resume(dev(tokens) if len(tokens) else empty(4, torch.int32), dev(tok_off),
                            dev(bo), B, dev(start), dev(seed), d_h)
    got = host(d_h)
    for r in range(R):
        lo, hi = int(bo[r]), int(bo[r + 1])
        assert (got[lo: lo + start[r]] == 0x7E7E7E7E7E7E7E7E).all(), r
        assert np.array_equal(got[lo + start[r]: hi], want[lo + start[r]: hi]), r
    assert aibx.status_fetch() == (0, 0)


@pytest.mark.parametrize("mk,num_blocks", [(W.cfg1_routing, None), (W.cfg2_routing, None),
                                           (W.cfg3_routing, None), (W.cfg5_routing, None),
                                           (W.cfg2_routing, 3000), (W.cfg1_routing, 300000)])
def test_route_head_collect_makes_the_matched_block_set(mk, num_blocks):
    """route_head_collect against the oracle's match_prefix + collect_blocks: same routing
    results and the same ascending set of matched blocks, twice in a row on the same scratch
    (filled with garbage first: the call clears it).  num_blocks 3000 puts some ids of the cfg2
    entries out of range (dropped, RANGE); 300,000 is a pool too large for the fused form, which
    takes the separate collect kernels with the list length read on the device."""
    w = W.build_routing(mk())
    s = w.spec
    B, P, R = s.block_tokens, s.num_pods, s.R
    nblk = s.id_space if num_blocks is None else num_blocks
    o = routing_oracle(w)
    h, bo = o["hashes"], o["blk_off"]
    rc, want_u, want_c = oracle.collect_blocks(o["block_ids"], nblk)
    keys, masks, ids = fill_entries(w, o["src_hashes"])
    g = aibx.Index(s.capacity, P)
    g.insert(dev(keys), dev(masks), dev(ids))
    nb = max(len(h), 1)
    d_tok, d_toff, d_bo = dev(w.tokens), dev(w.tok_off), dev(bo)
    scratch = torch.full((aibx.route_collect_scratch_bytes(nblk) // 4,), -1, dtype=torch.int32,
                         device="cuda")
    for rep in range(2):
        d_h = torch.zeros(nb, dtype=torch.uint64, device="cuda")
        d_ml, d_al, d_id = empty(R * P, torch.uint32), empty(R, torch.uint32), empty(nb, torch.uint32)
        d_bp, d_bs = empty(R, torch.int32), empty(R, torch.int64)
        d_dn, d_sd = empty(R, torch.uint32), empty(R, torch.uint64)
        d_un = torch.full((nb,), 0x55, dtype=torch.uint32, device="cuda")
        d_cnt = torch.full((1,), 0x55, dtype=torch.uint32, device="cuda")
        aibx.route_head_collect(g, d_tok, d_toff, d_bo, B, 0, dev(w.pod_load), w.ready_mask, None,
                                0, d_h, d_ml, d_al, d_id, d_bp, d_bs, d_dn, d_sd, nblk, scratch,
                                d_un, d_cnt)
        st = aibx.status_fetch()
        assert np.array_equal(host(d_ml).reshape(R, P), o["match_len"])
        assert np.array_equal(host(d_al), o["any_len"])
        assert np.array_equal(host(d_id)[: len(h)], o["block_ids"])
        assert np.array_equal(host(d_bp), o["best_pod"]) and np.array_equal(host(d_bs), o["best_score"])
        assert int(host(d_cnt)[0]) == want_c
        assert np.array_equal(host(d_un)[: len(h)], want_u)
        if rc == oracle.ERR_RANGE:
            assert st[0] == aibx.ERR_RANGE and st[1] > 0
        else:
            assert st == (0, 0)
        aibx.hash_blocks_resume(d_tok, d_toff, d_bo, B, d_dn, d_sd, d_h)
        assert np.array_equal(host(d_h)[: len(h)], h)
    assert want_c > 0
