"""GPU parity for the scan-resistant victim choice.  Which entries are taken among those AT the
threshold priority is unspecified, so the comparison with the oracle is: same number of victims,
same multiset of priorities, every entry strictly below the threshold present, every victim
live, distinct and carrying the priority the oracle assigns to it."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import dev, empty, fill_entries, gpu_hash, host
from paper_2504_03648_b200 import binding as aibx
import workloads as W

pytestmark = pytest.mark.gpu
ALL = (1 << 64) - 1


def gpu_victims(g, k):
    room = max(k, 1)
    d_k, d_p, d_c = empty(room, torch.uint64), empty(room, torch.uint32), empty(1, torch.uint64)
    g.pick_victims(k, d_k, d_p, d_c)
    cnt = int(host(d_c)[0])
    return host(d_k)[:cnt], host(d_p)[:cnt], cnt


def check_against_oracle(g, o, k):
    keys, prio, cnt = gpu_victims(g, k)
    wk, wp = o.pick_victims(k)
    assert cnt == len(wk)
    if cnt == 0:
        return
    assert len(set(keys.tolist())) == cnt                              # distinct
    assert np.array_equal(np.sort(prio), wp)                           # same priorities overall
    everyone_k, everyone_p = o.pick_victims(10**9)                     # priority of every live entry
    table = dict(zip(everyone_k.tolist(), everyone_p.tolist()))
    assert all(table.get(int(a)) == int(b) for a, b in zip(keys, prio))
    thr = int(wp[-1])
    below = set(kk for kk, pp in table.items() if pp < thr)
    assert below <= set(keys.tolist())                                 # nothing colder is left out


def test_hand_example():
    A, B, C, D, E = 11, 22, 33, 44, 55
    g, o = aibx.Index(16, 2), oracle.Index(16, 2)
    k5 = np.array([A, B, C, D, E], np.uint64)
    for ix in (o,):
        ix.insert(k5, np.ones(5, np.uint64), np.arange(5, dtype=np.uint32))
    g.insert(dev(k5), dev(np.ones(5, np.uint64)), dev(np.arange(5, dtype=np.uint32)))
    for batch, epoch in (([A, B, C, 999], 1), ([A, A, D], 2)):
        g.touch(dev(np.array(batch, np.uint64)), epoch)
        o.touch(batch, epoch)
    keys, prio, cnt = gpu_victims(g, 5)
    order = np.lexsort((keys, prio))
    assert keys[order].tolist() == [E, B, C, D, A]
    assert prio[order].tolist() == [0, 1, 1, 2, (1 << 30) + 2]
    keys, prio, cnt = gpu_victims(g, 1)
    assert keys.tolist() == [E]
    g.touch(dev(k5), 3); o.touch(k5, 3)                                # the scan
    keys, prio, cnt = gpu_victims(g, 1)
    assert keys.tolist() == [E] and prio.tolist() == [3]
    for k in (0, 2, 3, 5, 9):
        check_against_oracle(g, o, k)
    with pytest.raises(aibx.AibxError):
        g.touch(dev(k5), 0)
    with pytest.raises(aibx.AibxError):
        g.touch(dev(k5), 1 << 30)


@pytest.mark.parametrize("n_keys,capacity", [(300, 1024), (20000, 65536), (400000, 1 << 20)])
def test_random_traffic(n_keys, capacity):
    rng = np.random.default_rng(n_keys)
    keys = np.unique(rng.integers(1, 1 << 62, n_keys).astype(np.uint64))
    n = len(keys)
    masks = np.ones(n, np.uint64)
    ids = rng.integers(0, 1 << 20, n).astype(np.uint32)
    g, o = aibx.Index(capacity, 4), oracle.Index(capacity, 4)
    g.insert(dev(keys), dev(masks), dev(ids)); o.insert(keys, masks, ids)
    hot = keys[: n // 10]
    for epoch in range(1, 7):
        batch = np.concatenate([rng.choice(hot, n // 20), rng.choice(keys, n // 8)])
        g.touch(dev(batch), epoch); o.touch(batch, epoch)
    for k in (1, n // 100 + 1, n // 3, n, n + 5):
        check_against_oracle(g, o, k)
    # evicting the victims and asking again gives the next coldest; history survives rehash
    vk, vp, cnt = gpu_victims(g, n // 4)
    ones = np.full(cnt, ALL, dtype=np.uint64)
    g.evict(dev(vk), dev(ones)); o.evict(vk, ones)
    check_against_oracle(g, o, n // 4)
    g.rehash(capacity * 2); o.rehash(capacity * 2)
    check_against_oracle(g, o, n // 5)
    # re-inserting evicted keys starts them cold again; existing keys keep their history
    back = vk[: max(cnt // 2, 1)]
    some = keys[-5:]
    g.insert(dev(np.concatenate([back, some])), dev(np.ones(len(back) + 5, np.uint64)),
             dev(np.zeros(len(back) + 5, np.uint32)))
    o.insert(np.concatenate([back, some]), np.ones(len(back) + 5, np.uint64),
             np.zeros(len(back) + 5, np.uint32))
    check_against_oracle(g, o, len(back) + 3)
    assert aibx.status_fetch() == (0, 0)


@pytest.mark.parametrize("R", [40, 3000])          # several warps per request / one warp per request
def test_matching_stamps_the_matched_prefix(R):
    """match_prefix_touch and route_head_touch against the oracle's match_prefix followed by
    touch of the keys below any_len: same match results, and afterwards the same victims."""
    spec = W.scaled(W.cfg3_routing(), R=R, capacity=1 << 16, n_entries=1 << 15, n_prompts=40,
                    id_space=1 << 15, len_lo=64, len_hi=2048, len_mean=600.0, len_sd=300.0)
    w = W.build_routing(spec)
    B, P = spec.block_tokens, spec.num_pods
    h, bo = gpu_hash(w.tokens, w.tok_off, B)
    sh, _ = gpu_hash(w.src_tokens, w.src_tok_off, B)
    keys, masks, ids = fill_entries(w, sh)
    g, o = aibx.Index(spec.capacity, P), oracle.Index(spec.capacity, P)
    g.insert(dev(keys), dev(masks), dev(ids)); assert o.insert(keys, masks, ids) == oracle.OK
    d_h, d_bo = dev(h), dev(bo)
    d_tok, d_toff = dev(w.tokens), dev(w.tok_off)
    n_live = o.stats()[0]

    def oracle_step(epoch, lo, hi):
        sub_bo = bo[lo:hi + 1] - bo[lo]
        sub_h = h[bo[lo]:bo[hi]]
        ml, al, bid = o.match_prefix(sub_h, sub_bo)
        hit = np.concatenate([sub_h[sub_bo[r]: sub_bo[r] + al[r]] for r in range(hi - lo)])
        o.touch(hit, epoch)
        return ml, al, bid

    # epochs 1..3 over different slices of the batch through match_prefix_touch
    cuts = [0, R // 2, (3 * R) // 4, R]
    for epoch, (lo, hi) in enumerate(zip(cuts[:-1], cuts[1:]), start=1):
        n = hi - lo
        sub_bo = dev(bo[lo:hi + 1] - bo[lo])
        sub_h = dev(h[bo[lo]:bo[hi]]) if bo[hi] > bo[lo] else empty(1, torch.uint64)
        d_ml, d_al = empty(n * P, torch.uint32), empty(n, torch.uint32)
        d_id = empty(max(int(bo[hi] - bo[lo]), 1), torch.uint32)
        g.match_prefix_touch(sub_h, sub_bo, epoch, d_ml, d_al, d_id)
        ml, al, bid = oracle_step(epoch, lo, hi)
        assert np.array_equal(host(d_ml).reshape(n, P), ml) and np.array_equal(host(d_al), al)
        assert np.array_equal(host(d_id)[: len(bid)], bid)
        assert al.sum() > 0
    for k in (1, n_live // 50 + 1, n_live // 2, n_live):
        check_against_oracle(g, o, k)
    # epoch 4 over the whole batch through route_head_touch
    d_hh = torch.zeros(len(h), dtype=torch.uint64, device="cuda")
    d_ml, d_al, d_id = empty(R * P, torch.uint32), empty(R, torch.uint32), empty(len(h), torch.uint32)
    d_bp, d_bs = empty(R, torch.int32), empty(R, torch.int64)
    d_dn, d_sd = empty(R, torch.uint32), empty(R, torch.uint64)
    aibx.route_head_touch(g, d_tok, d_toff, d_bo, B, 0, dev(w.pod_load), w.ready_mask, None, 4, d_hh,
                          d_ml, d_al, d_id, d_bp, d_bs, d_dn, d_sd)
    ml, al, bid = oracle_step(4, 0, R)
    assert np.array_equal(host(d_ml).reshape(R, P), ml) and np.array_equal(host(d_al), al)
    for k in (1, n_live // 50 + 1, n_live // 2, n_live):
        check_against_oracle(g, o, k)
    # the plain calls leave the stamps alone
    g.match_prefix(d_h, d_bo, d_ml, d_al, d_id)
    check_against_oracle(g, o, n_live // 3)
    with pytest.raises(aibx.AibxError):
        g.match_prefix_touch(d_h, d_bo, 0, d_ml, d_al, d_id)
    assert aibx.status_fetch() == (0, 0)
