"""Pins for the oracle's residency index (CPU only): a Python dict model under hypothesis,
an operation-log brute force, and algebraic invariants.  The paper fixes none of this."""
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle

NO_BLOCK = 0xFFFFFFFF
ALL = (1 << 64) - 1


class DictModel:
    """The same batch semantics written with a dict, independently of the C code."""

    def __init__(self, P):
        self.d = {}
        self.all = (1 << P) - 1

    def insert(self, keys, masks, ids):
        for k, m, i in zip(keys, masks, ids):
            if k in (0, ALL) or (m & self.all) == 0:
                continue
            if k in self.d:
                om, oi = self.d[k]
                self.d[k] = (om | (m & self.all), min(oi, i))
            else:
                self.d[k] = (m & self.all, i)

    def evict(self, keys, masks):
        for k, m in zip(keys, masks):
            if k in self.d:
                om, oi = self.d[k]
                self.d[k] = (om & ~m & ALL, oi)
        freed = [self.d[k][1] if (k in self.d and self.d[k][0] == 0) else NO_BLOCK for k in keys]
        self.d = {k: v for k, v in self.d.items() if v[0] != 0}
        return freed

    def lookup(self, keys):
        return [self.d.get(k, (0, NO_BLOCK)) for k in keys]


small_keys = st.sampled_from([0, ALL, 1, 2, 3, 5, 8, 13, 21, 1 << 40, (1 << 63) + 5, ALL - 1])
op = st.tuples(
    st.sampled_from(["insert", "evict"]),
    st.lists(st.tuples(small_keys, st.integers(0, 255), st.integers(0, 40)), max_size=12),
)


@settings(max_examples=300, deadline=None)
@given(st.integers(1, 8), st.lists(op, max_size=10))
def test_against_dict_model(P, ops):
    ix = oracle.Index(64, P)
    model = DictModel(P)
    probe = [0, ALL, 1, 2, 3, 5, 8, 13, 21, 1 << 40, (1 << 63) + 5, ALL - 1, 77]
    for kind, items in ops:
        keys = [k for k, _, _ in items]
        masks = [m for _, m, _ in items]
        ids = [i for _, _, i in items]
        if kind == "insert":
            assert ix.insert(keys, masks, ids) == oracle.OK
            model.insert(keys, masks, ids)
        else:
            rc, freed = ix.evict(keys, masks)
            assert rc == oracle.OK
            assert freed.tolist() == model.evict(keys, masks)
        m, i = ix.lookup(probe)
        assert list(zip(m.tolist(), i.tolist())) == model.lookup(probe)
        assert ix.stats()[0] == len(model.d)


def test_operation_log_brute_force():
    """lookup(k) recomputed by scanning the raw log of inserts (no map of any kind)."""
    rng = np.random.default_rng(5)
    P = 6
    keys = rng.integers(1, 50, 400).astype(np.uint64)
    masks = rng.integers(0, 64, 400).astype(np.uint64)
    ids = rng.integers(0, 1000, 400).astype(np.uint32)
    ix = oracle.Index(1024, P)
    for lo in range(0, 400, 37):  # several batches
        assert ix.insert(keys[lo:lo + 37], masks[lo:lo + 37], ids[lo:lo + 37]) == oracle.OK
    probe = np.arange(0, 60, dtype=np.uint64)
    got_m, got_i = ix.lookup(probe)
    for q in range(60):
        m, i = 0, NO_BLOCK
        for k, mm, ii in zip(keys.tolist(), masks.tolist(), ids.tolist()):
            if k == q and (mm & 63):
                m |= mm & 63
                i = min(i, ii)
        if m == 0:
            i = NO_BLOCK
        assert (int(got_m[q]), int(got_i[q])) == (m, i), q


def test_order_and_capacity_independence_and_idempotence():
    rng = np.random.default_rng(9)
    keys = rng.integers(1, 1 << 62, 500).astype(np.uint64)
    keys[100:200] = keys[0:100]  # duplicates
    masks = rng.integers(1, 1 << 16, 500).astype(np.uint64)
    ids = rng.integers(0, 4096, 500).astype(np.uint32)
    a, b = oracle.Index(1024, 16), oracle.Index(4096, 16)
    perm = rng.permutation(500)
    a.insert(keys, masks, ids)
    b.insert(keys[perm], masks[perm], ids[perm])
    b.insert(keys[perm], masks[perm], ids[perm])  # idempotent
    ma, ia = a.lookup(keys)
    mb, ib = b.lookup(keys)
    assert np.array_equal(ma, mb) and np.array_equal(ia, ib)
    assert a.stats()[0] == b.stats()[0] == len(set(keys.tolist()))
    # evict with all ones removes outright and reports the id
    rc, freed = a.evict(keys[:50], np.full(50, ALL, dtype=np.uint64))
    assert np.array_equal(freed, ia[:50])
    m, i = a.lookup(keys[:50])
    assert not m.any() and (i == NO_BLOCK).all()


def test_no_id_sentinel_is_identity_of_min():
    ix = oracle.Index(8, 2)
    ix.insert([7], [1], [NO_BLOCK])
    assert ix.lookup([7])[1][0] == NO_BLOCK
    ix.insert([7], [2], [12])
    m, i = ix.lookup([7])
    assert (int(m[0]), int(i[0])) == (3, 12)


def test_full_and_invalid():
    ix = oracle.Index(8, 1)
    assert ix.insert(np.arange(1, 9), np.ones(8), np.zeros(8)) == oracle.OK
    assert ix.insert([100], [1], [0]) == oracle.ERR_FULL
    import pytest

    with pytest.raises(ValueError):
        oracle.Index(12, 4)      # not a power of two
    with pytest.raises(ValueError):
        oracle.Index(16, 65)


def test_export_and_rehash():
    rng = np.random.default_rng(17)
    keys = rng.integers(1, 1 << 62, 300).astype(np.uint64)
    masks = rng.integers(1, 1 << 8, 300).astype(np.uint64)
    ids = rng.integers(0, 5000, 300).astype(np.uint32)
    ix = oracle.Index(1024, 8)
    ix.insert(keys, masks, ids)
    ix.evict(keys[:40], np.full(40, ALL, dtype=np.uint64))
    ek, em, ei, cnt = ix.export()
    model = DictModel(8)
    model.insert(keys.tolist(), masks.tolist(), ids.tolist())
    model.evict(keys[:40].tolist(), [ALL] * 40)
    want = sorted(model.d.items())
    assert cnt == len(want) == ix.stats()[0]
    assert list(zip(ek.tolist(), zip(em.tolist(), ei.tolist()))) == want
    # truncated export still reports the full count
    k2, _, _, cnt2 = ix.export(max_entries=10)
    assert cnt2 == cnt and k2.tolist() == ek[:10].tolist()
    # export -> import into a fresh index reproduces every lookup
    other = oracle.Index(2048, 8)
    other.insert(ek, em, ei)
    probe = np.concatenate([keys, rng.integers(1, 1 << 62, 50).astype(np.uint64)])
    assert all(np.array_equal(a, b) for a, b in zip(ix.lookup(probe), other.lookup(probe)))
    # rehash keeps the content; too small a table is refused and changes nothing
    before = ix.lookup(probe)
    assert ix.rehash(4096) == oracle.OK and ix.stats() == (cnt, 4096)
    assert all(np.array_equal(a, b) for a, b in zip(before, ix.lookup(probe)))
    assert ix.rehash(256) == oracle.ERR_FULL and ix.stats() == (cnt, 4096)
    assert ix.rehash(300) == oracle.ERR_INVALID
    assert ix.rehash(512) == oracle.OK and ix.stats() == (cnt, 512)
    assert all(np.array_equal(a, b) for a, b in zip(before, ix.lookup(probe)))


def test_scan_resistant_victims_hand_example_and_model():
    # five entries; epoch 1 touches A B C, epoch 2 touches A (twice: counts once) and D,
    # epoch 3 is a "scan" touching everything once, epoch 4 touches B
    A, B, Cc, D, E = 11, 22, 33, 44, 55
    ix = oracle.Index(16, 2)
    ix.insert([A, B, Cc, D, E], [1] * 5, [0, 1, 2, 3, 4])
    assert ix.touch([A, B, Cc, 999], 1) == oracle.OK       # 999 is absent: ignored
    ix.touch([A, A, D], 2)
    # touches so far: A 2, B 1, C 1, D 1, E 0 -> cold first (E never, then B, C at epoch 1, D at 2)
    k, p = ix.pick_victims(5)
    assert k.tolist() == [E, B, Cc, D, A] and p.tolist() == [0, 1, 1, 2, (1 << 30) + 2]
    ix.touch([A, B, Cc, D, E], 3)                          # the scan
    k, p = ix.pick_victims(5)
    # E has been seen once only: it is still the first to go although it was touched last
    assert k.tolist() == [E, A, B, Cc, D]
    assert p.tolist() == [3] + [(1 << 30) + 3] * 4
    ix.touch([B], 4)
    k, _ = ix.pick_victims(3)
    assert k.tolist() == [E, A, Cc]
    # inserting an existing key again keeps its history; a new key starts cold
    ix.insert([A, 66], [2, 1], [9, 9])
    k, p = ix.pick_victims(2)
    assert k.tolist() == [66, E] and p.tolist() == [0, 3]
    assert ix.touch([A], 0) == oracle.ERR_INVALID and ix.touch([A], 1 << 30) == oracle.ERR_INVALID
    # Python model on random traffic
    rng = np.random.default_rng(23)
    keys = rng.integers(1, 1 << 60, 400).astype(np.uint64)
    ix = oracle.Index(1024, 4)
    ix.insert(keys, np.ones(400, np.uint64), np.zeros(400, np.uint32))
    model = {int(k): [0, 0] for k in keys}
    for epoch in range(1, 9):
        batch = rng.choice(keys, 120)
        ix.touch(batch, epoch)
        for kk in batch.tolist():
            t = model[kk]
            if t[1] != epoch:
                t[0], t[1] = min(t[0] + 1, 3), epoch
    want = sorted(((1 << 30 if t[0] >= 2 else 0) + t[1], kk) for kk, t in model.items())
    k, p = ix.pick_victims(150)
    assert list(zip(p.tolist(), k.tolist())) == want[:150]
    k, p = ix.pick_victims(10**6)
    assert len(k) == len(model)


def test_match_then_touch_marks_the_matched_prefix_only():
    """What the GPU's match-and-stamp calls are compared with: match_prefix followed by touch of
    the keys below any_len.  Hand example: the index holds A, B, C; the request [A, B, X, C] is
    cached up to B, so after the composition A and B carry the epoch and C, behind the hole, and
    the never-requested D stay cold."""
    A, B, Cc, D, X = 101, 202, 303, 404, 999
    ix = oracle.Index(16, 2)
    ix.insert(np.array([A, B, Cc, D], np.uint64), np.ones(4, np.uint64), np.arange(4, dtype=np.uint32))
    req = np.array([A, B, X, Cc], np.uint64)
    ml, al, ids = ix.match_prefix(req, np.array([0, 4], np.int64))
    assert al.tolist() == [2]
    ix.touch(req[: al[0]], 7)
    keys, prio = ix.pick_victims(4)
    assert dict(zip(keys.tolist(), prio.tolist())) == {Cc: 0, D: 0, A: 7, B: 7}
