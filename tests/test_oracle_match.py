"""Pins for longest-cached-prefix and the matched-block set (CPU only): brute-force rescan
over the raw entry list, a hand-worked example, invariants."""
import numpy as np

import oracle

NO_BLOCK = 0xFFFFFFFF
A, B, C, D = 0xA1, 0xB2, 0xC3, 0xD4


def test_hand_example():
    ix = oracle.Index(16, 3)
    ix.insert([A, B, C], [0b011, 0b001, 0b110], [5, 9, 2])
    ml, al, ids = ix.match_prefix([A, B, C, D], [0, 4])
    assert ml.tolist() == [[2, 1, 0]]
    assert al.tolist() == [3]
    assert ids.tolist() == [5, 9, 2, NO_BLOCK]


def _brute(entries, P, hashes, blk_off):
    """For every k from n_r down, test all blocks < k by scanning the entry list."""
    R = len(blk_off) - 1
    ml = np.zeros((R, P), dtype=np.uint32)
    al = np.zeros(R, dtype=np.uint32)

    def mask_of(h):
        m = 0
        for k, mm, _ in entries:
            if k == h:
                m |= mm
        return m

    for r in range(R):
        h = [int(x) for x in hashes[blk_off[r]:blk_off[r + 1]]]
        for p in range(P):
            for k in range(len(h), -1, -1):
                if all((mask_of(x) >> p) & 1 for x in h[:k]):
                    ml[r, p] = k
                    break
        for k in range(len(h), -1, -1):
            if all(mask_of(x) != 0 for x in h[:k]):
                al[r] = k
                break
    return ml, al


def test_brute_force_small():
    rng = np.random.default_rng(21)
    for trial in range(30):
        P = int(rng.integers(1, 7))
        universe = rng.integers(1, 1 << 60, 24).astype(np.uint64)
        n_e = int(rng.integers(0, 20))
        ek = rng.choice(universe, n_e)
        em = rng.integers(1, 1 << P, n_e).astype(np.uint64)
        ei = rng.integers(0, 99, n_e).astype(np.uint32)
        ix = oracle.Index(64, P)
        ix.insert(ek, em, ei)
        lens = rng.integers(0, 9, 5)
        blk_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
        hashes = rng.choice(universe, int(blk_off[-1]))
        # bias towards long runs of present keys
        if n_e:
            for r in range(5):
                run = int(rng.integers(0, lens[r] + 1))
                hashes[blk_off[r]:blk_off[r] + run] = rng.choice(ek, run)
        ml, al, ids = ix.match_prefix(hashes, blk_off)
        bml, bal = _brute(list(zip(ek.tolist(), em.tolist(), ei.tolist())), P, hashes, blk_off)
        assert np.array_equal(ml, bml) and np.array_equal(al, bal)
        lm, li = ix.lookup(hashes)
        for r in range(5):
            seg = slice(blk_off[r], blk_off[r + 1])
            a = int(al[r])
            assert np.array_equal(ids[seg][:a], li[seg][:a])
            assert (ids[seg][a:] == NO_BLOCK).all()
            assert (ml[r] <= a).all() and a <= lens[r]


def test_invariants():
    rng = np.random.default_rng(2)
    P = 5
    hashes = rng.integers(1, 1 << 62, 40).astype(np.uint64)
    blk_off = np.array([0, 10, 10, 25, 40], dtype=np.int64)
    ix = oracle.Index(128, P)
    ml, al, ids = ix.match_prefix(hashes, blk_off)                 # empty index
    assert not ml.any() and not al.any() and (ids == NO_BLOCK).all()
    ix.insert(hashes, np.full(40, 31), np.arange(40))              # everything everywhere
    ml, al, ids = ix.match_prefix(hashes, blk_off)
    n = np.diff(blk_off)
    assert np.array_equal(ml, np.repeat(n[:, None], P, 1)) and np.array_equal(al, n)
    assert ids.tolist() == list(range(40))
    # evicting pod 2 from one middle block cuts pod 2 there and nobody else
    ix.evict([hashes[14]], [0b00100])
    ml2, al2, _ = ix.match_prefix(hashes, blk_off)
    assert ml2[2].tolist() == [15, 15, 4, 15, 15] and al2[2] == 15
    assert (ml2 <= ml).all()                                       # monotone under evict
    # a hole: residency after it does not count
    ix.evict([hashes[3]], [(1 << 64) - 1])
    ml3, al3, ids3 = ix.match_prefix(hashes, blk_off)
    assert ml3[0].tolist() == [3] * 5 and al3[0] == 3
    assert (ids3[3:10] == NO_BLOCK).all()
    # pods >= P never appear: mask bits above P were dropped at insert
    ix2 = oracle.Index(16, 2)
    ix2.insert([9], [0b100], [1])
    assert ix2.stats()[0] == 0


def test_collect_blocks_is_sorted_set():
    rng = np.random.default_rng(4)
    ids = rng.integers(0, 50, 200).astype(np.uint32)
    ids[::7] = NO_BLOCK
    rc, out, cnt = oracle.collect_blocks(ids, 50)
    want = sorted(set(int(x) for x in ids if x != NO_BLOCK))
    assert rc == oracle.OK and cnt == len(want)
    assert out[:cnt].tolist() == want and (out[cnt:] == NO_BLOCK).all()
    rc, out, cnt = oracle.collect_blocks(ids, 30)                   # ids 30..49 now out of range
    want = [x for x in want if x < 30]
    assert rc == oracle.ERR_RANGE and out[:cnt].tolist() == want
    rc, out, cnt = oracle.collect_blocks(np.zeros(0, dtype=np.uint32), 10)
    assert rc == oracle.OK and cnt == 0
