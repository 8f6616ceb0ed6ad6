"""Pins for the integer prefix-and-load route score (CPU only): hand-worked example,
special cases that reduce to least-request / longest-match, independent recomputation."""
import numpy as np

import oracle

I64_MIN = -(1 << 63)


def test_hand_example():
    ml = np.array([[2, 1, 0]], dtype=np.uint32)      # n_r = 4, threshold 50 %: only hit=2 counts
    blk_off = [0, 4]
    bp, bs, sc = oracle.route_score(ml, blk_off, [10, 3, 0], 0b111, (4, 1, 50))
    assert sc.tolist() == [[-2, -3, 0]] and bp.tolist() == [2] and bs.tolist() == [0]
    bp, bs, sc = oracle.route_score(ml, blk_off, [5, 3, 9], 0b111, (4, 1, 50))
    assert sc.tolist() == [[3, -3, -9]] and bp.tolist() == [0] and bs.tolist() == [3]
    # defaults are (4, 1, 50)
    bp2, bs2, sc2 = oracle.route_score(ml, blk_off, [5, 3, 9], 0b111, None)
    assert sc2.tolist() == sc.tolist() and bp2.tolist() == bp.tolist()
    # pod 0 not ready -> next best
    bp, bs, _ = oracle.route_score(ml, blk_off, [5, 3, 9], 0b110, (4, 1, 50))
    assert bp.tolist() == [1] and bs.tolist() == [-3]
    bp, bs, _ = oracle.route_score(ml, blk_off, [5, 3, 9], 0, (4, 1, 50))
    assert bp.tolist() == [oracle.NO_POD] and bs.tolist() == [I64_MIN]


def test_threshold_edge_is_inclusive_and_zero_hit_never_counts():
    ml = np.array([[5, 4, 0]], dtype=np.uint32)       # n_r = 10: 50 % is exactly 5 blocks
    _, _, sc = oracle.route_score(ml, [0, 10], [0, 0, 0], 7, (1, 1, 50))
    assert sc.tolist() == [[5, 0, 0]]
    _, _, sc = oracle.route_score(ml, [0, 10], [0, 0, 0], 7, (1, 1, 0))
    assert sc.tolist() == [[5, 4, 0]]
    ml0 = np.zeros((1, 3), dtype=np.uint32)           # empty request, threshold 0: eff stays 0
    _, _, sc = oracle.route_score(ml0, [0, 0], [1, 2, 3], 7, (9, 1, 0))
    assert sc.tolist() == [[-1, -2, -3]]


def test_special_cases_and_recompute():
    rng = np.random.default_rng(8)
    R, P = 200, 13
    n = rng.integers(0, 50, R)
    blk_off = np.concatenate([[0], np.cumsum(n)]).astype(np.int64)
    ml = (rng.random((R, P)) * (n[:, None] + 1)).astype(np.uint32)
    load = rng.integers(0, 6, P).astype(np.int32)     # many ties
    ready = 0b1011111101111
    rd = np.array([(ready >> p) & 1 for p in range(P)], dtype=bool)
    # w_prefix = 0 -> least-request: argmin load over ready pods, lowest index on ties
    bp, bs, _ = oracle.route_score(ml, blk_off, load, ready, (0, 1, 50))
    masked = np.where(rd, load, 1 << 30)
    assert (bp == int(np.argmin(masked))).all()
    # w_load = 0, threshold 0 -> pod with the longest match (np.argmax takes the first max)
    bp, bs, _ = oracle.route_score(ml, blk_off, load, ready, (1, 0, 0))
    m2 = np.where(rd[None, :], ml.astype(np.int64), -1)
    assert np.array_equal(bp, np.argmax(m2, axis=1))
    # general parameters: argmax recomputed from the returned score matrix by numpy
    for prm in [(4, 1, 50), (7, 3, 25), (1, 100, 90), (-2, -1, 10)]:
        bp, bs, sc = oracle.route_score(ml, blk_off, load, ready, prm)
        s2 = np.where(rd[None, :], sc, I64_MIN)
        assert np.array_equal(bp, np.argmax(s2, axis=1))
        assert np.array_equal(bs, s2.max(axis=1))
        hit = ml.astype(np.int64)
        eff = np.where((hit > 0) & (100 * hit >= prm[2] * n[:, None]), hit, 0)
        assert np.array_equal(sc, prm[0] * eff - prm[1] * load.astype(np.int64)[None, :])


def test_sequential_assignment_hand_example_and_invariants():
    # three equal requests without any cached prefix, loads [1, 0, 0]: least-request with
    # ties to the lowest pod sends them to pod 1, pod 2, then pod 0 (all three at load 1)
    ml = np.zeros((3, 3), dtype=np.uint32)
    bo = [0, 4, 8, 12]
    bp, bs, load = oracle.route_assign(ml, bo, [1, 0, 0], 0b111, (4, 1, 50), 1)
    assert bp.tolist() == [1, 2, 0] and bs.tolist() == [0, 0, -1] and load.tolist() == [2, 1, 1]
    # a cached prefix outweighs load until the pod has taken enough requests: hit 2 of 4 blocks
    # on pod 0 is worth 8; each assignment adds 3 to its load
    ml = np.array([[2, 0]] * 4, dtype=np.uint32)
    bp, bs, load = oracle.route_assign(ml, [0, 4, 8, 12, 16], [0, 0], 0b11, (4, 1, 50), 3)
    assert bp.tolist() == [0, 0, 0, 1] and bs.tolist() == [8, 5, 2, 0] and load.tolist() == [9, 3]
    # increment 0 is the snapshot score; general case against a Python loop over numpy scores
    rng = np.random.default_rng(31)
    R, P = 300, 11
    n = rng.integers(0, 40, R)
    bo = np.concatenate([[0], np.cumsum(n)]).astype(np.int64)
    ml = (rng.random((R, P)) * (n[:, None] + 1)).astype(np.uint32)
    load0 = rng.integers(0, 20, P).astype(np.int32)
    ready = 0b10111011101
    bp0, bs0, _ = oracle.route_score(ml, bo, load0, ready, (4, 1, 50))
    bp, bs, load = oracle.route_assign(ml, bo, load0, ready, (4, 1, 50), 0)
    assert np.array_equal(bp, bp0) and np.array_equal(bs, bs0) and np.array_equal(load, load0)
    for inc in (1, 7):
        bp, bs, load = oracle.route_assign(ml, bo, load0, ready, (3, 2, 25), inc)
        cur = load0.astype(np.int64).copy()
        rd = np.array([(ready >> p) & 1 for p in range(P)], dtype=bool)
        for r in range(R):
            hit = ml[r].astype(np.int64)
            eff = np.where((hit > 0) & (100 * hit >= 25 * n[r]), hit, 0)
            sc = np.where(rd, 3 * eff - 2 * cur, I64_MIN)
            assert bp[r] == int(np.argmax(sc)) and bs[r] == sc.max()
            cur[bp[r]] += inc
        assert np.array_equal(load, cur) and load.sum() - load0.sum() == inc * R
    # nobody ready: nothing is assigned, loads stay
    bp, bs, load = oracle.route_assign(ml[:5], bo[:6], load0, 0, None, 1)
    assert (bp == oracle.NO_POD).all() and np.array_equal(load, load0)
