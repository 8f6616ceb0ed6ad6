"""Pins for the six routing policies of Section 3.2.2 (CPU only): a hand-worked example, numpy
argmin as the library special case of the four lowest-figure policies, plain list indexing for
the random policy, sorted tuples for the prefix-cache-aware policy, and its equality with the
(separately pinned) weighted route score under a prefix weight that dominates every load."""
import numpy as np

import oracle


def _ready_list(ready, P):
    return [p for p in range(P) if (ready >> p) & 1]


def test_hand_example():
    # three pods; figures chosen so that every policy picks a different pod where it can
    met = {"throughput": [900, 400, 650], "requests": [3, 5, 2], "kv_usage": [70, 10, 40],
           "queue_latency": [5, 50, 20], "serve_latency": [100, 40, 90]}
    ml = np.array([[2, 3, 0],      # n_r = 4: pods 0 and 1 pass 50 %; pod 1 has the longer hit
                   [2, 2, 0],      # equal hits: fewer requests wins -> pod 0 (3 < 5)
                   [1, 0, 0],      # 1 of 4 blocks is under the threshold -> least-request -> pod 2
                   [0, 0, 0]],     # nothing cached -> least-request -> pod 2
                  dtype=np.uint32)
    bo = [0, 4, 8, 12, 16]
    R, P, ready = 4, 3, 0b111
    assert oracle.route_policy("throughput", P, R, ready, met).tolist() == [1] * 4
    assert oracle.route_policy("least-request", P, R, ready, met).tolist() == [2] * 4
    assert oracle.route_policy("least-kv-cache", P, R, ready, met).tolist() == [1] * 4
    # latency sums: 105, 90, 110
    assert oracle.route_policy("least-latency", P, R, ready, met).tolist() == [1] * 4
    assert oracle.route_policy("prefix-cache-aware", P, R, ready, met, ml, bo).tolist() == [1, 0, 2, 2]
    # threshold 25 %: the third request's single block now counts
    assert oracle.route_policy("prefix-cache-aware", P, R, ready, met, ml, bo,
                               threshold_pct=25).tolist() == [1, 0, 0, 2]
    # pod 1 not ready: the others take over
    assert oracle.route_policy("throughput", P, R, 0b101, met).tolist() == [2] * 4
    assert oracle.route_policy("prefix-cache-aware", P, R, 0b101, met, ml, bo).tolist() == [0, 0, 2, 2]
    # random: draws index the ready pods in ascending order
    assert oracle.route_policy("random", P, 5, 0b101, draws=[0, 1, 2, 3, 2**64 - 1]).tolist() == \
        [0, 2, 0, 2, 2]                                   # (2^64 - 1) mod 2 = 1
    # nobody ready
    for pol in oracle.POLICIES:
        out = oracle.route_policy(pol, P, 2, 0, met, ml[:2], bo[:3], draws=[4, 9])
        assert out.tolist() == [oracle.NO_POD] * 2
    # bits of pods that do not exist are ignored
    assert oracle.route_policy("least-request", P, 1, 0b11000, met).tolist() == [oracle.NO_POD]


def test_lowest_figure_policies_are_numpy_argmin():
    rng = np.random.default_rng(17)
    for P in (1, 7, 32, 33, 64):
        for trial in range(20):
            met = {f: rng.integers(0, 9, P).astype(np.int32) for f in oracle._METRIC_FIELDS}  # ties
            if trial % 4 == 0:                     # whole int32 range: the latency sum needs 33 bits
                met = {f: rng.integers(-2**31, 2**31, P).astype(np.int32)
                       for f in oracle._METRIC_FIELDS}
                met["queue_latency"][: P // 2] = 2**31 - 1
                met["serve_latency"][: P // 2] = 2**31 - 1 - rng.integers(0, 3, P // 2)
            ready = int(rng.integers(1, 2**63)) & ((1 << P) - 1) if P < 64 else \
                int(rng.integers(1, 2**63)) * 2 + 1
            if ready == 0:
                ready = 1
            rd = np.array([(ready >> p) & 1 for p in range(P)], dtype=bool)
            for pol, fig in (("throughput", met["throughput"].astype(np.int64)),
                             ("least-request", met["requests"].astype(np.int64)),
                             ("least-kv-cache", met["kv_usage"].astype(np.int64)),
                             ("least-latency", met["queue_latency"].astype(np.int64)
                              + met["serve_latency"].astype(np.int64))):
                want = int(np.argmin(np.where(rd, fig, np.iinfo(np.int64).max)))
                got = oracle.route_policy(pol, P, 3, ready, met)
                assert got.tolist() == [want] * 3, (pol, P, trial)


def test_random_policy_is_list_indexing():
    rng = np.random.default_rng(23)
    for P in (1, 5, 64):
        for _ in range(10):
            ready = int.from_bytes(rng.bytes(8), "little") & ((1 << P) - 1 if P < 64 else 2**64 - 1)
            lst = _ready_list(ready, P)
            draws = np.frombuffer(rng.bytes(8 * 200), dtype=np.uint64)
            got = oracle.route_policy("random", P, 200, ready, draws=draws)
            want = [lst[int(d) % len(lst)] if lst else oracle.NO_POD for d in draws]
            assert got.tolist() == want
    # every ready pod is reachable and no other pod ever is
    got = oracle.route_policy("random", 8, 64, 0b10110100, draws=np.arange(64, dtype=np.uint64))
    assert sorted(set(got.tolist())) == [2, 4, 5, 7]


def _random_case(rng, R, P):
    n = rng.integers(0, 40, R)
    bo = np.concatenate([[0], np.cumsum(n)]).astype(np.int64)
    ml = (rng.random((R, P)) * (n[:, None] + 1)).astype(np.uint32)
    ml[rng.random((R, P)) < 0.3] = 0
    req = rng.integers(0, 5, P).astype(np.int32)
    return n, bo, ml, req


def test_prefix_cache_aware_is_a_sort_by_hit_then_requests_then_pod():
    rng = np.random.default_rng(29)
    for P in (3, 13, 64):
        R = 300
        n, bo, ml, req = _random_case(rng, R, P)
        ready = int.from_bytes(rng.bytes(8), "little") & ((1 << P) - 1 if P < 64 else 2**64 - 1) | 1
        lst = _ready_list(ready, P)
        for thr in (0, 30, 50, 100):
            got = oracle.route_policy("prefix-cache-aware", P, R, ready, {"requests": req}, ml, bo,
                                      threshold_pct=thr)
            for r in range(R):
                cands = [p for p in lst if ml[r, p] > 0 and 100 * int(ml[r, p]) >= thr * int(n[r])]
                if cands:
                    want = sorted(cands, key=lambda p: (-int(ml[r, p]), int(req[p]), p))[0]
                else:
                    want = sorted(lst, key=lambda p: (int(req[p]), p))[0]
                assert got[r] == want, (P, thr, r)


def test_prefix_cache_aware_equals_the_weighted_score_with_a_dominating_prefix_weight():
    # score = W*eff - requests with W above the spread of `requests` orders pods by (eff, then
    # fewer requests, then lower pod); with no qualifying pod every eff is 0 and the score is
    # least-request: the same choice as the policy
    rng = np.random.default_rng(31)
    for P in (4, 33, 64):
        R = 400
        n, bo, ml, req = _random_case(rng, R, P)
        ready = (1 << P) - 1 if P < 64 else 2**64 - 1
        ready &= ~0b100
        for thr in (0, 50, 80):
            got = oracle.route_policy("prefix-cache-aware", P, R, ready, {"requests": req}, ml, bo,
                                      threshold_pct=thr)
            bp, _, _ = oracle.route_score(ml, bo, req, ready, (1000, 1, thr))
            assert np.array_equal(got, bp)
    # and the four lowest-figure policies are the score with w_prefix = 0
    met = {f: rng.integers(0, 50, 9).astype(np.int32) for f in oracle._METRIC_FIELDS}
    ml = np.zeros((2, 9), dtype=np.uint32)
    for pol, fig in (("throughput", met["throughput"]), ("least-request", met["requests"]),
                     ("least-kv-cache", met["kv_usage"]),
                     ("least-latency", met["queue_latency"] + met["serve_latency"])):
        bp, _, _ = oracle.route_score(ml, [0, 3, 6], fig, 0b110111011, (0, 1, 50))
        assert np.array_equal(oracle.route_policy(pol, 9, 2, 0b110111011, met), bp)


def test_invalid_arguments():
    inv = oracle.ERR_INVALID
    met = {"requests": [1, 2]}
    assert oracle.route_policy(6, 2, 1, 3, met, expect=inv) == inv
    assert oracle.route_policy(-1, 2, 1, 3, met, expect=inv) == inv
    assert oracle.route_policy("least-request", 0, 1, 3, met, expect=inv) == inv
    assert oracle.route_policy("least-request", 65, 1, 3, met, expect=inv) == inv
    assert oracle.route_policy("throughput", 2, 1, 3, met, expect=inv) == inv      # array missing
    assert oracle.route_policy("least-latency", 2, 1, 3, {"queue_latency": [1, 2]}, expect=inv) == inv
    assert oracle.route_policy("random", 2, 1, 3, met, expect=inv) == inv          # no draws
    assert oracle.route_policy("prefix-cache-aware", 2, 1, 3, met, expect=inv) == inv
    assert oracle.route_policy("least-request", 2, 0, 3, met).tolist() == []       # R = 0
