"""The step that bench.py times, at the benchmark's full size and in its launch configuration
(route_head_collect, device-counted gather and scatter; the tail of the hash chains and the index
publish/expire on a second stream), checked against the oracle: routing outputs element by element, the gathered buffer
and the pool byte for byte, and the index back in its start state."""
import os
import sys

import numpy as np
import pytest
import torch

import oracle
from gpu_util import PoolModel, check_gather_full, check_pool_full, fill_entries, host
import workloads as W

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_step_matches_oracle():
    sys.path.insert(0, ROOT)
    import bench

    job = bench.GpuJob(0)
    w, kv = job.w, job.kv
    s = w.spec
    live0 = job.index.stats()[0]
    for _ in range(2):                       # twice: the second step sees the restored index
        job.step(record_copy_events=True)
    torch.cuda.synchronize()
    assert job.aibx.status_fetch() == (0, 0)

    h, bo = oracle.hash_blocks(w.tokens, w.tok_off, s.block_tokens, 0)
    sh, _ = oracle.hash_blocks(w.src_tokens, w.src_tok_off, s.block_tokens, 0)
    ox = oracle.Index(s.capacity, s.num_pods)
    ox.insert(*fill_entries(w, sh))
    ml, al, ids = ox.match_prefix(h, bo)
    bp, bs, _ = oracle.route_score(ml, bo, w.pod_load, w.ready_mask, None)
    rc, uniq, cnt = oracle.collect_blocks(ids, kv.num_blocks)

    assert np.array_equal(host(job.d_hashes), h)
    assert np.array_equal(host(job.d_match_len).reshape(s.R, s.num_pods), ml)
    assert np.array_equal(host(job.d_any_len), al)
    assert np.array_equal(host(job.d_block_ids), ids)
    assert np.array_equal(host(job.d_best_pod), bp) and np.array_equal(host(job.d_best_score), bs)
    assert int(host(job.d_count)[0]) == cnt == job.count
    assert np.array_equal(host(job.d_unique), uniq)

    # gathered buffer: sampled items against the oracle run on a one-block pool; the scatter put
    # the same bytes back, so the pool still holds its generated content there
    lay1 = oracle.kv_layout(0, kv.num_layers, kv.num_kv_heads, kv.block_tokens, kv.head_dim,
                            kv.elem_bytes, 1)
    buf = job.d_buf.view(cnt, kv.block_bytes)
    pool = job.d_pool.view(kv.num_blocks, kv.block_bytes)
    for i in (0, 1, cnt // 2, cnt - 1):
        mini = W.logical_blocks(kv, [uniq[i]])
        want = np.zeros(kv.block_bytes, dtype=np.uint8)
        oracle.kv_gather(mini, lay1, np.zeros(1, np.uint32), want)
        assert np.array_equal(host(buf[i]), want)
        assert np.array_equal(host(pool[int(uniq[i])]), mini)

    # every byte of the gathered buffer and of the pool (the scatter wrote the gathered bytes
    # back where they came from, so the pool must hold its generated content everywhere)
    model = PoolModel(kv)
    assert check_gather_full(model, uniq[:cnt], job.d_buf[: cnt * kv.block_bytes]) == []
    assert check_pool_full(model, job.d_pool) == []

    # the published batch was expired again: index as at the start
    assert job.index.stats()[0] == live0 == ox.stats()[0]
    d_m = torch.empty(job.nb, dtype=torch.uint64, device="cuda")
    job.index.lookup(job.d_new_keys, d_m, None)
    assert not host(d_m).any()
    assert job.aibx.status_fetch() == (0, 0)
