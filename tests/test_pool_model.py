"""The chunked whole-buffer / whole-pool comparison that the full-size GPU tests rely on, run
here on the CPU: the "device" pool is a host tensor on which gather and scatter are done by
plain numpy indexing (no oracle), so the model's regenerated content and the oracle's placement
of it are both checked against direct indexing, and a single flipped byte must be reported."""
import numpy as np
import pytest
import torch

import workloads as W
from gpu_util import NO_BLOCK, PoolModel, check_gather_full, check_pool_full
from workloads import build as synth_build


@pytest.mark.parametrize("layout", [0, 1, 2])
def test_model_follows_scatters_and_reports_a_flipped_byte(layout):
    synth_build.build()
    kv = W.KVSpec("pm", 21, layout, 3, 2, 4, 8, 1, 41)                 # 128-byte tiles, 384-byte blocks
    bb = kv.block_bytes
    pool = W.host_pool(kv).copy()
    logical = {0: lambda: pool.reshape(41, 3, -1),
               1: lambda: pool.reshape(3, 41, -1).transpose(1, 0, 2),
               2: lambda: pool.reshape(3, 2, 41, -1).transpose(2, 0, 1, 3)}[layout]().reshape(41, bb).copy()
    model = PoolModel(kv)
    for seed, n in ((700, 9), (701, 17)):
        ids = W.distinct_ids(seed, 41, n)
        ids[2] = NO_BLOCK
        content = W.pool_bytes(seed, 0, n * bb).reshape(n, bb)
        for i, b in enumerate(ids):
            if b != NO_BLOCK:
                logical[b] = content[i]
        model.scattered(ids, seed)
    phys = {0: lambda: logical.reshape(41, 3, -1),
            1: lambda: logical.reshape(41, 3, -1).transpose(1, 0, 2),
            2: lambda: logical.reshape(41, 3, 2, -1).transpose(1, 2, 0, 3)}[layout]().reshape(-1).copy()
    pool_t = torch.from_numpy(phys)
    assert check_pool_full(model, pool_t, chunk_bytes=5 * bb) == []
    ids = np.concatenate([W.distinct_ids(5, 41, 30), [NO_BLOCK, 7, 7]]).astype(np.uint32)
    buf = np.zeros((len(ids), bb), dtype=np.uint8)
    buf[ids != NO_BLOCK] = logical[ids[ids != NO_BLOCK]]
    buf_t = torch.from_numpy(buf.reshape(-1).copy())
    assert check_gather_full(model, ids, buf_t, chunk_bytes=4 * bb) == []
    buf_t[17 * bb + 5] ^= 1
    assert check_gather_full(model, ids, buf_t, chunk_bytes=4 * bb) == [("items", 16, 20)]
    pool_t[len(phys) - 3] ^= 0x80
    bad = check_pool_full(model, pool_t, chunk_bytes=5 * bb)
    assert bad == [("blocks", 40, 41)]
