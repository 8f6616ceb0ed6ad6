"""The synthetic input generator: determinism and the structure the configurations state."""
import os

import numpy as np

import workloads as W
from workloads import build as synth_build
from workloads import synth


def test_mix64_is_stateless_and_sliceable():
    a = W.pool_bytes(3, 0, 4096)
    b = W.pool_bytes(3, 1024, 512)
    assert np.array_equal(a[1024:1536], b)
    assert not np.array_equal(W.pool_bytes(4, 0, 64), a[:64])
    # splitmix64 with state GOLD (seed 0, counter 0): published first output of seed 0
    assert int(W.mix64(0, 0)) == 0xE220A8397B1DCDAF


def test_cfg1_shape():
    w = W.build_routing(W.cfg1_routing())
    s = w.spec
    lens = np.diff(w.tok_off)
    assert len(lens) == 8 and lens.min() >= 64 and lens.max() <= 512
    assert w.tokens.min() >= 0 and w.tokens.max() < 32000
    assert (np.diff(w.src_tok_off) == 128).all() and len(w.src_masks) == 16
    assert len(w.src_masks) + len(w.filler_keys) == 1024
    assert (w.src_masks != 0).all() and (w.src_masks < 16).all()
    assert len(set(w.src_ids.tolist())) == 16
    shared = w.prompt_of_request >= 0
    assert 2 <= shared.sum() <= 6
    for r in np.nonzero(shared)[0]:
        j = w.prompt_of_request[r]
        k = min(128, lens[r])
        assert np.array_equal(w.tokens[w.tok_off[r]:w.tok_off[r] + k],
                              w.src_tokens[w.src_tok_off[j]:w.src_tok_off[j] + k])
    w2 = W.build_routing(W.cfg1_routing())
    assert np.array_equal(w.tokens, w2.tokens) and np.array_equal(w.filler_keys, w2.filler_keys)


def test_prefix_closed_residency():
    spec = W.scaled(W.cfg2_routing(), R=4, n_entries=3000)
    w = W.build_routing(spec)
    nblk = np.diff(w.src_tok_off) // spec.block_tokens
    off = np.concatenate([[0], np.cumsum(nblk)])
    for j in range(spec.n_prompts):
        m = w.src_masks[off[j]:off[j + 1]]
        # each pod's residency is a prefix: masks only lose bits along the prompt
        assert all((int(m[i + 1]) & ~int(m[i])) == 0 for i in range(len(m) - 1))
        assert int(m[-1]) != 0                      # somebody holds the whole prompt
    assert len(set(w.src_ids.tolist())) == len(w.src_ids)


def test_long_context_block_table():
    spec = W.scaled(W.cfg5_routing(), R=3, len_lo=3200, len_hi=3200, id_space=300,
                    n_entries=400, capacity=1024)
    w = W.build_routing(spec)
    assert w.block_table.shape == (3, 100)
    for r in range(3):
        assert sorted(w.block_table[r].tolist()) == list(range(100 * r, 100 * r + 100))
    assert len(w.src_ids) == 3 * 75
    assert np.array_equal(w.src_ids[:75], w.block_table[0, :75])


def test_kv_specs_and_host_pool_layouts():
    assert W.cfg2_kv().block_bytes == 2 << 20 and W.cfg2_kv().pool_bytes == 8 << 30
    assert W.cfg4_kv().tile_bytes == 64 << 10 and W.cfg4_kv().block_bytes == 5 << 20
    assert W.cfg5_kv().block_bytes == 896 << 10
    assert W.cfg1_kv().block_bytes == 32 << 10
    kv0 = W.KVSpec("t", 9, 0, 3, 1, 2, 8, 1, 5)
    kv1 = W.scaled(kv0, layout=1)
    p0 = W.host_pool(kv0).reshape(5, 3, kv0.tile_bytes)
    p1 = W.host_pool(kv1).reshape(3, 5, kv0.tile_bytes)
    assert np.array_equal(p0.transpose(1, 0, 2), p1)            # same logical content
    assert np.array_equal(W.logical_blocks(kv1, [4, 1]).reshape(2, -1), p0[[4, 1]].reshape(2, -1))
    ids = W.distinct_ids(1, 100, 64)
    assert len(set(ids.tolist())) == 64
    bits = W.bf16_normal_bits(0, 10000).astype(np.uint32) << 16
    x = bits.view(np.float32)
    assert abs(x.mean()) < 0.05 and abs(x.std() - 1.0) < 0.05


def test_native_host_twin_equals_the_numpy_generator():
    synth_build.build()
    for seed, first, n in [(3, 0, 4096), (5003, 8 * 12345, 8 * 777), (2 ** 40 + 1, 5 << 33, 64)]:
        out = np.zeros(n, dtype=np.uint8)
        synth.fill_host(out, seed, first)
        assert np.array_equal(out, W.pool_bytes(seed, first, n))
    kv = W.KVSpec("t", 9, 1, 3, 1, 2, 8, 1, 5)
    p = W.physical_blocks(kv, 1, 4).reshape(3, 3, kv.tile_bytes)          # [layer][block][tile]
    whole = W.host_pool(kv).reshape(3, 5, kv.tile_bytes)
    assert np.array_equal(p, whole[:, 1:4])
    kv2 = W.scaled(kv, layout=2)
    p2 = W.physical_blocks(kv2, 1, 4).reshape(3, 2, 3, kv.tile_bytes // 2)   # [layer][K/V][block]
    assert np.array_equal(p2.transpose(0, 2, 1, 3).reshape(3, 3, kv.tile_bytes), p)
    assert np.array_equal(W.host_pool(kv2).reshape(3, 2, 5, -1)[:, :, 1:4], p2)
    kv0 = W.scaled(kv, layout=0)
    assert np.array_equal(W.physical_blocks(kv0, 1, 4), W.host_pool(kv0)[kv.block_bytes: 4 * kv.block_bytes])


def test_generators_hold_no_method_code():
    """The generator package is shared by the CPU checker's tests and the GPU tests, so it must
    name neither side."""
    pkg = os.path.dirname(os.path.abspath(W.__file__))
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "aibxo" not in text and "import oracle" not in text, f
                assert "paper_2504_03648_b200" not in text and "aibx.h" not in text, f
