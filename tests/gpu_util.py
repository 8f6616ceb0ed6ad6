"""Helpers shared by the GPU parity tests: run the same seeded workload through the C ABI
(device) and through the CPU oracle (host), and return both sets of results as numpy arrays."""
import numpy as np
import torch

import oracle
from paper_2504_03648_b200 import binding as aibx
from paper_2504_03648_b200 import workloads as W

NO_BLOCK = 0xFFFFFFFF


def dev(a, dtype=None):
    a = np.ascontiguousarray(a if dtype is None else np.asarray(a, dtype=dtype))
    return torch.from_numpy(a).cuda()


def host(t):
    return t.cpu().numpy()


def empty(n, dtype):
    return torch.empty(int(n), dtype=dtype, device="cuda")


def gpu_hash(tokens, tok_off, B, root=0):
    blk_off = oracle.block_offsets(tok_off, B)          # plain prefix sum of len // B
    d_h = empty(max(int(blk_off[-1]), 1), torch.uint64)
    aibx.hash_blocks(dev(tokens, np.int32) if len(tokens) else empty(4, torch.int32),
                     dev(tok_off, np.int64), dev(blk_off, np.int64), B, root, d_h)
    return host(d_h)[: int(blk_off[-1])], blk_off


def fill_entries(w: W.RoutingWorkload, src_hashes):
    keys = np.concatenate([src_hashes, w.filler_keys]).astype(np.uint64)
    masks = np.concatenate([w.src_masks, w.filler_masks]).astype(np.uint64)
    ids = np.concatenate([w.src_ids, w.filler_ids]).astype(np.uint32)
    return keys, masks, ids


def routing_oracle(w: W.RoutingWorkload, params=None, ready=None):
    s = w.spec
    h, bo = oracle.hash_blocks(w.tokens, w.tok_off, s.block_tokens, 0)
    sh, _ = oracle.hash_blocks(w.src_tokens, w.src_tok_off, s.block_tokens, 0)
    ix = oracle.Index(s.capacity, s.num_pods)
    assert ix.insert(*fill_entries(w, sh)) == oracle.OK
    ml, al, ids = ix.match_prefix(h, bo)
    bp, bs, sc = oracle.route_score(ml, bo, w.pod_load, w.ready_mask if ready is None else ready,
                                    params)
    rc, uniq, cnt = oracle.collect_blocks(ids, s.id_space)
    return dict(hashes=h, blk_off=bo, src_hashes=sh, match_len=ml, any_len=al, block_ids=ids,
                best_pod=bp, best_score=bs, scores=sc, unique=uniq, count=cnt, live=ix.stats()[0],
                index=ix)


def routing_gpu(w: W.RoutingWorkload, params=None, ready=None):
    s = w.spec
    B, P, R = s.block_tokens, s.num_pods, s.R
    h, bo = gpu_hash(w.tokens, w.tok_off, B)
    sh, _ = gpu_hash(w.src_tokens, w.src_tok_off, B)
    keys, masks, ids = fill_entries(w, sh)
    ix = aibx.Index(s.capacity, P)
    ix.insert(dev(keys), dev(masks), dev(ids))
    d_h, d_bo = dev(h), dev(bo)
    nb = max(len(h), 1)
    d_ml, d_al, d_ids = empty(R * P, torch.uint32), empty(R, torch.uint32), empty(nb, torch.uint32)
    ix.match_prefix(d_h, d_bo, d_ml, d_al, d_ids)
    d_bp, d_bs, d_sc = empty(R, torch.int32), empty(R, torch.int64), empty(R * P, torch.int64)
    aibx.route_score(d_ml, d_bo, P, dev(w.pod_load, np.int32),
                     w.ready_mask if ready is None else ready, params, d_bp, d_bs, d_sc)
    scratch = empty(max(aibx.collect_scratch_bytes(s.id_space) // 4, 1), torch.uint32)
    d_un, d_cnt = empty(nb, torch.uint32), empty(1, torch.uint32)
    aibx.collect_blocks(d_ids[: len(h)], s.id_space, scratch, d_un, d_cnt)
    st = aibx.status_fetch()
    live = ix.stats()[0]
    out = dict(hashes=h, blk_off=bo, src_hashes=sh, match_len=host(d_ml).reshape(R, P),
               any_len=host(d_al), block_ids=host(d_ids)[: len(h)], best_pod=host(d_bp),
               best_score=host(d_bs), scores=host(d_sc).reshape(R, P),
               unique=host(d_un)[: len(h)], count=int(host(d_cnt)[0]), live=live, status=st,
               index=ix)
    return out


def assert_routing_equal(g, o):
    for k in ("hashes", "src_hashes", "match_len", "any_len", "block_ids", "best_pod",
              "best_score", "scores", "unique"):
        assert np.array_equal(g[k], o[k]), k
    assert g["count"] == o["count"] and g["live"] == o["live"]
    assert g["status"] == (0, 0)


def kv_layout_gpu(kv: W.KVSpec, num_blocks=None):
    return aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens, kv.head_dim,
                         kv.elem_bytes, kv.num_blocks if num_blocks is None else num_blocks)


def kv_layout_oracle(kv: W.KVSpec, layout=None, num_blocks=None):
    return oracle.kv_layout(kv.layout if layout is None else layout, kv.num_layers,
                            kv.num_kv_heads, kv.block_tokens, kv.head_dim, kv.elem_bytes,
                            kv.num_blocks if num_blocks is None else num_blocks)


def read_block(pool_t: torch.Tensor, kv: W.KVSpec, b: int) -> np.ndarray:
    """Logical bytes [layer][tile] of block b of a device pool, whatever its physical layout."""
    if kv.layout == 0:
        return host(pool_t.view(kv.num_blocks, kv.block_bytes)[b])
    return host(pool_t.view(kv.num_layers, kv.num_blocks, kv.tile_bytes)[:, b].contiguous()).reshape(-1)
