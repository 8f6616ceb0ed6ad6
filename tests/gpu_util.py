"""Helpers shared by the GPU parity tests: run the same seeded workload through the C ABI
(device) and through the CPU oracle (host), and return both sets of results as numpy arrays."""
import numpy as np
import torch

import oracle
from paper_2504_03648_b200 import binding as aibx
import workloads as W

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
    if kv.layout == 1:
        return host(pool_t.view(kv.num_layers, kv.num_blocks, kv.tile_bytes)[:, b].contiguous()).reshape(-1)
    return host(pool_t.view(kv.num_layers * 2, kv.num_blocks, kv.tile_bytes // 2)[:, b].contiguous()).reshape(-1)


# ------------------------------------------------------------------------------------------
# whole-buffer / whole-pool comparison of pools far larger than host memory


class PoolModel:
    """What a device pool must hold at any moment: its generated content, then every scatter in
    order.  Nothing is kept but the id lists: content is regenerated for the blocks asked for,
    and the scattered bytes are put in place by the oracle's scatter."""

    def __init__(self, kv: W.KVSpec):
        self.kv = kv
        self.history = []                    # (position of each block in the id list or -1, seed)

    def scattered(self, ids: np.ndarray, seed: int) -> None:
        """A transfer buffer holding stream `seed` (item i = bytes [i, i+1) * block_bytes) was
        scattered to `ids`."""
        where = np.full(self.kv.num_blocks, -1, dtype=np.int64)
        ok = np.nonzero(ids < self.kv.num_blocks)[0]
        where[ids[ok]] = ok
        self.history.append((where, seed))

    def mini_pool(self, blocks: np.ndarray):
        """(bytes, oracle layout) of a pool of len(blocks) blocks, in the real pool's physical
        layout, holding what those blocks must hold now."""
        from workloads import synth

        kv, k = self.kv, len(blocks)
        bb = kv.block_bytes
        if k and int(blocks[-1]) - int(blocks[0]) == k - 1 and (np.diff(blocks) == 1).all():
            mini = W.physical_blocks(kv, int(blocks[0]), int(blocks[0]) + k)
        else:
            mini = W.to_physical(kv, W.logical_blocks(kv, blocks), k)
        lay = kv_layout_oracle(kv, num_blocks=k)
        for where, seed in self.history:
            pos = where[blocks]
            sel = np.nonzero(pos >= 0)[0]
            if len(sel) == 0:
                continue
            items = np.empty((len(sel), bb), dtype=np.uint8)
            for j, p in enumerate(pos[sel]):
                synth.fill_host(items[j], seed, int(p) * bb)
            rc, bad = oracle.kv_scatter(mini, lay, sel.astype(np.uint32), items.reshape(-1))
            assert rc == oracle.OK and bad == 0
        return mini, lay


def _same_bytes(a: np.ndarray, b: np.ndarray) -> bool:
    if a.size != b.size:
        return False
    if a.size % 8 == 0 and a.ctypes.data % 8 == 0 and b.ctypes.data % 8 == 0:
        return bool(np.array_equal(a.view(np.uint64), b.view(np.uint64)))
    return bool(np.array_equal(a, b))


class _ChunkedCompare:
    """Device bytes come back chunk by chunk through a ring of pinned host buffers (main
    thread) while worker threads regenerate what each chunk must hold and compare; the native
    generator, the oracle and numpy all release the interpreter lock."""

    def __init__(self, chunk_bytes: int, workers=None):
        import concurrent.futures
        import os
        import queue

        self.workers = workers or max(2, min(12, (os.cpu_count() or 4) - 2))
        self.pool = concurrent.futures.ThreadPoolExecutor(self.workers)
        self.free = queue.Queue()
        for _ in range(self.workers + 2):
            stage = torch.empty(chunk_bytes, dtype=torch.uint8)
            self.free.put(stage.pin_memory() if torch.cuda.is_available() else stage)
        self.pending = []
        self.bad = []

    def submit(self, dev_bytes: torch.Tensor, expect, tag):
        """expect() -> the bytes this chunk must hold (runs in a worker thread)."""
        stage = self.free.get()
        n = dev_bytes.numel()
        stage[:n].copy_(dev_bytes)                        # pinned: a plain synchronous copy

        def work():
            try:
                if not _same_bytes(stage[:n].numpy(), expect()):
                    self.bad.append(tag)
            finally:
                self.free.put(stage)

        self.pending.append(self.pool.submit(work))

    def finish(self):
        for f in self.pending:
            f.result()
        self.pool.shutdown()
        return self.bad


def check_gather_full(model: PoolModel, ids: np.ndarray, buf_d: torch.Tensor, chunk_bytes=160 << 20):
    """EVERY byte of a gathered transfer buffer against the oracle's gather from a regenerated
    mini pool of the blocks each chunk names.  Returns the list of failing chunks (empty = ok)."""
    kv = model.kv
    bb = kv.block_bytes
    per = max(1, chunk_bytes // bb)
    cmp = _ChunkedCompare(per * bb)

    def expect_for(sub):
        def expect():
            want = np.zeros(len(sub) * bb, dtype=np.uint8)
            valid = sub < kv.num_blocks
            mini, lay = model.mini_pool(sub[valid])
            local = np.full(len(sub), NO_BLOCK, dtype=np.uint32)
            local[valid] = np.arange(int(valid.sum()), dtype=np.uint32)
            rc, bad = oracle.kv_gather(mini, lay, local, want)
            assert rc == oracle.OK
            return want
        return expect

    for i0 in range(0, len(ids), per):
        i1 = min(i0 + per, len(ids))
        cmp.submit(buf_d[i0 * bb: i1 * bb], expect_for(ids[i0:i1]), ("items", i0, i1))
    return cmp.finish()


def check_pool_full(model: PoolModel, pool_d: torch.Tensor, chunk_bytes=160 << 20):
    """EVERY byte of a device pool against the model: generated content where nothing was
    scattered, the oracle's scatter of the regenerated buffers elsewhere."""
    kv = model.kv
    bb = kv.block_bytes
    per = max(1, chunk_bytes // bb)
    cmp = _ChunkedCompare(per * bb)
    for b0 in range(0, kv.num_blocks, per):
        b1 = min(b0 + per, kv.num_blocks)
        if kv.layout == 0:
            part = pool_d[b0 * bb: b1 * bb]
        elif kv.layout == 1:
            part = pool_d.view(kv.num_layers, kv.num_blocks, kv.tile_bytes)[:, b0:b1].contiguous().view(-1)
        else:
            part = pool_d.view(kv.num_layers * 2, kv.num_blocks, kv.tile_bytes // 2)[:, b0:b1].contiguous().view(-1)
        blocks = np.arange(b0, b1, dtype=np.int64)
        cmp.submit(part, (lambda bl: (lambda: model.mini_pool(bl)[0]))(blocks), ("blocks", b0, b1))
    return cmp.finish()
