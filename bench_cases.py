"""Single-kernel cases, microbenchmarks and the measurement functions behind the extra records
of the bench line (the largest KV configurations, the DRAM-resident index, the measured
random-access ceiling, the CPU oracle on all host cores).  `python bench.py --case NAME` runs one
of them alone and prints one JSON line; bench.py's default run calls the measure_* functions."""
from __future__ import annotations

import json
import os
import statistics
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))


# dram__bytes_read.sum + dram__bytes_write.sum per launch of kv_copy_bulk_kernel from the ncu
# captures summarised under profiles/ (256 blocks of each shape, `--case kv_small --shape ...`,
# mean of one gather and one scatter launch), valid only for the kernel source with this digest.
# On all three shapes the DRAM traffic is the bytes copied minus about 50 MB: what the kernel
# wrote last is still dirty in L2 when it ends.  That residue does not grow with the launch, so a
# full launch is taken as its own algorithmic bytes minus the residue measured on the small one.
NCU_TRAFFIC = {
    "kv_copy_sha1": "0ce289089085",
    "cfg2_shape": {"bytes_per_launch": 1021574272, "launch_algorithmic_bytes": 1073742848},
    "cfg4_shape": {"bytes_per_launch": 2634682112, "launch_algorithmic_bytes": 2684355584},
    "cfg5_shape": {"bytes_per_launch": 417690368, "launch_algorithmic_bytes": 469763072},
}


def kernel_digest() -> str:
    path = os.path.join(ROOT, "paper_2504_03648_b200", "csrc", "kv_copy.cuh")
    import hashlib

    return hashlib.sha1(open(path, "rb").read()).hexdigest()[:12]


def ncu_traffic(shape: str, launch_bytes: int):
    """DRAM bytes of one launch moving `launch_bytes`, from the captured small case of the same
    block shape; None when no capture exists for this shape or the kernel has changed since the
    counters were taken."""
    rec = NCU_TRAFFIC.get(shape)
    if not rec or NCU_TRAFFIC["kv_copy_sha1"] != kernel_digest():
        return None
    residue = rec["launch_algorithmic_bytes"] - rec["bytes_per_launch"]
    return float(max(launch_bytes - residue, 0))


def measured_peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"



# ---------------------------------------------------------------------------------------------
# small single-kernel cases (profiling targets and microbenchmarks; not the bench line)


def _event_times(torch, fn, reps, warm, before=None):
    """Event-timed calls of fn; `before` (an L2 eviction, say) runs ahead of every call on the
    same stream, outside the timed pair of events."""
    for _ in range(warm):
        if before:
            before()
        fn()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if before:
            before()
        a.record()
        fn()
        b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b))
    return ts


def case_kv_small(args):
    """Gather then scatter 256 blocks of one of the configured block shapes out of a 512-block
    pool (at least 0.45 GiB of traffic per launch, larger than L2): the capture target for
    kv_copy_bulk_kernel."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    from workloads import synth
    import workloads as W

    kv0 = {"cfg2": W.cfg2_kv, "cfg4": W.cfg4_kv, "cfg5": W.cfg5_kv}[args.shape]()
    kv = W.scaled(kv0, num_blocks=512)
    n = 256
    pool = torch.empty(kv.pool_bytes, dtype=torch.uint8, device="cuda")
    synth.fill_pool(pool, kv)
    ids_np = W.distinct_ids(7, kv.num_blocks, n)
    ids = torch.from_numpy(np.sort(ids_np) if args.shape == "cfg2" else ids_np).cuda()
    buf = torch.empty(n * kv.block_bytes, dtype=torch.uint8, device="cuda")
    lay = aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens, kv.head_dim,
                        kv.elem_bytes, kv.num_blocks)

    def both():
        aibx.kv_gather(pool, lay, ids, n, buf)
        aibx.kv_scatter(pool, lay, ids, n, buf)

    ts = _event_times(torch, both, max(args.steps, 1), max(args.warmup, 1))
    nbytes = 2 * (2 * n * kv.block_bytes + 4 * n)
    peak, kind = measured_peak_hbm()
    best = nbytes / (min(ts) * 1e-3) / 1e9
    print(json.dumps({"case": "kv_small", "shape": args.shape, "blocks": n,
                      "algorithmic_bytes_per_launch": nbytes // 2,
                      "ms_gather_plus_scatter_median": round(statistics.median(ts), 4),
                      "GBps_median": round(nbytes / (statistics.median(ts) * 1e-3) / 1e9, 1),
                      "GBps_best": round(best, 1), "peak": peak, "peak_kind": kind,
                      "status": aibx.status_fetch()}))


def index_table_bytes(slots: int, pods: int = 32) -> int:
    """Bytes a probe can touch: 16 bytes per slot with up to 32 pods, 32 bytes with more (the
    4-byte eviction stamps per entry are a separate array that lookups never read)."""
    return slots * (16 if pods <= 32 else 32)


def _big_index(torch, aibx, W, log2cap, P, seed):
    """Index of 2^log2cap slots at load 0.5 filled with random keys (all pods resident)."""
    cap = 1 << log2cap
    n = cap // 2
    st = W.Stream(seed, 31)
    keys = st.keys(n)
    ix = aibx.Index(cap, P)
    allm = (1 << P) - 1 if P < 64 else 0xFFFFFFFFFFFFFFFF
    ix.insert(torch.from_numpy(keys).cuda(),
              torch.from_numpy(np.full(n, allm, dtype=np.uint64)).cuda(),
              torch.from_numpy(np.arange(n, dtype=np.uint32)).cuda())
    return ix, keys


def _random_read_ceiling(torch, ws_bytes, gran, flush, n=1 << 24):
    """Measured ceiling for this access pattern: G reads/s of uniformly random, aligned reads of
    `gran` bytes over a working set of ws_bytes, L2 evicted before every launch (best of 1, 2
    and 4 independent reads per thread)."""
    from workloads import synth

    ws_bytes = (ws_bytes + 127) // 128 * 128
    base = torch.empty(ws_bytes // 8, dtype=torch.int64, device="cuda")
    base.zero_()
    best = 0.0
    for per in (1, 2, 4):
        sink = torch.empty(n // (32 * per) + 1, dtype=torch.int64, device="cuda")

        def run():
            synth.probe_random_reads(base, ws_bytes, gran, per, n, 17 + per, sink)

        t = statistics.median(_event_times(torch, run, 7, 2, before=flush.sum))
        best = max(best, n / (t * 1e-3) / 1e9)
    del base
    return best


def measure_match_large(log2cap, Rs=(262144,), steps=7, with_ceiling=True, P=32):
    """Prefix match at a size where a bandwidth roofline means something: an index of 2^log2cap
    slots (load 0.5, 32 pods), R requests of 64 blocks, every block resident, so all 64 lookups
    of a request are necessary.  Algorithmic bytes: 8 (key) + 32 (key, mask and id of one entry,
    rounded up to a sector) per lookup, 4*P + 4*64 + 4 out per request.  L2 is evicted by a
    256 MiB read before every launch (outside the timed events).  Two denominators: the measured
    stream bandwidth, and the measured rate of random 32-byte reads over a working set of the
    table's own size (one read per lookup is the least the method needs; on this GPU a read that
    misses L2 always moves a whole 128-byte line from DRAM, whatever it asked for)."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    import workloads as W

    nblk = 64
    ix, keys = _big_index(torch, aibx, W, log2cap, P, 11)
    flush = torch.empty(64 << 20, dtype=torch.int32, device="cuda")
    peak, kind = measured_peak_hbm()
    table_bytes = index_table_bytes(1 << log2cap, P)
    ceiling = _random_read_ceiling(torch, table_bytes, 32, flush) if with_ceiling else None
    out = []
    for R in Rs:
        st = W.Stream(12, R)
        pick = st.randint(0, len(keys), R * nblk)
        d_h = torch.from_numpy(keys[pick]).cuda()
        d_bo = torch.arange(0, (R + 1) * nblk, nblk, dtype=torch.int64, device="cuda")
        d_ml = torch.empty(R * P, dtype=torch.uint32, device="cuda")
        d_al = torch.empty(R, dtype=torch.uint32, device="cuda")
        d_ids = torch.empty(R * nblk, dtype=torch.uint32, device="cuda")

        def run():
            ix.match_prefix(d_h, d_bo, d_ml, d_al, d_ids)

        # a 256 MiB read evicts the table from L2 before every timed call
        ms = statistics.median(_event_times(torch, run, max(steps, 5), 3, before=flush.sum))
        assert int(d_al.cpu().numpy().min()) == nblk
        nbytes = R * nblk * 40 + R * (4 * P + 4 * nblk + 4)
        gbs = nbytes / (ms * 1e-3) / 1e9
        row = {"R": R, "lookups": R * nblk, "ms": round(ms, 4), "GBps": round(gbs, 1),
               "frac": round(gbs / peak, 4), "requests_per_s": round(R / (ms * 1e-3), 0),
               "lookups_per_s": round(R * nblk / (ms * 1e-3), 0)}
        if ceiling:
            row["frac_of_random_read_ceiling"] = round(R * nblk / (ms * 1e-3) / 1e9 / ceiling, 4)
        out.append(row)
        del d_h, d_bo, d_ml, d_al, d_ids
    status = aibx.status_fetch()
    ix.destroy()
    res = {"index_slots": 1 << log2cap, "table_MiB": round(table_bytes / 2 ** 20, 1), "pods": P,
           "blocks_per_request": nblk,
           "l2": "evicted before every launch (256 MiB read, outside the timed events)",
           "peak": peak, "peak_kind": kind, "results": out, "status": status}
    if ceiling:
        res["random_32B_read_ceiling_Greads_per_s"] = round(ceiling, 2)
    return res


def case_match_large(args):
    out = measure_match_large(args.log2cap, Rs=(4096, 32768, 262144), steps=args.steps, P=args.pods)
    out["case"] = "match_large"
    print(json.dumps(out))


def case_random_reads(args):
    """The memory system's own ceiling for the index's access pattern: uniformly random aligned
    reads of 32, 64 and 128 bytes (no keys, no table) over working sets from L2-resident to
    DRAM-resident, L2 evicted before every launch."""
    import torch

    flush = torch.empty(64 << 20, dtype=torch.int32, device="cuda")
    peak, kind = measured_peak_hbm()
    rows = []
    sizes = (args.ws_mib,) if args.ws_mib else (11, 16, 43, 64, 128, 171, 256, 1024, 4096)
    for ws_mib in sizes:
        for gran in ((args.read_bytes,) if args.read_bytes else (32, 64, 128)):
            g = _random_read_ceiling(torch, ws_mib << 20, gran, flush)
            rows.append({"working_set_MiB": ws_mib, "read_bytes": gran, "Greads_per_s": round(g, 2),
                         "GBps": round(g * gran, 1), "frac_of_stream": round(g * gran / peak, 4)})
    print(json.dumps({"case": "random_reads", "reads_per_launch": 1 << 24, "peak": peak,
                      "peak_kind": kind, "results": rows}))


def routing_batch_times(mk):
    """Event-timed routing calls (hash, match, score, head, tail, index fill) on one of the
    routing workloads, each call alone on an otherwise idle GPU."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    import workloads as W

    w = W.build_routing(mk())
    s = w.spec
    B, P, R = s.block_tokens, s.num_pods, s.R

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    def offsets(tok_off):
        n = (tok_off[1:] - tok_off[:-1]) // B
        o = np.zeros(len(tok_off), dtype=np.int64)
        np.cumsum(n, out=o[1:])
        return o

    bo, sbo = offsets(w.tok_off), offsets(w.src_tok_off)
    d_tok, d_toff, d_bo = dev(w.tokens), dev(w.tok_off), dev(bo)
    d_h = torch.empty(int(bo[-1]), dtype=torch.uint64, device="cuda")
    d_sh = torch.empty(int(sbo[-1]), dtype=torch.uint64, device="cuda")
    aibx.hash_blocks(dev(w.src_tokens), dev(w.src_tok_off), dev(sbo), B, 0, d_sh)
    ix = aibx.Index(s.capacity, P)
    d_keys = torch.cat([d_sh, dev(w.filler_keys)])
    d_masks = dev(np.concatenate([w.src_masks, w.filler_masks]))
    d_eids = dev(np.concatenate([w.src_ids, w.filler_ids]))

    def refill():
        ix.clear()
        ix.insert(d_keys, d_masks, d_eids)

    t_clear = statistics.median(_event_times(torch, lambda: ix.clear(), 5, 2))
    t_fill = statistics.median(_event_times(torch, refill, 5, 2)) - t_clear
    d_ml = torch.empty(R * P, dtype=torch.uint32, device="cuda")
    d_al = torch.empty(R, dtype=torch.uint32, device="cuda")
    d_ids = torch.empty(int(bo[-1]), dtype=torch.uint32, device="cuda")
    d_bp = torch.empty(R, dtype=torch.int32, device="cuda")
    d_bs = torch.empty(R, dtype=torch.int64, device="cuda")
    d_load = dev(w.pod_load)
    t_hash = statistics.median(_event_times(
        torch, lambda: aibx.hash_blocks(d_tok, d_toff, d_bo, B, 0, d_h), 10, 3))
    t_match = statistics.median(_event_times(
        torch, lambda: ix.match_prefix(d_h, d_bo, d_ml, d_al, d_ids), 10, 3))
    t_score = statistics.median(_event_times(
        torch, lambda: aibx.route_score(d_ml, d_bo, P, d_load, w.ready_mask, None, d_bp, d_bs,
                                        None), 10, 3))
    def twenty_matches():
        for _ in range(20):
            ix.match_prefix(d_h, d_bo, d_ml, d_al, d_ids)

    # a router matches batch after batch: 20 calls enqueued back to back, time per call
    t_match_stream = statistics.median(_event_times(torch, twenty_matches, 5, 2)) / 20
    # the same 20 calls captured once in a CUDA graph and replayed: what the GPU needs per batch
    # when the host's call path (Python, ctypes, launch) is out of the way
    t_match_graph = None
    try:
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            twenty_matches()                          # warm-up on the capture stream
        torch.cuda.current_stream().wait_stream(side)
        with torch.cuda.graph(graph, stream=side):
            twenty_matches()
        t_match_graph = statistics.median(_event_times(torch, graph.replay, 7, 2)) / 20
    except Exception:                                  # capture refused: the figure is left out
        t_match_graph = None
    d_dn = torch.empty(R, dtype=torch.uint32, device="cuda")
    d_sd = torch.empty(R, dtype=torch.uint64, device="cuda")
    t_head = statistics.median(_event_times(
        torch, lambda: aibx.route_head(ix, d_tok, d_toff, d_bo, B, 0, d_load, w.ready_mask, None,
                                       d_h, d_ml, d_al, d_ids, d_bp, d_bs, d_dn, d_sd), 10, 3))
    t_tail = statistics.median(_event_times(
        torch, lambda: aibx.hash_blocks_resume(d_tok, d_toff, d_bo, B, d_dn, d_sd, d_h), 10, 3))
    hashed_by_head = int(d_dn.cpu().numpy().astype(np.int64).sum())
    al = d_al.cpu().numpy().astype(np.int64)
    n_r = np.diff(bo)
    lookups = int(np.minimum(al + 1, n_r).sum())
    nbytes = lookups * 40 + int((4 * P + 4) * R + 4 * al.sum())
    out = {"config": s.name, "R": R, "blocks": int(bo[-1]), "necessary_lookups": lookups,
           "index_entries": int(d_keys.numel()),
           "insert_us": round(t_fill * 1e3, 1),
           "insert_Mkeys_per_s": round(d_keys.numel() / (t_fill * 1e-3) / 1e6, 1),
           "hash_us": round(t_hash * 1e3, 1), "match_us": round(t_match * 1e3, 1),
           "score_us": round(t_score * 1e3, 1),
           "route_head_us": round(t_head * 1e3, 1), "hash_tail_us": round(t_tail * 1e3, 1),
           "blocks_hashed_by_head": hashed_by_head,
           "hash_tokens_per_s": round(len(w.tokens) / (t_hash * 1e-3), 0),
           "hash_ns_per_block_longest_chain": round(t_hash * 1e6 / int(n_r.max()), 1),
           "match_requests_per_s": round(R / (t_match * 1e-3), 0),
           "match_us_back_to_back": round(t_match_stream * 1e3, 1),
           "match_requests_per_s_back_to_back": round(R / (t_match_stream * 1e-3), 0),
           "match_algorithmic_GBps": round(nbytes / (t_match * 1e-3) / 1e9, 2)}
    if t_match_graph:
        out["match_us_in_a_graph"] = round(t_match_graph * 1e3, 2)
        out["match_requests_per_s_in_a_graph"] = round(R / (t_match_graph * 1e-3), 0)
    ix.destroy()
    return out


def case_match_cfg(args):
    """The routing calls alone on the cfg2, routing-heavy (cfg3) and long-context (cfg5) batches."""
    from paper_2504_03648_b200 import binding as aibx
    import workloads as W

    res = [routing_batch_times(mk) for mk in (W.cfg2_routing, W.cfg3_routing, W.cfg5_routing)]
    print(json.dumps({"case": "match_cfg", "results": res, "status": aibx.status_fetch()}))


def _fit_pool(torch, W, kv, extra_bytes):
    """Shrink the pool (never the batch) when the device cannot hold the whole configuration."""
    free, _ = torch.cuda.mem_get_info()
    room = free - extra_bytes - (6 << 30)
    if kv.pool_bytes <= room:
        return kv
    return W.scaled(kv, num_blocks=int(room // kv.block_bytes))


def measure_cfg4(iters=100):
    """Llama-3-70B shape, layer-major pool of 20,000 x 5 MiB blocks: `iters` iterations
    alternating put (gather 2,048 blocks into the block-major buffer) and get (scatter them back
    out), every iteration with a fresh draw of ids.  Each iteration is one launch of the copy
    kernel timed by CUDA events on its stream; 20 GiB of traffic per launch evicts L2."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    from workloads import synth
    import workloads as W

    n = 2048
    kv = _fit_pool(torch, W, W.cfg4_kv(), n * W.cfg4_kv().block_bytes)
    pool = torch.empty(kv.pool_bytes, dtype=torch.uint8, device="cuda")
    synth.fill_pool(pool, kv)
    buf = torch.empty(n * kv.block_bytes, dtype=torch.uint8, device="cuda")
    synth.fill_linear(buf, 99)
    lay = aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens, kv.head_dim,
                        kv.elem_bytes, kv.num_blocks)
    ids = [torch.from_numpy(W.distinct_ids(1000 + j, kv.num_blocks, n)).cuda() for j in range(iters)]
    for j in range(3):
        aibx.kv_gather(pool, lay, ids[j], n, buf)
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(iters + 1)]
    ev[0].record()
    for j in range(iters):
        if j % 2 == 0:
            aibx.kv_gather(pool, lay, ids[j], n, buf)
        else:
            aibx.kv_scatter(pool, lay, ids[j], n, buf)
        ev[j + 1].record()
    torch.cuda.synchronize()
    ms = [ev[j].elapsed_time(ev[j + 1]) for j in range(iters)]
    status = aibx.status_fetch()
    nbytes = 2 * n * kv.block_bytes + 4 * n
    peak, kind = measured_peak_hbm()

    def gbs(t):
        return round(nbytes / (t * 1e-3) / 1e9, 1)

    g, sc = ms[0::2], ms[1::2]
    mean_ms = sum(ms) / len(ms)
    out = {"workload": "cfg4-llama3-70b: layer-major pool of %d x 5 MiB blocks (%.1f GiB), %d "
                       "iterations alternating put (gather) and get (scatter) of 2,048 fresh ids, "
                       "block-major buffer" % (kv.num_blocks, kv.pool_bytes / 2 ** 30, iters),
           "pool_blocks_effective": kv.num_blocks, "pool_blocks_configured": 20000,
           "blocks_per_iter": n, "tile_bytes": kv.tile_bytes, "iterations": iters,
           "gather_GBps_median": gbs(statistics.median(g)), "gather_GBps_best": gbs(min(g)),
           "scatter_GBps_median": gbs(statistics.median(sc)), "scatter_GBps_best": gbs(min(sc)),
           "all_iterations_GBps": round(nbytes * iters / (sum(ms) * 1e-3) / 1e9, 1),
           "roofline": {"bound": "hbm", "kernel": "kv_copy_bulk_kernel", "achieved": gbs(mean_ms),
                        "peak": peak, "peak_kind": kind, "unit": "GB/s",
                        "frac": round(gbs(mean_ms) / peak, 4),
                        "frac_of_nominal_8000": round(gbs(mean_ms) / 8000.0, 4),
                        "traffic": ncu_traffic("cfg4_shape", nbytes),
                        "algorithmic_bytes_per_launch": nbytes,
                        "avg_launch_ms": round(mean_ms, 4), "launches_timed": iters},
           "status": status}
    del pool, buf, ids
    torch.cuda.empty_cache()
    return out


def case_cfg4(args):
    out = measure_cfg4()
    out["case"] = "cfg4"
    print(json.dumps(out))


def measure_cfg5():
    """Long-context FP8 shape: per request gather its 3,000 cached blocks (get) and scatter its
    1,000 new blocks (put) in a block-major pool of 128,000 x 896 KiB blocks; 32 requests, so the
    get:put byte ratio is 3:1.  Every call is one launch of the copy kernel, event-timed."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    from workloads import synth
    import workloads as W

    kv0 = W.cfg5_kv()
    kv = _fit_pool(torch, W, kv0, 4000 * kv0.block_bytes)
    per = 4000 if kv.num_blocks == kv0.num_blocks else (kv.num_blocks // 32) // 4 * 4
    n_get, n_put = per * 3 // 4, per // 4
    pool = torch.empty(kv.pool_bytes, dtype=torch.uint8, device="cuda")
    synth.fill_pool(pool, kv)
    get_buf = torch.empty(n_get * kv.block_bytes, dtype=torch.uint8, device="cuda")
    put_buf = torch.empty(n_put * kv.block_bytes, dtype=torch.uint8, device="cuda")
    synth.fill_linear(put_buf, 77)
    lay = aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens, kv.head_dim,
                        kv.elem_bytes, kv.num_blocks)
    tables = [torch.from_numpy((r * per + W.Stream(4, 100 + r).permutation(per)).astype(np.uint32)).cuda()
              for r in range(32)]
    for r in range(3):
        aibx.kv_gather(pool, lay, tables[r][:n_get].contiguous(), n_get, get_buf)
    torch.cuda.synchronize()
    t_get, t_put = [], []
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for r in range(32):
        a, b, c = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        ids_get, ids_put = tables[r][:n_get].contiguous(), tables[r][n_get:].contiguous()
        a.record()
        aibx.kv_gather(pool, lay, ids_get, n_get, get_buf)
        b.record()
        aibx.kv_scatter(pool, lay, ids_put, n_put, put_buf)
        c.record()
        t_get.append((a, b))
        t_put.append((b, c))
    t1.record()
    torch.cuda.synchronize()
    g = [a.elapsed_time(b) for a, b in t_get]
    p = [a.elapsed_time(b) for a, b in t_put]
    status = aibx.status_fetch()
    gb, pb = 2 * n_get * kv.block_bytes + 4 * n_get, 2 * n_put * kv.block_bytes + 4 * n_put
    peak, kind = measured_peak_hbm()
    total = (gb + pb) * 32 / (t0.elapsed_time(t1) * 1e-3) / 1e9
    # the roofline object: all 64 launches, bytes and time summed (get launches weigh 3:1)
    mean_ms = (sum(g) + sum(p)) / 64.0
    mean_bytes = (gb + pb) / 2.0
    ach = mean_bytes / (mean_ms * 1e-3) / 1e9
    out = {"workload": "cfg5-long-context-fp8: block-major pool of %d x 896 KiB blocks (%.1f GiB), "
                       "32 requests, each gathers its %d cached blocks and scatters its %d new ones "
                       "(get:put bytes 3:1)" % (kv.num_blocks, kv.pool_bytes / 2 ** 30, n_get, n_put),
           "pool_blocks_effective": kv.num_blocks, "pool_blocks_configured": kv0.num_blocks,
           "get_blocks": n_get, "put_blocks": n_put, "block_bytes": kv.block_bytes,
           "get_GBps_median": round(gb / (statistics.median(g) * 1e-3) / 1e9, 1),
           "put_GBps_median": round(pb / (statistics.median(p) * 1e-3) / 1e9, 1),
           "mixed_GBps_all_32_requests": round(total, 1),
           "roofline": {"bound": "hbm", "kernel": "kv_copy_bulk_kernel", "achieved": round(ach, 1),
                        "peak": peak, "peak_kind": kind, "unit": "GB/s",
                        "frac": round(ach / peak, 4),
                        "frac_of_nominal_8000": round(ach / 8000.0, 4),
                        "traffic": ncu_traffic("cfg5_shape", int(mean_bytes)),
                        "algorithmic_bytes_per_launch": int(mean_bytes),
                        "avg_launch_ms": round(mean_ms, 4), "launches_timed": 64},
           "status": status}
    del pool, get_buf, put_buf, tables
    torch.cuda.empty_cache()
    return out


def case_cfg5(args):
    out = measure_cfg5()
    out["case"] = "cfg5"
    print(json.dumps(out))


def measure_lookup_flat(log2caps=(11, 19, 21, 23), reps=7, with_library=True):
    """Flat aibx_index_lookup of 2^24 keys, half of them present, against indexes of the four
    configured sizes, cold (L2 evicted by a 256 MiB read before each launch) and warm; next to
    it the measured ceiling for this access pattern (random 32-byte reads over a working set of
    the table's size) and a library gather of 32-byte rows (torch.index_select).  Algorithmic
    bytes per key: 8 in + 32 (one slot) + 12 out."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    import workloads as W

    n = 1 << 24
    peak, kind = measured_peak_hbm()
    flush = torch.empty(64 << 20, dtype=torch.int32, device="cuda")
    out = []
    for log2cap in log2caps:
        ix, keys = _big_index(torch, aibx, W, log2cap, 32, 20 + log2cap)
        st = W.Stream(40, log2cap)
        pick = st.randint(0, len(keys), n)
        q = keys[pick]
        miss = st.unit(n) < 0.5
        q[miss] = st.keys(int(miss.sum()))
        d_q = torch.from_numpy(q).cuda()
        d_m = torch.empty(n, dtype=torch.uint64, device="cuda")
        d_i = torch.empty(n, dtype=torch.uint32, device="cuda")

        def cold():
            ix.lookup(d_q, d_m, d_i)

        t_cold = statistics.median(_event_times(torch, cold, reps, 2, before=flush.sum))
        t_warm = statistics.median(_event_times(torch, lambda: ix.lookup(d_q, d_m, d_i), reps, 2))
        nbytes = n * (8 + 32 + 12)
        row = {"slots": 1 << log2cap, "table_MiB": round(index_table_bytes(1 << log2cap) / 2 ** 20, 2),
               "cold_ms": round(t_cold, 4), "warm_ms": round(t_warm, 4),
               "cold_Glookups_per_s": round(n / (t_cold * 1e-3) / 1e9, 2),
               "warm_Glookups_per_s": round(n / (t_warm * 1e-3) / 1e9, 2),
               "cold_GBps": round(nbytes / (t_cold * 1e-3) / 1e9, 1),
               "warm_GBps": round(nbytes / (t_warm * 1e-3) / 1e9, 1),
               "cold_frac": round(nbytes / (t_cold * 1e-3) / 1e9 / peak, 4),
               "warm_frac": round(nbytes / (t_warm * 1e-3) / 1e9 / peak, 4)}
        if log2cap >= 12:
            ceiling = _random_read_ceiling(torch, index_table_bytes(1 << log2cap), 32, flush)
            row["random_32B_read_ceiling_Greads_per_s"] = round(ceiling, 2)
            row["cold_frac_of_random_read_ceiling"] = round(n / (t_cold * 1e-3) / 1e9 / ceiling, 4)
        if with_library:
            # comparator: gather rows of the same table size with a library kernel
            table = torch.empty(((1 << log2cap), 4), dtype=torch.int64, device="cuda")
            idx = torch.from_numpy(W.Stream(41, log2cap).randint(0, 1 << log2cap, n)).cuda()
            dst = torch.empty((n, 4), dtype=torch.int64, device="cuda")
            t_lib = statistics.median(_event_times(
                torch, lambda: torch.index_select(table, 0, idx, out=dst), reps, 2))
            row["torch_index_select_32B_rows_Grows_per_s"] = round(n / (t_lib * 1e-3) / 1e9, 2)
            del table, idx, dst
        out.append(row)
        ix.destroy()
        del d_q, d_m, d_i
    return {"keys": n, "present": 0.5, "peak": peak, "peak_kind": kind, "results": out,
            "status": aibx.status_fetch()}


def case_lookup_flat(args):
    out = measure_lookup_flat()
    out["case"] = "lookup_flat"
    print(json.dumps(out))


def cpu_model() -> str:
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return ""


def case_oracle_cfg(args):
    """The CPU oracle on the routing halves of cfg2 / cfg3 / cfg5 at full size and on
    gather+scatter of 128 blocks of each KV shape (pool of 256 blocks on the host): on one host
    core, and the same oracle functions called from one thread per available core over disjoint
    request ranges (hash, match, score; the index is only read) or disjoint id ranges (gather,
    scatter).  The calls are ctypes calls, which release the interpreter lock."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    import workloads as W

    T = len(os.sched_getaffinity(0))
    pool_t = ThreadPoolExecutor(max_workers=T)

    def ranges(n):
        cuts = [n * i // T for i in range(T + 1)]
        return [(a, b) for a, b in zip(cuts[:-1], cuts[1:]) if b > a]

    def fan(fn, n):
        list(pool_t.map(lambda ab: fn(*ab), ranges(n)))

    def sub_off(off, a, b):
        return np.ascontiguousarray(off[a:b + 1] - off[a])

    def clock(fn, reps=3):
        ts = []
        for _ in range(reps):
            t0 = time.perf_counter()
            fn()
            ts.append(time.perf_counter() - t0)
        return min(ts)

    res = []
    for mk in (W.cfg2_routing, W.cfg3_routing, W.cfg5_routing):
        w = W.build_routing(mk())
        s = w.spec
        t_hash = clock(lambda: oracle.hash_blocks(w.tokens, w.tok_off, s.block_tokens, 0))
        h, bo = oracle.hash_blocks(w.tokens, w.tok_off, s.block_tokens, 0)
        sh, _ = oracle.hash_blocks(w.src_tokens, w.src_tok_off, s.block_tokens, 0)
        keys = np.concatenate([sh, w.filler_keys])
        masks = np.concatenate([w.src_masks, w.filler_masks])
        ids = np.concatenate([w.src_ids, w.filler_ids])
        ix = oracle.Index(s.capacity, s.num_pods)
        t0 = time.perf_counter()
        ix.insert(keys, masks, ids)
        t_ins = time.perf_counter() - t0
        t_match = clock(lambda: ix.match_prefix(h, bo))
        ml, al, _ = ix.match_prefix(h, bo)
        t_score = clock(lambda: oracle.route_score(ml, bo, w.pod_load, w.ready_mask, None))
        R = len(w.tok_off) - 1
        tok_parts = {ab: (np.ascontiguousarray(w.tokens[w.tok_off[ab[0]]:w.tok_off[ab[1]]]),
                          sub_off(w.tok_off, *ab)) for ab in ranges(R)}
        h_parts = {ab: (np.ascontiguousarray(h[bo[ab[0]]:bo[ab[1]]]), sub_off(bo, *ab),
                        np.ascontiguousarray(ml[ab[0]:ab[1]])) for ab in ranges(R)}
        tt_hash = clock(lambda: fan(lambda a, b: oracle.hash_blocks(
            *tok_parts[(a, b)], s.block_tokens, 0), R))
        tt_match = clock(lambda: fan(lambda a, b: ix.match_prefix(*h_parts[(a, b)][:2]), R))
        tt_score = clock(lambda: fan(lambda a, b: oracle.route_score(
            h_parts[(a, b)][2], h_parts[(a, b)][1], w.pod_load, w.ready_mask, None), R))
        res.append({"config": s.name, "hash_us": round(t_hash * 1e6, 1),
                    "insert_us": round(t_ins * 1e6, 1), "match_us": round(t_match * 1e6, 1),
                    "score_us": round(t_score * 1e6, 1),
                    "threads": {"hash_us": round(tt_hash * 1e6, 1),
                                "match_us": round(tt_match * 1e6, 1),
                                "score_us": round(tt_score * 1e6, 1)}})
    for kv0 in (W.cfg2_kv(), W.cfg4_kv(), W.cfg5_kv()):
        kv = W.scaled(kv0, num_blocks=256)
        pool = W.host_pool(kv)
        lay = oracle.kv_layout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens,
                               kv.head_dim, kv.elem_bytes, kv.num_blocks)
        ids = W.distinct_ids(5, 256, 128)
        buf = np.zeros(128 * kv.block_bytes, dtype=np.uint8)
        tg = clock(lambda: oracle.kv_gather(pool, lay, ids, buf))
        ts = clock(lambda: oracle.kv_scatter(pool, lay, ids, buf))
        nb = 2 * 128 * kv.block_bytes
        bb = kv.block_bytes
        ttg = clock(lambda: fan(lambda a, b: oracle.kv_gather(
            pool, lay, ids[a:b], buf[a * bb:b * bb]), 128))
        tts = clock(lambda: fan(lambda a, b: oracle.kv_scatter(
            pool, lay, ids[a:b], buf[a * bb:b * bb]), 128))
        res.append({"config": kv0.name, "gather_GBps": round(nb / tg / 1e9, 2),
                    "scatter_GBps": round(nb / ts / 1e9, 2),
                    "threads": {"gather_GBps": round(nb / ttg / 1e9, 2),
                                "scatter_GBps": round(nb / tts / 1e9, 2)}})
    pool_t.shutdown()
    print(json.dumps({"case": "oracle_cfg", "cores_used": 1, "threads_used": T,
                      "cores_available": T, "cpu": cpu_model(), "results": res}))


def case_hash_sweep(args):
    """hash_blocks alone: R equal-length requests, block sizes 8..64 tokens.  With few requests
    the time is the serial seed chain of one request, which separates the cost of a 32-byte
    stripe from the cost of a block end (fold + avalanche + reseed)."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    import workloads as W

    out = []
    for R, L in ((1, 32768), (64, 32768), (4096, 2048)):
        toks = torch.from_numpy(W.Stream(50, R).randint(0, 128256, R * L).astype(np.int32)).cuda()
        off = torch.arange(0, (R + 1) * L, L, dtype=torch.int64, device="cuda")
        for B in (8, 16, 32, 64):
            nb = L // B
            bo = torch.arange(0, (R + 1) * nb, nb, dtype=torch.int64, device="cuda")
            h = torch.empty(R * nb, dtype=torch.uint64, device="cuda")
            ms = statistics.median(_event_times(
                torch, lambda: aibx.hash_blocks(toks, off, bo, B, 0, h), 7, 3))
            out.append({"R": R, "tokens_per_request": L, "block_tokens": B,
                        "us": round(ms * 1e3, 1), "ns_per_block_of_a_chain": round(ms * 1e6 / nb, 1),
                        "ns_per_stripe_of_a_chain": round(ms * 1e6 / (nb * B // 8), 1),
                        "tokens_per_s": round(R * L / (ms * 1e-3), 0)})
    print(json.dumps({"case": "hash_sweep", "results": out, "status": aibx.status_fetch()}))


def case_kv_inner(args):
    """Gather/scatter with the head/token order of every tile swapped on the way (cfg2 block
    shape, 1,600 blocks = 3.4 GB per direction) next to the plain gather of the same blocks."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    from workloads import synth
    import workloads as W

    out = []
    for name, kv, n in (("cfg2 shape", W.scaled(W.cfg2_kv(), num_blocks=4096), 1600),
                        ("cfg4 shape", W.scaled(W.cfg4_kv(), num_blocks=2000), 640),
                        ("cfg5 shape", W.scaled(W.cfg5_kv(), num_blocks=8000), 3000)):
        pool = torch.empty(kv.pool_bytes, dtype=torch.uint8, device="cuda")
        synth.fill_pool(pool, kv)
        ids = torch.from_numpy(W.distinct_ids(7, kv.num_blocks, n)).cuda()
        buf = torch.empty(n * kv.block_bytes, dtype=torch.uint8, device="cuda")
        lay = aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens,
                            kv.head_dim, kv.elem_bytes, kv.num_blocks)
        nbytes = 2 * n * kv.block_bytes
        t_plain = statistics.median(_event_times(
            torch, lambda: aibx.kv_gather(pool, lay, ids, n, buf), 10, 3))
        row = {"shape": name, "blocks": n, "bytes_read_plus_written": nbytes,
               "plain_gather_GBps": round(nbytes / (t_plain * 1e-3) / 1e9, 1)}
        for engine, tag in ((2, "tensor_store"), (1, "storer_warps")):
            aibx.kv_set_inner_engine(engine)
            for pi, bi, order in ((0, 1, "head_token_to_token_head"),
                                  (1, 0, "token_head_to_head_token")):
                t_g = statistics.median(_event_times(
                    torch, lambda: aibx.kv_gather_inner(pool, lay, pi, bi, ids, n, buf), 10, 3))
                t_s = statistics.median(_event_times(
                    torch, lambda: aibx.kv_scatter_inner(pool, lay, pi, bi, ids, n, buf), 10, 3))
                row["%s_%s_gather_GBps" % (tag, order)] = round(nbytes / (t_g * 1e-3) / 1e9, 1)
                row["%s_%s_scatter_GBps" % (tag, order)] = round(nbytes / (t_s * 1e-3) / 1e9, 1)
        aibx.kv_set_inner_engine(0)
        out.append(row)
        del pool, buf
        torch.cuda.empty_cache()
    peak, kind = measured_peak_hbm()
    print(json.dumps({"case": "kv_inner", "peak": peak, "peak_kind": kind, "results": out,
                      "status": aibx.status_fetch()}))


def case_kv_inner_small(args):
    """Gather then scatter 256 blocks of the cfg2 shape out of a 1 GiB pool with the head/token
    order swapped (tensor-map store): the capture target for kv_permute_tma_kernel."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    from workloads import synth
    import workloads as W

    kv = W.scaled(W.cfg2_kv(), num_blocks=512)
    n = 256
    pool = torch.empty(kv.pool_bytes, dtype=torch.uint8, device="cuda")
    synth.fill_pool(pool, kv)
    ids = torch.from_numpy(np.sort(W.distinct_ids(7, kv.num_blocks, n))).cuda()
    buf = torch.empty(n * kv.block_bytes, dtype=torch.uint8, device="cuda")
    lay = aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens, kv.head_dim,
                        kv.elem_bytes, kv.num_blocks)
    aibx.kv_set_inner_engine(2)

    def both():
        aibx.kv_gather_inner(pool, lay, 0, 1, ids, n, buf)
        aibx.kv_scatter_inner(pool, lay, 0, 1, ids, n, buf)

    ts = _event_times(torch, both, max(args.steps, 1), max(args.warmup, 1))
    aibx.kv_set_inner_engine(0)
    nbytes = 2 * (2 * n * kv.block_bytes + 4 * n)
    peak, kind = measured_peak_hbm()
    print(json.dumps({"case": "kv_inner_small", "blocks": n,
                      "algorithmic_bytes_per_launch": nbytes // 2,
                      "ms_gather_plus_scatter_median": round(statistics.median(ts), 4),
                      "GBps_median": round(nbytes / (statistics.median(ts) * 1e-3) / 1e9, 1),
                      "GBps_best": round(nbytes / (min(ts) * 1e-3) / 1e9, 1), "peak": peak,
                      "peak_kind": kind, "status": aibx.status_fetch()}))


def case_kv_sweep(args):
    """Gather and scatter of n blocks, n = 1 ... 4,096, on the three KV shapes: where the
    bandwidth saturates (CUDA events around single calls, median of 15; L2 is evicted by a
    256 MiB read before every call and that read's time is subtracted)."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    from workloads import synth
    import workloads as W

    out = []
    flush = torch.empty(64 << 20, dtype=torch.int32, device="cuda")
    for name, kv in (("cfg2 shape (2 MiB blocks, block-major)", W.scaled(W.cfg2_kv(), num_blocks=4096)),
                     ("cfg4 shape (5 MiB blocks, layer-major)", W.scaled(W.cfg4_kv(), num_blocks=4096)),
                     ("cfg5 shape (896 KiB blocks, block-major)", W.scaled(W.cfg5_kv(), num_blocks=4096))):
        pool = torch.empty(kv.pool_bytes, dtype=torch.uint8, device="cuda")
        synth.fill_pool(pool, kv)
        buf = torch.empty(4096 * kv.block_bytes, dtype=torch.uint8, device="cuda")
        lay = aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens,
                            kv.head_dim, kv.elem_bytes, kv.num_blocks)
        all_ids = torch.from_numpy(W.distinct_ids(7, kv.num_blocks, 4096)).cuda()
        rows = []
        for n in (1, 2, 4, 8, 16, 32, 64, 128, 256, 512, 1024, 2048, 4096):
            ids = all_ids[:n].contiguous()

            def g():
                aibx.kv_gather(pool, lay, ids, n, buf)

            def sc():
                aibx.kv_scatter(pool, lay, ids, n, buf)

            tg = statistics.median(_event_times(torch, g, 15, 3, before=flush.sum))
            ts = statistics.median(_event_times(torch, sc, 15, 3, before=flush.sum))
            nbytes = 2 * n * kv.block_bytes
            rows.append({"n": n, "MB_moved": round(nbytes / 1e6, 1),
                         "gather_us": round(tg * 1e3, 1), "scatter_us": round(ts * 1e3, 1),
                         "gather_GBps": round(nbytes / (tg * 1e-3) / 1e9, 1),
                         "scatter_GBps": round(nbytes / (ts * 1e-3) / 1e9, 1)})
        out.append({"shape": name, "rows": rows})
        del pool, buf
        torch.cuda.empty_cache()
    peak, kind = measured_peak_hbm()
    print(json.dumps({"case": "kv_sweep", "peak": peak, "peak_kind": kind, "results": out,
                      "status": aibx.status_fetch()}))


def case_kv_layouts(args):
    """Gather and scatter of the same block shapes out of pools laid out block-major (0),
    layer-major (1) and layer-major with K and V of a layer as separate tensors (2): the three
    should move bytes at the same rate (cfg2 shape: 1,600 x 2 MiB of a 4,096-block pool; cfg4
    shape: 1,024 x 5 MiB of a 4,096-block pool; every launch moves more than L2 holds)."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    from workloads import synth
    import workloads as W

    out = []
    peak, kind = measured_peak_hbm()
    for name, kv0, n in (("cfg2 shape", W.cfg2_kv(), 1600), ("cfg4 shape", W.cfg4_kv(), 1024)):
        row = {"shape": name, "blocks": n}
        for layout in (0, 1, 2):
            kv = W.scaled(kv0, num_blocks=4096, layout=layout)
            pool = torch.empty(kv.pool_bytes, dtype=torch.uint8, device="cuda")
            synth.fill_pool(pool, kv)
            ids = torch.from_numpy(W.distinct_ids(7, kv.num_blocks, n)).cuda()
            buf = torch.empty(n * kv.block_bytes, dtype=torch.uint8, device="cuda")
            lay = aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens,
                                kv.head_dim, kv.elem_bytes, kv.num_blocks)
            nbytes = 2 * n * kv.block_bytes
            tg = statistics.median(_event_times(torch, lambda: aibx.kv_gather(pool, lay, ids, n, buf), 15, 3))
            ts = statistics.median(_event_times(torch, lambda: aibx.kv_scatter(pool, lay, ids, n, buf), 15, 3))
            row["layout%d_gather_GBps" % layout] = round(nbytes / (tg * 1e-3) / 1e9, 1)
            row["layout%d_scatter_GBps" % layout] = round(nbytes / (ts * 1e-3) / 1e9, 1)
            del pool, buf
            torch.cuda.empty_cache()
        out.append(row)
    print(json.dumps({"case": "kv_layouts", "peak": peak, "peak_kind": kind, "results": out,
                      "status": aibx.status_fetch()}))


def case_index_ops(args):
    """Operational index calls on the routing-heavy index (2^20 entries in 2^21 slots, 64 pods):
    touch, pick_victims, export, rehash, and the sequential assignment of 4,096 requests."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    import workloads as W

    ix, keys = _big_index(torch, aibx, W, 21, 64, 61)
    n = len(keys)
    d_keys = torch.from_numpy(keys).cuda()
    st = W.Stream(62, 0)
    res = {}
    for epoch in range(1, 5):
        batch = torch.from_numpy(keys[st.randint(0, n, n // 8)]).cuda()
        ts = _event_times(torch, lambda: ix.touch(batch, epoch), 3, 1)
        res["touch_%dk_keys_us" % (batch.numel() // 1000)] = round(statistics.median(ts) * 1e3, 1)
    for k in (1000, 100000):
        d_k = torch.empty(k, dtype=torch.uint64, device="cuda")
        d_p = torch.empty(k, dtype=torch.uint32, device="cuda")
        d_c = torch.empty(1, dtype=torch.uint64, device="cuda")
        ts = _event_times(torch, lambda: ix.pick_victims(k, d_k, d_p, d_c), 7, 2)
        res["pick_%d_victims_us" % k] = round(statistics.median(ts) * 1e3, 1)
        assert int(d_c.cpu().numpy()[0]) == k
    d_k = torch.empty(n, dtype=torch.uint64, device="cuda")
    d_m = torch.empty(n, dtype=torch.uint64, device="cuda")
    d_i = torch.empty(n, dtype=torch.uint32, device="cuda")
    d_c = torch.empty(1, dtype=torch.uint64, device="cuda")
    ts = _event_times(torch, lambda: ix.export(d_k, d_m, d_i, d_c), 7, 2)
    res["export_1M_entries_us"] = round(statistics.median(ts) * 1e3, 1)
    t0 = time.perf_counter()
    ix.rehash(1 << 22)
    torch.cuda.synchronize()
    res["rehash_2M_to_4M_slots_ms_wall"] = round((time.perf_counter() - t0) * 1e3, 2)
    R, P = 4096, 64
    ml = torch.from_numpy(st.randint(0, 100, R * P).astype(np.uint32)).cuda()
    bo = torch.arange(0, (R + 1) * 128, 128, dtype=torch.int64, device="cuda")
    load = torch.zeros(P, dtype=torch.int32, device="cuda")
    bp = torch.empty(R, dtype=torch.int32, device="cuda")
    bs = torch.empty(R, dtype=torch.int64, device="cuda")
    ts = _event_times(torch, lambda: aibx.route_assign(ml, bo, P, load, (1 << 64) - 1, None, 1, bp, bs), 7, 2)
    res["route_assign_4096_requests_64_pods_us"] = round(statistics.median(ts) * 1e3, 1)
    # matching alone against matching that also stamps the matched prefix (a new epoch per call,
    # so every call writes its stamps), on the routing-heavy batch
    w = W.build_routing(W.cfg3_routing())
    s3 = w.spec
    B, P3, R3 = s3.block_tokens, s3.num_pods, s3.R

    def offsets(tok_off):
        k = (tok_off[1:] - tok_off[:-1]) // B
        o = np.zeros(len(tok_off), dtype=np.int64)
        np.cumsum(k, out=o[1:])
        return o

    def dev(a):
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()

    bo3, sbo3 = offsets(w.tok_off), offsets(w.src_tok_off)
    d_bo3 = dev(bo3)
    d_h3 = torch.empty(int(bo3[-1]), dtype=torch.uint64, device="cuda")
    d_sh3 = torch.empty(int(sbo3[-1]), dtype=torch.uint64, device="cuda")
    aibx.hash_blocks(dev(w.tokens), dev(w.tok_off), d_bo3, B, 0, d_h3)
    aibx.hash_blocks(dev(w.src_tokens), dev(w.src_tok_off), dev(sbo3), B, 0, d_sh3)
    ix3 = aibx.Index(s3.capacity, P3)
    ix3.insert(torch.cat([d_sh3, dev(w.filler_keys)]),
               dev(np.concatenate([w.src_masks, w.filler_masks])),
               dev(np.concatenate([w.src_ids, w.filler_ids])))
    d_ml3 = torch.empty(R3 * P3, dtype=torch.uint32, device="cuda")
    d_al3 = torch.empty(R3, dtype=torch.uint32, device="cuda")
    d_id3 = torch.empty(int(bo3[-1]), dtype=torch.uint32, device="cuda")
    epoch = [0]

    def match_touch():
        epoch[0] += 1
        ix3.match_prefix_touch(d_h3, d_bo3, epoch[0], d_ml3, d_al3, d_id3)

    t_m = statistics.median(_event_times(
        torch, lambda: ix3.match_prefix(d_h3, d_bo3, d_ml3, d_al3, d_id3), 15, 3))
    t_mt = statistics.median(_event_times(torch, match_touch, 15, 3))
    hit = d_h3[:1]
    keys_hit = torch.cat([d_h3[int(bo3[r]): int(bo3[r]) + int(a)]
                          for r, a in enumerate(d_al3.cpu().numpy()) if a > 0] or [hit])

    def separate():
        epoch[0] += 1
        ix3.match_prefix(d_h3, d_bo3, d_ml3, d_al3, d_id3)
        ix3.touch(keys_hit, epoch[0])

    t_sep = statistics.median(_event_times(torch, separate, 15, 3))
    res["cfg3_match_us"] = round(t_m * 1e3, 1)
    res["cfg3_match_touch_us"] = round(t_mt * 1e3, 1)
    res["cfg3_match_then_touch_as_two_calls_us"] = round(t_sep * 1e3, 1)
    res["cfg3_matched_blocks_stamped"] = int(keys_hit.numel())
    res["cfg3_match_touch_over_match"] = round(t_mt / t_m, 3)
    print(json.dumps({"case": "index_ops", "entries": n, "results": res,
                      "status": aibx.status_fetch()}))


def case_kv_comparators(args):
    """Library comparators for the gather on the same GPU and bytes (cfg2 block shape, 1,600
    blocks): a plain device-to-device copy of the same size and torch.index_select over rows."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    from workloads import synth
    import workloads as W

    kv = W.cfg2_kv()
    n = 1600
    pool = torch.empty(kv.pool_bytes, dtype=torch.uint8, device="cuda")
    synth.fill_pool(pool, kv)
    ids_np = np.sort(W.distinct_ids(7, kv.num_blocks, n))
    ids = torch.from_numpy(ids_np).cuda()
    idx64 = torch.from_numpy(ids_np.astype(np.int64)).cuda()
    buf = torch.empty(n * kv.block_bytes, dtype=torch.uint8, device="cuda")
    lay = aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens, kv.head_dim,
                        kv.elem_bytes, kv.num_blocks)
    nbytes = 2 * n * kv.block_bytes
    rows = pool.view(torch.int32).view(kv.num_blocks, kv.block_bytes // 4)
    out_rows = buf.view(torch.int32).view(n, kv.block_bytes // 4)
    src = pool[: n * kv.block_bytes]

    def rate(fn):
        return round(nbytes / (statistics.median(_event_times(torch, fn, 10, 3)) * 1e-3) / 1e9, 1)

    res = {"aibx_kv_gather_GBps": rate(lambda: aibx.kv_gather(pool, lay, ids, n, buf)),
           "device_copy_same_bytes_GBps": rate(lambda: buf.copy_(src)),
           "torch_index_select_GBps": rate(lambda: torch.index_select(rows, 0, idx64, out=out_rows))}
    peak, kind = measured_peak_hbm()
    print(json.dumps({"case": "kv_comparators", "blocks": n, "bytes_read_plus_written": nbytes,
                      "peak": peak, "peak_kind": kind, "results": res,
                      "status": aibx.status_fetch()}))


CASES = {"kv_comparators": case_kv_comparators, "index_ops": case_index_ops, "kv_inner": case_kv_inner, "kv_inner_small": case_kv_inner_small, "kv_sweep": case_kv_sweep, "hash_sweep": case_hash_sweep, "oracle_cfg": case_oracle_cfg, "kv_small": case_kv_small, "match_large": case_match_large, "match_cfg": case_match_cfg,
         "cfg4": case_cfg4, "cfg5": case_cfg5, "lookup_flat": case_lookup_flat,
         "random_reads": case_random_reads, "kv_layouts": case_kv_layouts}


