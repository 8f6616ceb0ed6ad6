#!/usr/bin/env python
"""Benchmark of the KV-reuse hot path on B200.

One step = one pass of the whole path over one batch of the Llama-3-8B-shaped workload:
hash the 64 requests as far as matching needs, longest cached prefix against a 200k-entry index
and route score (one kernel) -> set of matched blocks -> gather them from the 8 GiB paged pool
into the transfer buffer -> scatter them back; beside the copies, on a second stream: the rest
of the hash chains, then publish and expire one batch of new index entries.

`value` is gather+scatter bytes (read + written) per second over the whole step, inputs
resident in HBM.  `e2e` is the same with host buffers: tokens come from pinned host memory,
routing results go back to the host, the matched blocks are put to pinned host memory
(aibx_kv_gather_to_host, the put to a DRAM cache) and got back from it
(aibx_kv_scatter_from_host).  The line also carries the prefix-match figures of the
routing-heavy batch (`prefix_match_routing_heavy`).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path has no exchange step.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "kv_gather_scatter_GBps_whole_step"
UNIT = "GB/s"
WORKLOAD = "cfg2-llama3-8b: 64 requests (1k-8k tokens, 32 Zipf prompts), index 200k/2^19 x 16 pods, " \
           "pool 4096 x 2 MiB bf16 blocks, gather+scatter of all matched blocks"
KERNELS_PER_STEP = 9    # head (hash+match+score), collect, gather, scatter, hash tail, insert, evict x3

# dram__bytes_read.sum + dram__bytes_write.sum per launch of kv_copy_bulk_kernel from the ncu
# capture summarised under profiles/, valid only for the kernel source with this digest.
NCU_TRAFFIC = {"kv_copy_sha1": "8e2d19eba677", "bytes_per_launch": 1026870016,
               "launch_algorithmic_bytes": 1073742848}


def kernel_digest() -> str:
    path = os.path.join(ROOT, "paper_2504_03648_b200", "csrc", "kv_copy.cuh")
    return hashlib.sha1(open(path, "rb").read()).hexdigest()[:12]


def measured_peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


# ---------------------------------------------------------------------------------------------
# clocks


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                      "sw_power_cap"), f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ---------------------------------------------------------------------------------------------
# the GPU arm


class GpuJob:
    """Everything resident on one GPU for the cfg2 workload, plus the step functions."""

    def __init__(self, device_index: int):
        import torch

        from paper_2504_03648_b200 import binding as aibx
        from workloads import synth
        import workloads as W

        self.torch, self.aibx = torch, aibx
        torch.cuda.set_device(device_index)
        aibx.lib()          # fails loudly when the CUDA library was not built
        self.w = w = W.build_routing(W.cfg2_routing())
        self.kv = kv = W.cfg2_kv()
        s = w.spec
        self.B, self.P, self.R = s.block_tokens, s.num_pods, s.R

        def dev(a):
            return torch.from_numpy(np.ascontiguousarray(a)).cuda()

        def offsets(tok_off):
            n = (tok_off[1:] - tok_off[:-1]) // self.B
            out = np.zeros(len(tok_off), dtype=np.int64)
            np.cumsum(n, out=out[1:])
            return out

        # requests: pinned on the host for the end-to-end leg, resident for the device leg
        self.h_tokens = torch.from_numpy(w.tokens).pin_memory()
        self.d_tokens = self.h_tokens.cuda()
        self.d_tok_off = dev(w.tok_off)
        blk_off = offsets(w.tok_off)
        self.nb = int(blk_off[-1])
        self.d_blk_off = dev(blk_off)
        self.d_hashes = torch.empty(self.nb, dtype=torch.uint64, device="cuda")

        # index content: the prompts' own chains (hashed on the GPU) plus filler entries
        src_off = offsets(w.src_tok_off)
        d_src_h = torch.empty(int(src_off[-1]), dtype=torch.uint64, device="cuda")
        aibx.hash_blocks(dev(w.src_tokens), dev(w.src_tok_off), dev(src_off), self.B, 0, d_src_h)
        self.index = aibx.Index(s.capacity, self.P)
        self.index.insert(torch.cat([d_src_h, dev(w.filler_keys)]),
                          dev(np.concatenate([w.src_masks, w.filler_masks])),
                          dev(np.concatenate([w.src_ids, w.filler_ids])))

        # one batch of new entries published and expired per step (state returns to the start)
        st = W.Stream(s.seed, 21)
        self.d_new_keys = dev(st.keys(self.nb))
        self.d_new_masks = dev(np.left_shift(np.uint64(1), (np.arange(self.nb) % self.P).astype(np.uint64)))
        self.d_new_ids = dev(st.randint(0, kv.num_blocks, self.nb).astype(np.uint32))
        self.d_all_ones = dev(np.full(self.nb, 0xFFFFFFFFFFFFFFFF, dtype=np.uint64))
        self.d_freed = torch.empty(self.nb, dtype=torch.uint32, device="cuda")

        # routing outputs
        R, P = self.R, self.P
        self.d_match_len = torch.empty(R * P, dtype=torch.uint32, device="cuda")
        self.d_any_len = torch.empty(R, dtype=torch.uint32, device="cuda")
        self.d_block_ids = torch.empty(self.nb, dtype=torch.uint32, device="cuda")
        self.d_best_pod = torch.empty(R, dtype=torch.int32, device="cuda")
        self.d_best_score = torch.empty(R, dtype=torch.int64, device="cuda")
        self.d_hashed = torch.empty(R, dtype=torch.uint32, device="cuda")
        self.d_next_seed = torch.empty(R, dtype=torch.uint64, device="cuda")
        self.d_pod_load = dev(w.pod_load)
        self.d_scratch = torch.empty(aibx.collect_scratch_bytes(kv.num_blocks) // 4 + 1,
                                     dtype=torch.int32, device="cuda")
        self.d_unique = torch.empty(self.nb, dtype=torch.uint32, device="cuda")
        self.d_count = torch.empty(1, dtype=torch.uint32, device="cuda")
        self.h_count = torch.empty(1, dtype=torch.uint32).pin_memory()
        self.h_best_pod = torch.empty(R, dtype=torch.int32).pin_memory()
        self.h_any_len = torch.empty(R, dtype=torch.uint32).pin_memory()
        self.h_unique = torch.empty(self.nb, dtype=torch.uint32).pin_memory()

        # KV pool and transfer buffer
        self.layout = aibx.KVLayout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens,
                                    kv.head_dim, kv.elem_bytes, kv.num_blocks)
        self.d_pool = torch.empty(kv.pool_bytes, dtype=torch.uint8, device="cuda")
        synth.fill_pool(self.d_pool, kv)
        self.count = self.routing()                      # how many blocks a step moves
        self.d_buf = torch.empty(self.count * kv.block_bytes, dtype=torch.uint8, device="cuda")
        self.h_buf = None
        self.side = None
        self.copy_events = []
        st_code = aibx.status_fetch()
        assert st_code == (0, 0), st_code

    # -- pieces of a step ------------------------------------------------------------------
    def routing_async(self) -> None:
        """Routing half of a step, enqueued only: the block count stays on the device.  Only
        the part of every chain that matching needs is hashed here (aibx_route_head); the rest
        is hashed by hash_tail() off the critical path."""
        aibx = self.aibx
        aibx.route_head(self.index, self.d_tokens, self.d_tok_off, self.d_blk_off, self.B, 0,
                        self.d_pod_load, self.w.ready_mask, None, self.d_hashes, self.d_match_len,
                        self.d_any_len, self.d_block_ids, self.d_best_pod, self.d_best_score,
                        self.d_hashed, self.d_next_seed)
        aibx.collect_blocks(self.d_block_ids, self.kv.num_blocks, self.d_scratch, self.d_unique,
                            self.d_count)

    def hash_tail(self) -> None:
        """The rest of every chain (the keys of the blocks that will be published)."""
        self.aibx.hash_blocks_resume(self.d_tokens, self.d_tok_off, self.d_blk_off, self.B,
                                     self.d_hashed, self.d_next_seed, self.d_hashes)

    def routing(self) -> int:
        aibx = self.aibx
        # hash -> match (+ score in the same kernel): one call, two launches
        aibx.route_batch(self.index, self.d_tokens, self.d_tok_off, self.d_blk_off, self.B, 0,
                         self.d_pod_load, self.w.ready_mask, None, self.d_hashes, self.d_match_len,
                         self.d_any_len, self.d_block_ids, self.d_best_pod, self.d_best_score)
        aibx.collect_blocks(self.d_block_ids, self.kv.num_blocks, self.d_scratch, self.d_unique,
                            self.d_count)
        # the host needs the size of the transfer: 4 bytes back, one stream sync
        self.h_count.copy_(self.d_count, non_blocking=True)
        self.torch.cuda.current_stream().synchronize()
        return int(self.h_count.numpy()[0])

    def publish_expire(self):
        self.index.insert(self.d_new_keys, self.d_new_masks, self.d_new_ids)
        self.index.evict(self.d_new_keys, self.d_all_ones, self.d_freed)

    def step(self, record_copy_events=False):
        """One pass of the whole path, enqueued without any host round trip: the number of
        matched blocks goes from aibx_collect_blocks to the copies on the device; the tail of
        the hash chains and the index publish/expire batch (both independent of the copies) run
        beside them on a second stream."""
        torch, aibx = self.torch, self.aibx
        main = torch.cuda.current_stream()
        if self.side is None:
            self.side = torch.cuda.Stream()
            self.ev_routed = torch.cuda.Event()
            self.ev_index = torch.cuda.Event()
        self.routing_async()
        self.ev_routed.record(main)
        self.side.wait_event(self.ev_routed)
        with torch.cuda.stream(self.side):
            self.hash_tail()
            self.publish_expire()
            self.ev_index.record(self.side)
        cap = self.count                                  # room in the transfer buffer, in blocks
        if record_copy_events:
            e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            e[0].record()
        aibx.kv_gather_counted(self.d_pool, self.layout, self.d_unique, cap, self.d_count, self.d_buf)
        if record_copy_events:
            e[1].record()
        aibx.kv_scatter_counted(self.d_pool, self.layout, self.d_unique, cap, self.d_count,
                                self.d_buf)
        if record_copy_events:
            e[2].record()
            self.copy_events.append(e)
        main.wait_event(self.ev_index)                    # the next step matches the restored index

    def step_e2e(self, pieces=32):
        """Same step with host buffers on both sides of every transfer: tokens come from pinned
        host memory, results go back to it, and the matched blocks go to pinned host memory (put:
        aibx_kv_gather_to_host) and come back from there (get: aibx_kv_scatter_from_host).  The
        block list is cut into `pieces`, consecutive pieces alternating between two streams per
        direction, so that gather, device->host, host->device and scatter of different pieces
        overlap and the two PCIe directions run at the same time.  With 32 pieces a step runs at
        the rate the link gives with both directions busy (measured 47.6 GB/s each way, against
        57 / 56 GB/s for one direction alone)."""
        torch, aibx = self.torch, self.aibx
        main = torch.cuda.current_stream()
        if self.h_buf is None:
            self.h_buf = torch.empty(self.d_buf.numel(), dtype=torch.uint8).pin_memory()
            self.d_buf_back = torch.empty_like(self.d_buf)
            self.s_put = [torch.cuda.Stream() for _ in range(2)]
            self.s_get = [torch.cuda.Stream() for _ in range(2)]
        self.d_tokens.copy_(self.h_tokens, non_blocking=True)
        n = self.routing()
        self.h_best_pod.copy_(self.d_best_pod, non_blocking=True)
        self.h_any_len.copy_(self.d_any_len, non_blocking=True)
        self.h_unique.copy_(self.d_unique, non_blocking=True)
        routed = torch.cuda.Event()
        routed.record(main)
        bb = self.kv.block_bytes
        per = (n + pieces - 1) // pieces
        done = []
        for k, c0 in enumerate(range(0, n, per)):
            m = min(per, n - c0)
            ids = self.d_unique[c0: c0 + m]
            lo, hi = c0 * bb, (c0 + m) * bb
            sp, sg = self.s_put[k % 2], self.s_get[k % 2]
            sp.wait_event(routed)
            with torch.cuda.stream(sp):
                aibx.kv_gather_to_host(self.d_pool, self.layout, ids, m, self.d_buf[lo:hi],
                                       self.h_buf[lo:hi])                       # put
                e_p = torch.cuda.Event()
                e_p.record(sp)
            sg.wait_event(e_p)
            with torch.cuda.stream(sg):
                aibx.kv_scatter_from_host(self.d_pool, self.layout, ids, m, self.d_buf_back[lo:hi],
                                          self.h_buf[lo:hi])                    # get
                e_g = torch.cuda.Event()
                e_g.record(sg)
            done.append(e_g)
        self.publish_expire()
        for e in done[-2:]:
            main.wait_event(e)
        main.synchronize()
        nbytes = n * bb
        h2d = self.h_tokens.numel() * 4 + nbytes
        d2h = 4 + self.R * 8 + self.nb * 4 + nbytes
        return h2d, d2h

    def stage_breakdown(self, reps=10):
        """Median device time of every call of the step, in microseconds (outside the timed run)."""
        torch, aibx = self.torch, self.aibx
        calls = {
            "hash_blocks": lambda: aibx.hash_blocks(self.d_tokens, self.d_tok_off, self.d_blk_off,
                                                    self.B, 0, self.d_hashes),
            "route_head": lambda: aibx.route_head(
                self.index, self.d_tokens, self.d_tok_off, self.d_blk_off, self.B, 0,
                self.d_pod_load, self.w.ready_mask, None, self.d_hashes, self.d_match_len,
                self.d_any_len, self.d_block_ids, self.d_best_pod, self.d_best_score,
                self.d_hashed, self.d_next_seed),
            "hash_tail": self.hash_tail,
            "match_prefix": lambda: self.index.match_prefix(self.d_hashes, self.d_blk_off,
                                                            self.d_match_len, self.d_any_len,
                                                            self.d_block_ids),
            "route_score": lambda: aibx.route_score(self.d_match_len, self.d_blk_off, self.P,
                                                    self.d_pod_load, self.w.ready_mask, None,
                                                    self.d_best_pod, self.d_best_score, None),
            "collect_blocks": lambda: aibx.collect_blocks(self.d_block_ids, self.kv.num_blocks,
                                                          self.d_scratch, self.d_unique, self.d_count),
            "kv_gather": lambda: aibx.kv_gather(self.d_pool, self.layout, self.d_unique, self.count,
                                                self.d_buf),
            "kv_scatter": lambda: aibx.kv_scatter(self.d_pool, self.layout, self.d_unique,
                                                  self.count, self.d_buf),
            "index_insert": lambda: self.index.insert(self.d_new_keys, self.d_new_masks,
                                                      self.d_new_ids),
            "index_evict": lambda: self.index.evict(self.d_new_keys, self.d_all_ones, self.d_freed),
        }
        out = {}
        for name, fn in calls.items():
            ts = []
            for _ in range(reps):
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                fn()
                b.record()
                b.synchronize()
                ts.append(a.elapsed_time(b) * 1e3)
            out[name] = round(statistics.median(ts), 2)
        return out


def max_over_ranks(value: float, dist, device) -> float:
    """Max of a per-rank scalar over all ranks (the timed interval of a multi-rank run)."""
    if dist is None:
        return float(value)
    import torch

    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(step_bytes_per_rank: int, world: int, ms_per_step: float) -> float:
    """Replicas only: every rank moves the same bytes; the job's rate uses the slowest rank."""
    return world * step_bytes_per_rank / (ms_per_step * 1e-3) / 1e9


def run_gpu(args):
    import torch

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist

        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (no CPU fallback exists)"

    job = GpuJob(local_rank)
    kv = job.kv
    step_bytes = 2 * 2 * job.count * kv.block_bytes        # gather + scatter, read + write

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        job.step()
    barrier()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for _ in range(args.steps):
        job.step(record_copy_events=True)
    t1.record()
    barrier()
    elapsed_ms = t0.elapsed_time(t1)
    clocks = sampler.stop() if rank == 0 else None
    elapsed_ms = max_over_ranks(elapsed_ms, dist, "cuda")
    status = job.aibx.status_fetch()
    assert status == (0, 0), status
    assert job.routing() == job.count, "the timed steps moved a different number of blocks"

    # dominant kernel: the bulk-copy kernel, two launches per step, timed inside the timed region
    durs = []
    for e in job.copy_events:
        durs += [e[0].elapsed_time(e[1]), e[1].elapsed_time(e[2])]
    launch_ms = sum(durs) / len(durs)
    launch_bytes = 2 * job.count * kv.block_bytes + 4 * job.count
    peak, peak_kind = measured_peak_hbm()
    achieved = launch_bytes / (launch_ms * 1e-3) / 1e9
    traffic = None
    if NCU_TRAFFIC["kv_copy_sha1"] == kernel_digest() and NCU_TRAFFIC["bytes_per_launch"]:
        traffic = NCU_TRAFFIC["bytes_per_launch"] * launch_bytes / NCU_TRAFFIC["launch_algorithmic_bytes"]

    # end-to-end leg (host buffers), fewer steps: PCIe-bound
    e2e_steps = max(2, min(5, args.steps))
    job.step_e2e()
    barrier()
    w0 = time.perf_counter()
    for _ in range(e2e_steps):
        h2d, d2h = job.step_e2e()
    torch.cuda.synchronize()
    e2e_s = (time.perf_counter() - w0) / e2e_steps
    e2e_s = max_over_ranks(e2e_s, dist, "cuda")

    stages = job.stage_breakdown() if rank == 0 else None
    cfg3 = None
    if rank == 0:
        # the other half of the metric: prefix match alone on the routing-heavy batch
        import workloads as W
        cfg3 = routing_batch_times(W.cfg3_routing)
    if dist is not None:
        dist.barrier()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = elapsed_ms / args.steps
    value = whole_job_value(step_bytes, world, ms_per_step)
    cpu = cpu_baseline(budget_s=12.0)
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "blocks_moved_per_step": job.count,
                   "bytes_moved_per_step": step_bytes, "parallelism": "replicas only" if world > 1 else "1 gpu",
                   "l2": "inputs larger than L2: 6.5 GB of KV traffic per step evicts it between steps",
                   "overlap": "hash chains past the first uncached block and index publish/expire on a second stream beside the copies; no host sync inside a step",
                   "kv_tuning": "bulk ring, loader + storer warp, 32 KiB x 3 stages, 1 CTA/SM"},
        "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_max_mhz", "reasons")},
        "e2e": {"value": round(world * step_bytes / e2e_s / 1e9, 2), "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": KERNELS_PER_STEP * args.steps,
        "roofline": {"bound": "hbm", "kernel": "kv_copy_bulk_kernel", "achieved": round(achieved, 1),
                     "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": round(achieved / peak, 4), "frac_of_nominal_8000": round(achieved / 8000.0, 4),
                     "traffic": traffic, "algorithmic_bytes_per_launch": launch_bytes,
                     "avg_launch_ms": round(launch_ms, 4), "launches_timed": len(durs)},
        "cpu_baseline": cpu,
        "match_requests_per_s": round(job.R / (stages["match_prefix"] * 1e-6), 1),
        "prefix_match_routing_heavy": {
            "workload": "cfg3: 4,096 requests, 527k blocks, index 2^20 entries / 2^21 slots, 64 pods",
            "match_requests_per_s": cfg3["match_requests_per_s"], "match_us": cfg3["match_us"],
            "match_requests_per_s_back_to_back": cfg3["match_requests_per_s_back_to_back"],
            "match_us_back_to_back": cfg3["match_us_back_to_back"],
            "hash_us": cfg3["hash_us"], "route_head_us": cfg3["route_head_us"],
            "decisions_per_s_via_route_head": round(cfg3["R"] / (cfg3["route_head_us"] * 1e-6), 0),
            "match_algorithmic_GBps": cfg3["match_algorithmic_GBps"]},
        "stage_us": stages,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# the CPU oracle: baseline leg and reference arm


class OracleSample:
    """The oracle on a bounded sample of the same workload: the whole routing batch, and
    gather+scatter of SAMPLE_BLOCKS blocks of the same shape out of a 512-block host pool."""

    SAMPLE_BLOCKS = 128
    POOL_BLOCKS = 512

    def __init__(self):
        import oracle
        import workloads as W

        self.oracle = oracle
        self.w = w = W.build_routing(W.cfg2_routing())
        s = w.spec
        kv = W.scaled(W.cfg2_kv(), num_blocks=self.POOL_BLOCKS)
        self.kv = kv
        sh, _ = oracle.hash_blocks(w.src_tokens, w.src_tok_off, s.block_tokens, 0)
        self.ix = oracle.Index(s.capacity, s.num_pods)
        self.ix.insert(np.concatenate([sh, w.filler_keys]),
                       np.concatenate([w.src_masks, w.filler_masks]),
                       np.concatenate([w.src_ids, w.filler_ids]))
        self.pool = W.host_pool(kv)
        self.lay = oracle.kv_layout(kv.layout, kv.num_layers, kv.num_kv_heads, kv.block_tokens,
                                    kv.head_dim, kv.elem_bytes, kv.num_blocks)
        self.ids = W.distinct_ids(5, kv.num_blocks, self.SAMPLE_BLOCKS)
        self.buf = np.zeros(self.SAMPLE_BLOCKS * kv.block_bytes, dtype=np.uint8)
        self.step_bytes = 2 * 2 * self.SAMPLE_BLOCKS * kv.block_bytes
        st = W.Stream(s.seed, 21)
        nb = int(oracle.block_offsets(w.tok_off, s.block_tokens)[-1])
        self.new_keys = st.keys(nb)
        self.new_masks = np.left_shift(np.uint64(1), (np.arange(nb) % s.num_pods).astype(np.uint64))
        self.new_ids = st.randint(0, 4096, nb).astype(np.uint32)
        self.all_ones = np.full(nb, 0xFFFFFFFFFFFFFFFF, dtype=np.uint64)

    def step(self):
        o, w, s = self.oracle, self.w, self.w.spec
        h, bo = o.hash_blocks(w.tokens, w.tok_off, s.block_tokens, 0)
        ml, al, ids = self.ix.match_prefix(h, bo)
        o.route_score(ml, bo, w.pod_load, w.ready_mask, None)
        o.collect_blocks(ids, 4096)
        o.kv_gather(self.pool, self.lay, self.ids, self.buf)
        o.kv_scatter(self.pool, self.lay, self.ids, self.buf)
        self.ix.insert(self.new_keys, self.new_masks, self.new_ids)
        self.ix.evict(self.new_keys, self.all_ones)

    describe = ("whole routing batch (64 requests, 200k-entry index) + gather and scatter of 128 of "
                "the 2 MiB blocks out of a 512-block host pool + one publish/expire batch, per step")


def cpu_baseline(budget_s: float):
    sample = OracleSample()
    sample.step()
    n, t0 = 0, time.perf_counter()
    while True:
        sample.step()
        n += 1
        dt = time.perf_counter() - t0
        if dt >= budget_s or n >= 2000:
            break
    return {"value": round(sample.step_bytes * n / dt / 1e9, 3), "unit": UNIT, "cores": 1,
            "kind": "oracle", "sample": OracleSample.describe, "steps": n,
            "seconds": round(dt, 2)}


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sample = OracleSample()
    for _ in range(max(args.warmup, 1)):
        sample.step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        sample.step()
    dt = time.perf_counter() - t0
    value = round(sample.step_bytes * args.steps / dt / 1e9, 3)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": max(args.warmup, 1),
        "ms_per_step": round(dt / args.steps * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "CPU oracle, one host core, bounded sample per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": OracleSample.describe},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------
# small single-kernel cases (profiling targets and microbenchmarks; not the bench line)


def _event_times(torch, fn, reps, warm):
    for _ in range(warm):
        fn()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b))
    return ts


def case_kv_small(args):
    """Gather then scatter 256 blocks of the cfg2 shape out of a 1 GiB pool (1 GiB of traffic
    per launch, larger than L2): the capture target for kv_copy_bulk_kernel."""
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

    def both():
        aibx.kv_gather(pool, lay, ids, n, buf)
        aibx.kv_scatter(pool, lay, ids, n, buf)

    ts = _event_times(torch, both, max(args.steps, 1), max(args.warmup, 1))
    nbytes = 2 * (2 * n * kv.block_bytes + 4 * n)
    peak, kind = measured_peak_hbm()
    best = nbytes / (min(ts) * 1e-3) / 1e9
    print(json.dumps({"case": "kv_small", "blocks": n, "algorithmic_bytes_per_launch": nbytes // 2,
                      "ms_gather_plus_scatter_median": round(statistics.median(ts), 4),
                      "GBps_median": round(nbytes / (statistics.median(ts) * 1e-3) / 1e9, 1),
                      "GBps_best": round(best, 1), "peak": peak, "peak_kind": kind,
                      "status": aibx.status_fetch()}))


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


def case_match_large(args):
    """Prefix match at a size where a bandwidth roofline means something: 2^23-slot index
    (256 MiB, load 0.5, 32 pods), R requests of 64 blocks, every block resident, so all
    64 lookups of a request are necessary.  Algorithmic bytes: 8 + 32 per lookup,
    4*P + 4*64 + 4 out per request."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    import workloads as W

    P, nblk = 32, 64
    ix, keys = _big_index(torch, aibx, W, args.log2cap, P, 11)
    out = []
    for R in (4096, 32768, 262144):
        st = W.Stream(12, R)
        pick = st.randint(0, len(keys), R * nblk)
        d_h = torch.from_numpy(keys[pick]).cuda()
        d_bo = torch.arange(0, (R + 1) * nblk, nblk, dtype=torch.int64, device="cuda")
        d_ml = torch.empty(R * P, dtype=torch.uint32, device="cuda")
        d_al = torch.empty(R, dtype=torch.uint32, device="cuda")
        d_ids = torch.empty(R * nblk, dtype=torch.uint32, device="cuda")
        flush = torch.empty(64 << 20, dtype=torch.int32, device="cuda")

        def run():
            flush.sum()                         # a 256 MiB read evicts the table from L2
            ix.match_prefix(d_h, d_bo, d_ml, d_al, d_ids)

        def only_flush():
            flush.sum()

        t_both = statistics.median(_event_times(torch, run, max(args.steps, 5), 3))
        t_flush = statistics.median(_event_times(torch, only_flush, max(args.steps, 5), 3))
        ms = t_both - t_flush
        assert int(d_al.cpu().numpy().min()) == nblk
        nbytes = R * nblk * 40 + R * (4 * P + 4 * nblk + 4)
        peak, kind = measured_peak_hbm()
        gbs = nbytes / (ms * 1e-3) / 1e9
        out.append({"R": R, "lookups": R * nblk, "ms": round(ms, 4), "GBps": round(gbs, 1),
                    "frac": round(gbs / peak, 4), "requests_per_s": round(R / (ms * 1e-3), 0),
                    "lookups_per_s": round(R * nblk / (ms * 1e-3), 0)})
    print(json.dumps({"case": "match_large", "index_slots": 1 << args.log2cap, "pods": P,
                      "blocks_per_request": nblk, "l2": "evicted before every launch (256 MiB read, "
                      "its time subtracted)", "peak": peak, "peak_kind": kind, "results": out,
                      "status": aibx.status_fetch()}))


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


def case_cfg4(args):
    """Llama-3-70B shape, layer-major pool of 20,000 x 5 MiB blocks: 100 iterations alternating
    put (gather 2,048 blocks into the block-major buffer) and get (scatter them back out)."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    from workloads import synth
    import workloads as W

    n, iters = 2048, 100
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
    nbytes = 2 * n * kv.block_bytes
    peak, kind = measured_peak_hbm()

    def gbs(t):
        return round(nbytes / (t * 1e-3) / 1e9, 1)

    g, sc = ms[0::2], ms[1::2]
    print(json.dumps({"case": "cfg4", "pool_blocks_effective": kv.num_blocks, "blocks_per_iter": n,
                      "tile_bytes": kv.tile_bytes, "bytes_per_iter": nbytes,
                      "gather_GBps_median": gbs(statistics.median(g)), "gather_GBps_best": gbs(min(g)),
                      "scatter_GBps_median": gbs(statistics.median(sc)), "scatter_GBps_best": gbs(min(sc)),
                      "all_100_GBps": round(nbytes * iters / (sum(ms) * 1e-3) / 1e9, 1),
                      "frac_of_measured_median": round(gbs(statistics.median(ms)) / peak, 4),
                      "frac_of_nominal_8000_median": round(gbs(statistics.median(ms)) / 8000.0, 4),
                      "peak": peak, "peak_kind": kind, "status": aibx.status_fetch()}))


def case_cfg5(args):
    """Long-context FP8 shape: per request gather its 3,000 cached blocks (get) and scatter its
    1,000 new blocks (put) in a block-major pool of 128,000 x 896 KiB blocks; 32 requests."""
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
    for r in range(2):
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
    gb, pb = 2 * n_get * kv.block_bytes, 2 * n_put * kv.block_bytes
    peak, kind = measured_peak_hbm()
    total = (gb + pb) * 32 / (t0.elapsed_time(t1) * 1e-3) / 1e9
    print(json.dumps({"case": "cfg5", "pool_blocks_effective": kv.num_blocks, "get_blocks": n_get,
                      "put_blocks": n_put, "block_bytes": kv.block_bytes,
                      "get_GBps_median": round(gb / (statistics.median(g) * 1e-3) / 1e9, 1),
                      "put_GBps_median": round(pb / (statistics.median(p) * 1e-3) / 1e9, 1),
                      "mixed_GBps_all_32_requests": round(total, 1),
                      "frac_of_measured": round(total / peak, 4),
                      "frac_of_nominal_8000": round(total / 8000.0, 4), "peak": peak,
                      "peak_kind": kind, "status": aibx.status_fetch()}))


def case_lookup_flat(args):
    """Flat aibx_index_lookup of 2^24 keys, half of them present, against indexes of the four
    configured sizes, cold (L2 evicted by a 256 MiB read before each launch) and warm; next to
    it a plain random gather of 32-byte rows (torch.index_select) as the hardware's own ceiling
    for this access pattern.  Algorithmic bytes per key: 8 in + 32 (one slot) + 12 out."""
    import torch

    from paper_2504_03648_b200 import binding as aibx
    import workloads as W

    n = 1 << 24
    peak, kind = measured_peak_hbm()
    flush = torch.empty(64 << 20, dtype=torch.int32, device="cuda")
    out = []
    for log2cap in (11, 19, 21, 23):
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
            flush.sum()
            ix.lookup(d_q, d_m, d_i)

        t_flush = statistics.median(_event_times(torch, lambda: flush.sum(), 7, 2))
        t_cold = statistics.median(_event_times(torch, cold, 7, 2)) - t_flush
        t_warm = statistics.median(_event_times(torch, lambda: ix.lookup(d_q, d_m, d_i), 7, 2))
        # comparator: gather the home rows of the same table size with a library kernel
        table = torch.empty(((1 << log2cap), 4), dtype=torch.int64, device="cuda")
        idx = torch.from_numpy(W.Stream(41, log2cap).randint(0, 1 << log2cap, n)).cuda()
        dst = torch.empty((n, 4), dtype=torch.int64, device="cuda")
        t_lib = statistics.median(_event_times(
            torch, lambda: torch.index_select(table, 0, idx, out=dst), 7, 2))
        nbytes = n * (8 + 32 + 12)
        out.append({"slots": 1 << log2cap, "table_MiB": (32 << log2cap) >> 20,
                    "cold_ms": round(t_cold, 4), "warm_ms": round(t_warm, 4),
                    "cold_Glookups_per_s": round(n / (t_cold * 1e-3) / 1e9, 2),
                    "warm_Glookups_per_s": round(n / (t_warm * 1e-3) / 1e9, 2),
                    "cold_GBps": round(nbytes / (t_cold * 1e-3) / 1e9, 1),
                    "warm_GBps": round(nbytes / (t_warm * 1e-3) / 1e9, 1),
                    "cold_frac": round(nbytes / (t_cold * 1e-3) / 1e9 / peak, 4),
                    "warm_frac": round(nbytes / (t_warm * 1e-3) / 1e9 / peak, 4),
                    "torch_index_select_32B_rows_Grows_per_s": round(n / (t_lib * 1e-3) / 1e9, 2)})
        ix.destroy()
        del table, idx, dst
    print(json.dumps({"case": "lookup_flat", "keys": n, "present": 0.5, "peak": peak,
                      "peak_kind": kind, "results": out, "status": aibx.status_fetch()}))


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
    cpu = ""
    try:
        for line in open("/proc/cpuinfo"):
            if line.startswith("model name"):
                cpu = line.split(":", 1)[1].strip()
                break
    except OSError:
        pass
    pool_t.shutdown()
    print(json.dumps({"case": "oracle_cfg", "cores_used": 1, "threads_used": T,
                      "cores_available": T, "cpu": cpu, "results": res}))


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
    t_flush = statistics.median(_event_times(torch, lambda: flush.sum(), 15, 3))
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
                flush.sum()
                aibx.kv_gather(pool, lay, ids, n, buf)

            def sc():
                flush.sum()
                aibx.kv_scatter(pool, lay, ids, n, buf)

            tg = statistics.median(_event_times(torch, g, 15, 3)) - t_flush
            ts = statistics.median(_event_times(torch, sc, 15, 3)) - t_flush
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
         "cfg4": case_cfg4, "cfg5": case_cfg5, "lookup_flat": case_lookup_flat}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default=None, choices=sorted(CASES),
                    help="run one small single-kernel case instead of the bench step")
    ap.add_argument("--log2cap", type=int, default=23)
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    args = ap.parse_args()
    if args.case:
        CASES[args.case](args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
