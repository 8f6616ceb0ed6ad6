#!/usr/bin/env python
"""Benchmark of the KV-reuse hot path on B200.

One step = one pass of the whole path over one batch of the Llama-3-8B-shaped workload:
hash the 64 requests as far as matching needs, longest cached prefix against a 200k-entry index
and route score (one kernel) -> set of matched blocks -> gather them from the 8 GiB paged pool
into the transfer buffer -> scatter them back; beside the copies, on a second stream: the rest
of the hash chains, then publish and expire one batch of new index entries; and on a third
stream, once the index is back in its start state, the routing of the next batch.

`value` is gather+scatter bytes (read + written) per second over the whole step, inputs
resident in HBM.  `e2e` is the same with host buffers: tokens come from pinned host memory,
routing results go back to the host, the matched blocks are put to pinned host memory
(aibx_kv_gather_to_host, the put to a DRAM cache) and got back from it
(aibx_kv_scatter_from_host).  Sibling records of the same line, each with its own roofline:
`kv_cfg4` (the largest configuration: 2,048 x 5 MiB blocks per call out of a 97.7 GiB layer-major
pool, put and get alternating), `kv_cfg5` (long-context FP8 pool, get:put 3:1),
`prefix_match_routing_heavy` (the routing-heavy batch), `prefix_match_large_index` (the match
kernel on indexes of 2^19 / 2^21 / 2^23 slots against the stream bandwidth and against the
measured random-read ceiling) and `index_lookup_flat`.  `cpu_baseline` times the CPU oracle on
one host core and on all of them.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun) runs N independent replicas, one per GPU: the path has no exchange step.
`--impl reference` times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
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
KERNELS_PER_STEP = 6    # head (hash+match+score+matched-block set), gather, scatter, hash tail, insert, evict

from bench_cases import CASES, cpu_model, measured_peak_hbm, ncu_traffic, routing_batch_times  # noqa: E402


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

        # routing outputs: two sets, used by alternate steps, so that the routing of the next
        # batch can run while the copies of this one still read this one's block list
        R, P = self.R, self.P
        self.d_pod_load = dev(w.pod_load)

        def routing_outputs():
            return dict(
                d_hashes=torch.empty(self.nb, dtype=torch.uint64, device="cuda"),
                d_match_len=torch.empty(R * P, dtype=torch.uint32, device="cuda"),
                d_any_len=torch.empty(R, dtype=torch.uint32, device="cuda"),
                d_block_ids=torch.empty(self.nb, dtype=torch.uint32, device="cuda"),
                d_best_pod=torch.empty(R, dtype=torch.int32, device="cuda"),
                d_best_score=torch.empty(R, dtype=torch.int64, device="cuda"),
                d_hashed=torch.empty(R, dtype=torch.uint32, device="cuda"),
                d_next_seed=torch.empty(R, dtype=torch.uint64, device="cuda"),
                d_scratch=torch.empty(aibx.route_collect_scratch_bytes(kv.num_blocks) // 4 + 1,
                                      dtype=torch.int32, device="cuda"),
                d_unique=torch.empty(self.nb, dtype=torch.uint32, device="cuda"),
                d_count=torch.empty(1, dtype=torch.uint32, device="cuda"))

        self._slots = [routing_outputs(), routing_outputs()]
        self._use(0)
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

    def _use(self, slot: int) -> None:
        """Make the routing outputs of one of the two sets the current ones (self.d_hashes ...)."""
        self._slot = slot
        for name, t in self._slots[slot].items():
            setattr(self, name, t)

    def release(self) -> None:
        """Give the device memory back (the index through its own destroy call)."""
        self.torch.cuda.synchronize()
        self.index.destroy()
        for name in [k for k, v in vars(self).items() if isinstance(v, self.torch.Tensor)]:
            delattr(self, name)

    # -- pieces of a step ------------------------------------------------------------------
    def routing_async(self) -> None:
        """Routing half of a step, enqueued only: the block count stays on the device.  Only
        the part of every chain that matching needs is hashed here (aibx_route_head_collect, which
        also leaves the set of matched blocks); the rest
        is hashed by hash_tail() off the critical path."""
        aibx = self.aibx
        aibx.route_head_collect(self.index, self.d_tokens, self.d_tok_off, self.d_blk_off, self.B, 0,
                                self.d_pod_load, self.w.ready_mask, None, 0, self.d_hashes,
                                self.d_match_len, self.d_any_len, self.d_block_ids, self.d_best_pod,
                                self.d_best_score, self.d_hashed, self.d_next_seed,
                                self.kv.num_blocks, self.d_scratch, self.d_unique, self.d_count)

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
        matched blocks goes from the routing kernel to the copies on the device; the tail of
        the hash chains and the index publish/expire batch (both independent of the copies) run
        beside them on a second stream; and as soon as the index is back in its start state the
        routing of the NEXT batch is enqueued on a third stream, beside this batch's copies
        (its outputs go to the other of two sets of buffers).  Every batch still goes through
        every stage in order; consecutive batches overlap as in any pipeline."""
        torch, aibx = self.torch, self.aibx
        main = torch.cuda.current_stream()
        if self.side is None:
            self.side = torch.cuda.Stream()
            self.route = torch.cuda.Stream()
            self.ev_routed = [torch.cuda.Event(), torch.cuda.Event()]
            self.ev_copied = [torch.cuda.Event(), torch.cuda.Event()]
            self.ev_index = torch.cuda.Event()
            self._routed_ahead = None
        if self._routed_ahead is not None:
            self._use(self._routed_ahead)                 # this batch was routed during the last step
        slot = self._slot
        if self._routed_ahead != slot:                    # first step: nothing was routed ahead
            self.route.wait_stream(main)
            with torch.cuda.stream(self.route):
                self.routing_async()
                self.ev_routed[slot].record(self.route)
        main.wait_event(self.ev_routed[slot])
        self.side.wait_event(self.ev_routed[slot])
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
        self.ev_copied[slot].record(main)
        main.wait_event(self.ev_index)                    # the index is back in its start state
        # the next batch's routing: needs the restored index and the other set of buffers, whose
        # last reader was the previous step's scatter
        nxt = 1 - slot
        self.route.wait_event(self.ev_index)
        self.route.wait_event(self.ev_copied[nxt])
        self._use(nxt)
        with torch.cuda.stream(self.route):
            self.routing_async()
            self.ev_routed[nxt].record(self.route)
        self._routed_ahead = nxt
        self._use(slot)                                   # results of the step just enqueued

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
            "route_head_collect": self.routing_async,
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
    traffic = ncu_traffic("cfg2_shape", launch_bytes)

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
    extras = {}
    count, R_job = job.count, job.R
    if rank == 0:
        # the other half of the metric: prefix match alone on the routing-heavy batch
        import workloads as W
        cfg3 = routing_batch_times(W.cfg3_routing)
    if rank == 0 and world == 1:
        # sibling records, each a measurement of its own on the now idle GPU: the cfg2 job's
        # pool and buffers are given back first so that the 97.7 and 109 GiB pools fit
        import gc

        import bench_cases as BC

        job.release()
        del job
        gc.collect()
        torch.cuda.empty_cache()
        extras["kv_cfg4"] = BC.measure_cfg4()
        extras["kv_cfg5"] = BC.measure_cfg5()
        extras["prefix_match_large_index"] = [BC.measure_match_large(c) for c in (19, 21, 23)]
        extras["index_lookup_flat"] = BC.measure_lookup_flat(with_library=False, reps=5)
    if dist is not None:
        dist.barrier()
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    ms_per_step = elapsed_ms / args.steps
    value = whole_job_value(step_bytes, world, ms_per_step)
    cpu = cpu_baseline(budget_s=6.0)
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": round(ms_per_step, 4),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "blocks_moved_per_step": count,
                   "bytes_moved_per_step": step_bytes, "parallelism": "replicas only" if world > 1 else "1 gpu",
                   "l2": "inputs larger than L2: 6.5 GB of KV traffic per step evicts it between steps",
                   "overlap": "hash chains past the first uncached block and index publish/expire on a second stream beside the copies; the next batch's routing on a third stream beside them once the index is restored (two sets of routing outputs); no host sync inside a step",
                   "kv_tuning": "bulk ring, loader + storer warp, 32 KiB x 3 stages, 1 CTA/SM",
                   "sibling_records": "kv_cfg4 (largest configuration), kv_cfg5, prefix_match_large_index, index_lookup_flat: measured at n_gpus = 1 only"},
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
        "match_requests_per_s": round(R_job / (stages["match_prefix"] * 1e-6), 1),
        "prefix_match_routing_heavy": {
            "workload": "cfg3: 4,096 requests, 527k blocks, index 2^20 entries / 2^21 slots, 64 pods",
            "match_requests_per_s": cfg3["match_requests_per_s"], "match_us": cfg3["match_us"],
            "match_requests_per_s_back_to_back": cfg3["match_requests_per_s_back_to_back"],
            "match_us_back_to_back": cfg3["match_us_back_to_back"],
            "match_us_in_a_graph": cfg3.get("match_us_in_a_graph"),
            "match_requests_per_s_in_a_graph": cfg3.get("match_requests_per_s_in_a_graph"),
            "hash_us": cfg3["hash_us"], "route_head_us": cfg3["route_head_us"],
            "decisions_per_s_via_route_head": round(cfg3["R"] / (cfg3["route_head_us"] * 1e-6), 0),
            "match_algorithmic_GBps": cfg3["match_algorithmic_GBps"]},
        "stage_us": stages,
    }
    line.update(extras)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# the CPU oracle: baseline leg and reference arm


class OracleSample:
    """The oracle on a bounded sample of the same workload: the whole routing batch and one
    publish/expire batch as they are, and gather+scatter of SAMPLE_BLOCKS blocks of the same
    shape out of a 512-block host pool.  The GPU step moves `count` blocks per routing batch, so
    a like-for-like step time is routing + index update + the copy time per block x count (the
    copies stream far more bytes than the caches hold, so their time is proportional)."""

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
        self.sample_bytes = 2 * 2 * self.SAMPLE_BLOCKS * kv.block_bytes
        st = W.Stream(s.seed, 21)
        nb = int(oracle.block_offsets(w.tok_off, s.block_tokens)[-1])
        self.new_keys = st.keys(nb)
        self.new_masks = np.left_shift(np.uint64(1), (np.arange(nb) % s.num_pods).astype(np.uint64))
        self.new_ids = st.randint(0, 4096, nb).astype(np.uint32)
        self.all_ones = np.full(nb, 0xFFFFFFFFFFFFFFFF, dtype=np.uint64)
        self.count = None                 # matched blocks of the batch, from the oracle itself
        self.threads = None

    # the three parts of a step, each returning its wall time
    def routing(self) -> float:
        o, w, s = self.oracle, self.w, self.w.spec
        t0 = time.perf_counter()
        h, bo = o.hash_blocks(w.tokens, w.tok_off, s.block_tokens, 0)
        ml, al, ids = self.ix.match_prefix(h, bo)
        o.route_score(ml, bo, w.pod_load, w.ready_mask, None)
        _, _, self.count = o.collect_blocks(ids, 4096)
        return time.perf_counter() - t0

    def copies(self) -> float:
        o = self.oracle
        t0 = time.perf_counter()
        o.kv_gather(self.pool, self.lay, self.ids, self.buf)
        o.kv_scatter(self.pool, self.lay, self.ids, self.buf)
        return time.perf_counter() - t0

    def index_update(self) -> float:
        t0 = time.perf_counter()
        self.ix.insert(self.new_keys, self.new_masks, self.new_ids)
        self.ix.evict(self.new_keys, self.all_ones)
        return time.perf_counter() - t0

    # the same oracle functions called from T threads over disjoint request / id ranges (the
    # index is only read; the calls are ctypes calls, which release the interpreter lock)
    def use_threads(self, T: int):
        from concurrent.futures import ThreadPoolExecutor

        o, w, s = self.oracle, self.w, self.w.spec
        self.T = T
        self.threads = ThreadPoolExecutor(max_workers=T)
        R = len(w.tok_off) - 1
        cuts = [R * i // T for i in range(T + 1)]
        self.req_parts = []
        for a, b in zip(cuts[:-1], cuts[1:]):
            if b > a:
                toks = np.ascontiguousarray(w.tokens[w.tok_off[a]:w.tok_off[b]])
                self.req_parts.append((toks, np.ascontiguousarray(w.tok_off[a:b + 1] - w.tok_off[a])))
        cuts = [self.SAMPLE_BLOCKS * i // T for i in range(T + 1)]
        self.id_parts = [(a, b) for a, b in zip(cuts[:-1], cuts[1:]) if b > a]

    def routing_threads(self) -> float:
        o, w, s = self.oracle, self.w, self.w.spec

        def part(p):
            h, bo = o.hash_blocks(p[0], p[1], s.block_tokens, 0)
            ml, al, ids = self.ix.match_prefix(h, bo)
            o.route_score(ml, bo, w.pod_load, w.ready_mask, None)
            return ids

        t0 = time.perf_counter()
        ids = np.concatenate(list(self.threads.map(part, self.req_parts)))
        o.collect_blocks(ids, 4096)
        return time.perf_counter() - t0

    def copies_threads(self) -> float:
        o, bb = self.oracle, self.kv.block_bytes
        t0 = time.perf_counter()
        list(self.threads.map(lambda ab: o.kv_gather(self.pool, self.lay, self.ids[ab[0]:ab[1]],
                                                     self.buf[ab[0] * bb:ab[1] * bb]), self.id_parts))
        list(self.threads.map(lambda ab: o.kv_scatter(self.pool, self.lay, self.ids[ab[0]:ab[1]],
                                                      self.buf[ab[0] * bb:ab[1] * bb]), self.id_parts))
        return time.perf_counter() - t0

    def step(self, threaded=False):
        """One sample step; returns (routing s, copies s, index update s)."""
        if threaded:
            return self.routing_threads(), self.copies_threads(), self.index_update()
        return self.routing(), self.copies(), self.index_update()

    def like_for_like(self, t_route, t_copy, t_update):
        """GB/s of a full step (count blocks gathered and scattered) at the sampled rates."""
        full_bytes = 2 * 2 * self.count * self.kv.block_bytes
        est = t_route + t_update + t_copy * self.count / self.SAMPLE_BLOCKS
        return full_bytes / est / 1e9

    describe = ("per step: the whole routing batch (64 requests, 200k-entry index) and one "
                "publish/expire batch as they are, gather and scatter of 128 of the 2 MiB blocks "
                "out of a 512-block host pool; value = bytes of a full step (all matched blocks) "
                "over routing + index update + copy time scaled from 128 blocks to the full count")


def _oracle_leg(sample, budget_s, threaded):
    sample.step(threaded)
    tr = tc = tu = 0.0
    n, t0 = 0, time.perf_counter()
    while True:
        a, b, c = sample.step(threaded)
        tr, tc, tu = tr + a, tc + b, tu + c
        n += 1
        if time.perf_counter() - t0 >= budget_s or n >= 2000:
            break
    return {"value": round(sample.like_for_like(tr / n, tc / n, tu / n), 3),
            "kv_copies_alone_GBps": round(sample.sample_bytes * n / tc / 1e9, 3),
            "routing_ms": round(tr / n * 1e3, 3), "index_update_ms": round(tu / n * 1e3, 3),
            "steps": n, "seconds": round(time.perf_counter() - t0, 2)}


def cpu_baseline(budget_s: float):
    sample = OracleSample()
    one = _oracle_leg(sample, budget_s, False)
    T = len(os.sched_getaffinity(0))
    sample.use_threads(T)
    many = _oracle_leg(sample, budget_s, True)
    sample.threads.shutdown()
    out = {"value": one["value"], "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": OracleSample.describe, "cpu": cpu_model(), "cores_available": T}
    out.update({k: one[k] for k in ("kv_copies_alone_GBps", "routing_ms", "index_update_ms",
                                    "steps", "seconds")})
    many.update({"unit": UNIT, "cores": T,
                 "how": "the same oracle functions called from one thread per available core over "
                        "disjoint request ranges (hash, match, score) and id ranges (gather, "
                        "scatter); the index update stays on one thread"})
    out["all_cores"] = many
    return out


def run_reference(args):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    sample = OracleSample()
    for _ in range(max(args.warmup, 1)):
        sample.step()
    tr = tc = tu = 0.0
    t0 = time.perf_counter()
    for _ in range(args.steps):
        a, b, c = sample.step()
        tr, tc, tu = tr + a, tc + b, tu + c
    dt = time.perf_counter() - t0
    n = args.steps
    value = round(sample.like_for_like(tr / n, tc / n, tu / n), 3)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": args.gpus, "steps": args.steps, "warmup": max(args.warmup, 1),
        "ms_per_step": round(dt / args.steps * 1e3, 3), "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u8", "data": "synthetic",
        "config": {"workload": WORKLOAD},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": OracleSample.describe, "cpu": cpu_model(),
                         "kv_copies_alone_GBps": round(sample.sample_bytes * n / tc / 1e9, 3),
                         "routing_ms": round(tr / n * 1e3, 3),
                         "index_update_ms": round(tu / n * 1e3, 3)},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", default=None, choices=sorted(CASES),
                    help="run one small single-kernel case instead of the bench step")
    ap.add_argument("--log2cap", type=int, default=23)
    ap.add_argument("--pods", type=int, default=32, help="match_large: pods of the index (up to 32: "
                    "16-byte entries, beyond: 32-byte entries)")
    ap.add_argument("--ws-mib", type=int, default=0, help="random_reads: one working-set size")
    ap.add_argument("--read-bytes", type=int, default=0, choices=[0, 32, 64, 128],
                    help="random_reads: one read size")
    ap.add_argument("--shape", default="cfg2", choices=["cfg2", "cfg4", "cfg5"],
                    help="block shape of the kv_small case")
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
