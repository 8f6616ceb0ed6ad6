"""The multi-rank side of bench.py (replicas only): two gloo ranks on CPU agree on the max of
their timed intervals and rank 0's whole-job value sums both replicas' bytes."""
import os
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist

    import bench

    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 2.0 + rank          # rank 1 is the slow one
    slowest = bench.max_over_ranks(mine, dist, "cpu")
    out.put((rank, slowest, bench.whole_job_value(10**9, world, slowest)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_interval():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, slowest, value in got:
        assert slowest == 3.0
        assert abs(value - 2 * 1e9 / 3e-3 / 1e9) < 1e-9


def test_single_rank_passthrough():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.max_over_ranks(1.25, None, "cpu") == 1.25
    assert bench.whole_job_value(6 * 10**9, 1, 2.0) == 3000.0
