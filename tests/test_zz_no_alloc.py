"""The allocation-free variant of collect_blocks (GPU).

Some users of this library run where device memory cannot be requested: inside an inference
engine that has already handed almost all of HBM to its KV pool, or in a callback where a
cudaMalloc (which may fail, and synchronises the device) is not acceptable.  For them
aibx_collect_blocks_static keeps its scratch bitmap in a fixed array inside the library.  This
file checks, through the C ABI, that it returns exactly what aibx_collect_blocks returns with
caller-provided scratch - on two calls in a row, because the array is shared between calls and
still holds the first call's marks when the second one starts - that both calls also agree with
the CPU oracle's own definition of the matched-block set, that the device's free memory is the
same before and after a call (the point of the entry point), and that it refuses pools larger
than the array.  Collected last so that a failure here cannot hide another test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2504_03648_b200 import binding as aibx

pytestmark = pytest.mark.gpu
NO_BLOCK = 0xFFFFFFFF


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _both(ids, num_blocks):
    n = len(ids)
    d_ids = _dev(ids)
    scratch = torch.full((aibx.collect_scratch_bytes(num_blocks) // 4 + 1,), -1, dtype=torch.int32,
                         device="cuda")
    ref_u = torch.empty(n, dtype=torch.uint32, device="cuda")
    ref_c = torch.empty(1, dtype=torch.uint32, device="cuda")
    aibx.collect_blocks(d_ids, num_blocks, scratch, ref_u, ref_c)
    ref_status = aibx.status_fetch()
    got_u = torch.empty(n, dtype=torch.uint32, device="cuda")
    got_c = torch.empty(1, dtype=torch.uint32, device="cuda")
    aibx.collect_blocks_static(d_ids, num_blocks, got_u, got_c)
    got_status = aibx.status_fetch()
    return (ref_u.cpu().numpy(), int(ref_c.cpu()[0]), ref_status), \
           (got_u.cpu().numpy(), int(got_c.cpu()[0]), got_status)


def test_static_scratch_matches_caller_scratch_twice_in_a_row():
    rng = np.random.default_rng(2024)
    # first call: a large pool, dense marks all over the array
    big = aibx.collect_static_max_blocks()
    ids1 = rng.integers(0, big, 300000).astype(np.uint32)
    ids1[::11] = NO_BLOCK
    ref, got = _both(ids1, big)
    assert got[1] == ref[1] > 0 and np.array_equal(got[0], ref[0]) and got[2] == ref[2] == (0, 0)
    rc, want_u, want_c = oracle.collect_blocks(ids1, big)              # independent of both GPU paths
    assert rc == oracle.OK and got[1] == want_c and np.array_equal(got[0], want_u)
    # second call right after it: a small pool whose ids the first call also marked, plus ids
    # that are out of range for this pool (they must be dropped and counted, as in the original)
    ids2 = rng.integers(0, 5000, 4000).astype(np.uint32)
    ids2[::7] = NO_BLOCK
    ids2[5] = 4096
    ids2[6] = 70000
    ref, got = _both(ids2, 4096)
    assert got[1] == ref[1] and np.array_equal(got[0], ref[0])
    assert got[2] == ref[2] and got[2][0] == aibx.ERR_RANGE
    want = sorted(set(int(x) for x in ids2 if x < 4096))
    assert got[0][: got[1]].tolist() == want and (got[0][got[1]:] == NO_BLOCK).all()
    rc, want_u, want_c = oracle.collect_blocks(ids2, 4096)
    assert rc == oracle.ERR_RANGE and got[1] == want_c and np.array_equal(got[0], want_u)


def test_static_variant_takes_no_device_memory():
    """Inputs and outputs are made first; across the call itself (large pool, so the built-in
    array is really used) neither the driver's free memory nor torch's own counters move."""
    rng = np.random.default_rng(7)
    big = aibx.collect_static_max_blocks()
    d_ids = _dev(rng.integers(0, big, 200000).astype(np.uint32))
    out = torch.empty(200000, dtype=torch.uint32, device="cuda")
    cnt = torch.empty(1, dtype=torch.uint32, device="cuda")
    aibx.collect_blocks_static(d_ids, big, out, cnt)                   # first call: resolves the array
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        aibx.collect_blocks_static(d_ids, big, out, cnt)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
    assert int(cnt.cpu()[0]) == len(np.unique(d_ids.cpu().numpy())) and aibx.status_fetch() == (0, 0)


def test_static_scratch_rejects_pools_beyond_its_array():
    ids = _dev(np.arange(8, dtype=np.uint32))
    out = torch.full((8,), 7, dtype=torch.int32, device="cuda").view(torch.uint32)
    cnt = torch.full((1,), 7, dtype=torch.int32, device="cuda").view(torch.uint32)
    with pytest.raises(aibx.AibxError) as e:
        aibx.collect_blocks_static(ids, aibx.collect_static_max_blocks() + 1, out, cnt)
    assert e.value.code == aibx.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert int(cnt.cpu()[0]) == 7 and (out.cpu().numpy() == 7).all()       # nothing was enqueued
    # empty input is fine and reports zero blocks
    aibx.collect_blocks_static(torch.empty(0, dtype=torch.uint32, device="cuda"), 64,
                               torch.empty(0, dtype=torch.uint32, device="cuda"), cnt)
    assert int(cnt.cpu()[0]) == 0 and aibx.status_fetch() == (0, 0)
