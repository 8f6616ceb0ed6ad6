"""The JSON line bench.py prints: one line, the keys the measurement contract names, and
values that hang together (whole-job value against ms_per_step and the bytes moved, roofline
fraction against achieved and peak, end-to-end bytes counted, launches counted)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_contract():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "4", "--warmup", "3"],
                       cwd=ROOT, stdout=subprocess.PIPE, stderr=subprocess.PIPE, timeout=600)
    assert r.returncode == 0, r.stderr.decode()[-2000:]
    lines = [ln for ln in r.stdout.decode().splitlines() if ln.strip()]
    assert len(lines) == 1, lines
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step",
                "higher_is_better", "scaling", "vs_baseline", "dtype", "data", "config", "clocks",
                "e2e", "gpu_launches", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["n_gpus"] == 1 and d["steps"] == 4 and d["warmup"] >= 3 and d["higher_is_better"] is True
    assert d["scaling"] == "weak" and d["vs_baseline"] is None and d["dtype"] == "u8"
    assert d["data"] == "synthetic" and "workload" in d["config"] and "model" not in d["config"]
    # value = bytes moved per step / time per step
    moved = d["config"]["bytes_moved_per_step"]
    assert abs(d["value"] - moved / (d["ms_per_step"] * 1e-3) / 1e9) < 0.01 * d["value"]
    rf = d["roofline"]
    assert rf["bound"] == "hbm" and rf["unit"] == "GB/s" and rf["peak"] > 1000
    assert abs(rf["frac"] - rf["achieved"] / rf["peak"]) < 1e-3
    assert 0.3 < rf["frac"] < 1.2                        # a copy kernel cannot be far above a plain copy
    assert rf["traffic"] is None or 0.8 < rf["traffic"] / rf["algorithmic_bytes_per_launch"] < 1.3
    assert d["value"] < rf["achieved"]                    # the whole step cannot beat its copy kernel
    e = d["e2e"]
    assert e["unit"] == d["unit"] and 0 < e["value"] < d["value"]
    assert e["h2d_bytes_per_step"] > moved // 4 and e["d2h_bytes_per_step"] > moved // 4
    assert d["gpu_launches"] == 6 * d["steps"]
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] == 1 and c["value"] > 0 and c["unit"] == d["unit"]
    assert c["cpu"] and c["all_cores"]["cores"] == c["cores_available"] >= 1
    assert c["all_cores"]["value"] > 0 and c["all_cores"]["unit"] == d["unit"]
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"} and d["clocks"]["sm_max_mhz"] > 0
    # sibling records: the largest KV configurations, each with a roofline of its own
    for key, kernel_launches in (("kv_cfg4", 100), ("kv_cfg5", 64)):
        k = d[key]
        assert k["status"] == [0, 0] and "workload" in k
        assert k["pool_blocks_effective"] <= k["pool_blocks_configured"]
        r = k["roofline"]
        assert r["bound"] == "hbm" and r["launches_timed"] == kernel_launches
        assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-3 and 0.3 < r["frac"] < 1.2
        assert abs(r["achieved"] - r["algorithmic_bytes_per_launch"] / (r["avg_launch_ms"] * 1e-3) / 1e9) \
            < 0.01 * r["achieved"]
    big = d["prefix_match_large_index"]
    assert [b["index_slots"] for b in big] == [1 << 19, 1 << 21, 1 << 23]
    for b in big:
        row = b["results"][-1]
        assert row["lookups"] == row["R"] * 64 and 0 < row["frac"] < 1.2
        assert b["random_32B_read_ceiling_Greads_per_s"] > 1
        assert 0 < row["frac_of_random_read_ceiling"] < 1.5
    assert len(d["index_lookup_flat"]["results"]) == 4
