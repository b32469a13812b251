"""`bench.py` on a small case: the JSON line carries every key of the contract and sane values."""
import json
import os
import subprocess
import sys

import pytest

from gpu_util import require_gpu

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_on_a_small_case():
    require_gpu()
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "4", "--warmup", "3",
                          "--blocks", "256", "--pool-blocks", "4096", "--cpu-seconds", "1", "--hash-prompts", "64"],
                         capture_output=True, text=True, timeout=900, cwd=ROOT)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better",
                "scaling", "vs_baseline", "dtype", "data", "config", "clocks", "e2e", "gpu_launches",
                "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["metric"] == "kv_store_load_gbps" and d["unit"] == "GB/s" and d["n_gpus"] == 1
    assert d["steps"] == 4 and d["warmup"] == 3 and d["scaling"] == "weak" and d["dtype"] == "u8"
    assert d["config"]["workload"].startswith("c1_store_load_microbench") and d["config"]["self_check"] is True
    assert d["value"] > 0 and d["gpu_launches"] > 0
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and r["peak"] > 0
    assert abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and r["kernel"] == "copy_blocks_bulk_kernel"
    e = d["e2e"]
    assert e["value"] > 0 and e["h2d_bytes_per_step"] > 0 and e["d2h_bytes_per_step"] > 0
    assert len(e["passes_gbps"]) == 2 and e["value"] == max(e["passes_gbps"])
    # every host-link strategy and both device copy paths side by side, and the microbench's curve
    assert set(e["by_strategy"]) == {"staged", "zero_copy", "copy_engine"}
    assert all(v["value"] > 0 for v in e["by_strategy"].values())
    assert set(r["by_copy_path"]) == {"bulk", "vector"} and all(v["achieved"] > 0 for v in r["by_copy_path"].values())
    assert r["tp8_rank_shape"]["piece_bytes"] == 4096 and r["tp8_rank_shape"]["achieved"] > 0
    rows = e["curve"]["rows"]
    assert {(x["tier"], x["op"], x["ids"], x["mask"]) for x in rows} >= {
        ("host", "store", "random", "bernoulli"), ("host", "load", "contiguous", "ones"), ("hbm", "store", "random", "ones")}
    assert {x["blocks"] for x in rows} == {1, 16, 256} and all(x["gbps"] > 0 for x in rows)
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["value"] > 0 and c["cores"] == 1
    assert set(d["clocks"]) >= {"sm_mhz", "sm_max_mhz", "reasons"}
