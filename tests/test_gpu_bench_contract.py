"""The benchmark prints one JSON line with the keys the measurement contract asks for (short run on the GPU)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "8", "--warmup", "3", "--no-extras"],
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "e2e", "gpu_launches", "clocks", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["value"] > 0 and d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 8 and d["vs_baseline"] is None
    assert d["config"]["workload"].startswith("c2_") and "l2" in d["config"]
    assert d["matches_oracle"] is True and d["e2e"]["matches_oracle"] is True
    assert d["e2e"]["h2d_bytes_per_step"] == 8 * 26214400 and d["e2e"]["value"] < d["value"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and r["traffic"] > 0
    # per step: seven SUM launches, and the empty ordering kernels of the two graphs: one in front of each graph's first
    # copies, one behind each of the seven copy stages of the ring all-gather
    assert d["gpu_launches"] == (7 + 2 + 7) * 8
    ds = d["direct_schedule"]
    assert ds["matches_oracle"] is True and ds["sum_launches_per_step"] == 1 and ds["value"] > d["value"]
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0
