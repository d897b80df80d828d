"""The benchmark prints one JSON line with the keys the measurement contract asks for (short run on the GPU)."""
import json
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_bench_line_has_the_contract_keys():
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "8", "--warmup", "3", "--no-extras", "--no-large"],
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0, out.stderr[-3000:]
    lines = [l for l in out.stdout.strip().splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    for key in ("metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
                "dtype", "data", "config", "e2e", "gpu_launches", "clocks", "roofline", "cpu_baseline"):
        assert key in d, key
    assert d["value"] > 0 and d["unit"] == "GB/s" and d["n_gpus"] == 1 and d["steps"] == 8 and d["vs_baseline"] is None
    # the workload is the largest single-GPU configuration: the gradient stream in 40 MiB buckets
    assert d["config"]["workload"].startswith("c4_") and "l2" in d["config"] and d["config"]["bytes_per_rank"] == 40 << 20
    assert d["matches_oracle"] is True and d["e2e"]["matches_oracle"] is True and d["last_bucket"]["matches_oracle"] is True
    assert d["e2e"]["h2d_bytes_per_step"] == 8 * (40 << 20) and d["e2e"]["value"] < d["value"]
    r = d["roofline"]
    assert r["bound"] == "hbm" and r["unit"] == "GB/s" and abs(r["frac"] - r["achieved"] / r["peak"]) < 1e-9 and r["traffic"] > 0
    # per step of the default (stage-decomposed) schedule: one chain sum launch per piece (the copy route cuts a 5 MiB ring
    # chunk into 4 pieces so that copies and sums overlap) and the empty ordering kernels of the graphs
    assert d["sms_used"]["sum_launches_per_step"] == d["config"]["pieces_per_chunk"] == 4 and d["sms_used"]["sum_ctas"] == 8
    assert d["gpu_launches"] == (4 + d["sms_used"]["ordering_kernels_per_step"]) * 8
    rs = d["ring_schedule"]
    assert rs["matches_oracle"] is True and rs["sum_launches_per_step"] == 7 and rs["value"] < d["value"]
    assert rs["roofline"]["kernel"].startswith("sum2_kernel")
    c = d["cpu_baseline"]
    assert c["kind"] == "oracle" and c["cores"] >= 1 and c["value"] > 0


def test_large_message_and_gemm_rows_carry_oracle_flags():
    """The two evidence blocks of the full run, on their own sizes: every row says whether its output matched the oracle."""
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--steps", "5", "--warmup", "3", "--no-extras"],
                         capture_output=True, text=True, timeout=1500)
    assert out.returncode == 0, out.stderr[-3000:]
    d = json.loads([l for l in out.stdout.strip().splitlines() if l.startswith("{")][0])
    lm = d["large_messages"]
    assert lm["all_match_oracle"] is True
    seen = {(r["op"], r["MiB_per_rank"], r["config"]) for r in lm["rows"] if "config" in r}
    for mib in (64, 256, 1024):
        for op in ("allreduce", "reduce_scatter", "allgather", "sendrecv"):
            assert (op, mib, "CE_sum8") in seen and (op, mib, "SM_copy148_sum148") in seen
    gm = d["gemm_loss_matched"]
    names = [r["config"] for r in gm["rows"]]
    assert "CE_sum8" in names and all("SM_copy%d_sum8" % b in names for b in (8, 16, 32, 64, 148))
    assert all(r["matches_oracle"] is True and -0.05 < r["gemm_loss"] < 1.0 for r in gm["rows"])      # a loss of zero is measured within ~1 %
