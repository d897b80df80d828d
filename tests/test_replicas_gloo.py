"""The N > 1 plumbing of the benchmark (replicas, barrier, max/sum over ranks) on CPU with gloo, world size 2."""
import os
import socket
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import json, os, sys
    sys.path.insert(0, %r)
    from paper_2609_34334_b200 import replicas
    w = replicas.init_from_env(backend="gloo")
    assert w.distributed and w.size == 2 and w.backend == "gloo"
    replicas.barrier(w)
    t = 1.0 + w.rank * 0.5                      # rank 1 is the slow replica
    slowest = replicas.max_over_ranks(w, t)
    units = replicas.sum_over_ranks(w, 10.0)    # every replica processed 10 units
    thr = replicas.whole_job_throughput(w, 10.0, t)
    replicas.barrier(w)
    print(json.dumps({"rank": w.rank, "slowest": slowest, "units": units, "thr": thr}), flush=True)
    replicas.shutdown(w)
""") % ROOT


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_replicas_aggregate_with_gloo(tmp_path):
    port = _free_port()
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), CUDA_VISIBLE_DEVICES="")
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(out.strip().splitlines()[-1])
    import json
    for line in outs:
        d = json.loads(line)
        assert d["slowest"] == 1.5          # max over ranks
        assert d["units"] == 20.0           # sum over ranks
        assert abs(d["thr"] - 20.0 / 1.5) < 1e-12


def test_single_process_is_identity():
    from paper_2609_34334_b200 import replicas
    env_backup = {k: os.environ.pop(k, None) for k in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    try:
        w = replicas.init_from_env()
        assert not w.distributed and w.size == 1
        assert replicas.max_over_ranks(w, 2.5) == 2.5 and replicas.sum_over_ranks(w, 4.0) == 4.0
        assert replicas.whole_job_throughput(w, 8.0, 2.0) == 4.0
        replicas.barrier(w)
    finally:
        for k, v in env_backup.items():
            if v is not None:
                os.environ[k] = v


def test_reference_arm_prints_one_json_line():
    """`bench.py --impl reference` times the oracle on the host and needs no GPU."""
    import json
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "2", "--warmup", "1"],
                         capture_output=True, text=True, timeout=600)
    assert out.returncode == 0, out.stderr[-2000:]
    d = json.loads(out.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["value"] > 0 and d["unit"] == "GB/s"
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["value"] == d["value"]
    # other ranks of a multi-process launch print nothing and exit 0
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0", "--gpus", "2"],
                         capture_output=True, text=True, timeout=600, env=env)
    assert out.returncode == 0 and out.stdout.strip() == ""
