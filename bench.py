#!/usr/bin/env python
"""Benchmark of the ring hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras]

Workload (N = 1): the data-parallel gradient bucket of the second benchmark configuration:
reduce-scatter then all-gather over R = 8 logical ranks, 25 MiB of bf16 per rank (13,107,200
elements, normal(0, 1e-3), seed 1), fp32 accumulation, 8 ring chunks.  One step = one pass of the
whole path over one bucket: plan lookup, fork/join ordering, 7 x 8 reduce-scatter moves, 7 batched
SUM steps, 7 x 8 all-gather moves.  Four bucket sets (1.6 GiB) are used in rotation so that no step
finds its inputs in the 126 MB L2.

Reported value: all-reduce bus bandwidth, S * 2(R-1)/R / t_step in GB/s (nccl-tests convention), for the
copy-route path with at most 8 CTAs for sums; with N GPUs, N independent replicas run and the value
is the sum of their units over the slowest replica's time.  One JSON line on stdout (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "allreduce bus GB/s vs 8 TB/s HBM roofline; SMs used; co-run GEMM TFLOP/s loss"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
FALLBACK_BF16_TFLOPS = 1590.0
N_BUCKET_SETS = 4

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one SUM launch, from the ncu capture summarised in
# profiles/sum2_kernel_bf16_8cta_200MiB.md: 573.88 MB of traffic for 629.15 MB of algorithmic bytes (operands of
# 200 MiB, larger than L2; part of the output is still in L2 when the kernel ends).  Traffic grows in proportion to
# the bytes a launch processes, so it is scaled to this workload's launch (8 segments x 3,276,800 B x 3).
NCU_TRAFFIC_PER_ALGORITHMIC_BYTE = 573.88 / 629.15
SM_PORT_GBPS = 123.0   # measured mixed 2:1 read/write ceiling of one SM's memory port (bulk loads + bulk stores)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the variant table, GEMM probe and p2p lines")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d.get("bf16_tflops", FALLBACK_BF16_TFLOPS)),
                "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 1400.0)), "source": "measured"}
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": FALLBACK_BF16_TFLOPS, "bf16_tflops_sustained": 1400.0,
                "source": "fallback"}


# ---------------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML (read only) while a timed region runs."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, index: int, period_s: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml

            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def _reasons(self):
        nv = self.nv
        for fn in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            if hasattr(nv, fn):
                try:
                    return int(getattr(nv, fn)(self.h))
                except Exception:
                    continue
        return 0

    def run(self):
        if not self.ok:
            return
        while not self._halt.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                mask = self._reasons()
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                self.power.append(self.nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=1.0)
        s = sorted(self.samples)
        med = s[len(s) // 2] if s else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(s),
                "power_w_max": max(self.power) if self.power else None}


# ---------------------------------------------------------------------------------------------------
def bus_factor(R):
    return 2.0 * (R - 1) / R


def algorithmic_hbm_bytes_allreduce(S, R):
    """Rank-local ring on one device: every wire byte is read+written by a MOVE in both phases (2+2) and read
    twice + written once by a SUM (3): 7 * S * (R-1)."""
    return 7.0 * S * (R - 1)


def reference_arm(args, world):
    """Times the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if world.rank != 0:
        return
    from oracle import ring
    from paper_2609_34334_b200 import workloads as W

    c = W.C2_DP_BUCKET
    R, dtype = c.R, c.dtype
    threads = ring.max_threads()
    n = c.count
    xs = W.rank_inputs(c.dist, c.seed, R, n, dtype, c.sigma)
    t0 = time.perf_counter()
    ring.ring_allreduce(xs, threads=threads)
    t_one = time.perf_counter() - t0
    budget = 150.0
    frac = 1.0
    if t_one * (args.steps + args.warmup) > budget:       # bounded sample: a prefix of every rank's bucket
        frac = budget / (t_one * (args.steps + args.warmup))
        n = max(R * 1024, int(n * frac) // (R * 8) * (R * 8))
        xs = [x[:n].copy() for x in xs]
    for _ in range(args.warmup):
        ring.ring_allreduce(xs, threads=threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ring.ring_allreduce(xs, threads=threads)
    dt = (time.perf_counter() - t0) / args.steps
    S = n * W.elem_size(dtype)
    val = S * bus_factor(R) / dt / 1e9
    sample = "all %d elements per rank" % n if frac == 1.0 else "first %d of %d elements per rank (%.1f%%)" % (n, c.count, 100.0 * n / c.count)
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": c.name, "R": R, "elements_per_rank": n, "step": "ring all-reduce by the CPU oracle"},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------------
def main():
    args = parse_args()
    from paper_2609_34334_b200 import replicas

    if args.impl == "reference":
        world = replicas.World(rank=int(os.environ.get("RANK", "0")), size=int(os.environ.get("WORLD_SIZE", "1")))
        reference_arm(args, world)
        return 0

    import numpy as np
    import torch

    from paper_2609_34334_b200 import binding as hb
    from paper_2609_34334_b200 import diag as hd
    from paper_2609_34334_b200 import workloads as W

    if not torch.cuda.is_available():
        sys.stderr.write("bench.py: no CUDA device; the hot path has no CPU fallback\n")
        return 2
    world = replicas.init_from_env()
    dev = world.local_rank if world.distributed else 0
    torch.cuda.set_device(dev)
    hb.lib()
    peaks = measured_peaks()
    steps, warmup = max(1, args.steps), max(3, args.warmup)

    c = W.C2_DP_BUCKET
    R, n, dtype, e = c.R, c.count, c.dtype, 2
    S = n * e
    count = n // R
    stream = torch.cuda.Stream()

    # ---- inputs: bucket set 0 is the seeded workload; sets 1.. are the same values rotated (only timing uses them)
    xs = W.rank_inputs(c.dist, c.seed, R, n, dtype, c.sigma)
    send_sets, recv_sets = [], []
    for b in range(N_BUCKET_SETS):
        if b == 0:
            send = [torch.from_numpy(x.view(np.int16)).to("cuda", non_blocking=False) for x in xs]
        else:
            send = [torch.roll(t, 4099 * b) for t in send_sets[0]]
        send_sets.append(send)
        recv_sets.append([torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)])
    scratch = torch.empty(hb.scratch_bytes_direct(R, n, dtype) + 256, dtype=torch.uint8, device="cuda")   # covers every variant
    spad = (-scratch.data_ptr()) % 256

    def new_comm(path=hb.PATH_CE, **params):
        cm = hb.Comm(R, dev)
        cm.set_scratch(scratch.data_ptr() + spad, scratch.numel() - 256)
        cm.set_path(path)
        for k, v in params.items():
            cm.set_param(k, v)
        return cm

    def step(cm, b, st):
        """reduce-scatter into chunk r of recv[r], then all-gather in place: the two calls of the workload."""
        recv = recv_sets[b]
        rs_out = [recv[r].data_ptr() + r * count * e for r in range(R)]
        cm.reduce_scatter(send_sets[b], rs_out, count, dtype, st)
        cm.allgather(rs_out, recv, count, dtype, st)

    def timed(cm, k_steps, k_warm, fn=step, sampler=None):
        # warm-up touches every bucket set at least once, so every cached graph exists before the timed region
        for k in range(max(k_warm, N_BUCKET_SETS)):
            fn(cm, k % N_BUCKET_SETS, stream)
        stream.synchronize()
        replicas.barrier(world)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if sampler:
            sampler.start()
        e0.record(stream)
        for k in range(k_steps):
            fn(cm, k % N_BUCKET_SETS, stream)
        e1.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        clocks = sampler.stop() if sampler else None
        replicas.barrier(world)
        return e0.elapsed_time(e1) / 1e3 / k_steps, clocks

    # ---- headline: copy-route path, <= 8 CTAs for sums
    comm = new_comm(hb.PATH_CE, sum_ctas=8)
    sampler = ClockSampler(dev)
    t_step, clocks = timed(comm, steps, warmup, sampler=sampler)
    st = comm.last_stats()
    # spread: ten more windows of steps/10 steps each (median and best), same launch configuration
    win = []
    for _ in range(10):
        tw, _ = timed(comm, max(5, steps // 10), 0)
        win.append(tw * 1e3)
    win.sort()
    windows = {"n": 10, "steps_each": max(5, steps // 10), "median_ms_per_step": win[len(win) // 2], "best_ms_per_step": win[0],
               "worst_ms_per_step": win[-1]}
    # launches of our kernels per step: the SUM launches of the reduce-scatter, plus the empty one-warp kernels that order
    # copy nodes inside the two graphs (in front of each graph's first copies and behind each all-gather stage)
    rs_out0 = [recv_sets[0][r].data_ptr() + r * count * e for r in range(R)]
    comm.allgather(rs_out0, recv_sets[0], count, dtype, stream)
    stream.synchronize()
    ag_stats = comm.last_stats()
    comm.reduce_scatter(send_sets[0], rs_out0, count, dtype, stream)
    stream.synchronize()
    rs_stats = comm.last_stats()
    launches_per_step = (rs_stats["n_sum_launches"] + rs_stats["n_move_launches"] + rs_stats["n_order_launches"] +
                         ag_stats["n_sum_launches"] + ag_stats["n_move_launches"] + ag_stats["n_order_launches"])

    # results of the timed configuration on bucket set 0 (ranks 0 and 5, full vectors), kept for the comparison with the
    # oracle, which happens where the oracle runs: in the CPU-baseline leg below
    parity = None
    step(comm, 0, stream)
    stream.synchronize()
    got_parity = {r: recv_sets[0][r].cpu().numpy().view(np.uint16).copy() for r in (0, 5)}

    t_slowest = replicas.max_over_ranks(world, t_step)
    units = replicas.sum_over_ranks(world, S * bus_factor(R))
    value = units / t_slowest / 1e9

    # ---- the same workload, constraints and bits as the stage-decomposed ("direct") schedule: the reduce-scatter as R-1
    # independent permutation stages into R-1 inbox slots and one chain sum per rank in the ring's order, the all-gather as
    # R-1 independent stages; copy route, 8 SUM CTAs.  Timed like the headline (same steps, same bucket sets).
    comm_d = new_comm(hb.PATH_CE, sum_ctas=8, rs_direct=1, ag_direct=1)
    t_direct, _ = timed(comm_d, steps, warmup)
    step(comm_d, 0, stream)
    stream.synchronize()
    got_direct = {r: recv_sets[0][r].cpu().numpy().view(np.uint16).copy() for r in (0, 5)}
    comm_d.reduce_scatter(send_sets[0], rs_out0, count, dtype, stream)
    stream.synchronize()
    direct_sum_launches = int(comm_d.last_stats()["n_sum_launches"])
    comm_d.destroy()
    t_direct_slowest = replicas.max_over_ranks(world, t_direct)
    direct_line = {"schedule": "rs_direct + ag_direct (rank local; the ring's order of addition and rounding)", "path": "CE (driver copy route)",
                   "sum_ctas": 8, "value": units / t_direct_slowest / 1e9, "unit": "GB/s", "ms_per_step": t_direct_slowest * 1e3,
                   "sum_launches_per_step": direct_sum_launches,
                   "algorithmic_bytes_per_step": 2.0 * S * (R - 1) + 1.0 * S * (R + 1) + 2.0 * S * (R - 1), "matches_oracle": None}

    # ---- end to end: host buffers through hoccl_host_allreduce (H2D and D2H inside the timed region)
    per = (S + 255) // 256 * 256
    staging = torch.empty(2 * R * per + 256, dtype=torch.uint8, device="cuda")
    gpad = (-staging.data_ptr()) % 256
    comm.set_staging(staging.data_ptr() + gpad, 2 * R * per)
    h_send = [torch.from_numpy(x.view(np.int16)).pin_memory() for x in xs]
    h_recv = [torch.zeros(n, dtype=torch.int16).pin_memory() for _ in range(R)]

    def e2e_step(cm, b, st):
        cm.host_allreduce(h_send, h_recv, n, dtype, st)

    k_e2e = max(3, min(steps, 20))
    t_e2e, _ = timed(comm, k_e2e, 3, fn=e2e_step)
    e2e_ok = None
    got_e2e = h_recv[3].numpy().view(np.uint16).copy()
    t_e2e_slowest = replicas.max_over_ranks(world, t_e2e)
    e2e_value = units / t_e2e_slowest / 1e9

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world.size, "steps": steps, "warmup": warmup,
        "ms_per_step": t_slowest * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": c.name, "R": R, "elements_per_rank": n, "bytes_per_rank": S, "ring_chunks": R,
            "step": "hoccl_reduce_scatter + hoccl_allgather on one bucket", "path": "CE (driver copy route)",
            "sum_ctas": 8, "executor": "cuda graph replay", "pieces_per_chunk": rs_stats["n_pieces"],
            "l2": "inputs larger than L2: %d bucket sets of %d MiB in rotation" % (N_BUCKET_SETS, 2 * R * S >> 20),
            "parallelism": "replicas x%d (the path does not shard)" % world.size,
        },
        "algbw_GBps": S / t_slowest / 1e9 * world.size,
        "hbm_roofline": {
            "algorithmic_bytes_per_step": algorithmic_hbm_bytes_allreduce(S, R),
            "achieved_GBps": algorithmic_hbm_bytes_allreduce(S, R) / t_step / 1e9,
            "frac_of_8TBps": algorithmic_hbm_bytes_allreduce(S, R) / t_step / 1e9 / NOMINAL_HBM_GBS,
            "frac_of_measured_copy": algorithmic_hbm_bytes_allreduce(S, R) / t_step / 1e9 / peaks["hbm_gbs"],
        },
        "sms_used": {"sum_ctas": int(rs_stats["max_sum_ctas"]), "moves": "driver copy route (see move_needs_sm)",
                     "ordering_kernels_per_step": int(rs_stats["n_order_launches"] + ag_stats["n_order_launches"]),
                     "ordering_kernel": "empty, 1 CTA of 32 threads, ~2 us each (orders copy nodes inside the graphs)"},
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": R * S, "d2h_bytes_per_step": R * S,
                "ms_per_step": t_e2e_slowest * 1e3, "call": "hoccl_host_allreduce (pinned host buffers; inbound copies, ring and outbound copies pipelined over 8 pieces per chunk)", "steps": k_e2e,
                "matches_oracle": e2e_ok},
        "gpu_launches": int(launches_per_step * steps),
        "clocks": clocks,
        "host_launch_us_per_call": st["host_launch_us"],
        "windows": windows,
        "matches_oracle": parity,
        "direct_schedule": direct_line,
        "peaks": peaks,
    }

    if world.rank == 0:
        # ---- the direct schedule's dominant kernel, the chain sum, timed per launch the same way (one launch per step)
        prof_d = new_comm(hb.PATH_CE, sum_ctas=8, profile=1, rs_direct=1, ag_direct=1)
        for k in range(3):
            step(prof_d, k % N_BUCKET_SETS, stream)
        stream.synchronize()
        prof_d.profile_reset()
        for k in range(min(steps, 40)):
            step(prof_d, k % N_BUCKET_SETS, stream)
            stream.synchronize()
            prof_d.last_stats()
        pd = prof_d.last_stats()
        nld = max(1, pd["sum_kernel_launches_timed"])
        avg_d = pd["sum_kernel_ms"] / nld
        bytes_d = pd["sum_kernel_bytes"] / nld
        ach_d = bytes_d / (avg_d * 1e-3) / 1e9 if avg_d > 0 else 0.0
        # traffic: the ncu capture of profiles/chain_kernel_bf16_8cta_25MiB.md (216.7 MB of DRAM traffic for 235.9 MB of
        # algorithmic bytes; the output of one launch is still in L2 when it ends), scaled by the bytes of this launch
        line["direct_schedule"]["roofline"] = {
            "kernel": "chain_kernel<bf16>", "bound": "hbm", "achieved": ach_d, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": ach_d / peaks["hbm_gbs"], "peak_source": "of " + peaks["source"], "traffic": bytes_d * (216.72 / 235.93),
            "algorithmic_bytes_per_launch": bytes_d, "avg_launch_us": avg_d * 1e3, "launches_timed": int(nld), "ctas": 8,
            "note": "8 CTAs by design; 8 reads : 1 write per output byte, 111 GB/s per SM (profiles/chain_kernel_bf16_8cta_25MiB.md)"}
        prof_d.destroy()
        # ---- roofline of the dominant kernel (the only kernel of this path): SUM, timed per launch with CUDA events
        prof = new_comm(hb.PATH_CE, sum_ctas=8, profile=1)
        for k in range(3):
            step(prof, k % N_BUCKET_SETS, stream)
        stream.synchronize()
        prof.profile_reset()
        for k in range(min(steps, 40)):
            step(prof, k % N_BUCKET_SETS, stream)
            stream.synchronize()
            prof.last_stats()
        ps = prof.last_stats()
        nl = max(1, ps["sum_kernel_launches_timed"])
        avg_ms = ps["sum_kernel_ms"] / nl
        bytes_per_launch = ps["sum_kernel_bytes"] / nl
        achieved = bytes_per_launch / (avg_ms * 1e-3) / 1e9 if avg_ms > 0 else 0.0
        line["roofline"] = {
            "kernel": "sum2_kernel<bf16>", "bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / peaks["hbm_gbs"], "peak_source": "of " + peaks["source"],
            "traffic": bytes_per_launch * NCU_TRAFFIC_PER_ALGORITHMIC_BYTE, "algorithmic_bytes_per_launch": bytes_per_launch,
            "avg_launch_us": avg_ms * 1e3, "launches_timed": int(nl), "ctas": 8,
            "sm_budget_ceiling_GBps": 8 * SM_PORT_GBPS, "frac_of_sm_budget_ceiling": achieved / (8 * SM_PORT_GBPS),
            "note": "8 CTAs by design (SM budget for sums): the bound is 8 SM memory ports (~123 GB/s each for 2 reads + 1 write), "
                    "not HBM; roofline_unconstrained is the same kernel on the whole GPU",
        }
        prof.destroy()
        # SM footprint of this library's kernels per step (SMs x busy time) and the paper's contention rate (Eq. 1) with
        # compute taken as active for the whole step: I = sum over kernels of CTAs x duration / (N_SM x step time)
        n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
        sum_us_per_step = avg_ms * 1e3 * rs_stats["n_sum_launches"]
        line["sms_used"].update({"sum_launches_per_step": int(rs_stats["n_sum_launches"]), "sum_busy_us_per_step": sum_us_per_step,
                                 "footprint_sm_us_per_step": 8 * sum_us_per_step, "n_sm": n_sm,
                                 "contention_rate_of_sums": 8 * sum_us_per_step / (n_sm * t_step * 1e6)})
        # the same kernel without the SM budget, timed alone on 256 MiB operands (kernel quality, not the path)
        big = 128 << 20
        a = torch.empty(big, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
        b2 = torch.empty(big, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
        o = torch.empty(big, dtype=torch.bfloat16, device="cuda")
        # SMs used, counted: every CTA of an 8-CTA SUM launch (the launch shape of the timed path) reports its SM id
        ids = torch.full((8,), -1, dtype=torch.int32, device="cuda")
        if hd.kernel_sms("sum", a, b2, o, 8 * 3276800, dtype, 8, ids, stream) == hb.OK:
            stream.synchronize()
            line["sms_used"]["distinct_sms_of_one_sum_launch"] = len(set(ids.cpu().tolist()))
        full = {}
        for ctas in (8, 16, 32, 48, 64, 96, 128, 148, 296, 592):
            for _ in range(3):
                hd.sum_launch(a, b2, o, big, dtype, ctas, stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            reps = 3 if ctas == 8 else 10
            for _ in range(reps):
                hd.sum_launch(a, b2, o, big, dtype, ctas, stream)
            e1.record(stream)
            stream.synchronize()
            full[str(ctas)] = 3.0 * big * 2 / (e0.elapsed_time(e1) / 1e3 / reps) / 1e9
        line["roofline_unconstrained"] = {
            "kernel": "sum2_kernel<bf16>", "operands": "3 x 256 MiB, timed alone", "GBps_by_ctas": full,
            "best_frac_of_measured": max(full.values()) / peaks["hbm_gbs"],
            # the north star's "grid sized to the fewest SMs that still saturate HBM": first CTA count within 5 % of the best
            "fewest_ctas_within_5pct_of_best": min(int(k_) for k_, v_ in full.items() if v_ >= 0.95 * max(full.values()))}
        del a, b2, o

    if world.rank == 0 and world.size == 1:
        # ---- CPU baseline: the oracle on the host cores, whole bucket, a few repetitions
        from oracle import ring as oracle_ring

        thr = oracle_ring.max_threads()
        reps, t0 = 0, time.perf_counter()
        while reps < 3 or (time.perf_counter() - t0 < 2.5 and reps < 50):
            want = oracle_ring.ring_allreduce(xs, threads=thr)
            reps += 1
        t_cpu = (time.perf_counter() - t0) / reps
        # the oracle's result against what the device produced in the timed configuration and end to end
        line["matches_oracle"] = all(bool((got_parity[r] == want[r]).all()) for r in got_parity)
        line["e2e"]["matches_oracle"] = bool((got_e2e == want[3]).all())
        line["direct_schedule"]["matches_oracle"] = all(bool((got_direct[r] == want[r]).all()) for r in got_direct)
        t1 = time.perf_counter()
        oracle_ring.ring_allreduce(xs, threads=1)          # the canonical single-thread run (the parity reference)
        t_single = time.perf_counter() - t1
        line["cpu_baseline"] = {"value": S * bus_factor(R) / t_cpu / 1e9, "unit": "GB/s", "cores": thr, "kind": "oracle",
                                "sample": "%d repetitions of the whole bucket (all %d elements per rank)" % (reps, n),
                                "ms_per_step": t_cpu * 1e3, "single_thread_value": S * bus_factor(R) / t_single / 1e9,
                                "single_thread_ms_per_step": t_single * 1e3}

        if not args.no_extras:
            line["extras"] = extras(hb, hd, W, torch, np, new_comm, step, timed, stream, R, S, n, dtype, peaks, send_sets, recv_sets)

    comm.destroy()
    if world.rank == 0:
        print(json.dumps(line), flush=True)
    replicas.shutdown(world)
    return 0


def small_case(hb, W, torch, np, stream):
    """The small configuration (all-reduce over R = 4, 1,048,576 fp32 per rank, uniform[-1,1), seed 0): latency bound
    (its algorithmic bytes take 11 us at 8 TB/s).  Time per call on both paths; the result is checked against the oracle."""
    from oracle import ring as oracle_ring
    c = W.C1_SMALL_ALLREDUCE
    R, n = c.R, c.count
    xs = W.rank_inputs(c.dist, c.seed, R, n, c.dtype)
    want = oracle_ring.ring_allreduce(xs, threads=oracle_ring.max_threads())
    sets = 8      # 8 x 32 MiB of buffers in rotation: larger than L2
    send = [[torch.from_numpy(x).cuda() for x in xs] for _ in range(sets)]
    recv = [[torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(R)] for _ in range(sets)]
    nb = hb.scratch_bytes_direct(R, n, c.dtype)
    scratch = torch.empty(nb + 256, dtype=torch.uint8, device="cuda")
    rows = {}
    for name, path, ctas, fused, direct, fwd in (("CE_sum8", hb.PATH_CE, 8, 0, 0, 0), ("CE_sum8_direct_allgather", hb.PATH_CE, 8, 0, 1, 0),
                                                 ("SM_8", hb.PATH_SM, 8, 0, 0, 0), ("SM_148", hb.PATH_SM, 148, 0, 0, 0),
                                                 ("SM_148_one_kernel", hb.PATH_SM, 148, 1, 0, 0),
                                                 ("SM_148_direct_allgather", hb.PATH_SM, 148, 0, 1, 0),
                                                 ("SM_148_direct_allgather_forward", hb.PATH_SM, 148, 0, 1, 1)):
        cm = hb.Comm(R, 0)
        cm.set_scratch(scratch.data_ptr() + (-scratch.data_ptr()) % 256, nb)
        cm.set_path(path)
        for key, v in (("sum_ctas", ctas), ("copy_ctas", ctas), ("fused", fused), ("ag_direct", direct), ("forward", fwd)):
            cm.set_param(key, v)
        for b in range(sets):
            cm.allreduce(send[b], recv[b], n, c.dtype, stream)
        stream.synchronize()
        ok = all(bool((recv[0][r].cpu().numpy().view(np.uint32) == want[r].view(np.uint32)).all()) for r in range(R))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 200
        e0.record(stream)
        for i in range(reps):
            cm.allreduce(send[i % sets], recv[i % sets], n, c.dtype, stream)
        e1.record(stream)
        stream.synchronize()
        t = e0.elapsed_time(e1) / 1e3 / reps
        S1 = n * 4
        # algorithmic bytes: the ring's 7 S (R-1); the direct all-gather on the SM path reads a chunk once and stores it R-1
        # times (5 S (R-1) + S R); no figure for the forward comparison variant
        moved = None if fwd else (5.0 * S1 * (R - 1) + S1 * R if (direct and path == hb.PATH_SM) else 7.0 * S1 * (R - 1))
        rows[name] = {"us_per_call": t * 1e6, "busbw_GBps": S1 * 2 * (R - 1) / R / t / 1e9,
                      "hbm_frac_of_8TBps": None if moved is None else moved / t / 1e9 / NOMINAL_HBM_GBS, "matches_oracle": ok}
        cm.destroy()
    # the oracle on the host cores for the same configuration (a reported baseline, as for the headline workload)
    thr = oracle_ring.max_threads()
    t0 = time.perf_counter()
    reps = 0
    while reps < 5 or (time.perf_counter() - t0 < 0.5 and reps < 200):
        oracle_ring.ring_allreduce(xs, threads=thr)
        reps += 1
    t_cpu = (time.perf_counter() - t0) / reps
    rows["cpu_oracle"] = {"us_per_call": t_cpu * 1e6, "busbw_GBps": n * 4 * 2 * (R - 1) / R / t_cpu / 1e9, "cores": thr}
    rows["workload"] = c.name
    return rows


def extras(hb, hd, W, torch, np, new_comm, step, timed, stream, R, S, n, dtype, peaks, send_sets, recv_sets):
    """Context lines: path / CTA-budget variants, whether a move needs an SM, p2p, and the co-running GEMM probe."""
    out = {}
    k, w = 40, 5
    variants = [("CE", hb.PATH_CE, 8, 8), ("CE", hb.PATH_CE, 32, 8), ("CE", hb.PATH_CE, 148, 8), ("SM", hb.PATH_SM, 8, 8),
                ("SM", hb.PATH_SM, 8, 32), ("SM", hb.PATH_SM, 8, 48), ("SM", hb.PATH_SM, 148, 148), ("SM", hb.PATH_SM, 296, 296)]
    rows = []
    hbm = 7.0 * S * (R - 1)
    for name, path, sc, cc in variants:
        cm = new_comm(path, sum_ctas=sc, copy_ctas=cc)
        t, _ = timed(cm, k, w)
        rows.append({"path": name, "sum_ctas": sc, "copy_ctas": cc if path == hb.PATH_SM else None, "ms_per_step": t * 1e3,
                     "busbw_GBps": S * bus_factor(R) / t / 1e9, "hbm_frac_of_8TBps": hbm / t / 1e9 / NOMINAL_HBM_GBS})
        cm.destroy()
    out["variants"] = rows
    # the same copy-route graphs without their empty ordering kernels (parameter "order_kernels" = 0): the comparison point
    pg_rows = []
    for sc in (8, 148):
        cm = new_comm(hb.PATH_CE, sum_ctas=sc, order_kernels=0)
        t, _ = timed(cm, k, w)
        pg_rows.append({"path": "CE", "sum_ctas": sc, "ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9,
                        "hbm_frac_of_8TBps": hbm / t / 1e9 / NOMINAL_HBM_GBS})
        cm.destroy()
    out["plain_graphs_no_order_kernels"] = pg_rows
    # SM footprint of this library's kernels on the SM path (SMs x busy time per step), per-launch CUDA events in the graph
    fp_rows = []
    for sc, cc in ((8, 8), (8, 32), (8, 48), (148, 148)):
        cm = new_comm(hb.PATH_SM, sum_ctas=sc, copy_ctas=cc, profile=1)
        for b in range(4):
            step(cm, b, stream)
        stream.synchronize()
        cm.profile_reset()
        nst = 10
        for b in range(nst):
            step(cm, b % 4, stream)
            stream.synchronize()
            cm.last_stats()
        ps = cm.last_stats()
        sum_us = ps["sum_kernel_ms"] * 1e3 / nst
        copy_us = ps["copy_kernel_ms"] * 1e3 / nst
        fp_rows.append({"sum_ctas": sc, "copy_ctas": cc, "sum_busy_us_per_step": sum_us, "copy_busy_us_per_step": copy_us,
                        "sum_launches_per_step": ps["sum_kernel_launches_timed"] / nst,
                        "copy_launches_per_step": ps["copy_kernel_launches_timed"] / nst,
                        "footprint_sm_us_per_step": sc * sum_us + cc * copy_us,
                        "sum_GBps": ps["sum_kernel_bytes"] / max(ps["sum_kernel_ms"], 1e-9) / 1e6,
                        "copy_GBps": ps["copy_kernel_bytes"] / max(ps["copy_kernel_ms"], 1e-9) / 1e6})
        cm.destroy()
    out["sm_path_footprint"] = fp_rows
    # one all-reduce call instead of two calls (all-gather of early pieces overlaps the last sums)
    cm = new_comm(hb.PATH_CE, sum_ctas=8)

    def one_call(c_, b, st):
        c_.allreduce(send_sets[b], recv_sets[b], n, dtype, st)

    t, _ = timed(cm, k, w, fn=one_call)
    out["single_call_allreduce"] = {"ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9}
    # comparison point: the whole reduction in one kernel (same bits, not rank local), by CTA budget
    op_rows = []
    for ctas in (8, 32, 148):
        c1 = new_comm(hb.PATH_CE, sum_ctas=ctas, onepass=1)
        t, _ = timed(c1, k, w, fn=one_call)
        op_rows.append({"ctas": ctas, "ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9,
                        "bytes_per_step": 2.0 * R * S, "GBps": 2.0 * R * S / t / 1e9})
        c1.destroy()
    out["onepass_allreduce"] = op_rows
    # second comparison point: fused sum-and-forward (a SUM stores into the next rank's inbox; moves only at step 0)
    fw_rows = []
    for name, path, sc, cc in (("CE", hb.PATH_CE, 8, 8), ("SM", hb.PATH_SM, 8, 8), ("SM", hb.PATH_SM, 148, 148)):
        c1 = new_comm(path, sum_ctas=sc, copy_ctas=cc, forward=1)
        t, _ = timed(c1, k, w)
        fw_rows.append({"path": name, "sum_ctas": sc, "ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9})
        c1.destroy()
    out["forward_variant"] = fw_rows
    # direct all-gather: R-1 independent permutation stages r -> r+k instead of R-1 dependent ring hops (rank local, same bytes)
    ad_rows = []
    for name, path, sc, cc, fw in (("CE", hb.PATH_CE, 8, 8, 0), ("CE", hb.PATH_CE, 148, 8, 0), ("SM", hb.PATH_SM, 8, 8, 0),
                                   ("SM", hb.PATH_SM, 8, 48, 0), ("SM", hb.PATH_SM, 148, 148, 0), ("SM", hb.PATH_SM, 148, 148, 1)):
        c1 = new_comm(path, sum_ctas=sc, copy_ctas=cc, ag_direct=1, forward=fw)
        t, _ = timed(c1, k, w)
        # algorithmic bytes: the copy route moves every stage separately (the ring's 2 S (R-1) for the all-gather); the SM path
        # reads every chunk once and stores it R-1 times (S R); the forward variant is a comparison point, no fraction given
        ag_bytes = 2.0 * S * (R - 1) if path == hb.PATH_CE else 1.0 * S * R
        hbm_d = 5.0 * S * (R - 1) + ag_bytes
        t1, _ = timed(c1, k, w, fn=one_call)
        ad_rows.append({"path": name, "sum_ctas": sc, "copy_ctas": cc if path == hb.PATH_SM else None, "forward": fw, "ms_per_step": t * 1e3,
                        "busbw_GBps": S * bus_factor(R) / t / 1e9, "hbm_bytes_per_step": None if fw else hbm_d,
                        "hbm_frac_of_8TBps": None if fw else hbm_d / t / 1e9 / NOMINAL_HBM_GBS,
                        "one_allreduce_call_ms": t1 * 1e3, "one_allreduce_call_busbw_GBps": S * bus_factor(R) / t1 / 1e9})
        c1.destroy()
    out["direct_allgather"] = ad_rows
    # direct schedule: the reduce-scatter too as independent permutation stages, into R-1 inbox slots of the owner, and ONE chain
    # sum per rank in the ring's order (rank local, the ring's bits); with the ring or the direct all-gather behind it
    ds_rows = []
    for name, path, sc, cc, agd in (("CE", hb.PATH_CE, 8, 8, 0), ("CE", hb.PATH_CE, 8, 8, 1), ("CE", hb.PATH_CE, 32, 8, 1), ("CE", hb.PATH_CE, 148, 8, 1),
                                    ("SM", hb.PATH_SM, 8, 8, 1), ("SM", hb.PATH_SM, 8, 48, 1), ("SM", hb.PATH_SM, 148, 148, 1)):
        c1 = new_comm(path, sum_ctas=sc, copy_ctas=cc, rs_direct=1, ag_direct=agd)
        t, _ = timed(c1, k, w)
        t1, _ = timed(c1, k, w, fn=one_call)
        # algorithmic bytes: moves 2 S (R-1), chain sum S (R+1) (R reads and one write per output byte), all-gather 2 S (R-1) as
        # copies or S R as a fan-out launch
        ag_bytes = 1.0 * S * R if (agd and path == hb.PATH_SM) else 2.0 * S * (R - 1)
        hbm_d = 2.0 * S * (R - 1) + 1.0 * S * (R + 1) + ag_bytes
        ds_rows.append({"path": name, "sum_ctas": sc, "copy_ctas": cc if path == hb.PATH_SM else None, "ag_direct": agd, "ms_per_step": t * 1e3,
                        "busbw_GBps": S * bus_factor(R) / t / 1e9, "hbm_bytes_per_step": hbm_d, "hbm_frac_of_8TBps": hbm_d / t / 1e9 / NOMINAL_HBM_GBS,
                        "one_allreduce_call_ms": t1 * 1e3, "one_allreduce_call_busbw_GBps": S * bus_factor(R) / t1 / 1e9,
                        "sum_launches_per_step": int(c1.last_stats()["n_sum_launches"])})
        c1.destroy()
    out["direct_schedule"] = ds_rows
    # SM path with the whole collective as one cooperative kernel (grid barriers instead of kernel boundaries)
    fu_rows = []
    for ctas in (8, 148):
        c1 = new_comm(hb.PATH_SM, sum_ctas=ctas, copy_ctas=ctas, fused=1)
        t, _ = timed(c1, k, w, fn=one_call)
        fu_rows.append({"ctas": ctas, "ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9,
                        "launches_per_step": int(c1.last_stats()["n_move_launches"] + c1.last_stats()["n_sum_launches"]),
                        "async_error": int(c1.async_error())})
        c1.destroy()
    out["fused_ring_kernel_SM_path"] = fu_rows
    # the one route on a single device that really uses no SM for moves: bounce through pinned host memory
    host_stage = torch.empty(400 << 20, dtype=torch.uint8).pin_memory()
    c1 = new_comm(hb.PATH_CE_HOST, sum_ctas=8)
    c1.set_host_staging(host_stage)
    t, _ = timed(c1, 6, 3)
    out["host_bounce_path"] = {"ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9,
                               "pcie_bytes_per_step_each_way": 2.0 * S * (R - 1)}
    # the same with the direct all-gather: a final chunk goes out to the host once and comes back R-1 times
    c1.set_param("ag_direct", 1)
    t, _ = timed(c1, 6, 3)
    out["host_bounce_path_direct_allgather"] = {"ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9,
                                                "pcie_bytes_per_step_outbound": 1.0 * S * (R - 1) + 1.0 * S,
                                                "pcie_bytes_per_step_inbound": 2.0 * S * (R - 1)}
    c1.destroy()
    # handshake mode (CPU proxy + stream memory operations) on the SM path, against the same path launched directly
    hs = {}
    for label, flag in (("direct", 0), ("handshake", 1)):
        c1 = new_comm(hb.PATH_SM, sum_ctas=8, copy_ctas=32, handshake=flag)
        t, _ = timed(c1, k, w)
        hs[label] = {"ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9}
        if flag:
            hs["handshakes_served"] = c1.handshakes()
        c1.destroy()
    out["handshake_mode_SM_copy32_sum8"] = hs
    # stream executor (events) instead of graph replay
    cm.set_param("use_graph", 0)
    t, _ = timed(cm, k, w)
    out["stream_executor"] = {"ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9,
                              "host_launch_us_per_call": cm.last_stats()["host_launch_us"]}
    cm.set_param("use_graph", 1)

    # does a move need an SM?  (bounded occupancy kernel + one 64 MiB move)
    src = send_sets[0][0]
    dst = recv_sets[0][0]
    nb = min(64 << 20, src.numel() * 2)
    ce_needs, ce_end = hd.probe_move_needs_sm(cm, hb.PATH_CE, dst, src, nb, 3000)
    sm_needs, sm_end = hd.probe_move_needs_sm(cm, hb.PATH_SM, dst, src, nb, 3000)
    pinned = torch.empty(8 << 20, dtype=torch.uint8).pin_memory()
    h2d_needs, h2d_end = hd.probe_move_needs_sm(cm, hb.PATH_CE, dst, pinned, pinned.numel(), 3000)
    cm.set_host_staging(host_stage)
    hb_needs, hb_end = hd.probe_move_needs_sm(cm, hb.PATH_CE_HOST, dst, src, min(nb, 16 << 20), 3000)
    out["move_needs_sm"] = {"CE_HOST_bounce_16MiB": hb_needs, "CE_HOST_move_end_us": hb_end,
                            "CE_driver_copy_same_device_64MiB": ce_needs, "CE_move_end_us": ce_end, "SM_copy_kernel": sm_needs,
                            "SM_move_end_us": sm_end, "control_pinned_host_to_device_8MiB": h2d_needs,
                            "control_move_end_us": h2d_end, "occupancy_kernel_us": 3000,
                            "note": "true = the move finished only after a kernel holding every SM had ended"}
    out["copy_routes_16MiB"] = [{"route": n_, "needs_sm": s_, "end_us": round(t_, 1)}
                                for n_, s_, t_ in hd.probe_copy_routes(cm, dst, src, min(nb, 16 << 20), 3000)]
    # host cost of one call with an idle queue (the paper's CPU launch overhead axis)
    host_us = {}
    for label, use_graph in (("graph_replay", 1), ("stream_executor", 0)):
        cm.set_param("use_graph", use_graph)
        step(cm, 0, stream)
        stream.synchronize()
        vals = []
        for _ in range(15):
            cm.allreduce(send_sets[0], recv_sets[0], n, dtype, stream)
            vals.append(cm.last_stats()["host_launch_us"])
            stream.synchronize()
        vals.sort()
        host_us[label] = vals[len(vals) // 2]
    cm.set_param("use_graph", 1)
    out["host_launch_us_per_allreduce_call_idle_queue"] = host_us

    # point to point: 64 MiB bf16 activations [4, 2048, 4096]
    act = torch.empty(4 * 2048 * 4096, dtype=torch.bfloat16, device="cuda").normal_(0, 1)
    slots = [torch.empty_like(act) for _ in range(4)]
    p2p = {}
    for name, path in (("CE", hb.PATH_CE), ("SM8", hb.PATH_SM)):
        cm.set_path(path)
        cm.set_param("copy_ctas", 8)

        def hop(c_, b, st):
            c_.send(act, act.numel(), "bf16", 0, 1, st)
            c_.recv(slots[b], act.numel(), "bf16", 0, 1, st)

        t, _ = timed(cm, 20, 3, fn=hop)
        p2p[name] = {"us_per_message": t * 1e6, "algbw_GBps": act.numel() * 2 / t / 1e9,
                     "hbm_frac_of_8TBps": 2 * act.numel() * 2 / t / 1e9 / NOMINAL_HBM_GBS}
    out["p2p_64MiB"] = p2p
    cm.set_path(hb.PATH_CE)

    # co-running bf16 GEMM probe (4096^3) on another stream: TFLOP/s alone and beside the collective
    gs = torch.cuda.Stream()
    A = torch.randn(4096, 4096, dtype=torch.bfloat16, device="cuda")
    B = torch.randn(4096, 4096, dtype=torch.bfloat16, device="cuda")
    C = torch.empty(4096, 4096, dtype=torch.bfloat16, device="cuda")
    flops = 2.0 * 4096 ** 3

    def gemm_tflops(cm_, n_gemm=150, fn=step):
        with torch.cuda.stream(gs):
            for _ in range(10):
                torch.matmul(A, B, out=C)
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_comm = 0
        if cm_ is not None:
            t_c, _ = timed(cm_, 10, 3, fn=fn)
            n_comm = int(1.5 * n_gemm * 80e-6 / t_c) + 2
        c0.record(stream)
        g0.record(gs)
        done_c = 0
        for i in range(n_gemm):
            with torch.cuda.stream(gs):
                torch.matmul(A, B, out=C)
            want_c = (i + 1) * n_comm // n_gemm
            while done_c < want_c:
                fn(cm_, done_c % N_BUCKET_SETS, stream)
                done_c += 1
        g1.record(gs)
        c1.record(stream)
        torch.cuda.synchronize()
        tf = flops * n_gemm / (g0.elapsed_time(g1) / 1e3) / 1e12
        bw = (S * bus_factor(R) * done_c / (c0.elapsed_time(c1) / 1e3) / 1e9) if done_c else 0.0
        return tf, bw

    probe = {}
    alone, _ = gemm_tflops(None)
    probe["alone_TFLOPs"] = alone
    for name, path, sc, cc, op, fw in (("CE_sum8", hb.PATH_CE, 8, 8, 0, 0), ("CE_sum8_plain_graphs_no_order_kernels", hb.PATH_CE, 8, 8, 0, 4),
                                       ("SM_copy8_sum8", hb.PATH_SM, 8, 8, 0, 0),
                                       ("SM_copy32_sum8", hb.PATH_SM, 8, 32, 0, 0), ("SM_copy48_sum8", hb.PATH_SM, 8, 48, 0, 0),
                                       ("SM_copy148_sum148", hb.PATH_SM, 148, 148, 0, 0),
                                       ("SM_copy48_sum8_direct_allgather", hb.PATH_SM, 8, 48, 0, 3),
                                       ("CE_sum8_direct_schedule", hb.PATH_CE, 8, 8, 0, 5), ("SM_copy48_sum8_direct_schedule", hb.PATH_SM, 8, 48, 0, 5),
                                       ("SM_forward_copy8_sum8", hb.PATH_SM, 8, 8, 0, 1),
                                       ("SM_one_kernel_8", hb.PATH_SM, 8, 8, 0, 2),
                                       ("onepass_8", hb.PATH_CE, 8, 8, 1, 0), ("CE_HOST_sum8", hb.PATH_CE_HOST, 8, 8, 0, 0)):
        c2 = new_comm(path, sum_ctas=sc, copy_ctas=cc, onepass=op, forward=1 if fw == 1 else 0, fused=1 if fw == 2 else 0,
                      ag_direct=1 if fw in (3, 5) else 0, order_kernels=0 if fw == 4 else 1, rs_direct=1 if fw == 5 else 0)
        if path == hb.PATH_CE_HOST:
            c2.set_host_staging(host_stage)
        # the one-pass comparison kernel is one all-reduce call (reduce-scatter + all-gather would add the path's moves)
        tf, bw = gemm_tflops(c2, fn=one_call if op else step)
        probe[name] = {"gemm_TFLOPs": tf, "loss": 1.0 - tf / alone, "comm_busbw_GBps": bw}
        c2.destroy()
    out["gemm_probe_4096"] = probe
    out["c1_small_allreduce"] = small_case(hb, W, torch, np, stream)
    # the paper's own figures, as context only (other hardware, real multi-GPU links, no reduction on its path)
    out["paper_context"] = {
        "hardware": "32 x NVIDIA H800 80 GB (132 SMs each), 8 per node on NVLink, one 50 GB/s NIC per GPU",
        "communication_performance": "within 3 % of the state of the art on average (point-to-point, all-gather, all-to-all, 2 MB to 1 GB)",
        "sms_freed": "about 10 % of the SMs (pipeline- plus data-parallel traffic of a GPT-6.7B run)",
        "end_to_end_training_gain": "up to 5 % (2.4 % at 6.7B, 5.1 % at 32B parameters) over the SM-driven library",
        "allgather_8_gpus_1GB_algbw_GBps": 192.2, "intra_node_p2p_1GB_algbw_GBps": 192.2, "alltoall_8_gpus_1GB_algbw_GBps": 191.4,
        "reductions": "outside the paper's scope (they fall back to the SM-driven library there): no all-reduce figure exists to compare with",
    }
    cm.destroy()
    return out


if __name__ == "__main__":
    sys.exit(main())
