#!/usr/bin/env python
"""Benchmark of the collective hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras] [--no-large]

Workload (N = 1): the largest single-GPU configuration, the GPT-6.7B-shaped data-parallel gradient stream: 32 layers of
hidden 4096 / FFN 16384 bf16 gradients, normal(0, 1e-3), seed 3, cut flat into 40 MiB buckets (307 of them and one of
8 MiB) and all-reduced over R = 8 logical ranks.  One step = one pass of the whole path over one bucket: one
hoccl_allreduce call (plan lookup, ordering into the caller's stream, the reduce-scatter's moves, the sum, the
all-gather's moves), on the copy route with at most 8 CTAs for sums, default settings otherwise.  Three bucket sets
(640 MiB each, every one larger than the 126 MB L2) are used in rotation.

Reported value: all-reduce bus bandwidth, S * 2(R-1)/R / t_step in GB/s (nccl-tests convention).  With N GPUs, N
independent replicas run and the value is the sum of their units over the slowest replica's time.  One JSON line on
stdout (rank 0).  Beside the headline the line carries: the same workload on the ring schedule step by step
(`ring_schedule`), the per-launch roofline of the dominant kernel of each, the end-to-end figure through host buffers,
the CPU oracle timed on the host cores, `large_messages` (64 MiB to 1 GiB per rank, every collective, copy route against
SM path, each checked against the oracle), `gemm_loss_matched` (what a co-running GEMM loses against the collective's
throughput beside it, copy route and copy-kernel budgets) and `extras` (the smaller configurations and comparison points).
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
MiB = 1 << 20

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per algorithmic byte of one launch, from one ncu capture of each
# kernel on operands larger than L2 with 8 CTAs (part of a launch's output is still in L2 when it ends).  Traffic of these
# streaming kernels grows in proportion to the bytes a launch processes, so it is scaled to the launch timed here.
NCU_TRAFFIC_PER_BYTE_SUM = 573.88 / 629.15       # sum2_kernel<bf16>, 3 x 200 MiB
NCU_TRAFFIC_PER_BYTE_CHAIN = 217.56 / 235.93     # chain_pipe_kernel<bf16, 8 operands>, 25 MiB each
SM_PORT_GBPS_SUM = 123.0     # measured ceiling of one SM's memory port at 2 reads : 1 write
SM_PORT_GBPS_CHAIN = 163.0   # the same at 8 reads : 1 write (every in-flight depth tried ends there)


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the smaller configurations and comparison points")
    ap.add_argument("--no-large", action="store_true", help="skip large_messages and gemm_loss_matched")
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


def ring_bytes_allreduce(S, R):
    """Rank-local ring on one device: every wire byte is read+written by a MOVE in both phases (2+2) and read twice + written
    once by a SUM (3): 7 * S * (R-1)."""
    return 7.0 * S * (R - 1)


def direct_bytes_allreduce(S, R):
    """Stage-decomposed schedule: moves 2 S (R-1) into the owners' inbox slots, one chain sum per rank (R reads and one write per
    output byte: S (R+1)), all-gather moves 2 S (R-1)."""
    return 4.0 * S * (R - 1) + S * (R + 1)


def reference_arm(args, world):
    """Times the CPU oracle, as it stands, on the host cores (rank 0 only): the ring all-reduce of one 40 MiB bucket."""
    if world.rank != 0:
        return
    from oracle import ring
    from paper_2609_34334_b200 import workloads as W

    g = W.C4_GRADIENTS
    R, dtype = g.R, g.dtype
    threads = ring.max_threads()
    xs = W.gradient_bucket(g, 0)
    n = xs[0].size
    t0 = time.perf_counter()
    ring.ring_allreduce(xs, threads=threads)
    t_one = time.perf_counter() - t0
    budget = 150.0
    full = n
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
    sample = ("all %d elements per rank of one bucket" % n if n == full else
              "first %d of %d elements per rank of one bucket (%.1f%%)" % (n, full, 100.0 * n / full))
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "GB/s", "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": g.name, "R": R, "elements_per_rank": n, "bytes_per_rank": S,
                   "step": "ring all-reduce of one bucket by the CPU oracle"},
        "cpu_baseline": {"value": val, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------------
class Bench:
    """Buffers, communicators and timing for all-reduce over R ranks of n elements of bf16, several buffer sets in rotation."""

    def __init__(self, torch, hb, replicas, world, dev, R, n, nsets, first_set_host=None):
        import numpy as np

        self.torch, self.hb, self.replicas, self.world, self.dev = torch, hb, replicas, world, dev
        self.R, self.n, self.dtype, self.e = R, n, "bf16", 2
        self.S = n * 2
        self.nsets = nsets
        self.stream = torch.cuda.Stream()
        self.send_sets, self.recv_sets = [], []
        for b in range(nsets):
            if b == 0 and first_set_host is not None:
                send = [torch.from_numpy(x.view(np.int16)).to("cuda") for x in first_set_host]
            elif b == 0:
                send = [torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3).view(torch.int16) for _ in range(R)]
            else:
                send = [torch.roll(t, 4099 * b) for t in self.send_sets[0]]      # the same values rotated: only timing uses them
            self.send_sets.append(send)
            self.recv_sets.append([torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)])
        self.scratch = torch.empty(hb.scratch_bytes_direct(R, n, self.dtype) + 256, dtype=torch.uint8, device="cuda")   # covers every variant
        self.spad = (-self.scratch.data_ptr()) % 256

    def comm(self, path, **params):
        cm = self.hb.Comm(self.R, self.dev)
        cm.set_scratch(self.scratch.data_ptr() + self.spad, self.scratch.numel() - 256)
        cm.set_path(path)
        for k, v in params.items():
            cm.set_param(k, v)
        return cm

    def allreduce(self, cm, b, st):
        cm.allreduce(self.send_sets[b], self.recv_sets[b], self.n, self.dtype, st)

    def two_calls(self, cm, b, st):
        """reduce-scatter into chunk r of recv[r], then all-gather in place: the gradient bucket as two calls."""
        count = self.n // self.R
        recv = self.recv_sets[b]
        rs_out = [recv[r].data_ptr() + r * count * self.e for r in range(self.R)]
        cm.reduce_scatter(self.send_sets[b], rs_out, count, self.dtype, st)
        cm.allgather(rs_out, recv, count, self.dtype, st)

    def timed(self, cm, k_steps, k_warm, fn=None, sampler=None):
        torch, stream = self.torch, self.stream
        fn = fn or self.allreduce
        # warm-up touches every buffer set at least once, so every cached graph exists before the timed region
        for k in range(max(k_warm, self.nsets)):
            fn(cm, k % self.nsets, stream)
        stream.synchronize()
        self.replicas.barrier(self.world)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if sampler:
            sampler.start()
        e0.record(stream)
        for k in range(k_steps):
            fn(cm, k % self.nsets, stream)
        e1.record(stream)
        stream.synchronize()
        torch.cuda.synchronize()
        clocks = sampler.stop() if sampler else None
        self.replicas.barrier(self.world)
        return e0.elapsed_time(e1) / 1e3 / k_steps, clocks

    def kernel_roofline(self, peaks, steps, fn=None, **params):
        """Per-launch time of the SUM kernels of this configuration, from CUDA events recorded around every SUM node."""
        cm = self.comm(self.hb.PATH_CE, profile=1, **params)
        fn = fn or self.allreduce
        for k in range(3):
            fn(cm, k % self.nsets, self.stream)
        self.stream.synchronize()
        cm.profile_reset()
        for k in range(min(steps, 40)):
            fn(cm, k % self.nsets, self.stream)
            self.stream.synchronize()
            cm.last_stats()
        ps = cm.last_stats()
        cm.destroy()
        nl = max(1, ps["sum_kernel_launches_timed"])
        avg_ms = ps["sum_kernel_ms"] / nl
        per_launch = ps["sum_kernel_bytes"] / nl
        ach = per_launch / (avg_ms * 1e-3) / 1e9 if avg_ms > 0 else 0.0
        return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                "peak_source": "of " + peaks["source"], "algorithmic_bytes_per_launch": per_launch, "avg_launch_us": avg_ms * 1e3,
                "launches_timed": int(nl), "ctas": int(params.get("sum_ctas", 8))}

    def result(self, ranks=(0, 5)):
        import numpy as np

        return {r: self.recv_sets[0][r].cpu().numpy().view(np.uint16).copy() for r in ranks}

    def free(self):
        self.send_sets, self.recv_sets, self.scratch = [], [], None
        self.torch.cuda.empty_cache()


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
    oracle_here = world.rank == 0 and world.size == 1      # the one leg that may run the CPU oracle

    g = W.C4_GRADIENTS
    R, dtype = g.R, g.dtype
    sizes = g.buckets()
    n = sizes[0]
    S = n * 2
    xs = W.gradient_bucket(g, 0)                           # bucket 0 of every rank: the seeded workload
    B = Bench(torch, hb, replicas, world, dev, R, n, 3, first_set_host=xs)
    stream = B.stream

    # ---- headline: copy route, <= 8 CTAs for sums, default settings (the schedule is chosen automatically)
    comm = B.comm(hb.PATH_CE, sum_ctas=8)
    sampler = ClockSampler(dev)
    t_step, clocks = B.timed(comm, steps, warmup, sampler=sampler)
    st = comm.last_stats()
    win = sorted(B.timed(comm, max(5, steps // 10), 0)[0] * 1e3 for _ in range(10))
    windows = {"n": 10, "steps_each": max(5, steps // 10), "median_ms_per_step": win[len(win) // 2], "best_ms_per_step": win[0],
               "worst_ms_per_step": win[-1]}
    launches_per_step = int(st["n_sum_launches"] + st["n_move_launches"] + st["n_order_launches"])
    rc, opt = hd.options_resolve(hd.PLAN_ALLREDUCE, R, n, dtype, hb.PATH_CE, scratch_bytes=B.scratch.numel() - 256)
    direct = bool(opt and opt["plan_kind"] & hd.PLAN_FLAG_RS_DIRECT)
    B.allreduce(comm, 0, stream)
    stream.synchronize()
    got_head = B.result()

    t_slowest = replicas.max_over_ranks(world, t_step)
    units = replicas.sum_over_ranks(world, S * bus_factor(R))
    value = units / t_slowest / 1e9
    own_bytes = direct_bytes_allreduce(S, R) if direct else ring_bytes_allreduce(S, R)

    # ---- the same workload on the ring schedule, step by step (R-1 moves and R-1 sums per chunk, then R-1 hops)
    comm_r = B.comm(hb.PATH_CE, sum_ctas=8, rs_direct=0, ag_direct=0)
    t_ring, _ = B.timed(comm_r, steps, warmup)
    str_ = comm_r.last_stats()
    B.allreduce(comm_r, 0, stream)
    stream.synchronize()
    got_ring = B.result()
    comm_r.destroy()
    t_ring_slowest = replicas.max_over_ranks(world, t_ring)
    ring_line = {"schedule": "ring reduce-scatter (R-1 steps of move + sum) and ring all-gather (R-1 hops)", "path": "CE (driver copy route)",
                 "sum_ctas": 8, "value": units / t_ring_slowest / 1e9, "unit": "GB/s", "ms_per_step": t_ring_slowest * 1e3,
                 "sum_launches_per_step": int(str_["n_sum_launches"]), "algorithmic_bytes_per_step": ring_bytes_allreduce(S, R),
                 "hbm_frac_of_8TBps": ring_bytes_allreduce(S, R) / t_ring / 1e9 / NOMINAL_HBM_GBS, "matches_oracle": None}

    # ---- end to end: host buffers through hoccl_host_allreduce (H2D and D2H inside the timed region)
    per = (S + 255) // 256 * 256
    staging = torch.empty(2 * R * per + 256, dtype=torch.uint8, device="cuda")
    gpad = (-staging.data_ptr()) % 256
    comm.set_staging(staging.data_ptr() + gpad, 2 * R * per)
    h_send = [torch.from_numpy(x.view(np.int16)).pin_memory() for x in xs]
    h_recv = [torch.zeros(n, dtype=torch.int16).pin_memory() for _ in range(R)]

    def e2e_step(cm, b, st_):
        cm.host_allreduce(h_send, h_recv, n, dtype, st_)

    k_e2e = max(3, min(steps, 20))
    t_e2e, _ = B.timed(comm, k_e2e, 3, fn=e2e_step)
    got_e2e = h_recv[3].numpy().view(np.uint16).copy()
    t_e2e_slowest = replicas.max_over_ranks(world, t_e2e)
    del staging, h_send, h_recv

    line = {
        "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": world.size, "steps": steps, "warmup": warmup,
        "ms_per_step": t_slowest * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": g.name, "R": R, "elements_per_rank": n, "bytes_per_rank": S, "ring_chunks": R,
            "stream": "%d buckets of %d MiB and one of %d MiB per rank (%.1f GiB); every bucket is the same work, %d are timed" %
                      (len(sizes) - 1, S >> 20, sizes[-1] * 2 >> 20, sum(sizes) * 2 / 2 ** 30, steps),
            "step": "one hoccl_allreduce call on one bucket", "path": "CE (driver copy route)", "sum_ctas": 8,
            "schedule": ("stage-decomposed reduce-scatter and all-gather, one chain sum per rank in the ring's order (chosen automatically: "
                         "the attached scratch holds its R-1 inbox slots per rank)") if direct else "ring, step by step",
            "executor": "cuda graph replay", "pieces_per_chunk": st["n_pieces"],
            "l2": "inputs larger than L2: %d bucket sets of %d MiB in rotation" % (B.nsets, 2 * R * S >> 20),
            "gemm_probe": "not running during the timed steps; gemm_loss_matched times the same stream beside it",
            "parallelism": "replicas x%d (the path does not shard)" % world.size,
        },
        "algbw_GBps": S / t_slowest / 1e9 * world.size,
        "full_stream_ms_estimate": t_step * 1e3 * (len(sizes) - 1 + sizes[-1] / n),
        "hbm_roofline": {
            "definition": "bytes the rank-local RING must move, 7 S (R-1), over the step time, against 8 TB/s (the target's definition)",
            "ring_bytes_per_step": ring_bytes_allreduce(S, R),
            "frac_of_8TBps": ring_bytes_allreduce(S, R) / t_step / 1e9 / NOMINAL_HBM_GBS,
            "frac_of_measured_copy": ring_bytes_allreduce(S, R) / t_step / 1e9 / peaks["hbm_gbs"],
            "bytes_this_schedule_moves": own_bytes, "achieved_GBps_own_bytes": own_bytes / t_step / 1e9,
            "frac_of_8TBps_own_bytes": own_bytes / t_step / 1e9 / NOMINAL_HBM_GBS,
        },
        "sms_used": {"sum_ctas": int(st["max_sum_ctas"]), "sum_launches_per_step": int(st["n_sum_launches"]),
                     "moves": "driver copy route (see extras.move_needs_sm)",
                     "ordering_kernels_per_step": int(st["n_order_launches"]),
                     "ordering_kernel": "empty, 1 CTA of 32 threads, ~2 us each (orders copy nodes inside the graph)"},
        "e2e": {"value": units / t_e2e_slowest / 1e9, "unit": "GB/s", "h2d_bytes_per_step": R * S, "d2h_bytes_per_step": R * S,
                "ms_per_step": t_e2e_slowest * 1e3, "steps": k_e2e, "matches_oracle": None,
                "call": "hoccl_host_allreduce (pinned host buffers; inbound copies, the collective and outbound copies pipelined over 8 pieces per chunk)"},
        "gpu_launches": int(launches_per_step * steps),
        "clocks": clocks,
        "host_launch_us_per_call": st["host_launch_us"],
        "windows": windows,
        "matches_oracle": None,
        "ring_schedule": ring_line,
        "peaks": peaks,
    }

    if world.rank == 0:
        # ---- roofline of the dominant kernel of the timed configuration, per launch, CUDA events around every SUM node
        r = B.kernel_roofline(peaks, steps, sum_ctas=8)
        if direct:
            r.update({"kernel": "chain_pipe_kernel<bf16, 8 operands>", "traffic": r["algorithmic_bytes_per_launch"] * NCU_TRAFFIC_PER_BYTE_CHAIN,
                      "sm_budget_ceiling_GBps": 8 * SM_PORT_GBPS_CHAIN, "frac_of_sm_budget_ceiling": r["achieved"] / (8 * SM_PORT_GBPS_CHAIN),
                      "note": "8 CTAs by design (the SM budget for sums): R reads and 1 write per output byte; the bound is 8 SM memory ports "
                              "(~163 GB/s each at this mix), not HBM; with the whole GPU the same sum runs at 5.7 TB/s"})
        else:
            r.update({"kernel": "sum2_kernel<bf16>", "traffic": r["algorithmic_bytes_per_launch"] * NCU_TRAFFIC_PER_BYTE_SUM,
                      "sm_budget_ceiling_GBps": 8 * SM_PORT_GBPS_SUM, "frac_of_sm_budget_ceiling": r["achieved"] / (8 * SM_PORT_GBPS_SUM)})
        line["roofline"] = r
        rr = B.kernel_roofline(peaks, steps, sum_ctas=8, rs_direct=0, ag_direct=0)
        rr.update({"kernel": "sum2_kernel<bf16>", "traffic": rr["algorithmic_bytes_per_launch"] * NCU_TRAFFIC_PER_BYTE_SUM,
                   "sm_budget_ceiling_GBps": 8 * SM_PORT_GBPS_SUM, "frac_of_sm_budget_ceiling": rr["achieved"] / (8 * SM_PORT_GBPS_SUM),
                   "note": "8 CTAs by design: the bound is 8 SM memory ports (~123 GB/s each for 2 reads + 1 write), not HBM; "
                           "roofline_unconstrained is the same kernel on the whole GPU"})
        line["ring_schedule"]["roofline"] = rr
        n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
        sum_us = r["avg_launch_us"] * st["n_sum_launches"]
        # SM footprint of this library's kernels per step (SMs x busy time) and the paper's contention rate (Eq. 1) with compute
        # taken as active for the whole step: sum over kernels of CTAs x duration / (N_SM x step time)
        line["sms_used"].update({"sum_busy_us_per_step": sum_us, "footprint_sm_us_per_step": 8 * sum_us, "n_sm": n_sm,
                                 "contention_rate_of_sums": 8 * sum_us / (n_sm * t_step * 1e6)})
        # the SUM kernel without the SM budget, timed alone on 256 MiB operands (kernel quality, not the path)
        big = 128 << 20
        a = torch.empty(big, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
        b2 = torch.empty(big, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
        o = torch.empty(big, dtype=torch.bfloat16, device="cuda")
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
            # "grid sized to the fewest SMs that still saturate HBM": first CTA count within 5 % of the best
            "fewest_ctas_within_5pct_of_best": min(int(k_) for k_, v_ in full.items() if v_ >= 0.95 * max(full.values()))}
        del a, b2, o

    want = None
    if oracle_here:
        # ---- CPU baseline: the oracle on the host cores, one whole bucket, a few repetitions; and the comparison of what the
        # device produced with the oracle's bits, which happens where the oracle runs
        from oracle import ring as oracle_ring

        thr = oracle_ring.max_threads()
        reps, t0 = 0, time.perf_counter()
        while reps < 3 or (time.perf_counter() - t0 < 2.5 and reps < 50):
            want = oracle_ring.ring_allreduce(xs, threads=thr)
            reps += 1
        t_cpu = (time.perf_counter() - t0) / reps
        line["matches_oracle"] = all(bool((got_head[r] == want[r]).all()) for r in got_head)
        line["ring_schedule"]["matches_oracle"] = all(bool((got_ring[r] == want[r]).all()) for r in got_ring)
        line["e2e"]["matches_oracle"] = bool((got_e2e == want[3]).all())
        t1 = time.perf_counter()
        oracle_ring.ring_allreduce(xs, threads=1)          # the canonical single-thread run (the parity reference)
        t_single = time.perf_counter() - t1
        line["cpu_baseline"] = {"value": S * bus_factor(R) / t_cpu / 1e9, "unit": "GB/s", "cores": thr, "kind": "oracle",
                                "sample": "%d repetitions of one whole bucket (all %d elements per rank)" % (reps, n),
                                "ms_per_step": t_cpu * 1e3, "single_thread_value": S * bus_factor(R) / t_single / 1e9,
                                "single_thread_ms_per_step": t_single * 1e3}
        # the ragged last bucket of the stream (8 MiB) through the same communicator
        xl = W.gradient_bucket(g, len(sizes) - 1)
        nl = xl[0].size
        sl = [torch.from_numpy(x.view(np.int16)).cuda() for x in xl]
        rl = [torch.zeros(nl, dtype=torch.int16, device="cuda") for _ in range(R)]
        comm.allreduce(sl, rl, nl, dtype, stream)
        stream.synchronize()
        wl = oracle_ring.ring_allreduce(xl, threads=thr)
        line["last_bucket"] = {"elements_per_rank": nl, "bytes_per_rank": nl * 2,
                               "matches_oracle": all(bool((rl[r].cpu().numpy().view(np.uint16) == wl[r]).all()) for r in range(R))}
        del sl, rl, xl, wl

        if not args.no_large:
            want_dev = torch.from_numpy(want[0].view(np.int16)).cuda()
            line["gemm_loss_matched"] = gemm_loss_matched(torch, hb, W, B, want_dev)
            del want_dev

    comm.destroy()
    B.free()
    if oracle_here and not args.no_large:
        line["large_messages"] = large_messages(torch, hb, W, np, peaks)
    if oracle_here and not args.no_extras:
        line["extras"] = extras(torch, hb, hd, W, np, replicas, world, dev, peaks)
    if world.rank == 0:
        print(json.dumps(line), flush=True)
    replicas.shutdown(world)
    return 0


# ---------------------------------------------------------------------------------------------------
def gemm_loss_matched(torch, hb, W, B, want_dev):
    """What a co-running bf16 GEMM (8192 x 4096 x 16384, on another stream) loses while the gradient stream's buckets are
    all-reduced back to back, against the collective's bus bandwidth beside it: the copy route, and the SM-copy path under
    copy-kernel budgets of 8 to 148 CTAs (and as one kernel with roles, 8 + 40 CTAs), every one with 8-CTA sums and the default
    schedule.  `interpolated` reads the SM
    path's loss at the copy route's throughput, so that the two are compared at equal bandwidth."""
    g = W.C4_GRADIENTS
    R, S, stream = B.R, B.S, B.stream
    gs = torch.cuda.Stream()
    M, K, N = g.gemm_probe
    A = torch.randn(M, K, dtype=torch.bfloat16, device="cuda")
    Bm = torch.randn(K, N, dtype=torch.bfloat16, device="cuda")
    C = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    flops = 2.0 * M * N * K

    def corun(n_gemm, cm=None, n_bucket=0):
        with torch.cuda.stream(gs):
            for _ in range(3):
                torch.matmul(A, Bm, out=C)
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(stream)
        g0.record(gs)
        done = 0
        for i in range(n_gemm):
            with torch.cuda.stream(gs):
                torch.matmul(A, Bm, out=C)
            while cm is not None and done < (i + 1) * n_bucket // n_gemm:
                B.allreduce(cm, done % B.nsets, stream)
                done += 1
        g1.record(gs)
        c1.record(stream)
        torch.cuda.synchronize()
        return flops * n_gemm / (g0.elapsed_time(g1) / 1e3) / 1e12, c0.elapsed_time(c1) / 1e3, done

    n_gemm = 40
    alone, _, _ = corun(n_gemm)
    rows = []
    configs = [("CE_sum8", hb.PATH_CE, 8, 8, {}), ("CE_sum8_ring", hb.PATH_CE, 8, 8, {"rs_direct": 0, "ag_direct": 0}),
               ("CE_sum8_plain_graphs", hb.PATH_CE, 8, 8, {"order_kernels": 0, "ce_overlap": 0})]
    configs += [("SM_copy%d_sum8" % b, hb.PATH_SM, 8, b, {}) for b in (8, 16, 32, 40, 64, 148)]
    configs += [("SM_roles_copy40_sum8", hb.PATH_SM, 8, 40, {"roles": 1}), ("SM_copy148_sum148", hb.PATH_SM, 148, 148, {})]
    for name, path, sc, cc, extra in configs:
        cm = B.comm(path, sum_ctas=sc, copy_ctas=cc, **extra)
        time.sleep(0.5)   # the stand-alone figure must not inherit the clocks the previous row's GEMM left behind (power cap)
        t, _ = B.timed(cm, 12, 3)
        t_g = n_gemm * flops / (alone * 1e12)
        n_bucket = max(1, int(1.3 * t_g / t) + 1)
        tf, tc, done = corun(n_gemm, cm, n_bucket)
        # the bits of what ran beside the GEMM: bucket set 0 once more, compared on the device with the oracle's result
        for t_ in B.recv_sets[0]:
            t_.zero_()
        torch.cuda.synchronize()
        B.allreduce(cm, 0, stream)
        stream.synchronize()
        ok = all(bool(torch.equal(t_, want_dev)) for t_ in B.recv_sets[0])
        rows.append({"config": name, "path": "CE" if path == hb.PATH_CE else "SM", "sum_ctas": sc,
                     "copy_ctas": cc if path == hb.PATH_SM else None, "busbw_alone_GBps": S * bus_factor(R) / t / 1e9,
                     "gemm_TFLOPs_beside": tf, "gemm_loss": 1.0 - tf / alone, "busbw_beside_GBps": done * S * bus_factor(R) / tc / 1e9,
                     "matches_oracle": ok})
        cm.destroy()
    # the SM path's loss at the copy route's throughput (piecewise linear over the budget rows, by bandwidth beside the GEMM)
    sm = sorted((r["busbw_beside_GBps"], r["gemm_loss"]) for r in rows if r["config"].startswith("SM_copy") and r["sum_ctas"] == 8)
    ce = next(r for r in rows if r["config"] == "CE_sum8")
    x = ce["busbw_beside_GBps"]
    interp = None
    if sm and sm[0][0] <= x <= sm[-1][0]:
        for (x0, y0), (x1, y1) in zip(sm, sm[1:]):
            if x0 <= x <= x1:
                interp = y0 if x1 == x0 else y0 + (y1 - y0) * (x - x0) / (x1 - x0)
                break
    near = min((r for r in rows if r["config"].startswith("SM_copy") and r["sum_ctas"] == 8), key=lambda r: abs(r["busbw_beside_GBps"] - x))
    return {"workload": g.name, "gemm_probe": [M, K, N], "gemm_alone_TFLOPs": alone, "gemms_per_run": n_gemm, "rows": rows,
            "interpolated": {"at_busbw_beside_GBps": x, "copy_route_gemm_loss": ce["gemm_loss"], "sm_copy_path_gemm_loss_at_that_bandwidth": interp,
                             "nearest_sm_copy_row": {"config": near["config"], "busbw_beside_GBps": near["busbw_beside_GBps"],
                                                     "gemm_loss": near["gemm_loss"]},
                             "note": "null: the copy route's bandwidth lies outside the range the copy-kernel budgets cover; the nearest "
                                     "budget row is given beside it"}}


def large_messages(torch, hb, W, np, peaks):
    """All-reduce, reduce-scatter, all-gather and send/recv at 64 MiB, 256 MiB and 1 GiB per rank (R = 8, bf16, per-rank sizes in
    the nccl-tests convention), copy route against SM path (graphs of kernels, and the one kernel with roles).  Inputs depend on (rank, position), generated on the device; every
    row's output is compared, on the device, with what the CPU oracle computes from the same bytes."""
    from oracle import ring as oracle_ring

    R, dtype, e = 8, "bf16", 2
    stream = torch.cuda.Stream()
    thr = oracle_ring.max_threads()
    configs = [("CE_sum8", hb.PATH_CE, 8, 8, {}), ("CE_sum8_ring", hb.PATH_CE, 8, 8, {"rs_direct": 0, "ag_direct": 0}),
               ("CE_sum148", hb.PATH_CE, 148, 8, {}), ("SM_copy8_sum8", hb.PATH_SM, 8, 8, {}), ("SM_copy40_sum8", hb.PATH_SM, 8, 40, {}),
               ("SM_roles_copy40_sum8", hb.PATH_SM, 8, 40, {"roles": 1}), ("SM_copy148_sum148", hb.PATH_SM, 148, 148, {})]
    rows = []

    def bits(t):
        return t.view(torch.int16)

    for mib in (64, 256, 1024):
        S = mib * MiB
        n = S // e
        q = n // R
        send = [W.hashed_device("uniform", 4, r, n, dtype) for r in range(R)]
        recv = [torch.empty_like(s) for s in send]
        small = [torch.empty(q, dtype=send[0].dtype, device="cuda") for _ in range(R)]
        xs = [bits(s).cpu().numpy().view(np.uint16) for s in send]
        t0 = time.perf_counter()
        want_ar = oracle_ring.ring_allreduce(xs, threads=thr)[0]
        t_oracle = time.perf_counter() - t0
        want_ag = oracle_ring.allgather([x[:q] for x in xs], threads=thr)[0]
        want_p2p = oracle_ring.sendrecv(xs[2])
        d_ar = torch.from_numpy(want_ar.view(np.int16)).cuda()
        d_ag = torch.from_numpy(want_ag.view(np.int16)).cuda()
        d_p2p = torch.from_numpy(want_p2p.view(np.int16)).cuda()
        del xs, want_ar, want_ag, want_p2p
        scratch = torch.empty(hb.scratch_bytes_direct(R, n, dtype) + 256, dtype=torch.uint8, device="cuda")
        pad = (-scratch.data_ptr()) % 256
        torch.cuda.synchronize()
        for name, path, sc, cc, extra in configs:
            cm = hb.Comm(R, 0)
            cm.set_scratch(scratch.data_ptr() + pad, scratch.numel() - 256)
            cm.set_path(path)
            for k, v in dict(sum_ctas=sc, copy_ctas=cc, **extra).items():
                cm.set_param(k, v)

            def ar():
                cm.allreduce(send, recv, n, dtype, stream)

            def rs():
                cm.reduce_scatter(send, small, q, dtype, stream)

            def ag():
                cm.allgather([s[:q] for s in send], recv, q, dtype, stream)

            def p2p():
                cm.send(send[2], n, dtype, 2, 5, stream)
                cm.recv(recv[5], n, dtype, 2, 5, stream)

            def check_ar():
                return all(bool(torch.equal(bits(t), d_ar)) for t in recv)

            def check_rs():
                return all(bool(torch.equal(bits(small[r]), d_ar[r * q:(r + 1) * q])) for r in range(R))

            def check_ag():
                return all(bool(torch.equal(bits(t), d_ag)) for t in recv)

            def check_p2p():
                return bool(torch.equal(bits(recv[5]), d_p2p))

            ops = [("allreduce", ar, check_ar, ring_bytes_allreduce(S, R), bus_factor(R)),
                   ("reduce_scatter", rs, check_rs, 5.0 * S * (R - 1), (R - 1) / R),
                   ("allgather", ag, check_ag, 2.0 * S * (R - 1), (R - 1) / R)]
            if name in ("CE_sum8", "SM_copy8_sum8", "SM_copy148_sum148"):
                ops.append(("sendrecv", p2p, check_p2p, 2.0 * S, 1.0))
            for op, fn, check, ring_bytes, bf in ops:
                if op in ("allgather", "sendrecv") and name in ("CE_sum148", "SM_roles_copy40_sum8"):
                    continue                     # no sums in these: the row would repeat CE_sum8 / SM_copy40_sum8
                for t in recv + small:
                    t.zero_()
                torch.cuda.synchronize()
                fn()
                stream.synchronize()
                ok = check()
                fn()
                stream.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                reps = 3 if mib >= 1024 else 5
                e0.record(stream)
                for _ in range(reps):
                    fn()
                e1.record(stream)
                stream.synchronize()
                t = e0.elapsed_time(e1) / 1e3 / reps
                stt = cm.last_stats()
                rows.append({"op": op, "MiB_per_rank": mib, "config": name, "sum_ctas": sc if op in ("allreduce", "reduce_scatter") else None,
                             "copy_ctas": cc if path == hb.PATH_SM else None, "ms": t * 1e3, "algbw_GBps": S / t / 1e9,
                             "busbw_GBps": S * bf / t / 1e9,
                             # bytes the rank-local ring must move for this operation over the time, against 8 TB/s and the measured copy peak
                             "hbm_frac_of_8TBps": ring_bytes / t / 1e9 / NOMINAL_HBM_GBS,
                             "hbm_frac_of_measured": ring_bytes / t / 1e9 / peaks["hbm_gbs"],
                             "pieces_per_chunk": int(stt["n_pieces"]), "matches_oracle": ok})
            cm.destroy()
        rows.append({"op": "cpu_oracle_allreduce", "MiB_per_rank": mib, "ms": t_oracle * 1e3, "busbw_GBps": S * bus_factor(R) / t_oracle / 1e9,
                     "cores": thr})
        del send, recv, small, d_ar, d_ag, d_p2p, scratch
        torch.cuda.empty_cache()
    return {"R": R, "dtype": dtype, "inputs": "uniform[-1,1) hashed from (rank, position), generated on the device",
            "hbm_frac": "the ring's algorithmic bytes (all-reduce 7 S (R-1), reduce-scatter 5 S (R-1), all-gather 2 S (R-1), send/recv 2 S) over the time",
            "all_match_oracle": all(r.get("matches_oracle", True) for r in rows), "rows": rows}


def small_case(torch, hb, W, np, stream):
    """The small configuration (all-reduce over R = 4, 1,048,576 fp32 per rank, uniform[-1,1), seed 0): latency bound (its
    algorithmic bytes take 11 us at 8 TB/s), and a 4 KiB all-reduce over R = 8.  Time per call; every result is checked against
    the oracle."""
    from oracle import ring as oracle_ring
    c = W.C1_SMALL_ALLREDUCE
    out = {}
    for label, R, n, dtype, dist, seed in ((c.name, c.R, c.count, c.dtype, c.dist, c.seed), ("allreduce_r8_bf16_4KiB", 8, 2048, "bf16", "uniform", 4)):
        xs = W.rank_inputs(dist, seed, R, n, dtype)
        want = oracle_ring.ring_allreduce(xs, threads=oracle_ring.max_threads())
        e = W.elem_size(dtype)
        S1 = n * e
        sets = 8      # buffers in rotation (larger than L2 for the 4 MiB case)
        view = (lambda x: x) if dtype == "fp32" else (lambda x: x.view(np.int16))
        send = [[torch.from_numpy(view(x)).cuda() for x in xs] for _ in range(sets)]
        recv = [[torch.zeros_like(s) for s in send[0]] for _ in range(sets)]
        nb = hb.scratch_bytes_direct(R, n, dtype)
        scratch = torch.empty(nb + 256, dtype=torch.uint8, device="cuda")
        rows = {}
        for name, path, params in (
                ("CE_sum8", hb.PATH_CE, {}),                                            # defaults: small-message rule, automatic schedule
                ("CE_sum8_driver_copies", hb.PATH_CE, {"ce_small_bytes": 0}),
                ("CE_sum8_driver_copies_ring", hb.PATH_CE, {"ce_small_bytes": 0, "rs_direct": 0, "ag_direct": 0}),
                ("SM_8", hb.PATH_SM, {"copy_ctas": 8}), ("SM_8_ring", hb.PATH_SM, {"copy_ctas": 8, "rs_direct": 0, "ag_direct": 0}),
                ("SM_148", hb.PATH_SM, {"sum_ctas": 148, "copy_ctas": 148}),
                ("SM_148_ring", hb.PATH_SM, {"sum_ctas": 148, "copy_ctas": 148, "rs_direct": 0, "ag_direct": 0}),
                ("SM_148_ring_one_kernel", hb.PATH_SM, {"sum_ctas": 148, "copy_ctas": 148, "fused": 1})):
            cm = hb.Comm(R, 0)
            cm.set_scratch(scratch.data_ptr() + (-scratch.data_ptr()) % 256, nb)
            cm.set_path(path)
            for key, v in params.items():
                cm.set_param(key, v)
            for b in range(sets):
                cm.allreduce(send[b], recv[b], n, dtype, stream)
            stream.synchronize()
            ok = all(bool((recv[0][r].cpu().numpy().view(np.uint8) == want[r].view(np.uint8)).all()) for r in range(R))
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = 200
            e0.record(stream)
            for i in range(reps):
                cm.allreduce(send[i % sets], recv[i % sets], n, dtype, stream)
            e1.record(stream)
            stream.synchronize()
            t = e0.elapsed_time(e1) / 1e3 / reps
            stt = cm.last_stats()
            rows[name] = {"us_per_call": t * 1e6, "busbw_GBps": S1 * 2 * (R - 1) / R / t / 1e9,
                          "hbm_frac_of_8TBps": 7.0 * S1 * (R - 1) / t / 1e9 / NOMINAL_HBM_GBS, "sum_launches": int(stt["n_sum_launches"]),
                          "copy_kernel_launches": int(stt["n_move_launches"]), "matches_oracle": ok}
            cm.destroy()
        thr = oracle_ring.max_threads()
        t0 = time.perf_counter()
        reps = 0
        while reps < 5 or (time.perf_counter() - t0 < 0.5 and reps < 200):
            oracle_ring.ring_allreduce(xs, threads=thr)
            reps += 1
        t_cpu = (time.perf_counter() - t0) / reps
        rows["cpu_oracle"] = {"us_per_call": t_cpu * 1e6, "busbw_GBps": S1 * 2 * (R - 1) / R / t_cpu / 1e9, "cores": thr}
        out[label] = rows
        del send, recv, scratch
    return out


def extras(torch, hb, hd, W, np, replicas, world, dev, peaks):
    """Context lines on the 25 MiB gradient bucket (R = 8, bf16, reduce-scatter + all-gather as two calls): schedules, paths and
    CTA budgets, comparison points, whether a move needs an SM, send/recv, the proxy, and the small configurations."""
    from oracle import ring as oracle_ring

    out = {}
    c = W.C2_DP_BUCKET
    R, n, dtype = c.R, c.count, c.dtype
    S = n * 2
    xs = W.rank_inputs(c.dist, c.seed, R, n, dtype, c.sigma)
    want = oracle_ring.ring_allreduce(xs, threads=oracle_ring.max_threads())
    want_dev = torch.from_numpy(want[0].view(np.int16)).cuda()
    B = Bench(torch, hb, replicas, world, dev, R, n, 4, first_set_host=xs)
    stream = B.stream
    step = B.two_calls
    k, w = 40, 5
    hbm = ring_bytes_allreduce(S, R)

    def bits_ok(cm, fn):
        for t in B.recv_sets[0]:
            t.zero_()
        torch.cuda.synchronize()
        fn(cm, 0, stream)
        stream.synchronize()
        return all(bool(torch.equal(t, want_dev)) for t in B.recv_sets[0])

    def row(cm, fn=step, own_bytes=None, **tags):
        t, _ = B.timed(cm, k, w, fn=fn)
        r = dict(tags)
        r.update({"ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9, "hbm_frac_of_8TBps": hbm / t / 1e9 / NOMINAL_HBM_GBS,
                  "matches_oracle": bits_ok(cm, fn)})
        if own_bytes:
            r["bytes_this_schedule_moves"] = own_bytes
        return r

    # ---- schedules x paths x budgets (default = automatic direct schedule; ring = rs_direct 0, ag_direct 0)
    sched = []
    for name, path, sc, cc in (("CE", hb.PATH_CE, 8, 8), ("CE", hb.PATH_CE, 32, 8), ("CE", hb.PATH_CE, 148, 8), ("SM", hb.PATH_SM, 8, 8),
                               ("SM", hb.PATH_SM, 8, 32), ("SM", hb.PATH_SM, 8, 48), ("SM", hb.PATH_SM, 148, 148)):
        for label, extra in (("direct", {}), ("ring", {"rs_direct": 0, "ag_direct": 0}), ("ring_direct_allgather", {"rs_direct": 0, "ag_direct": 1})):
            cm = B.comm(path, sum_ctas=sc, copy_ctas=cc, **extra)
            r = row(cm, path=name, sum_ctas=sc, copy_ctas=cc if path == hb.PATH_SM else None, schedule=label)
            # the sums are in the first of the two calls: its statistics, not the all-gather's
            cnt = B.n // R
            rs_out = [B.recv_sets[0][q].data_ptr() + q * cnt * B.e for q in range(R)]
            cm.reduce_scatter(B.send_sets[0], rs_out, cnt, B.dtype, stream)
            stream.synchronize()
            r["sum_launches_per_step"] = int(cm.last_stats()["n_sum_launches"])
            sched.append(r)
            cm.destroy()
    out["c2_dp_bucket"] = {"workload": c.name, "step": "hoccl_reduce_scatter + hoccl_allgather on one 25 MiB bucket", "rows": sched}

    def one_call(c_, b, st):
        c_.allreduce(B.send_sets[b], B.recv_sets[b], n, dtype, st)

    cm = B.comm(hb.PATH_CE, sum_ctas=8)
    out["single_call_allreduce"] = row(cm, fn=one_call)
    # the copy-route graphs without their empty ordering kernels (parameter "order_kernels" = 0): the comparison point
    pg = []
    for sc in (8, 148):
        c1 = B.comm(hb.PATH_CE, sum_ctas=sc, order_kernels=0, rs_direct=0, ag_direct=0)
        pg.append(row(c1, path="CE", sum_ctas=sc, schedule="ring"))
        c1.destroy()
    out["plain_graphs_no_order_kernels"] = pg
    # comparison points that are not rank local: the whole reduction in one kernel; sum-and-forward
    op_rows = []
    for ctas in (8, 32, 148):
        c1 = B.comm(hb.PATH_CE, sum_ctas=ctas, onepass=1, rs_direct=0, ag_direct=0)
        op_rows.append(row(c1, fn=one_call, ctas=ctas, own_bytes=2.0 * R * S))
        c1.destroy()
    out["onepass_allreduce"] = op_rows
    fw_rows = []
    for name, path, sc, cc in (("CE", hb.PATH_CE, 8, 8), ("SM", hb.PATH_SM, 8, 8), ("SM", hb.PATH_SM, 148, 148)):
        c1 = B.comm(path, sum_ctas=sc, copy_ctas=cc, forward=1)
        fw_rows.append(row(c1, path=name, sum_ctas=sc))
        c1.destroy()
    out["forward_variant"] = fw_rows
    # SM path with the whole ring as one cooperative kernel (grid barriers instead of kernel boundaries)
    fu_rows = []
    for ctas in (8, 148):
        c1 = B.comm(hb.PATH_SM, sum_ctas=ctas, copy_ctas=ctas, fused=1)
        r = row(c1, fn=one_call, ctas=ctas)
        r["async_error"] = int(c1.async_error())
        fu_rows.append(r)
        c1.destroy()
    out["fused_ring_kernel_SM_path"] = fu_rows
    # the one route on a single device that really uses no SM for moves: bounce through pinned host memory
    host_stage = torch.empty(400 << 20, dtype=torch.uint8).pin_memory()
    c1 = B.comm(hb.PATH_CE_HOST, sum_ctas=8, rs_direct=0)
    c1.set_host_staging(host_stage)
    t, _ = B.timed(c1, 6, 3, fn=step)
    out["host_bounce_path"] = {"ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9, "matches_oracle": bits_ok(c1, step),
                               "schedule": "ring reduce-scatter, direct all-gather (a final chunk goes out to the host once and comes back R-1 times)",
                               "pcie_bytes_per_step_outbound": 1.0 * S * (R - 1) + 1.0 * S, "pcie_bytes_per_step_inbound": 2.0 * S * (R - 1)}
    c1.destroy()
    # handshake mode (CPU proxy + stream memory operations) on the SM path, against the same path launched directly, and how
    # busy the proxy thread was (the analogue of the paper's CPU slack)
    hs = {}
    for label, flag in (("direct_launch", 0), ("handshake", 1)):
        c1 = B.comm(hb.PATH_SM, sum_ctas=8, copy_ctas=32, handshake=flag)
        for b in range(B.nsets):
            step(c1, b, stream)
        stream.synchronize()
        h0 = 0
        if flag:
            c1.proxy_stats(reset=True)
            h0 = c1.handshakes()
        t, _ = B.timed(c1, k, 0, fn=step)
        hs[label] = {"ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9}
        if flag:
            busy, span = c1.proxy_stats()
            served = c1.handshakes() - h0
            hs[label].update({"handovers": served, "proxy_busy_us_per_handover": busy / max(1, served), "proxy_span_us": span,
                              "proxy_busy_us": busy, "proxy_slack": 1.0 - busy / span if span > 0 else None,
                              "matches_oracle": bits_ok(c1, step)})
        c1.destroy()
    out["handshake_mode_SM_copy32_sum8"] = hs
    # stream executor (events) instead of graph replay
    cm.set_param("use_graph", 0)
    t, _ = B.timed(cm, k, w, fn=step)
    out["stream_executor"] = {"ms_per_step": t * 1e3, "busbw_GBps": S * bus_factor(R) / t / 1e9,
                              "host_launch_us_per_call": cm.last_stats()["host_launch_us"]}
    cm.set_param("use_graph", 1)

    # does a move need an SM?  (bounded occupancy kernel + one 64 MiB move)
    src = B.send_sets[0][0]
    dst = B.recv_sets[0][0]
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
        one_call(cm, 0, stream)
        stream.synchronize()
        vals = []
        for _ in range(15):
            one_call(cm, 0, stream)
            vals.append(cm.last_stats()["host_launch_us"])
            stream.synchronize()
        vals.sort()
        host_us[label] = vals[len(vals) // 2]
    cm.set_param("use_graph", 1)
    out["host_launch_us_per_allreduce_call_idle_queue"] = host_us

    # point to point: 64 MiB bf16 activations [4, 2048, 4096], one message at a time and the pipeline wave (8 stages x 16 microbatches)
    act = torch.empty(4 * 2048 * 4096, dtype=torch.bfloat16, device="cuda").normal_(0, 1)
    slots = [torch.empty_like(act) for _ in range(4)]
    p2p = {}
    for name, path in (("CE", hb.PATH_CE), ("SM8", hb.PATH_SM)):
        cm.set_path(path)
        cm.set_param("copy_ctas", 8)

        def hop(c_, b, st):
            c_.send(act, act.numel(), "bf16", 0, 1, st)
            c_.recv(slots[b], act.numel(), "bf16", 0, 1, st)

        t, _ = B.timed(cm, 20, 3, fn=hop)
        p2p[name] = {"us_per_message": t * 1e6, "algbw_GBps": act.numel() * 2 / t / 1e9,
                     "hbm_frac_of_8TBps": 2 * act.numel() * 2 / t / 1e9 / NOMINAL_HBM_GBS, "delivered_bit_exact": bool(torch.equal(slots[0], act))}
    out["p2p_64MiB"] = p2p
    cm.set_path(hb.PATH_CE)
    cm.destroy()
    del act, slots
    B.free()
    out["pipeline_wave"] = pipeline_wave(torch, hb, W)
    out["small_messages"] = small_case(torch, hb, W, np, stream)
    # the paper's own figures, as context only (other hardware, real multi-GPU links, no reduction on its path)
    out["paper_context"] = {
        "hardware": "32 x NVIDIA H800 80 GB (132 SMs each), 8 per node on NVLink, one 50 GB/s NIC per GPU",
        "communication_performance": "within 3 % of the state of the art on average (point-to-point, all-gather, all-to-all, 2 MB to 1 GB)",
        "sms_freed": "about 10 % of the SMs (pipeline- plus data-parallel traffic of a GPT-6.7B run)",
        "end_to_end_training_gain": "up to 5 % (2.4 % at 6.7B, 5.1 % at 32B parameters) over the SM-driven library",
        "allgather_8_gpus_1GB_algbw_GBps": 192.2, "intra_node_p2p_1GB_algbw_GBps": 192.2, "alltoall_8_gpus_1GB_algbw_GBps": 191.4,
        "reductions": "outside the paper's scope (they fall back to the SM-driven library there): no all-reduce figure exists to compare with",
    }
    return out


def pipeline_wave(torch, hb, W):
    """Pipeline-parallel send/recv: bf16 activations [4, 2048, 4096] (64 MiB) forwarded stage to stage across 8 logical stages,
    16 microbatches (112 hops), every stage on its own stream, alone and beside a 4096^3 bf16 GEMM on another stream."""
    c = W.C3_PIPELINE
    n, S, M = c.count, c.count * 2, c.microbatches
    stream, gs = torch.cuda.Stream(), torch.cuda.Stream()
    slots = [[torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(M)] for _ in range(c.stages)]
    for m in range(M):
        slots[0][m].normal_(0, 1)
    A = torch.randn(4096, 4096, dtype=torch.bfloat16, device="cuda")
    Bm = torch.randn(4096, 4096, dtype=torch.bfloat16, device="cuda")
    C = torch.empty(4096, 4096, dtype=torch.bfloat16, device="cuda")
    flops = 2.0 * 4096 ** 3
    stage_streams = [torch.cuda.Stream() for _ in range(c.stages)]
    hops = (c.stages - 1) * M

    def wave(comm):
        for m in range(M):
            for s in range(c.stages - 1):
                comm.send(slots[s][m], n, "bf16", s, s + 1, stage_streams[s])
                comm.recv(slots[s + 1][m], n, "bf16", s, s + 1, stage_streams[s + 1])

    def fork():
        ev = torch.cuda.Event()
        ev.record(stream)
        for st in stage_streams:
            st.wait_event(ev)

    def join():
        for st in stage_streams:
            ev = torch.cuda.Event()
            ev.record(st)
            stream.wait_event(ev)

    n_gemm = 150
    torch.cuda.synchronize()
    with torch.cuda.stream(gs):
        for _ in range(10):
            torch.matmul(A, Bm, out=C)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(gs)
        for _ in range(n_gemm):
            torch.matmul(A, Bm, out=C)
        g1.record(gs)
    torch.cuda.synchronize()
    alone = flops * n_gemm / (g0.elapsed_time(g1) / 1e3) / 1e12
    rows = []
    for name, path, cc in (("CE", hb.PATH_CE, 8), ("SM8", hb.PATH_SM, 8), ("SM32", hb.PATH_SM, 32), ("SMall", hb.PATH_SM, 148)):
        comm = hb.Comm(c.stages, 0)
        comm.set_path(path)
        comm.set_param("copy_ctas", cc)
        wave(comm)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        fork()
        wave(comm)
        join()
        e1.record(stream)
        torch.cuda.synchronize()
        t = e0.elapsed_time(e1) / 1e3
        waves = max(1, int(1.3 * n_gemm * flops / (alone * 1e12) / t) + 1)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(stream)
        fork()
        g0.record(gs)
        done = 0
        for i in range(n_gemm):
            with torch.cuda.stream(gs):
                torch.matmul(A, Bm, out=C)
            while done < (i + 1) * waves // n_gemm:
                wave(comm)
                done += 1
        g1.record(gs)
        join()
        c1.record(stream)
        torch.cuda.synchronize()
        tf = flops * n_gemm / (g0.elapsed_time(g1) / 1e3) / 1e12
        tc = c0.elapsed_time(c1) / 1e3
        ok = all(bool(torch.equal(slots[c.stages - 1][m], slots[0][m])) for m in range(M))
        rows.append({"config": name, "copy_ctas": cc if path == hb.PATH_SM else None, "wave_ms": t * 1e3, "algbw_GBps": hops * S / t / 1e9,
                     "hbm_frac_of_8TBps": 2.0 * hops * S / t / 1e9 / NOMINAL_HBM_GBS, "gemm_TFLOPs_beside": tf, "gemm_loss": 1 - tf / alone,
                     "algbw_beside_GBps": done * hops * S / tc / 1e9 if done else 0.0, "delivered_bit_exact": ok})
        comm.destroy()
    return {"workload": c.name, "hops": hops, "message_MiB": S >> 20, "gemm_alone_TFLOPs": alone, "rows": rows}


if __name__ == "__main__":
    sys.exit(main())
