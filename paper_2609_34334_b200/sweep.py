"""Message-size sweep of every operation on both paths (the fifth benchmark configuration) and the
pipeline / gradient-stream workloads (third and fourth), through the C ABI.

    python -m paper_2609_34334_b200.sweep sizes   [--min-log2 12 --max-log2 30 --ranks 2,4,8 --dtypes bf16 --ops all --out FILE]
    python -m paper_2609_34334_b200.sweep pipeline [--microbatches 16]
    python -m paper_2609_34334_b200.sweep gradients [--buckets 32] [--budgets 1,2,4,8,16,32,64]
    python -m paper_2609_34334_b200.sweep launch-cost
    python -m paper_2609_34334_b200.sweep alltoallv [--mib 4,64,256] [--model 4,2]

Sizes are per-rank buffer bytes S in the nccl-tests convention (all-reduce: send = recv = S; reduce-scatter:
send = S; all-gather: recv = S; all-to-all: send = recv = S; send/recv: S), like the sweeps the paper reports (Sec. 5 "Communication
benchmarks").  Timing: CUDA events around back-to-back calls on one stream after warm-up, buffers rotated
when the working set is smaller than L2.  Prints one JSON object per line.
"""
from __future__ import annotations

import argparse
import json
import sys
import time

import torch

from . import binding as hb
from . import workloads as W

NOMINAL_HBM = 8.0e12
L2_BYTES = 126 << 20


def _hbm_bytes(op, S, R):
    """Algorithmic HBM bytes of the rank-local ring on one device: S(R-1) wire bytes in total over all ranks per
    phase; a MOVE reads and writes each (2 B), a SUM reads two and writes one (3 B)."""
    return {"allreduce": 7.0 * S * (R - 1), "reduce_scatter": 5.0 * S * (R - 1), "allgather": 2.0 * S * (R - 1) + 2.0 * S,
            "alltoall": 2.0 * S * R, "sendrecv": 2.0 * S}[op]


def _bus_factor(op, R):
    return {"allreduce": 2.0 * (R - 1) / R, "reduce_scatter": (R - 1) / R, "allgather": (R - 1) / R, "alltoall": (R - 1) / R,
            "sendrecv": 1.0}[op]


class Arena:
    """Per-rank device buffers for one operation, several rotating sets when small."""

    def __init__(self, op, R, S, dtype, nsets):
        e = W.elem_size(dtype)
        tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
        self.op, self.R, self.S, self.dtype, self.e = op, R, S, dtype, e
        n = S // e
        if op == "allreduce":
            self.count, send_n, recv_n = n, n, n
        elif op == "reduce_scatter":
            self.count, send_n, recv_n = n // R, n, n // R
        elif op == "allgather":
            self.count, send_n, recv_n = n // R, n // R, n
        elif op == "alltoall":
            self.count, send_n, recv_n = n // R, n, n
        else:
            self.count, send_n, recv_n = n, n, n
        ranks = R if op != "sendrecv" else 1
        self.sets = []
        for _ in range(nsets):
            send = [torch.empty(max(send_n, 1), dtype=tdt, device="cuda").normal_(0, 1e-3) for _ in range(ranks)]
            recv = [torch.zeros(max(recv_n, 1), dtype=tdt, device="cuda") for _ in range(ranks)]
            self.sets.append((send, recv))

    def call(self, comm, k, stream):
        send, recv = self.sets[k % len(self.sets)]
        if self.op == "allreduce":
            comm.allreduce(send, recv, self.count, self.dtype, stream)
        elif self.op == "reduce_scatter":
            comm.reduce_scatter(send, recv, self.count, self.dtype, stream)
        elif self.op == "allgather":
            comm.allgather(send, recv, self.count, self.dtype, stream)
        elif self.op == "alltoall":
            comm.alltoall(send, recv, self.count, self.dtype, stream)
        else:
            comm.send(send[0], self.count, self.dtype, 0, 1, stream)
            comm.recv(recv[0], self.count, self.dtype, 0, 1, stream)


def time_op(comm, arena, stream, min_window_s=0.01, max_iters=200):
    nsets = len(arena.sets)
    for k in range(max(3, nsets)):
        arena.call(comm, k, stream)
    stream.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    arena.call(comm, 0, stream)
    e1.record(stream)
    stream.synchronize()
    one = max(e0.elapsed_time(e1) / 1e3, 1e-6)
    iters = int(min(max_iters, max(3, min_window_s / one)))
    e0.record(stream)
    for k in range(iters):
        arena.call(comm, k, stream)
    e1.record(stream)
    stream.synchronize()
    return e0.elapsed_time(e1) / 1e3 / iters


def sweep_sizes(args):
    torch.cuda.set_device(0)
    stream = torch.cuda.Stream()
    ops = ["allreduce", "reduce_scatter", "allgather", "alltoall", "sendrecv"] if args.ops == "all" else args.ops.split(",")
    # name -> (path, SUM CTAs, copy CTAs, further parameters).  Default schedule unless "ring" is in the name.
    ring = {"rs_direct": 0, "ag_direct": 0}
    table = {
        "CE": (hb.PATH_CE, 8, 8, {}),                                   # copy route as a new communicator has it
        "CEring": (hb.PATH_CE, 8, 8, dict(ring)),                       # the ring step by step
        "CEdriver": (hb.PATH_CE, 8, 8, {"ce_small_bytes": 0}),          # driver copies at every size (no small-message rule)
        "CEonegraph": (hb.PATH_CE, 8, 8, {"ce_overlap": 0}),            # the direct schedule as one graph (no overlap of copies and sums)
        "CEplain": (hb.PATH_CE, 8, 8, {"order_kernels": 0, "ce_overlap": 0}),   # plain graphs: no empty ordering kernels
        "CEall": (hb.PATH_CE, 148, 8, {}),                              # copy route with whole-GPU sums
        "SM8": (hb.PATH_SM, 8, 8, {}), "SM8ring": (hb.PATH_SM, 8, 8, dict(ring)),
        "SM40": (hb.PATH_SM, 8, 40, {}),                                # 8-CTA sums beside 40 copy CTAs
        "SMroles40": (hb.PATH_SM, 8, 40, {"roles": 1}),                 # the same as one cooperative kernel with roles
        "SMall": (hb.PATH_SM, 148, 148, {}), "SMallring": (hb.PATH_SM, 148, 148, dict(ring)),
        "SMallfused": (hb.PATH_SM, 148, 148, {"fused": 1}),             # the ring as one cooperative kernel
        "SM8fused": (hb.PATH_SM, 8, 8, {"fused": 1}),
    }
    names = ["CE", "SM8", "SMall"] if args.configs == "all" else args.configs.split(",")
    configs = [(nm,) + table[nm] for nm in names]
    out = open(args.out, "w") if args.out else None
    for dtype in args.dtypes.split(","):
        for R in [int(r) for r in args.ranks.split(",")]:
            for lg in range(args.min_log2, args.max_log2 + 1):
                S = 1 << lg
                e = W.elem_size(dtype)
                if S // e < R:
                    continue
                for op in ops:
                    if op == "sendrecv" and R != 2:
                        continue            # point to point does not depend on R
                    ranks = R if op != "sendrecv" else 1
                    footprint = 2 * ranks * S
                    nsets = 1 if footprint > 2 * L2_BYTES else int(min(8, max(2, (3 * L2_BYTES) // max(footprint, 1))))
                    if footprint * nsets > (48 << 30):
                        nsets = 1
                    arena = Arena(op, R, S, dtype, nsets)
                    scratch = torch.empty(hb.scratch_bytes_direct(R, S // e, dtype) + 256, dtype=torch.uint8, device="cuda")
                    pad = (-scratch.data_ptr()) % 256
                    for name, path, sc, cc, extra in configs:
                        comm = hb.Comm(R, 0)
                        if scratch.numel() > 256:
                            comm.set_scratch(scratch.data_ptr() + pad, scratch.numel() - 256)
                        comm.set_path(path)
                        comm.set_param("sum_ctas", sc)
                        comm.set_param("copy_ctas", cc)
                        for k_, v_ in extra.items():
                            comm.set_param(k_, v_)
                        t = time_op(comm, arena, stream)
                        row = {"op": op, "R": R, "dtype": dtype, "S": S, "config": name, "sum_ctas": sc,
                               "copy_ctas": cc if path == hb.PATH_SM else None, "us": t * 1e6, "algbw_GBps": S / t / 1e9,
                               "busbw_GBps": S * _bus_factor(op, R) / t / 1e9,
                               # the bytes the rank-local RING must move for this operation, over the time
                               "hbm_frac_of_8TBps": _hbm_bytes(op, S, R) / t / NOMINAL_HBM, "buffer_sets": nsets,
                               "pieces": int(comm.last_stats()["n_pieces"])}
                        line = json.dumps(row)
                        print(line, flush=True)
                        if out:
                            out.write(line + "\n")
                        comm.destroy()
                    del arena, scratch
                    torch.cuda.empty_cache()
    if out:
        out.close()


def pipeline(args):
    """Stage-to-stage forwarding of bf16 activations [4, 2048, 4096] over 8 logical stages while a 4096^3 bf16
    GEMM probe loops on another stream (the third benchmark configuration; forward wave only)."""
    torch.cuda.set_device(0)
    c = W.C3_PIPELINE
    n, S = c.count, c.count * 2
    M = args.microbatches
    stream, gs = torch.cuda.Stream(), torch.cuda.Stream()
    slots = [[torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(M)] for _ in range(c.stages)]
    for m in range(M):
        slots[0][m].normal_(0, 1)
    A = torch.randn(4096, 4096, dtype=torch.bfloat16, device="cuda")
    B = torch.randn(4096, 4096, dtype=torch.bfloat16, device="cuda")
    C = torch.empty(4096, 4096, dtype=torch.bfloat16, device="cuda")
    flops = 2.0 * 4096 ** 3

    stage_streams = [torch.cuda.Stream() for _ in range(c.stages)]

    def wave(comm):
        # every stage posts on its own stream: the send of hop s -> s+1 on stage s's stream, the matching recv on
        # stage s+1's stream; hop (m, s) follows hop (m, s-1) through the order of stage s's stream
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

    def gemm_alone(n_gemm=200):
        with torch.cuda.stream(gs):
            for _ in range(10):
                torch.matmul(A, B, out=C)
            g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            g0.record(gs)
            for _ in range(n_gemm):
                torch.matmul(A, B, out=C)
            g1.record(gs)
        torch.cuda.synchronize()
        return flops * n_gemm / (g0.elapsed_time(g1) / 1e3) / 1e12

    alone = gemm_alone()
    print(json.dumps({"workload": c.name, "gemm_alone_TFLOPs": alone}), flush=True)
    for name, path, cc, split in (("CE", hb.PATH_CE, 8, 1), ("SM8", hb.PATH_SM, 8, 1),
                                  ("SM32", hb.PATH_SM, 32, 1), ("SMall", hb.PATH_SM, 148, 1)):
        comm = hb.Comm(c.stages, 0)
        comm.set_path(path)
        comm.set_param("copy_ctas", cc)
        comm.set_param("p2p_split", split)
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
        hops = (c.stages - 1) * M
        # beside the GEMM probe: keep waves going while 200 GEMMs run
        n_gemm = 200
        waves = max(1, int(1.3 * n_gemm * flops / (alone * 1e12) / t) + 1)
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(stream)
        fork()
        g0.record(gs)
        done = 0
        for i in range(n_gemm):
            with torch.cuda.stream(gs):
                torch.matmul(A, B, out=C)
            while done < (i + 1) * waves // n_gemm:
                wave(comm)
                done += 1
        g1.record(gs)
        join()
        c1.record(stream)
        torch.cuda.synchronize()
        tf = flops * n_gemm / (g0.elapsed_time(g1) / 1e3) / 1e12
        tc = c0.elapsed_time(c1) / 1e3
        ok = all(torch.equal(slots[c.stages - 1][m], slots[0][m]) for m in range(M))
        print(json.dumps({"workload": c.name, "config": name, "copy_ctas": cc if path == hb.PATH_SM else None, "hops": hops,
                          "message_MiB": S >> 20, "wave_ms": t * 1e3, "algbw_GBps": hops * S / t / 1e9,
                          "hbm_frac_of_8TBps": 2.0 * hops * S / t / NOMINAL_HBM, "gemm_TFLOPs_beside": tf,
                          "gemm_loss": 1 - tf / alone, "algbw_beside_GBps": done * hops * S / tc / 1e9 if done else 0.0,
                          "delivered_bit_exact": ok}), flush=True)
        comm.destroy()


def gradients(args):
    """GPT-6.7B shaped data-parallel all-reduce: 40 MiB bf16 buckets over R = 8 back to back, beside an
    8192 x 4096 x 16384 bf16 GEMM probe (the fourth benchmark configuration).  A window of `--buckets` buckets is
    timed (the full stream is 307 buckets + one of 8 MiB; every bucket is the same work)."""
    torch.cuda.set_device(0)
    g = W.C4_GRADIENTS
    R, dtype = g.R, g.dtype
    sizes = g.buckets()
    per = sizes[0]
    S = per * 2
    nb = min(args.buckets, len(sizes))
    stream, gs = torch.cuda.Stream(), torch.cuda.Stream()
    pool = 3     # reusable per-rank bucket buffers
    send = [[torch.empty(per, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3) for _ in range(R)] for _ in range(pool)]
    recv = [[torch.empty(per, dtype=torch.bfloat16, device="cuda") for _ in range(R)] for _ in range(pool)]
    scratch = torch.empty(hb.scratch_bytes_direct(R, per, dtype) + 256, dtype=torch.uint8, device="cuda")
    pad = (-scratch.data_ptr()) % 256
    M, K, N = g.gemm_probe
    A = torch.randn(M, K, dtype=torch.bfloat16, device="cuda")
    B = torch.randn(K, N, dtype=torch.bfloat16, device="cuda")
    C = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    flops = 2.0 * M * N * K

    def gemm_tflops(n_gemm, comm=None, n_bucket=0):
        with torch.cuda.stream(gs):
            for _ in range(3):
                torch.matmul(A, B, out=C)
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record(stream)
        g0.record(gs)
        done = 0
        for i in range(n_gemm):
            with torch.cuda.stream(gs):
                torch.matmul(A, B, out=C)
            while comm is not None and done < (i + 1) * n_bucket // n_gemm:
                comm.allreduce(send[done % pool], recv[done % pool], per, dtype, stream)
                done += 1
        g1.record(gs)
        c1.record(stream)
        torch.cuda.synchronize()
        return flops * n_gemm / (g0.elapsed_time(g1) / 1e3) / 1e12, c0.elapsed_time(c1) / 1e3, done

    alone, _, _ = gemm_tflops(40)
    print(json.dumps({"workload": g.name, "buckets_total": len(sizes), "bucket_MiB": S >> 20, "last_bucket_MiB": sizes[-1] * 2 >> 20,
                      "gemm_probe": [M, K, N], "gemm_alone_TFLOPs": alone}), flush=True)
    configs = [("CE_sum8", hb.PATH_CE, 8, 8), ("CE_sum8_plain_graphs", hb.PATH_CE, 8, 8), ("SM_copy8_sum8", hb.PATH_SM, 8, 8),
               ("SM_copy32_sum8", hb.PATH_SM, 8, 32), ("SM_copy148_sum148", hb.PATH_SM, 148, 148)]
    if getattr(args, "budgets", ""):
        # the copy-route path, then the SM-copy path under every CTA budget (SUM budget: the same, at most 8), then the whole GPU
        configs = [("CE_sum8", hb.PATH_CE, 8, 8), ("CE_sum8_plain_graphs", hb.PATH_CE, 8, 8)]
        for b in [int(x) for x in args.budgets.split(",")]:
            configs.append(("SM_copy%d_sum%d" % (b, min(b, 8)), hb.PATH_SM, min(b, 8), b))
        configs.append(("SM_copy148_sum148", hb.PATH_SM, 148, 148))
    if getattr(args, "ring", False):   # every configuration once more on the ring schedule, step by step
        configs = configs + [(n_ + "_ring", p_, s_, c_) for n_, p_, s_, c_ in configs if not n_.endswith("_plain_graphs")]
    for name, path, sc, cc in configs:
        comm = hb.Comm(R, 0)
        comm.set_scratch(scratch.data_ptr() + pad, scratch.numel() - 256)
        comm.set_path(path)
        comm.set_param("sum_ctas", sc)
        comm.set_param("copy_ctas", cc)
        if name.endswith("_ring"):
            comm.set_param("ag_direct", 0)
            comm.set_param("rs_direct", 0)
        comm.set_param("order_kernels", 0 if name.endswith("_plain_graphs") else 1)   # the copy-route graphs without ordering kernels
        for k in range(pool):
            comm.allreduce(send[k], recv[k], per, dtype, stream)
        stream.synchronize()
        # the stand-alone figure must not inherit the clocks the previous configuration's GEMM left behind (power cap)
        time.sleep(0.5)
        for k in range(pool):
            comm.allreduce(send[k], recv[k], per, dtype, stream)
        stream.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for k in range(nb):
            comm.allreduce(send[k % pool], recv[k % pool], per, dtype, stream)
        e1.record(stream)
        stream.synchronize()
        t = e0.elapsed_time(e1) / 1e3 / nb
        n_gemm = 40
        t_g = n_gemm * flops / (alone * 1e12)
        n_bucket = max(1, int(1.3 * t_g / t) + 1)
        tf, tc, done = gemm_tflops(n_gemm, comm, n_bucket)
        print(json.dumps({"workload": g.name, "config": name, "ms_per_bucket": t * 1e3, "busbw_GBps": S * 2 * (R - 1) / R / t / 1e9,
                          "hbm_frac_of_8TBps": 7.0 * S * (R - 1) / t / NOMINAL_HBM,
                          "full_stream_ms_estimate": t * 1e3 * (len(sizes) - 1 + sizes[-1] / per),
                          "gemm_TFLOPs_beside": tf, "gemm_loss": 1 - tf / alone,
                          "busbw_beside_GBps": done * S * 2 * (R - 1) / R / tc / 1e9}), flush=True)
        comm.destroy()


def launch_cost(args):
    """Host time of one all-reduce call against the number of operations it issues (the paper's CPU launch overhead
    axis, Sec. 5): R = 8, 64 MiB bf16 per rank, chunks cut into 1..64 pieces, stream executor against graph replay, with
    an idle queue (the stream is synchronised after every call)."""
    torch.cuda.set_device(0)
    R, dtype = 8, "bf16"
    n = (64 << 20) // 2
    stream = torch.cuda.Stream()
    send = [torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3) for _ in range(R)]
    recv = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(R)]
    scratch = torch.empty(hb.scratch_bytes(R, n, dtype) + 256, dtype=torch.uint8, device="cuda")
    pad = (-scratch.data_ptr()) % 256
    chunk = n * 2 // R
    for path_name, path in (("CE", hb.PATH_CE), ("SM", hb.PATH_SM)):
        for pieces in (1, 2, 4, 8, 16, 32, 64):
            for label, use_graph in (("stream_executor", 0), ("graph_replay", 1)):
                comm = hb.Comm(R, 0)
                comm.set_scratch(scratch.data_ptr() + pad, scratch.numel() - 256)
                comm.set_path(path)
                comm.set_param("use_graph", use_graph)
                comm.set_param("max_pieces", pieces)
                comm.set_param("piece_bytes", max(1024, chunk // pieces))
                vals, dev = [], []
                for k in range(12):
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record(stream)
                    comm.allreduce(send, recv, n, dtype, stream)
                    e1.record(stream)
                    st = comm.last_stats()
                    stream.synchronize()
                    if k >= 2:
                        vals.append(st["host_launch_us"])
                        dev.append(e0.elapsed_time(e1) * 1e3)
                vals.sort()
                dev.sort()
                print(json.dumps({"path": path_name, "executor": label, "pieces_per_chunk": int(st["n_pieces"]),
                                  "operations": int(st["n_moves"] + st["n_sum_launches"]), "moves": int(st["n_moves"]),
                                  "sum_launches": int(st["n_sum_launches"]), "host_us_per_call_median": vals[len(vals) // 2],
                                  "device_us_per_call_median": dev[len(dev) // 2]}), flush=True)
                comm.destroy()


def alltoallv(args):
    """User-defined pattern (the paper's collective scheduler, Sec. 3.4, driving hoccl_alltoallv): an expert-parallel
    dispatch where every rank sends S bytes in total, split over the destinations either uniformly or with a skew
    (destination weights 1/(1+k) in a per-source random order, seeded).  Time per call on both paths, host time
    per call, and the schedule's stage count.  The uniform case is compared with hoccl_alltoall."""
    import numpy as np
    torch.cuda.set_device(0)
    R, dtype, e = 8, "bf16", 2
    stream = torch.cuda.Stream()
    rng = np.random.default_rng(5)
    for S in [int(x) << 20 for x in args.mib.split(",")]:
        n = S // e
        send = [torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1) for _ in range(R)]
        for pattern in ("uniform", "skewed"):
            if pattern == "uniform":
                counts = np.full((R, R), n // R, dtype=np.int64)
            else:
                counts = np.zeros((R, R), dtype=np.int64)
                for u in range(R):
                    w = 1.0 / (1.0 + rng.permutation(R))
                    counts[u] = np.floor(w / w.sum() * n).astype(np.int64) // 8 * 8
            sdispls = np.concatenate([np.zeros((R, 1), dtype=np.int64), np.cumsum(counts, axis=1)[:, :-1]], axis=1)
            recv_counts = counts.T                         # recv_counts[v][u] = what v gets from u
            rdispls = np.concatenate([np.zeros((R, 1), dtype=np.int64), np.cumsum(recv_counts, axis=1)[:, :-1]], axis=1)
            recv = [torch.zeros(int(recv_counts[v].sum()) + 8, dtype=torch.bfloat16, device="cuda") for v in range(R)]
            moved = int(counts.sum()) * e
            configs = [("CE", hb.PATH_CE, 8, 0, 0), ("SM8", hb.PATH_SM, 8, 0, 0), ("SMall", hb.PATH_SM, 148, 0, 0)]
            # the same pattern over a modelled topology of two (or four) nodes: forwarding copies and "RDMA" legs as real copies
            for gpn in [int(x) for x in args.model.split(",") if x]:
                configs += [("CE_model%d" % gpn, hb.PATH_CE, 8, gpn, 0), ("CE_model%d_sub256K" % gpn, hb.PATH_CE, 8, gpn, 256 << 10),
                            ("SMall_model%d" % gpn, hb.PATH_SM, 148, gpn, 0)]
            stage_buf = None
            for name, path, ctas, gpn, sub in configs:
                comm = hb.Comm(R, 0)
                comm.set_path(path)
                comm.set_param("copy_ctas", ctas)
                tau = None
                if gpn:
                    comm.set_param("model_gpus_per_node", gpn)
                    comm.set_param("model_rdma_sub_bytes", sub)
                    if stage_buf is None:
                        stage_buf = torch.empty(2 * moved + 2 * R * R * 256 + 256, dtype=torch.uint8, device="cuda")
                    comm.set_staging(stage_buf.data_ptr() + (-stage_buf.data_ptr()) % 256, stage_buf.numel() - 256)
                    sch = hb.Schedule(counts.astype(np.uint64) * e, gpn, chunk_bytes=4 << 20)
                    tau = {"stages_host": len(sch.stages), "total_tau_us_at_400_and_50_GBps": sch.total_tau * 1e6,
                           "lower_bound_us": sch.lower_bound * 1e6}

                def call():
                    comm.alltoallv(send, counts.reshape(-1), sdispls.reshape(-1), recv, rdispls.reshape(-1), dtype, stream)

                for _ in range(3):
                    call()
                stream.synchronize()
                ok = all(torch.equal(recv[v][int(rdispls[v][u]):int(rdispls[v][u] + counts[u][v])],
                                     send[u][int(sdispls[u][v]):int(sdispls[u][v] + counts[u][v])]) for u in range(R) for v in range(R))
                iters = 10
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                for _ in range(iters):
                    call()
                e1.record(stream)
                stream.synchronize()
                t = e0.elapsed_time(e1) / 1e3 / iters
                st = comm.last_stats()
                row = {"op": "alltoallv", "pattern": pattern, "S": S, "config": name, "us": t * 1e6, "GBps_moved": moved / t / 1e9,
                       "hbm_frac_of_8TBps": 2.0 * moved / t / NOMINAL_HBM, "stages": int(st["n_pieces"]), "moves": int(st["n_moves"]),
                       "launches": int(st["n_move_launches"]), "host_us_per_call": st["host_launch_us"], "delivered_bit_exact": ok,
                       "largest_flow_MiB": float(counts.max() * e / 2 ** 20), "smallest_flow_MiB": float(counts.min() * e / 2 ** 20)}
                if tau:
                    row.update(tau)
                    row["model_gpus_per_node"] = gpn
                    row["model_rdma_sub_bytes"] = sub
                if pattern == "uniform":
                    r2 = [torch.zeros(n, dtype=torch.bfloat16, device="cuda") for _ in range(R)]
                    for _ in range(3):
                        comm.alltoall(send, r2, n // R, dtype, stream)
                    stream.synchronize()
                    e0.record(stream)
                    for _ in range(iters):
                        comm.alltoall(send, r2, n // R, dtype, stream)
                    e1.record(stream)
                    stream.synchronize()
                    row["alltoall_us"] = e0.elapsed_time(e1) * 1e3 / iters
                    del r2
                print(json.dumps(row), flush=True)
                comm.destroy()
            del recv
        del send
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    s = sub.add_parser("sizes")
    s.add_argument("--min-log2", type=int, default=12)
    s.add_argument("--max-log2", type=int, default=30)
    s.add_argument("--ranks", default="2,4,8")
    s.add_argument("--dtypes", default="bf16")
    s.add_argument("--ops", default="all")
    s.add_argument("--configs", default="all")
    s.add_argument("--out", default="")
    p = sub.add_parser("pipeline")
    p.add_argument("--microbatches", type=int, default=16)
    g = sub.add_parser("gradients")
    g.add_argument("--buckets", type=int, default=32)
    g.add_argument("--budgets", default="", help="comma list of copy-kernel CTA budgets, e.g. 1,2,4,8,16,32,64")
    g.add_argument("--ring", action="store_true", help="repeat every configuration on the ring schedule (rs_direct = 0, ag_direct = 0)")
    sub.add_parser("launch-cost")
    a2 = sub.add_parser("alltoallv")
    a2.add_argument("--mib", default="4,64,256", help="comma list of MiB sent per rank")
    a2.add_argument("--model", default="", help="comma list of modelled GPUs per node (e.g. 4,2): also run the pattern over that topology")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        sys.stderr.write("sweep: no CUDA device\n")
        return 2
    {"sizes": sweep_sizes, "pipeline": pipeline, "gradients": gradients, "launch-cost": launch_cost, "alltoallv": alltoallv}[args.cmd](args)
    return 0


if __name__ == "__main__":
    sys.exit(main())
