"""Kernel microbenchmarks through the C ABI (hoccl_sum_launch / hoccl_copy_launch), one kernel at a time.

    python -m paper_2609_34334_b200.microbench --kernel sum --dtype bf16 --mib 200 --ctas 8 --reps 5
    python -m paper_2609_34334_b200.microbench --kernel routes --mib 16      # which same-device copy routes need an SM
    python -m paper_2609_34334_b200.microbench --kernel ring --mib 32 --ctas 148   # all-reduce, R = 8, as one cooperative kernel
    python -m paper_2609_34334_b200.microbench --kernel port --mib 256 --ctas 8    # what the memory ports of `ctas` SMs carry
    python -m paper_2609_34334_b200.microbench --kernel fan --mib 25 --ctas 148    # one source to 7 destinations: fan-out against 7 copies
    python -m paper_2609_34334_b200.microbench --kernel chain --mib 25 --ctas 8    # 7 inbox operands + the local one into one output
    python -m paper_2609_34334_b200.microbench --kernel beside --mib 40 --ctas 8   # the chain sum while a 1 GiB copy runs on another stream

Operands are larger than L2 by default; timing uses CUDA events on the launching stream after warm-up.
Prints one JSON line.  This is the small case used for ncu captures of a single kernel.
"""
from __future__ import annotations

import argparse
import json

import torch

from . import binding as hb
from . import diag as hd


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--kernel", default="sum", choices=["sum", "copy", "routes", "ring", "port", "fan", "chain", "beside"])
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "fp32"])
    ap.add_argument("--mib", type=int, default=200, help="MiB per operand")
    ap.add_argument("--ctas", type=int, default=8)
    ap.add_argument("--reps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    args = ap.parse_args()
    torch.cuda.set_device(0)
    nbytes = args.mib << 20
    if args.kernel == "port":
        # read only, write only, 1 : 1 copy and 2 : 1 sum with the same number of CTAs (one CTA occupies one SM)
        n = nbytes // 2
        a = torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
        b = torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
        o = torch.empty(n, dtype=torch.bfloat16, device="cuda")
        sink = torch.zeros(1, dtype=torch.int32, device="cuda")
        st = torch.cuda.Stream()
        cases = {"read_only": (lambda: hd.port_probe("read", a, nbytes, args.ctas, sink, st), nbytes),
                 "write_only": (lambda: hd.port_probe("write", o, nbytes, args.ctas, sink, st), nbytes),
                 "copy_1r_1w": (lambda: hd.copy_launch(a, o, nbytes, args.ctas, st), 2 * nbytes),
                 "sum_2r_1w": (lambda: hd.sum_launch(a, b, o, n, "bf16", args.ctas, st), 3 * nbytes)}
        out = {"probe": "memory ports of %d SMs (one 1024-thread CTA each), %d MiB operands" % (args.ctas, args.mib), "ctas": args.ctas}
        for name, (fn, moved) in cases.items():
            for _ in range(args.warmup):
                assert fn() == hb.OK
            st.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            for _ in range(args.reps):
                fn()
            e1.record(st)
            st.synchronize()
            sec = e0.elapsed_time(e1) / 1e3 / args.reps
            out[name] = {"GBps": moved / sec / 1e9, "GBps_per_sm": moved / sec / 1e9 / args.ctas, "us": sec * 1e6}
        print(json.dumps(out))
        return
    if args.kernel == "beside":
        # what concurrent copies cost a sum under a CTA budget: the chain sum (7 inbox operands + the local one) is timed while a
        # 1 GiB copy runs on another stream, as copy_kernel launches of several CTA budgets and as one driver copy
        nsrc = 7
        n = nbytes // 2
        inbox = torch.empty(nsrc * n, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
        local = torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
        out_t = torch.empty(n, dtype=torch.bfloat16, device="cuda")
        big = 1 << 30
        src = torch.empty(big, dtype=torch.uint8, device="cuda")
        dst = torch.empty(big, dtype=torch.uint8, device="cuda")
        sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
        torch.cuda.synchronize()

        def chain():
            assert hd.chain_launch(inbox, nbytes, nsrc, local, out_t, n, "bf16", args.ctas, sa) == hb.OK

        rows = []
        for what in ("none", "copy_16", "copy_32", "copy_48", "copy_64", "copy_100", "copy_140", "driver"):
            best = None
            for _ in range(max(1, args.reps)):
                chain()
                torch.cuda.synchronize()
                k0, k1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                c0.record(sb)
                if what == "driver":
                    with torch.cuda.stream(sb):
                        dst.copy_(src, non_blocking=True)
                elif what != "none":
                    assert hd.copy_launch(src, dst, big, int(what.split("_")[1]), sb) == hb.OK
                c1.record(sb)
                k0.record(sa)
                chain()
                k1.record(sa)
                torch.cuda.synchronize()
                row = {"background": what, "chain_us": k0.elapsed_time(k1) * 1e3, "background_us": c0.elapsed_time(c1) * 1e3}
                if best is None or row["chain_us"] < best["chain_us"]:
                    best = row
            best["background_GBps"] = 2.0 * big / best["background_us"] / 1e3 if what != "none" else 0.0
            rows.append(best)
        print(json.dumps({"probe": "chain sum (%d CTAs, output of %d MiB, 8 operands) beside a 1 GiB copy on another stream" % (args.ctas, args.mib),
                          "rows": rows}))
        return
    if args.kernel == "chain":
        # the sum of the direct reduce-scatter for R = 8: seven inbox operands and the local one, one output (8 reads : 1 write)
        nsrc, sets = 7, 3
        tdt = torch.bfloat16 if args.dtype == "bf16" else torch.float32
        e = 2 if args.dtype == "bf16" else 4
        n = nbytes // e
        st = torch.cuda.Stream()
        inbox = [torch.empty(nsrc * n, dtype=tdt, device="cuda").normal_(0, 1e-3) for _ in range(sets)]
        local = [torch.empty(n, dtype=tdt, device="cuda").normal_(0, 1e-3) for _ in range(sets)]
        out_t = [torch.empty(n, dtype=tdt, device="cuda") for _ in range(sets)]
        torch.cuda.synchronize()

        def chain(k):
            assert hd.chain_launch(inbox[k], nbytes, nsrc, local[k], out_t[k], n, args.dtype, args.ctas, st) == hb.OK

        for k in range(max(args.warmup, sets)):
            chain(k % sets)
        st.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for k in range(args.reps):
            chain(k % sets)
        e1.record(st)
        st.synchronize()
        sec = e0.elapsed_time(e1) / 1e3 / args.reps
        acc = inbox[0][:n].clone()
        for j in range(1, nsrc):
            acc = (acc.float() + inbox[0][j * n:(j + 1) * n].float()).to(tdt)
        acc = (acc.float() + local[0].float()).to(tdt)
        assert torch.equal(out_t[0], acc), "kernel result differs from torch's fp32 add + RNE, taken step by step"
        moved = (nsrc + 2) * nbytes
        print(json.dumps({"kernel": "chain", "dtype": args.dtype, "mib_per_operand": args.mib, "inbox_operands": nsrc, "ctas": args.ctas,
                          "us_per_launch": sec * 1e6, "algorithmic_bytes_per_launch": moved, "GBps": moved / sec / 1e9,
                          "GBps_per_cta": moved / sec / 1e9 / args.ctas, "output_GBps_per_cta": nbytes / sec / 1e9 / args.ctas}))
        return
    if args.kernel == "fan":
        # the move of the direct all-gather: one chunk to R - 1 = 7 peers, as one fan-out launch and as 7 copy launches
        nd, sets = 7, 3
        srcs = [torch.randint(0, 255, (nbytes,), dtype=torch.uint8, device="cuda") for _ in range(sets)]
        dsts = [[torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(nd)] for _ in range(sets)]
        st = torch.cuda.Stream()

        def fan(k):
            assert hd.fanout_launch(srcs[k], dsts[k], nbytes, args.ctas, st) == hb.OK

        def copies(k):
            for d in dsts[k]:
                assert hd.copy_launch(srcs[k], d, nbytes, args.ctas, st) == hb.OK

        out = {"kernel": "fan", "mib_per_operand": args.mib, "destinations": nd, "ctas": args.ctas}
        for name, fn, moved in (("fan_out", fan, (1 + nd) * nbytes), ("separate_copies", copies, 2 * nd * nbytes)):
            for k in range(max(args.warmup, sets)):
                fn(k % sets)
            st.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(st)
            for k in range(args.reps):
                fn(k % sets)
            e1.record(st)
            st.synchronize()
            sec = e0.elapsed_time(e1) / 1e3 / args.reps
            out[name] = {"us": sec * 1e6, "algorithmic_bytes": moved, "GBps": moved / sec / 1e9, "delivered_GBps": nd * nbytes / sec / 1e9}
            assert all(torch.equal(d, srcs[0]) for d in dsts[0])
        print(json.dumps(out))
        return
    if args.kernel == "ring":
        R = 8
        e = 2 if args.dtype == "bf16" else 4
        n = nbytes // e
        tdt = torch.bfloat16 if args.dtype == "bf16" else torch.float32
        send = [torch.empty(n, dtype=tdt, device="cuda").normal_(0, 1e-3) for _ in range(R)]
        recv = [torch.empty(n, dtype=tdt, device="cuda") for _ in range(R)]
        nb = hb.scratch_bytes(R, n, args.dtype)
        scratch = torch.empty(nb + 256, dtype=torch.uint8, device="cuda")
        comm = hb.Comm(R, 0)
        comm.set_path(hb.PATH_SM)
        comm.set_scratch(scratch.data_ptr() + (-scratch.data_ptr()) % 256, nb)
        for k, v in (("fused", 1), ("sum_ctas", args.ctas), ("copy_ctas", args.ctas)):
            comm.set_param(k, v)
        st = torch.cuda.Stream()
        for _ in range(args.warmup):
            comm.allreduce(send, recv, n, args.dtype, st)
        st.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(st)
        for _ in range(args.reps):
            comm.allreduce(send, recv, n, args.dtype, st)
        e1.record(st)
        st.synchronize()
        sec = e0.elapsed_time(e1) / 1e3 / args.reps
        moved = 7.0 * nbytes * (R - 1)
        assert all(torch.equal(recv[0], recv[r]) for r in range(1, R)), "ranks disagree"
        assert comm.async_error() == hb.OK
        stats = comm.last_stats()
        print(json.dumps({"kernel": "ring_kernel (all-reduce, R = 8, one cooperative launch)", "dtype": args.dtype,
                          "mib_per_rank": args.mib, "ctas": int(stats["max_copy_ctas"]), "us_per_launch": sec * 1e6,
                          "algorithmic_bytes_per_launch": moved, "GBps": moved / sec / 1e9,
                          "busbw_GBps": nbytes * 2 * (R - 1) / R / sec / 1e9}))
        comm.destroy()
        return
    if args.kernel == "routes":
        src = torch.full((nbytes,), 7, dtype=torch.uint8, device="cuda")
        dst = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
        host = torch.empty(nbytes, dtype=torch.uint8).pin_memory()
        comm = hb.Comm(2, 0)
        comm.set_param("copy_ctas", args.ctas)
        comm.set_host_staging(host)
        rows = hd.probe_copy_routes(comm, dst, src, nbytes, 3000)
        comm.destroy()
        print(json.dumps({"probe": "copy routes under a kernel that holds every SM for 3000 us", "mib": args.mib,
                          "routes": [{"route": n, "needs_sm": s, "end_us": round(t, 1)} for n, s, t in rows]}))
        return
    e = 2 if args.dtype == "bf16" else 4
    n = nbytes // e
    tdt = torch.bfloat16 if args.dtype == "bf16" else torch.float32
    a = torch.empty(n, dtype=tdt, device="cuda").normal_(0, 1e-3)
    b = torch.empty(n, dtype=tdt, device="cuda").normal_(0, 1e-3)
    o = torch.empty(n, dtype=tdt, device="cuda")
    st = torch.cuda.Stream()

    def launch():
        if args.kernel == "sum":
            rc = hd.sum_launch(a, b, o, n, args.dtype, args.ctas, st)
        else:
            rc = hd.copy_launch(a, o, nbytes, args.ctas, st)
        assert rc == hb.OK, rc

    for _ in range(args.warmup):
        launch()
    st.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(st)
    for _ in range(args.reps):
        launch()
    e1.record(st)
    st.synchronize()
    sec = e0.elapsed_time(e1) / 1e3 / args.reps
    moved = (3 if args.kernel == "sum" else 2) * nbytes
    if args.kernel == "sum":
        assert torch.equal(o, (a.float() + b.float()).to(tdt)), "kernel result differs from torch's fp32 add + RNE"
    else:
        assert torch.equal(o, a)
    print(json.dumps({"kernel": args.kernel, "dtype": args.dtype, "mib_per_operand": args.mib, "ctas": args.ctas,
                      "us_per_launch": sec * 1e6, "algorithmic_bytes_per_launch": moved, "GBps": moved / sec / 1e9,
                      "GBps_per_cta": moved / sec / 1e9 / args.ctas}))


if __name__ == "__main__":
    main()
