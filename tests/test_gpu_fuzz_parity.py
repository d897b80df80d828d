"""Randomised GPU parity (hypothesis, derandomised so that every run draws the same cases): operation, rank count,
element count, dtype, path, executor, piece settings, variants, in-place form and per-rank byte offsets are drawn
together, values include signed zeros, subnormals, infinities and NaNs, and every result is compared with the
oracle bit for bit (any NaN matches any NaN).  What must hold: no setting and no layout changes a bit, and a combination
of settings that does not fit together (as the host-only option rules say) is refused with nothing enqueued."""
import numpy as np
import pytest
import torch
from hypothesis import given, settings, strategies as st, HealthCheck

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import diag as hd
from paper_2609_34334_b200 import workloads as W
from gpu_util import DevBuf, np_dtype, same_bits
from test_gpu_parity import make_comm

pytestmark = pytest.mark.gpu


def _values(rng, n, dtype, flavour):
    """n elements of `dtype` as the arrays the library sees (fp32: float32; bf16: uint16 bit patterns)."""
    if flavour == "normal":
        x = rng.standard_normal(n).astype(np.float32) * np.float32(1e-3)
    elif flavour == "wide":        # magnitudes across the whole exponent range: overflow to inf, cancellation, subnormal sums
        with np.errstate(over="ignore"):
            x = (rng.standard_normal(n) * np.exp2(rng.integers(-140, 127, n))).astype(np.float32)
    else:                           # special values sprinkled over small integers
        x = rng.integers(-4, 5, n).astype(np.float32)
        pick = rng.integers(0, 12, n)
        x[pick == 0] = np.float32("inf")
        x[pick == 1] = np.float32("-inf")
        x[pick == 2] = np.float32("nan")
        x[pick == 3] = np.float32(-0.0)
        x[pick == 4] = np.float32(1e-41)      # subnormal in fp32 and in bf16
    if dtype == "fp32":
        return x
    u = x.view(np.uint32)
    return (u >> 16).astype(np.uint16)        # truncation is enough for test inputs: any bf16 pattern is a legal input


case = st.fixed_dictionaries({
    "op": st.sampled_from(["allreduce", "allreduce", "reduce_scatter", "allgather", "alltoall"]),
    "R": st.integers(1, 9),
    "n": st.one_of(st.integers(0, 40), st.integers(41, 5000), st.integers(5001, 300_000), st.integers(300_001, 2_500_000)),
    "dtype": st.sampled_from(["fp32", "bf16"]),
    "path": st.sampled_from([hb.PATH_CE, hb.PATH_SM]),
    "use_graph": st.integers(0, 1),
    "piece_kib": st.sampled_from([1, 4, 64, 256, 4096]),
    "max_pieces": st.integers(1, 6),
    "variant": st.sampled_from(["plain", "plain", "fused", "forward", "onepass", "roles"]),
    "piece_grade": st.integers(-1, 1),
    "ctas": st.sampled_from([1, 3, 8, 148]),
    "in_place": st.booleans(),
    "offs": st.lists(st.integers(0, 3), min_size=9, max_size=9),
    "flavour": st.sampled_from(["normal", "wide", "special"]),
    "seed": st.integers(0, 2 ** 31 - 1),
    "ag_direct": st.integers(0, 2),
    "rs_direct": st.integers(0, 2),
    "ce_small_kib": st.sampled_from([0, 0, 64, 8192]),
})


@settings(max_examples=300, deadline=None, derandomize=True, suppress_health_check=list(HealthCheck))
@given(c=case)
def test_random_cases_match_the_oracle(oracle, c):
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    torch.cuda.set_device(0)
    R, dtype, op = c["R"], c["dtype"], c["op"]
    e = W.elem_size(dtype)
    rng = np.random.default_rng(c["seed"])
    count = c["n"]                       # allreduce: elements per rank; other operations: elements per block
    total = count if op == "allreduce" else count * R
    offs = [o * e for o in c["offs"][:R]]
    params = dict(use_graph=c["use_graph"], piece_bytes=c["piece_kib"] << 10, max_pieces=c["max_pieces"], sum_ctas=c["ctas"],
                  copy_ctas=c["ctas"], ag_direct=c["ag_direct"], rs_direct=c["rs_direct"], ce_small_bytes=c["ce_small_kib"] << 10,
                  piece_grade=c["piece_grade"])
    if c["variant"] != "plain":
        params[c["variant"]] = 1
    comm = make_comm(R, max(total, 1), dtype, c["path"], **params)
    npd = np_dtype(dtype)
    # what the option rules say about this combination, without a device
    kind = {"allreduce": hd.PLAN_ALLREDUCE, "reduce_scatter": hd.PLAN_REDUCE_SCATTER, "allgather": hd.PLAN_ALLGATHER,
            "alltoall": hd.PLAN_ALLTOALL}[op]
    verdict, _ = hd.options_resolve(kind, R, count, dtype, c["path"], **{k: v for k, v in params.items()
                                                                     if k in ("use_graph", "ag_direct", "rs_direct", "onepass", "forward",
                                                                              "fused", "roles", "ce_small_bytes", "copy_ctas")})
    if verdict != hb.OK:
        assert verdict == hb.ERR_UNSUPPORTED
        send = [DevBuf(max(total, 1) * e) for _ in range(R)]
        recv = [DevBuf(max(total, 1) * e, fill=0x3C) for _ in range(R)]
        fn = {"allreduce": comm.allreduce_rc, "reduce_scatter": comm.reduce_scatter_rc, "allgather": comm.allgather_rc,
              "alltoall": comm.alltoall_rc}[op]
        assert fn(send, recv, count, dtype) == hb.ERR_UNSUPPORTED, c
        torch.cuda.synchronize()
        for b in recv:
            assert (b.get(np.uint8) == 0x3C).all() and b.guards_intact(), c      # nothing was enqueued
        assert comm.destroy() == hb.OK
        return
    if op == "allreduce":
        xs = [_values(rng, count, dtype, c["flavour"]) for _ in range(R)]
        want = oracle.ring_allreduce(xs)
        send = [DevBuf(count * e, offs[r]).put(xs[r]) for r in range(R)]
        recv = send if c["in_place"] else [DevBuf(count * e, offs[(r + 1) % R]) for r in range(R)]
        comm.allreduce(send, recv, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert same_bits(recv[r].get(npd), want[r], dtype), (c, r)
    elif op == "reduce_scatter":
        xs = [_values(rng, total, dtype, c["flavour"]) for _ in range(R)]
        want = oracle.ring_reduce_scatter(xs)
        send = [DevBuf(total * e, offs[r]).put(xs[r]) for r in range(R)]
        if c["in_place"]:
            comm.reduce_scatter(send, [send[r].ptr + r * count * e for r in range(R)], count, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert same_bits(send[r].get(npd)[r * count:(r + 1) * count], want[r], dtype), (c, r)
            recv = []
        else:
            recv = [DevBuf(count * e, offs[(r + 2) % R]) for r in range(R)]
            comm.reduce_scatter(send, recv, count, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert same_bits(recv[r].get(npd), want[r], dtype), (c, r)
    elif op == "allgather":
        xs = [_values(rng, count, dtype, c["flavour"]) for _ in range(R)]
        cat = np.concatenate(xs) if count else np.zeros(0, dtype=npd)
        recv = [DevBuf(total * e, offs[r]) for r in range(R)]
        if c["in_place"]:
            for r in range(R):
                recv[r].view[r * count * e:(r + 1) * count * e].copy_(torch.from_numpy(xs[r].view(np.uint8).copy()))
            send = []
            comm.allgather([recv[r].ptr + r * count * e for r in range(R)], recv, count, dtype)
        else:
            send = [DevBuf(count * e, offs[(r + 1) % R]).put(xs[r]) for r in range(R)]
            comm.allgather(send, recv, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert (recv[r].get(npd).view(np.uint8) == cat.view(np.uint8)).all(), (c, r)
    else:
        xs = [_values(rng, total, dtype, c["flavour"]) for _ in range(R)]
        want = oracle.alltoall(xs)
        send = [DevBuf(total * e, offs[r]).put(xs[r]) for r in range(R)]
        recv = [DevBuf(total * e, offs[(r + 1) % R]) for r in range(R)]
        comm.alltoall(send, recv, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert (recv[r].get(npd).view(np.uint8) == want[r].view(np.uint8)).all(), (c, r)
    for b in list(send) + list(recv) + [comm._scratch_keep]:
        assert b.guards_intact(), c
    assert comm.async_error() == hb.OK
    assert comm.destroy() == hb.OK
