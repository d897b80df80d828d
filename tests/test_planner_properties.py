"""Property-based checks of the ring planner (hypothesis): for arbitrary rank counts, element counts, piece settings and
send-pointer phases, interpreting the plan in a random topological order reproduces the oracle's bits, every SUM is
rank local in the standard plans, and scratch pieces never overlap."""
import random

import numpy as np
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import diag as hd
from paper_2609_34334_b200 import workloads as W
from test_planner import _run_plan


@settings(max_examples=60, deadline=None, suppress_health_check=[HealthCheck.function_scoped_fixture])
@given(R=st.integers(1, 9), n=st.integers(0, 6000), piece_kib=st.integers(1, 8), max_pieces=st.integers(1, 9),
       in_place=st.booleans(), forward=st.booleans(), seed=st.integers(0, 10 ** 6))
def test_allreduce_plans(oracle, R, n, piece_kib, max_pieces, in_place, forward, seed):
    rng = random.Random(seed)
    xs = W.rank_inputs("uniform", seed % 1000, R, n, "fp32")
    want = oracle.ring_allreduce(xs)
    align = [4 * rng.randrange(4) for _ in range(R)]
    kind = hd.PLAN_ALLREDUCE_FWD if forward else hd.PLAN_ALLREDUCE
    plan = hd.Plan(kind, R, n, "fp32", in_place, piece_kib * 1024, max_pieces, align)
    if n == 0:
        assert plan.ops == []
        return
    by = {}
    for op in plan.ops:
        assert op["bytes"] > 0
        if op["kind"] == hd.OP_SUM and not forward:
            assert op["rank"] == op["dst_rank"]
        for buf, rank, off in ((op["src_buf"], op["rank"], op["src_off"]), (op["dst_buf"], op["dst_rank"], op["dst_off"])):
            if buf in (hd.BUF_INBOX, hd.BUF_PARTIAL):
                assert off + op["bytes"] <= plan.slot_bytes
        if op["kind"] == hd.OP_SUM:                      # pieces of one (step, rank) never overlap in the inbox slot
            by.setdefault((op["step"], op["rank"]), []).append((op["src_off"], op["bytes"]))
    for spans in by.values():
        spans.sort()
        for (o1, b1), (o2, _) in zip(spans, spans[1:]):
            assert o1 + b1 <= o2
    got = _run_plan(plan, kind, R, n, "fp32", xs, in_place, rng)
    for r in range(R):
        assert (got[r].view(np.uint32) == want[r].view(np.uint32)).all()


@settings(max_examples=40, deadline=None, suppress_health_check=[HealthCheck.function_scoped_fixture])
@given(R=st.integers(1, 9), count=st.integers(1, 1500), kind=st.sampled_from(["rs", "ag", "a2a"]), in_place=st.booleans(),
       seed=st.integers(0, 10 ** 6))
def test_other_collective_plans(oracle, R, count, kind, in_place, seed):
    rng = random.Random(seed)
    if kind == "rs":
        xs = W.rank_inputs("uniform", seed % 997, R, R * count, "fp32")
        want = oracle.ring_reduce_scatter(xs)
        plan = hd.Plan(hd.PLAN_REDUCE_SCATTER, R, count, "fp32", in_place, 2048, 5)
        got = _run_plan(plan, hd.PLAN_REDUCE_SCATTER, R, count, "fp32", xs, in_place, rng)
    elif kind == "ag":
        xs = W.rank_inputs("uniform", seed % 997, R, count, "bf16")
        want = oracle.allgather(xs)
        plan = hd.Plan(hd.PLAN_ALLGATHER, R, count, "bf16", in_place, 1024, 4)
        got = _run_plan(plan, hd.PLAN_ALLGATHER, R, count, "bf16", xs, in_place, rng)
    else:
        xs = W.rank_inputs("uniform", seed % 997, R, R * count, "bf16")
        want = oracle.alltoall(xs)
        plan = hd.Plan(hd.PLAN_ALLTOALL, R, count, "bf16", False, 1024, 4)
        got = _run_plan(plan, hd.PLAN_ALLTOALL, R, count, "bf16", xs, False, rng)
    for r in range(R):
        assert (got[r].view(np.uint8) == want[r].view(np.uint8)).all()
