"""The whole grid of schedule options, on the CPU: every combination is either refused (HOCCL_ERR_UNSUPPORTED) or resolves
to a plan that, executed by the numpy interpreter of test_planner.py in a random topological order, gives the oracle's bits.

hoccl_options_resolve is the function every entry point of the library applies before it plans a call, so what this test
sees is what a call does.  The refusal rules are restated here independently (`_must_refuse`), so that a rule dropped in
the library shows up as a disagreement, not as a silently different schedule.
"""
import itertools
import random

import numpy as np
import pytest

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import diag as hd
from paper_2609_34334_b200 import workloads as W
from test_planner import _run_plan

KINDS = {"allreduce": hd.PLAN_ALLREDUCE, "reduce_scatter": hd.PLAN_REDUCE_SCATTER, "allgather": hd.PLAN_ALLGATHER,
         "alltoall": hd.PLAN_ALLTOALL}


def _must_refuse(kind, path, o):
    """The rules as the header states them."""
    reduction = kind in ("allreduce", "reduce_scatter")
    if o["handshake"] and path != hb.PATH_SM:
        return True                       # the proxy cannot issue driver copies behind a parked stream
    if o["handshake"] and (o["onepass"] or o["fused"]):
        return True                       # the proxy replays graphs
    if o["fused"] and path != hb.PATH_SM:
        return True                       # the one-kernel form is an SM-path executor
    if reduction and o["onepass"]:
        if o["forward"] or o["fused"] or o["rs_direct"] == 1 or (o["ag_direct"] == 1 and kind == "allreduce"):
            return True                   # the one-pass kernel replaces the whole schedule
    if reduction and o["rs_direct"] == 1 and (o["forward"] or o["fused"]):
        return True                       # no chain phase in the ring kernel, no steps to forward between
    if reduction and o.get("roles"):
        if path != hb.PATH_SM or o["handshake"] or o["onepass"] or o["forward"] or o["fused"] or o["rs_direct"] == 0:
            return True                   # the roles kernel runs the direct schedule on the SM path, nothing else
        if kind == "allreduce" and o["ag_direct"] == 0:
            return True
    return False


GRID = list(itertools.product([0, 1], [0, 1], [0, 1], [0, 1, 2], [0, 1, 2], [0, 1], [0, 1], [0, 1]))   # onepass forward fused rs ag handshake graph roles


@pytest.mark.parametrize("kind", sorted(KINDS))
@pytest.mark.parametrize("path", [hb.PATH_CE, hb.PATH_SM, hb.PATH_CE_HOST])
def test_every_combination_is_served_as_asked_or_refused(oracle, kind, path):
    R, dtype = 4, "fp32"
    count = 1030 if kind == "allreduce" else 258
    n_send = count if kind in ("allreduce", "allgather") else R * count
    xs = W.rank_inputs("uniform", 23, R, n_send, dtype)
    if kind == "allreduce":
        want = oracle.ring_allreduce(xs)
    elif kind == "reduce_scatter":
        want = oracle.ring_reduce_scatter(xs)
    elif kind == "allgather":
        want = oracle.allgather(xs)
    else:
        want = oracle.alltoall(xs)
    rng = random.Random(7)
    big = hb.scratch_bytes_direct(R, n_send, dtype)
    small = hb.scratch_bytes(R, n_send, dtype)
    served = refused = 0
    plans = {}
    for onepass, forward, fused, rs, ag, handshake, graph, roles in GRID:
        o = dict(onepass=onepass, forward=forward, fused=fused, rs_direct=rs, ag_direct=ag, handshake=handshake, use_graph=graph,
                 roles=roles, ce_small_bytes=0)
        for scratch in (big, small):
            rc, res = hd.options_resolve(KINDS[kind], R, count, dtype, path, scratch_bytes=scratch, **o)
            if _must_refuse(kind, path, o):
                assert rc == hb.ERR_UNSUPPORTED and res is None, (kind, path, o)
                refused += 1
                continue
            assert rc == hb.OK, (kind, path, o)
            served += 1
            pk = res["plan_kind"]
            assert pk & 15 == KINDS[kind]
            reduction = kind in ("allreduce", "reduce_scatter")
            if roles and reduction:       # the roles kernel: the direct schedule, whatever the scratch (a call fails later if it is too small)
                assert pk & hd.PLAN_FLAG_RS_DIRECT and res["executor"] == hd.EXEC_ROLES and res["path"] == hb.PATH_SM
                assert kind != "allreduce" or pk & hd.PLAN_FLAG_AG_DIRECT
                continue
            # what was asked for is in the plan; "automatic" yields to it
            assert bool(pk & hd.PLAN_FLAG_FORWARD) == bool(forward and reduction)
            if rs == 1 and reduction:
                assert pk & hd.PLAN_FLAG_RS_DIRECT
            if rs == 0 or not reduction:
                assert not pk & hd.PLAN_FLAG_RS_DIRECT
            if rs == 2 and reduction:
                assert bool(pk & hd.PLAN_FLAG_RS_DIRECT) == (scratch == big and not forward and not fused and not onepass)
            if kind in ("allreduce", "allgather"):
                if ag == 1:
                    assert pk & hd.PLAN_FLAG_AG_DIRECT
                if ag == 0:
                    assert not pk & hd.PLAN_FLAG_AG_DIRECT
            else:
                assert not pk & hd.PLAN_FLAG_AG_DIRECT
            want_exec = (hd.EXEC_ONEPASS if (onepass and reduction) else hd.EXEC_PROXY if handshake else hd.EXEC_ONE_KERNEL if fused
                         else hd.EXEC_GRAPH if graph else hd.EXEC_STREAMS)
            assert res["executor"] == want_exec, (kind, path, o, res)
            assert res["path"] == path and res["small_switch"] == 0
            if res["executor"] == hd.EXEC_ONEPASS:
                continue                  # one kernel, no plan (its bits are checked on the GPU)
            if pk not in plans:           # the plan of this schedule, executed once per distinct schedule
                plan = hd.Plan(pk, R, count, dtype, False, 1024, 4)
                got = _run_plan(plan, pk, R, count, dtype, xs, False, rng)
                for r in range(R):
                    assert (got[r].view(np.uint32) == want[r].view(np.uint32)).all(), (kind, pk, r)
                if pk & hd.PLAN_FLAG_RS_DIRECT:
                    assert plan.scratch_bytes <= big
                else:
                    assert plan.scratch_bytes <= small
                plans[pk] = True
    assert served > 0 and refused > 0
    assert len(plans) >= (4 if kind == "allreduce" else 2 if kind != "alltoall" else 1)


def test_small_messages_on_the_copy_route_take_the_copy_kernel():
    """ce_small_bytes: per-rank message size (the collective's own convention) up to which HOCCL_PATH_CE issues its moves as
    batched copy-kernel launches with ce_small_ctas CTAs; the other paths and larger messages are untouched."""
    R, dtype = 8, "bf16"
    lim = 1 << 20
    for kind, count_at_limit in (("allreduce", lim // 2), ("reduce_scatter", lim // 2 // R), ("allgather", lim // 2 // R),
                                 ("alltoall", lim // 2 // R)):
        for count, switched in ((count_at_limit, 1), (count_at_limit + 8, 0), (1, 1)):
            rc, res = hd.options_resolve(KINDS[kind], R, count, dtype, hb.PATH_CE, ce_small_bytes=lim, ce_small_ctas=148, copy_ctas=8)
            assert rc == hb.OK
            assert res["small_switch"] == switched, (kind, count)
            assert res["path"] == (hb.PATH_SM if switched else hb.PATH_CE)
            assert res["copy_ctas"] == (148 if switched else 8)
            if kind in ("allreduce", "allgather"):
                assert bool(res["plan_kind"] & hd.PLAN_FLAG_AG_DIRECT)      # automatic: small chunks, and always on the SM route
        for path in (hb.PATH_SM, hb.PATH_CE_HOST):
            rc, res = hd.options_resolve(KINDS[kind], R, 16, dtype, path, ce_small_bytes=lim, copy_ctas=8)
            assert rc == hb.OK and res["small_switch"] == 0 and res["path"] == path and res["copy_ctas"] == 8
        rc, res = hd.options_resolve(KINDS[kind], R, 16, dtype, hb.PATH_CE, ce_small_bytes=0)
        assert rc == hb.OK and res["small_switch"] == 0 and res["path"] == hb.PATH_CE
    # the host entry keeps its route: its pieces are pipelined against host copies
    rc, res = hd.options_resolve(hd.PLAN_ALLREDUCE, R, 16, dtype, hb.PATH_CE, ce_small_bytes=lim, host_call=1)
    assert rc == hb.OK and res["small_switch"] == 0


def test_argument_errors():
    assert hd.options_resolve(7, 4, 10, "fp32")[0] == hb.ERR_INVALID_ARG
    assert hd.options_resolve(0, 0, 10, "fp32")[0] == hb.ERR_INVALID_ARG
    assert hd.options_resolve(0, 4, 10, 9)[0] == hb.ERR_UNSUPPORTED
    # the roles kernel has chain loops for 2 to 8 ranks
    assert hd.options_resolve(0, 9, 1000, "fp32", hb.PATH_SM, roles=1)[0] == hb.ERR_UNSUPPORTED
    assert hd.options_resolve(0, 1, 1000, "fp32", hb.PATH_SM, roles=1)[0] == hb.ERR_UNSUPPORTED
    assert hd.options_resolve(0, 8, 1000, "fp32", hb.PATH_SM, roles=1)[0] == hb.OK
    assert hd.options_resolve(0, 8, 1000, "fp32", hb.PATH_SM, roles=1, host_call=1)[1]["executor"] == hd.EXEC_GRAPH
    assert hd.lib().hoccl_options_resolve(None, None) == hb.ERR_INVALID_ARG
