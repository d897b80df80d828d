"""Host-only checks of the ring planner through the C ABI (hoccl_plan_*).

The plan is executed here by a small interpreter (numpy copies for MOVE, numpy float32 adds for SUM)
in RANDOM topological orders of its group DAG and compared bit for bit with the CPU oracle: a missing
dependency, a wrong offset or a wrong chunk index shows up as a wrong result.  Structural rules are
checked as well: rank locality of every SUM, every ring MOVE crosses exactly one rank boundary, every
byte of every chunk is covered exactly once per step, scratch slots are never exceeded.
"""
import random

import numpy as np
import pytest

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import diag as hd
from paper_2609_34334_b200 import workloads as W

PHASE_RS, PHASE_AG, PHASE_OWN = 0, 1, 2


def _topo_order(num_groups, deps, rng):
    indeg = [len(d) for d in deps]
    users = [[] for _ in range(num_groups)]
    for g, ds in enumerate(deps):
        for d in ds:
            assert 0 <= d < g, "dependencies must point to earlier groups (acyclic by construction)"
            users[d].append(g)
    ready = [g for g in range(num_groups) if indeg[g] == 0]
    order = []
    while ready:
        g = ready.pop(rng.randrange(len(ready)))
        order.append(g)
        for u in users[g]:
            indeg[u] -= 1
            if indeg[u] == 0:
                ready.append(u)
    assert len(order) == num_groups
    return order


def _run_plan(plan, kind, R, count, dtype, xs, in_place, rng):
    e = W.elem_size(dtype)
    npdt = np.float32 if dtype == "fp32" else np.uint16
    base = {hd.PLAN_ALLREDUCE_FWD: hd.PLAN_ALLREDUCE, hd.PLAN_REDUCE_SCATTER_FWD: hd.PLAN_REDUCE_SCATTER, hd.PLAN_ALLREDUCE_AGD: hd.PLAN_ALLREDUCE,
            hd.PLAN_ALLREDUCE_FWD_AGD: hd.PLAN_ALLREDUCE, hd.PLAN_ALLGATHER_DIRECT: hd.PLAN_ALLGATHER}.get(kind, kind)
    kind = base if base < 16 else (base & 15)
    if kind == hd.PLAN_ALLREDUCE:
        send_n, recv_n = count, count
    elif kind == hd.PLAN_ALLTOALL:
        send_n, recv_n = R * count, R * count
    elif kind == hd.PLAN_REDUCE_SCATTER:
        send_n, recv_n = R * count, count
    else:
        send_n, recv_n = count, R * count
    slot = plan.slot_bytes
    if R > 1 and count > 0 and kind in (hd.PLAN_ALLREDUCE, hd.PLAN_REDUCE_SCATTER):
        assert 0 < slot <= hb.scratch_bytes(R, send_n, dtype) // (2 * R)      # the advertised bound covers any piece setting
        bound = hb.scratch_bytes_direct(R, send_n, dtype) if plan.inbox_slots > 1 else hb.scratch_bytes(R, send_n, dtype)
        assert plan.scratch_bytes <= bound
    send = [x.copy().view(np.uint8) for x in xs]
    if in_place:
        if kind == hd.PLAN_ALLREDUCE:
            recv = send
        elif kind == hd.PLAN_REDUCE_SCATTER:
            recv = [send[r][r * count * e:(r + 1) * count * e] for r in range(R)]
        else:
            recv = [np.zeros(recv_n * e, dtype=np.uint8) for _ in range(R)]
            for r in range(R):
                recv[r][r * count * e:(r + 1) * count * e] = send[r]
                send[r] = recv[r][r * count * e:(r + 1) * count * e]
    else:
        recv = [np.full(recv_n * e, 0xAB, dtype=np.uint8) for _ in range(R)]
    inbox = [np.full(slot * plan.inbox_slots, 0xCD, dtype=np.uint8) for _ in range(R)]
    partial = [np.full(slot, 0xEF, dtype=np.uint8) for _ in range(R)]
    bufs = {hd.BUF_SEND: send, hd.BUF_RECV: recv, hd.BUF_INBOX: inbox, hd.BUF_PARTIAL: partial}
    by_group = {}
    for op in plan.ops:
        by_group.setdefault(op["group"], []).append(op)
    for g in _topo_order(plan.num_groups, plan.deps, rng):
        ops = by_group[g]
        rng.shuffle(ops)           # ops of one group are independent of each other
        for op in ops:
            n = op["bytes"]
            assert n > 0 and n % e == 0
            src = bufs[op["src_buf"]][op["rank"]][op["src_off"]:op["src_off"] + n]
            assert src.size == n
            if op["kind"] == hd.OP_MOVE:
                dst = bufs[op["dst_buf"]][op["dst_rank"]]
                assert op["dst_off"] + n <= dst.size
                dst[op["dst_off"]:op["dst_off"] + n] = src
            elif op["kind"] == hd.OP_CHAIN:
                assert dtype == "fp32" and op["rank"] == op["dst_rank"] and op["src_buf"] == hd.BUF_INBOX
                box = bufs[hd.BUF_INBOX][op["rank"]]
                acc = box[op["src_off"]:op["src_off"] + n].view(np.float32).copy()
                for j in range(1, op["nsrc"]):
                    lo = op["src_off"] + j * op["src_stride"]
                    assert lo + n <= box.size
                    acc = acc + box[lo:lo + n].view(np.float32)
                loc = bufs[op["local_buf"]][op["rank"]][op["local_off"]:op["local_off"] + n]
                res = (acc + loc.view(np.float32)).view(np.uint8)
                out = bufs[op["dst_buf"]][op["dst_rank"]]
                assert op["dst_off"] + n <= out.size
                out[op["dst_off"]:op["dst_off"] + n] = res
            else:
                assert dtype == "fp32"
                loc = bufs[op["local_buf"]][op["rank"]][op["local_off"]:op["local_off"] + n]
                out = bufs[op["dst_buf"]][op["dst_rank"]]
                assert op["dst_off"] + n <= out.size
                res = (src.view(np.float32) + loc.view(np.float32)).view(np.uint8)
                out[op["dst_off"]:op["dst_off"] + n] = res
    return [r.view(npdt) for r in recv]


CASES = [(R, n, pb, mp) for R in (1, 2, 3, 4, 8) for (n, pb, mp) in
         ((0, 4096, 8), (1, 4096, 8), (5, 1024, 4), (R * 1024, 1024, 3), (R * 1024 + 3, 1024, 8), (4099, 2048, 2), (70001, 8192, 8))]


@pytest.mark.parametrize("R,n,piece_bytes,max_pieces", CASES)
def test_allreduce_plan_executes_to_oracle_bits(oracle, R, n, piece_bytes, max_pieces):
    rng = random.Random(R * 1000 + n)
    xs = W.rank_inputs("uniform", 17, R, n, "fp32")
    want = oracle.ring_allreduce(xs)
    for in_place in (False, True):
        align = [(4 * rng.randrange(4)) for _ in range(R)] if in_place else None
        plan = hd.Plan(hd.PLAN_ALLREDUCE, R, n, "fp32", in_place, piece_bytes, max_pieces, align)
        # SUM operands share their 16-byte phase (vector path), whatever the send pointers' alignment
        for op in plan.ops:
            if op["kind"] == hd.OP_SUM:
                a = align[op["rank"]] if align else 0
                assert op["src_off"] % 16 == (a + op["local_off"]) % 16
                if op["dst_buf"] == hd.BUF_PARTIAL:
                    assert op["dst_off"] % 16 == op["src_off"] % 16
        for trial in range(2):
            got = _run_plan(plan, hd.PLAN_ALLREDUCE, R, n, "fp32", xs, in_place, rng)
            for r in range(R):
                assert (got[r].view(np.uint32) == want[r].view(np.uint32)).all(), (R, n, in_place, r)


@pytest.mark.parametrize("R", [1, 2, 4, 8])
@pytest.mark.parametrize("count", [1, 7, 1024, 3001])
def test_reduce_scatter_and_allgather_plans(oracle, R, count):
    rng = random.Random(R * 77 + count)
    xs = W.rank_inputs("uniform", 23, R, R * count, "fp32")
    want = oracle.ring_reduce_scatter(xs)
    for in_place in (False, True):
        plan = hd.Plan(hd.PLAN_REDUCE_SCATTER, R, count, "fp32", in_place, 2048, 4)
        got = _run_plan(plan, hd.PLAN_REDUCE_SCATTER, R, count, "fp32", xs, in_place, rng)
        for r in range(R):
            assert (got[r].view(np.uint32) == want[r].view(np.uint32)).all()
    for dtype in ("fp32", "bf16"):
        ys = W.rank_inputs("uniform", 29, R, count, dtype)
        cat = np.concatenate(ys)
        for in_place in (False, True):
            plan = hd.Plan(hd.PLAN_ALLGATHER, R, count, dtype, in_place, 1024, 8)
            assert all(op["kind"] == hd.OP_MOVE for op in plan.ops)
            got = _run_plan(plan, hd.PLAN_ALLGATHER, R, count, dtype, ys, in_place, rng)
            for r in range(R):
                assert (got[r] == cat).all()


@pytest.mark.parametrize("R,n", [(2, 100), (4, 1 << 20), (8, 13_107_200), (8, 1001), (5, 12345)])
def test_structure_rules(R, n):
    e = 4
    plan = hd.Plan(hd.PLAN_ALLREDUCE, R, n, "fp32", False, 1 << 20, 8)
    q = -(-n // R)
    lo = [min(c * q, n) for c in range(R)]
    hi = [min((c + 1) * q, n) for c in range(R)]
    sums = [op for op in plan.ops if op["kind"] == hd.OP_SUM]
    moves = [op for op in plan.ops if op["kind"] == hd.OP_MOVE]
    # rank locality: a SUM touches one rank only; its operands are inbox + own send data
    for op in sums:
        assert op["rank"] == op["dst_rank"]
        assert op["src_buf"] == hd.BUF_INBOX and op["local_buf"] == hd.BUF_SEND
        assert op["chunk"] == (op["rank"] - 2 - op["step"]) % R
        assert op["dst_buf"] == (hd.BUF_RECV if op["step"] == R - 2 else hd.BUF_PARTIAL)
        assert op["src_off"] + op["bytes"] <= plan.slot_bytes
    # every ring MOVE crosses exactly one rank boundary, towards rank+1
    for op in moves:
        assert op["phase"] in (PHASE_RS, PHASE_AG)
        assert op["dst_rank"] == (op["rank"] + 1) % R and op["dst_rank"] != op["rank"]
        if op["phase"] == PHASE_RS:
            assert op["chunk"] == (op["rank"] - 1 - op["step"]) % R
            assert op["dst_buf"] == hd.BUF_INBOX
            assert op["src_buf"] == (hd.BUF_SEND if op["step"] == 0 else hd.BUF_PARTIAL)
        else:
            assert op["chunk"] == (op["rank"] - op["step"]) % R
            assert op["src_buf"] == hd.BUF_RECV and op["dst_buf"] == hd.BUF_RECV and op["src_off"] == op["dst_off"]
    # coverage: per (phase, step, rank) the pieces tile the chunk exactly once
    for kind_ops, phase in ((moves, PHASE_RS), (moves, PHASE_AG), (sums, PHASE_RS)):
        seen = {}
        for op in kind_ops:
            if op["phase"] != phase:
                continue
            seen.setdefault((op["step"], op["rank"], op["chunk"]), []).append(op)
        assert len({(s, r) for s, r, _ in seen}) == len(seen)          # one chunk per (step, rank)
        for (s, r, c), ops in seen.items():
            total = sum(o["bytes"] for o in ops)
            assert total == (hi[c] - lo[c]) * e
            if all(o["dst_buf"] == hd.BUF_RECV for o in ops):
                spans = sorted((o["dst_off"] - lo[c] * e, o["bytes"]) for o in ops)
                pos = 0
                for off, b in spans:
                    assert off == pos
                    pos += b
            else:       # scratch: pieces must not overlap inside the slot
                spans = sorted((o["dst_off"], o["bytes"]) for o in ops)
                for (o1, b1), (o2, _) in zip(spans, spans[1:]):
                    assert o1 + b1 <= o2
    steps = {op["step"] for op in sums}
    assert steps == set(range(R - 1))
    # SUM groups form one chain (the SM budget for sums is global): each has the previous SUM group among its deps
    sum_groups = sorted({op["group"] for op in sums})
    for a, b in zip(sum_groups, sum_groups[1:]):
        assert a in plan.deps[b]
    # counts: (R-1) steps x R ranks x pieces for each of RS-move, SUM, AG-move when nothing is empty
    if n % R == 0:
        pieces = len({op["piece"] for op in plan.ops})
        assert len(sums) == (R - 1) * R * pieces
        assert len(moves) == 2 * (R - 1) * R * pieces


def test_piece_geometry():
    # 25 MiB bf16 bucket over 8 ranks: chunk 3,276,800 B
    plan = hd.Plan(hd.PLAN_ALLREDUCE, 8, 13_107_200, "bf16", False, 1 << 20, 8)
    pieces = sorted({op["piece"] for op in plan.ops})
    assert pieces == [0, 1, 2, 3]
    sizes = {op["bytes"] for op in plan.ops}
    assert max(sizes) % 1024 == 0 and sum(sorted({(op["piece"], op["bytes"]) for op in plan.ops if op["rank"] == 0 and op["step"] == 0 and op["kind"] == 1}, key=lambda t: t[0])[k][1] for k in range(4)) == 3_276_800
    one = hd.Plan(hd.PLAN_ALLREDUCE, 8, 13_107_200, "bf16", False, 64 << 20, 8)
    assert {op["piece"] for op in one.ops} == {0}
    capped = hd.Plan(hd.PLAN_ALLREDUCE, 2, 1 << 28, "fp32", False, 1 << 20, 8)
    assert len({op["piece"] for op in capped.ops}) == 8


@pytest.mark.parametrize("R", [1, 2, 5, 8])
@pytest.mark.parametrize("count", [1, 33, 4099])
def test_alltoall_plan(oracle, R, count):
    rng = random.Random(R * 31 + count)
    for dtype in ("fp32", "bf16"):
        xs = W.rank_inputs("uniform", 37, R, R * count, dtype)
        want = oracle.alltoall(xs)
        plan = hd.Plan(hd.PLAN_ALLTOALL, R, count, dtype, False, 1024, 8)
        assert all(op["kind"] == hd.OP_MOVE for op in plan.ops) and all(len(d) == 0 for d in plan.deps)
        # every stage is a permutation: each rank sends one block and receives one block
        stages = {}
        for op in plan.ops:
            stages.setdefault((op["phase"], op["step"], op["piece"]), []).append(op)
        for (phase, k, _), ops in stages.items():
            assert sorted(o["rank"] for o in ops) == list(range(R)) and sorted(o["dst_rank"] for o in ops) == list(range(R))
            for o in ops:
                assert o["dst_rank"] == (o["rank"] + (k if phase == 3 else 0)) % R
        got = _run_plan(plan, hd.PLAN_ALLTOALL, R, count, dtype, xs, False, rng)
        for r in range(R):
            assert (got[r] == want[r]).all()
    with pytest.raises(hb.HocclError):
        hd.Plan(hd.PLAN_ALLTOALL, R, count, "fp32", True, 1024, 8)      # no in-place form


@pytest.mark.parametrize("R,n,piece_bytes,max_pieces", [c for c in CASES if c[0] > 1 and c[1] > 0])
def test_forward_variant_plans_execute_to_oracle_bits(oracle, R, n, piece_bytes, max_pieces):
    """Fused sum-and-forward: no moves after step 0, a SUM stores into the next rank's other slot; same bits."""
    rng = random.Random(R * 999 + n)
    xs = W.rank_inputs("uniform", 19, R, n, "fp32")
    want = oracle.ring_allreduce(xs)
    for in_place in (False, True):
        plan = hd.Plan(hd.PLAN_ALLREDUCE_FWD, R, n, "fp32", in_place, piece_bytes, max_pieces)
        rs_moves = [op for op in plan.ops if op["kind"] == hd.OP_MOVE and op["phase"] == 0]
        assert all(op["step"] == 0 for op in rs_moves)
        for op in plan.ops:
            if op["kind"] == hd.OP_SUM and op["step"] < R - 2:
                assert op["dst_rank"] == (op["rank"] + 1) % R and op["dst_buf"] != op["src_buf"]
        for trial in range(2):
            got = _run_plan(plan, hd.PLAN_ALLREDUCE_FWD, R, n, "fp32", xs, in_place, rng)
            for r in range(R):
                assert (got[r].view(np.uint32) == want[r].view(np.uint32)).all(), (R, n, in_place, r)
    if n % R == 0:
        wrs = oracle.ring_reduce_scatter(xs)
        plan = hd.Plan(hd.PLAN_REDUCE_SCATTER_FWD, R, n // R, "fp32", False, piece_bytes, max_pieces)
        got = _run_plan(plan, hd.PLAN_REDUCE_SCATTER_FWD, R, n // R, "fp32", xs, False, rng)
        for r in range(R):
            assert (got[r].view(np.uint32) == wrs[r].view(np.uint32)).all()


@pytest.mark.parametrize("R,n,piece_bytes,max_pieces", [c for c in CASES if c[0] > 1 and c[1] > 0])
def test_direct_allgather_plans(oracle, R, n, piece_bytes, max_pieces):
    """The all-gather as the R-1 permutation stages r -> r+k of its traffic matrix: every rank sends only its own chunk, the
    stages wait for nothing but the chunk being final, the bytes moved equal the ring's, and any legal order gives the bits."""
    rng = random.Random(R * 4242 + n)
    xs = W.rank_inputs("uniform", 29, R, n, "fp32")
    want = oracle.ring_allreduce(xs)
    for kind in (hd.PLAN_ALLREDUCE_AGD, hd.PLAN_ALLREDUCE_FWD_AGD):
        for in_place in (False, True):
            plan = hd.Plan(kind, R, n, "fp32", in_place, piece_bytes, max_pieces)
            ring = hd.Plan(hd.PLAN_ALLREDUCE_FWD if kind == hd.PLAN_ALLREDUCE_FWD_AGD else hd.PLAN_ALLREDUCE, R, n, "fp32", in_place, piece_bytes, max_pieces)
            ag = [op for op in plan.ops if op["phase"] == 1]
            ring_ag = [op for op in ring.ops if op["phase"] == 1]
            assert sum(op["bytes"] for op in ag) == sum(op["bytes"] for op in ring_ag)
            # the reduce-scatter half is the ring's, op for op
            strip = lambda ops: [{k: v for k, v in op.items() if k != "group"} for op in ops if op["phase"] != 1]
            assert strip(plan.ops) == strip(ring.ops)
            sum_groups = {op["group"] for op in plan.ops if op["kind"] == hd.OP_SUM and op["step"] == R - 2}
            for op in ag:
                assert op["kind"] == hd.OP_MOVE and op["chunk"] == op["rank"]                  # a rank sends what it owns
                assert op["dst_rank"] == (op["rank"] + op["step"] + 1) % R != op["rank"]        # stage k = step + 1
                assert op["src_buf"] == hd.BUF_RECV and op["dst_buf"] == hd.BUF_RECV and op["src_off"] == op["dst_off"]
                deps = plan.deps[op["group"]]
                assert len(deps) == 1 and deps[0] in sum_groups                               # no stage waits for another stage
            # every (destination, chunk) pair is served exactly once per piece
            seen = {}
            for op in ag:
                seen.setdefault((op["dst_rank"], op["chunk"]), []).append((op["dst_off"], op["bytes"]))
            q = -(-n // R)
            for d in range(R):
                for c in range(R):
                    size = (min((c + 1) * q, n) - min(c * q, n)) * 4
                    if c == d or size == 0:
                        assert (d, c) not in seen
                        continue
                    spans = sorted(seen[(d, c)])
                    assert spans[0][0] == min(c * q, n) * 4 and sum(b for _, b in spans) == size
                    assert all(a[0] + a[1] == b[0] for a, b in zip(spans, spans[1:]))
            for trial in range(2):
                got = _run_plan(plan, kind, R, n, "fp32", xs, in_place, rng)
                for r in range(R):
                    assert (got[r].view(np.uint32) == want[r].view(np.uint32)).all(), (kind, R, n, in_place, r)


@pytest.mark.parametrize("R", [2, 3, 8])
@pytest.mark.parametrize("count", [1, 7, 3001])
def test_direct_standalone_allgather_plan(oracle, R, count):
    rng = random.Random(R * 31 + count)
    xs = W.rank_inputs("uniform", 37, R, count, "fp32")
    want = oracle.allgather(xs)
    for in_place in (False, True):
        plan = hd.Plan(hd.PLAN_ALLGATHER_DIRECT, R, count, "fp32", in_place, 1024, 8)
        assert all(not d for d in plan.deps)                     # nothing waits for anything
        assert plan.slot_bytes == 0
        for op in plan.ops:
            assert op["kind"] == hd.OP_MOVE and op["chunk"] == op["rank"]
            assert op["src_buf"] == (hd.BUF_RECV if in_place else hd.BUF_SEND)
        for trial in range(2):
            got = _run_plan(plan, hd.PLAN_ALLGATHER_DIRECT, R, count, "fp32", xs, in_place, rng)
            for r in range(R):
                assert (got[r].view(np.uint32) == want[r].view(np.uint32)).all()


@pytest.mark.parametrize("R,n,piece_bytes,max_pieces", [c for c in CASES if c[0] > 1 and c[1] > 0])
def test_direct_reduce_scatter_plans(oracle, R, n, piece_bytes, max_pieces):
    """The reduce-scatter as the R-1 permutation stages of its traffic matrix plus one chain sum per rank: every move leaves
    the sender's own send buffer for the owner's inbox slot (the slot order is the ring's order of addition), nothing waits
    for anything but the moves of its own piece, and any legal order gives the ring's bits."""
    rng = random.Random(R * 515 + n)
    xs = W.rank_inputs("uniform", 41, R, n, "fp32")
    want = oracle.ring_allreduce(xs)
    for flags in (hd.PLAN_FLAG_RS_DIRECT, hd.PLAN_FLAG_RS_DIRECT | hd.PLAN_FLAG_AG_DIRECT):
        kind = hd.PLAN_ALLREDUCE | flags
        for in_place in (False, True):
            align = [(4 * rng.randrange(4)) for _ in range(R)] if in_place else None
            plan = hd.Plan(kind, R, n, "fp32", in_place, piece_bytes, max_pieces, align)
            assert plan.inbox_slots == R - 1
            q = -(-n // R)
            rs_moves = [op for op in plan.ops if op["kind"] == hd.OP_MOVE and op["phase"] == 0]
            chains = [op for op in plan.ops if op["kind"] == hd.OP_CHAIN]
            assert not [op for op in plan.ops if op["kind"] == hd.OP_SUM]
            for op in rs_moves:
                k = op["step"] + 1
                assert op["dst_rank"] == (op["rank"] + k) % R == op["chunk"] and op["src_buf"] == hd.BUF_SEND and op["dst_buf"] == hd.BUF_INBOX
                assert not plan.deps[op["group"]]
                slot = op["dst_off"] // plan.slot_bytes
                assert (op["dst_rank"] + 1 + slot) % R == op["rank"]            # slot j holds source d+1+j: the ring's order
            for op in chains:
                assert op["rank"] == op["dst_rank"] == op["chunk"] and op["nsrc"] == R - 1 and op["src_stride"] == plan.slot_bytes
                assert op["local_buf"] == hd.BUF_SEND and op["dst_buf"] == hd.BUF_RECV
                a = align[op["rank"]] if align else 0
                assert op["src_off"] % 16 == (a + op["local_off"]) % 16          # operands share their 16-byte phase
            moved = sum(op["bytes"] for op in rs_moves)
            assert moved == sum((min((c + 1) * q, n) - min(c * q, n)) * 4 for c in range(R)) * (R - 1)
            for trial in range(2):
                got = _run_plan(plan, kind, R, n, "fp32", xs, in_place, rng)
                for r in range(R):
                    assert (got[r].view(np.uint32) == want[r].view(np.uint32)).all(), (flags, R, n, in_place, r)
    if n % R == 0:
        wrs = oracle.ring_reduce_scatter(xs)
        kind = hd.PLAN_REDUCE_SCATTER | hd.PLAN_FLAG_RS_DIRECT
        for in_place in (False, True):
            plan = hd.Plan(kind, R, n // R, "fp32", in_place, piece_bytes, max_pieces)
            got = _run_plan(plan, kind, R, n // R, "fp32", xs, in_place, rng)
            for r in range(R):
                res = got[r] if not in_place else got[r]
                assert (res.view(np.uint32) == wrs[r].view(np.uint32)).all(), (R, n, in_place, r)
    # flags that do not apply are ignored, unknown ones refused
    assert hd.Plan(hd.PLAN_ALLGATHER | hd.PLAN_FLAG_RS_DIRECT, R, 8, "fp32").inbox_slots == 1
    with pytest.raises(hb.HocclError):
        hd.Plan(hd.PLAN_ALLREDUCE | 256, R, 8, "fp32")


@pytest.mark.parametrize("R,n,piece_bytes,max_pieces", [(4, 4 * (3 << 20) // 4 + 5, 256 << 10, 64), (8, 8 * 700_000 + 3, 384 << 10, 6),
                                                        (2, 2 * 1_000_000, 512 << 10, 3), (3, 3 * 90_000, 256 << 10, 8)])
def test_graded_pieces_cover_the_chunk_and_give_the_ring_bits(oracle, R, n, piece_bytes, max_pieces):
    """PLAN_FLAG_GRADED: the same operations on pieces of unequal size (the outer ones a third and two thirds of a middle one, in
    units of 128 KiB).  The pieces still tile every chunk exactly, every piece keeps its own region of the scratch slots (no
    two regions overlap, every region starts on a 128-byte line), and any legal order gives the ring's bits."""
    rng = random.Random(R * 77 + max_pieces)
    dtype, e = "fp32", 4
    xs = W.rank_inputs("uniform", 43, R, n, dtype)
    want = oracle.ring_allreduce(xs)
    q = -(-n // R)
    for flags in (hd.PLAN_FLAG_RS_DIRECT | hd.PLAN_FLAG_AG_DIRECT, 0):
        kind = hd.PLAN_ALLREDUCE | flags
        plain = hd.Plan(kind, R, n, dtype, False, piece_bytes, max_pieces)
        plan = hd.Plan(kind | hd.PLAN_FLAG_GRADED, R, n, dtype, False, piece_bytes, max_pieces)
        assert plan.scratch_bytes <= hb.scratch_bytes_direct(R, n, dtype) if flags else plan.scratch_bytes <= hb.scratch_bytes(R, n, dtype)
        # the pieces of chunk 0 as the sums see them: contiguous, complete, and (when the chunk is large enough) graded
        sums = sorted((op["local_off"], op["bytes"]) for op in plan.ops if op["kind"] in (hd.OP_CHAIN, hd.OP_SUM) and op["chunk"] == 0
                      and op["rank"] == 0 and (op["kind"] == hd.OP_CHAIN or op["step"] == R - 2))
        assert sums[0][0] == 0 and sum(b for _, b in sums) == min(q, n) * e
        for (o0, b0), (o1, _) in zip(sums, sums[1:]):
            assert o0 + b0 == o1
        sizes = [b for _, b in sums]
        if len(sizes) >= 3 and q * e // len(sizes) >= 256 << 10:
            assert sizes[0] < sizes[1] and sizes[-1] < sizes[-2] and all(b % (128 << 10) == 0 for b in sizes[:-1])
            assert len(sizes) == len([1 for op in plain.ops if op["kind"] in (hd.OP_CHAIN, hd.OP_SUM) and op["chunk"] == 0 and op["rank"] == 0
                                      and (op["kind"] == hd.OP_CHAIN or op["step"] == R - 2)])
        else:
            assert [op for op in plan.ops] == [op for op in plain.ops]          # too small to grade: the plain plan
        # regions of one inbox slot do not overlap and start on 128-byte lines
        regions = sorted((op["dst_off"], op["bytes"]) for op in plan.ops if op["kind"] == hd.OP_MOVE and op["dst_buf"] == hd.BUF_INBOX
                         and op["dst_rank"] == 1 and op["dst_off"] < plan.slot_bytes and (flags or op["step"] == 0))
        for (o0, b0), (o1, _) in zip(regions, regions[1:]):
            assert o0 + b0 <= o1
            if len(sizes) > 1 and min(sizes[:-1]) >= 16 << 10:
                assert (o1 - regions[0][0]) % 128 == 0                 # regions[0][0] is the 16-byte phase of this rank's operand
        got = _run_plan(plan, kind, R, n, dtype, xs, False, rng)
        for r in range(R):
            assert (got[r].view(np.uint32) == want[r].view(np.uint32)).all(), (R, n, flags, r)
