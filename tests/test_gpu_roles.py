"""GPU parity for the "roles" setting: all-reduce and reduce-scatter of the stage-decomposed schedule (paper Sec. 3.4: the traffic
matrix cut into permutation stages; Sec. 3.3: chunk pipelining) as ONE cooperative kernel whose first CTAs only sum and whose
other CTAs only move, pipelined over pieces through counters in device memory.

The order of the adds and every rounding are the ring's, so every result must carry the oracle's bits: for both dtypes, in
place, with ragged sizes, misaligned buffers, one piece and many pieces, few and many CTAs of either role, on the first call and
on the replay.  The waits of the kernel are bounded: a wait for a mover that does not exist runs out, the kernel ends by itself
and the communicator reports it (no GPU fault involved)."""
import time

import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import diag as hd
from paper_2609_34334_b200 import workloads as W
from gpu_util import DevBuf, np_dtype, same_bits
from test_gpu_parity import make_comm, run_allreduce

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    torch.cuda.set_device(0)
    yield
    torch.cuda.synchronize()


def roles_comm(R, n, dtype, **params):
    params.setdefault("sum_ctas", 8)
    params.setdefault("copy_ctas", 16)
    return make_comm(R, n, dtype, hb.PATH_SM, roles=1, rs_direct=1, **params)


BUDGETS = [dict(), dict(sum_ctas=1, copy_ctas=1), dict(sum_ctas=3, copy_ctas=5), dict(sum_ctas=8, copy_ctas=40), dict(sum_ctas=64, copy_ctas=84)]


@pytest.mark.parametrize("budget", BUDGETS)
def test_allreduce_in_one_kernel_with_roles(oracle, budget):
    for dtype in ("fp32", "bf16"):
        e = W.elem_size(dtype)
        for R, n, piece in [(2, 1, 0), (2, 100_003, 65536), (3, 5, 0), (4, 262_144 + 9, 65536), (8, 8 * 70_000 + 3, 32768), (8, 7, 0), (5, 99_999, 4096),
                            (8, 8 * 600_000 + 5, 0), (7, 7 * 3000, 1024)]:
            xs = W.rank_inputs("uniform", 290 + R, R, n, dtype)
            want = oracle.ring_allreduce(xs)
            extra = dict(piece_bytes=piece) if piece else {}
            comm = roles_comm(R, n, dtype, **budget, **extra)
            for in_place in (False, True):
                offs = [(r % 4) * e for r in range(R)] if in_place else None
                got = run_allreduce(comm, xs, dtype, in_place=in_place, offs=offs)
                for r in range(R):
                    assert same_bits(got[r], want[r], dtype), (dtype, R, n, in_place, r)
                st = comm.last_stats()
                assert st["n_move_launches"] == 1 and st["n_sum_launches"] == 0, st          # one launch carries everything
                assert st["max_sum_ctas"] == budget.get("sum_ctas", 8) and st["max_copy_ctas"] == budget.get("copy_ctas", 16), st
            if piece and n * e // R > piece:
                assert st["n_pieces"] > 1, st
            assert comm.async_error() == hb.OK
            assert comm.destroy() == hb.OK


def test_replays_and_back_to_back_calls(oracle):
    """The second call of a signature replays the cached table; calls on one stream follow each other without a host wait, each
    with its own table in the same device area, and the counters of one launch are clean for the next."""
    R, dtype = 8, "bf16"
    e = W.elem_size(dtype)
    sizes = [8 * 300_000 + 1, 8 * 40_000, 8 * 300_000 + 1, 13, 8 * 40_000]
    comm = roles_comm(R, max(sizes), dtype, copy_ctas=24)
    stream = torch.cuda.Stream()
    cases = []
    for k, n in enumerate(sizes):
        xs = W.rank_inputs("uniform", 300 + (k % 3), R, n, dtype)
        send = [DevBuf(n * e).put(xs[r]) for r in range(R)]
        recv = [DevBuf(n * e) for r in range(R)]
        cases.append((n, xs, send, recv))
    hits = []
    for rep in range(2):
        for n, xs, send, recv in cases:
            comm.allreduce(send, recv, n, dtype, stream)
            hits.append(comm.last_stats()["graph_hit"])
    stream.synchronize()
    assert hits == [0] * len(sizes) + [1] * len(sizes)
    for n, xs, send, recv in cases:
        want = oracle.ring_allreduce(xs)
        for r in range(R):
            assert same_bits(recv[r].get(np_dtype(dtype)), want[r], dtype), (n, r)
            assert recv[r].guards_intact() and send[r].guards_intact()
    assert comm.async_error() == hb.OK
    assert comm.destroy() == hb.OK


def test_reduce_scatter_in_one_kernel_with_roles(oracle):
    for dtype in ("fp32", "bf16"):
        e = W.elem_size(dtype)
        for R, count, piece in [(2, 1, 0), (4, 1025, 2048), (8, 4099, 2048), (3, 77, 0), (8, 250_000, 0)]:
            xs = W.rank_inputs("uniform", 241, R, R * count, dtype)
            want = oracle.ring_reduce_scatter(xs)
            comm = roles_comm(R, R * count, dtype, **(dict(piece_bytes=piece) if piece else {}))
            send = [DevBuf(R * count * e).put(xs[r]) for r in range(R)]
            recv = [DevBuf(count * e, (r % 2) * e) for r in range(R)]
            comm.reduce_scatter(send, recv, count, dtype)
            torch.cuda.synchronize()
            assert comm.last_stats()["n_move_launches"] == 1 and comm.last_stats()["n_sum_launches"] == 0
            for r in range(R):
                assert same_bits(recv[r].get(np_dtype(dtype)), want[r], dtype), (dtype, R, count, r)
                assert recv[r].guards_intact() and send[r].guards_intact()
                assert (send[r].get(np_dtype(dtype)).view(np.uint8) == xs[r].view(np.uint8)).all(), "send buffer was written"
            comm.reduce_scatter(send, [send[r].ptr + r * count * e for r in range(R)], count, dtype)      # in place
            torch.cuda.synchronize()
            for r in range(R):
                assert same_bits(send[r].get(np_dtype(dtype))[r * count:(r + 1) * count], want[r], dtype)
            assert comm.destroy() == hb.OK


def test_special_values(oracle):
    for dtype in ("fp32", "bf16"):
        R, n = 4, 4 * 2048 + 3
        xs = W.rank_inputs("uniform", 295, R, n, dtype)
        special = np.array([np.nan, np.inf, -np.inf, 0.0, -0.0, 1e-40, -1e-40, 3.0e38, -3.0e38, 1.0], dtype=np.float32)
        for r in range(R):
            v = np.roll(special, r)
            if dtype == "fp32":
                xs[r][:v.size] = v
            else:
                xs[r][:v.size] = (v.view(np.uint32) >> 16).astype(np.uint16)
        want = oracle.ring_allreduce(xs)
        comm = roles_comm(R, n, dtype)
        got = run_allreduce(comm, xs, dtype)
        for r in range(R):
            assert same_bits(got[r], want[r], dtype)
        assert comm.destroy() == hb.OK


def test_what_the_roles_kernel_does_not_serve_is_refused_or_left_to_the_graph(oracle):
    R, n, dtype = 4, 4096, "fp32"
    send = [DevBuf(n * 4) for _ in range(R)]
    recv = [DevBuf(n * 4, fill=0x3C) for _ in range(R)]
    # contradictions: nothing is enqueued
    for path, extra in ((hb.PATH_CE, {}), (hb.PATH_SM, dict(fused=1)), (hb.PATH_SM, dict(forward=1)), (hb.PATH_SM, dict(onepass=1)),
                        (hb.PATH_SM, dict(handshake=1)), (hb.PATH_SM, dict(rs_direct=0)), (hb.PATH_SM, dict(ag_direct=0))):
        params = dict(roles=1, rs_direct=2)
        params.update(extra)
        comm = make_comm(R, n, dtype, path, **params)
        assert comm.allreduce_rc(send, recv, n, dtype) == hb.ERR_UNSUPPORTED, (path, extra)
        torch.cuda.synchronize()
        assert all((b.get(np.uint8) == 0x3C).all() for b in recv)
        comm.destroy()
    # the scratch of the ring form is too small for the direct form's R - 1 inbox slots
    comm = make_comm(R, n, dtype, hb.PATH_SM, roles=1)
    assert comm.allreduce_rc(send, recv, n, dtype) == hb.ERR_SCRATCH
    comm.destroy()
    # more CTAs than can be resident together: the same schedule runs as a graph of kernels, same bits
    xs = W.rank_inputs("uniform", 296, R, n, dtype)
    want = oracle.ring_allreduce(xs)
    comm = roles_comm(R, n, dtype, sum_ctas=8, copy_ctas=512)
    got = run_allreduce(comm, xs, dtype)
    assert comm.last_stats()["n_sum_launches"] >= 1
    for r in range(R):
        assert same_bits(got[r], want[r], dtype)
    # calls without a reduction ignore the setting
    count = n // R
    gs = [DevBuf(count * 4).put(xs[r][:count]) for r in range(R)]
    gr = [DevBuf(n * 4) for _ in range(R)]
    comm.allgather(gs, gr, count, dtype)
    torch.cuda.synchronize()
    for r in range(R):
        assert (gr[r].get(np.float32).view(np.uint32) == np.concatenate([xs[j][:count] for j in range(R)]).view(np.uint32)).all()
    assert comm.destroy() == hb.OK


def test_a_wait_that_nobody_answers_runs_out_and_is_reported(oracle):
    """Failure detection without a GPU fault: the summing CTAs wait for one mover more than the grid has.  They give up after their
    bounded number of polls, the movers that wait for those sums see the give-up flag and leave, the kernel ends by itself, the
    status says TIMEOUT, and the communicator works normally afterwards (the counters were cleaned)."""
    R, n, dtype = 4, 4 * 50_000 + 1, "fp32"
    comm = roles_comm(R, n, dtype)
    xs = W.rank_inputs("uniform", 297, R, n, dtype)
    send = [DevBuf(n * 4).put(xs[r]) for r in range(R)]
    recv = [DevBuf(n * 4, fill=0x3C) for _ in range(R)]
    assert comm.async_error() == hb.OK
    t0 = time.time()
    assert hd.selftest_roles_timeout(comm, send, recv, n, dtype) == hb.OK
    torch.cuda.synchronize()
    waited = time.time() - t0
    assert 0.05 < waited < 30.0, waited                       # it really waited, and it really stopped by itself
    assert comm.async_error() == hb.ERR_TIMEOUT
    assert all((b.get(np.uint8) == 0x3C).all() for b in recv)  # no sum ran, so no all-gather move ran either
    assert all(b.guards_intact() for b in send + recv)
    assert comm.async_error(clear=True) == hb.ERR_TIMEOUT
    assert comm.async_error() == hb.OK
    want = oracle.ring_allreduce(xs)
    comm.allreduce(send, recv, n, dtype)
    torch.cuda.synchronize()
    for r in range(R):
        assert same_bits(recv[r].get(np.float32), want[r], dtype)
    assert comm.async_error() == hb.OK
    assert comm.destroy() == hb.OK
