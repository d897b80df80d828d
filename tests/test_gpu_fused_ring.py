"""GPU parity for the "fused" setting of the SM path: the whole collective as ONE cooperative kernel that walks
the ring steps with grid barriers between them.  Same bits as the oracle for every operation, CTA budget, rank
count, alignment and size class; the collective really is one launch; the barrier words are clean afterwards."""
import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import diag as hd
from paper_2609_34334_b200 import workloads as W
from gpu_util import DevBuf, np_dtype, same_bits
from test_gpu_parity import make_comm, run_allreduce, SMALL

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    torch.cuda.set_device(0)
    yield
    torch.cuda.synchronize()


def fused_comm(R, n, dtype, ctas):
    return make_comm(R, n, dtype, hb.PATH_SM, fused=1, sum_ctas=ctas, copy_ctas=ctas)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("ctas", [1, 8, 148])
def test_fused_allreduce_small_and_ragged(oracle, dtype, ctas):
    for R, n in SMALL:
        xs = W.rank_inputs("uniform", 100 + n % 13, R, n, dtype)
        want = oracle.ring_allreduce(xs)
        comm = fused_comm(R, n, dtype, ctas)
        for in_place in (False, True):
            got = run_allreduce(comm, xs, dtype, in_place)
            for r in range(R):
                assert same_bits(got[r], want[r], dtype), (R, n, r, in_place)
            st = comm.last_stats()
            if R > 1 and n > 0:
                assert st["n_move_launches"] == 1 and st["n_sum_launches"] == 0, st      # one launch for the collective
                assert st["max_copy_ctas"] <= ctas
        assert comm.async_error() == hb.OK
        assert comm.destroy() == hb.OK


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_fused_unaligned_rank_buffers(oracle, dtype):
    e = W.elem_size(dtype)
    R, n = 4, 4 * 3000 + 2
    xs = W.rank_inputs("normal", 5, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    comm = fused_comm(R, n, dtype, 8)
    for offs in ([e, e, e, e], [0, e, 2 * e, 3 * e]):
        got = run_allreduce(comm, xs, dtype, False, offs)
        for r in range(R):
            assert same_bits(got[r], want[r], dtype)
    comm.destroy()


@pytest.mark.parametrize("ctas", [8, 148])
def test_fused_bucket_spans_many_tiles(oracle, ctas):
    """The gradient-bucket workload (R = 8, 25 MiB bf16 per rank): every CTA walks many tiles per phase; replayed."""
    c = W.C2_DP_BUCKET
    R, n = c.R, c.count
    xs = W.rank_inputs(c.dist, c.seed, R, n, c.dtype, c.sigma)
    want = oracle.ring_allreduce(xs, threads=oracle.max_threads())
    comm = fused_comm(R, n, c.dtype, ctas)
    send = [DevBuf(n * 2).put(xs[r]) for r in range(R)]
    recv = [DevBuf(n * 2) for _ in range(R)]
    for rep in range(3):
        for b in recv:
            b.view.fill_(rep)
        comm.allreduce(send, recv, n, c.dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert same_bits(recv[r].get(np.uint16), want[r], c.dtype), (rep, r)
            assert recv[r].guards_intact() and send[r].guards_intact()
    assert comm.last_stats()["graph_hit"] == 1
    assert comm.async_error() == hb.OK
    comm.destroy()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_fused_reduce_scatter_allgather_alltoall(oracle, dtype):
    e = W.elem_size(dtype)
    for R, count in [(1, 9), (2, 1), (4, 1025), (8, 40_003), (3, 77)]:
        xs = W.rank_inputs("uniform", 41, R, R * count, dtype)
        want = oracle.ring_reduce_scatter(xs)
        comm = fused_comm(R, R * count, dtype, 8)
        send = [DevBuf(R * count * e).put(xs[r]) for r in range(R)]
        recv = [DevBuf(count * e) for _ in range(R)]
        comm.reduce_scatter(send, recv, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert same_bits(recv[r].get(np_dtype(dtype)), want[r], dtype)
            assert recv[r].guards_intact() and send[r].guards_intact()
        ys = W.rank_inputs("uniform", 43, R, count, dtype)
        cat = np.concatenate(ys)
        gs = [DevBuf(count * e).put(ys[r]) for r in range(R)]
        gr = [DevBuf(R * count * e) for _ in range(R)]
        comm.allgather(gs, gr, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert (gr[r].get(np_dtype(dtype)).view(np.uint8) == cat.view(np.uint8)).all()
            assert gr[r].guards_intact()
        wa = oracle.alltoall(xs)
        ar = [DevBuf(R * count * e) for _ in range(R)]
        comm.alltoall(send, ar, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert (ar[r].get(np_dtype(dtype)).view(np.uint8) == wa[r].view(np.uint8)).all()
            assert ar[r].guards_intact()
        assert comm.async_error() == hb.OK
        comm.destroy()


@pytest.mark.parametrize("R", [10, 16])
def test_fused_many_ranks(oracle, R):
    """10 ranks need the large parameter block; 16 ranks do not fit one launch and fall back to the graph."""
    for dtype, n in (("bf16", R * 1000 + 5), ("fp32", R * 257)):
        xs = W.rank_inputs("uniform", 500 + R, R, n, dtype)
        want = oracle.ring_allreduce(xs)
        comm = fused_comm(R, n, dtype, 8)
        got = run_allreduce(comm, xs, dtype)
        for r in range(R):
            assert same_bits(got[r], want[r], dtype), (R, dtype, r)
        st = comm.last_stats()
        assert (st["n_sum_launches"] == 0) == (R == 10), st
        comm.destroy()


def test_fused_forward_variant_and_stream_order(oracle):
    """forward = 1 inside the one kernel (a SUM stores into the next rank's inbox), and ordering against
    neighbouring work on the caller's stream."""
    R, n, dtype = 8, 8 * 50_000 + 3, "bf16"
    xs = W.rank_inputs("normal", 9, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    comm = make_comm(R, n, dtype, hb.PATH_SM, fused=1, forward=1, sum_ctas=8, copy_ctas=8)
    got = run_allreduce(comm, xs, dtype)
    for r in range(R):
        assert same_bits(got[r], want[r], dtype)
    comm.destroy()
    comm = fused_comm(R, n, dtype, 8)
    stream = torch.cuda.Stream()
    send = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    recv = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    host = [torch.from_numpy(x.view(np.int16)).cuda() for x in xs]
    torch.cuda.synchronize()
    with torch.cuda.stream(stream):
        for r in range(R):
            send[r].copy_(host[r])                       # producer on the same stream, just before the call
        comm.allreduce(send, recv, n, dtype, stream)
        outs = [recv[r].clone() for r in range(R)]       # consumer on the same stream, just after
    stream.synchronize()
    for r in range(R):
        assert same_bits(outs[r].cpu().numpy().view(np.uint16), want[r], dtype)
    comm.destroy()


def test_bounded_barrier_wait_runs_out_and_is_reported(oracle):
    """Failure detection without a GPU fault: a barrier that waits for an arrival nobody makes.  Every CTA gives up
    after its bounded number of polls, the kernel ends by itself, the phase behind the barrier does not run, the
    status says TIMEOUT, and the communicator works normally afterwards (the barrier words were cleaned)."""
    import time
    R, n, dtype = 4, 4 * 5000 + 1, "fp32"
    comm = fused_comm(R, n, dtype, 8)
    nbytes = 1 << 20
    src = torch.full((nbytes,), 7, dtype=torch.uint8, device="cuda")
    dst = torch.zeros(nbytes, dtype=torch.uint8, device="cuda")
    assert comm.async_error() == hb.OK
    t0 = time.time()
    assert hd.selftest_barrier_timeout(comm, dst, src, nbytes) == hb.OK
    torch.cuda.synchronize()
    waited = time.time() - t0
    assert 0.05 < waited < 30.0, waited                       # it really waited, and it really stopped by itself
    assert comm.async_error() == hb.ERR_TIMEOUT
    assert bool((dst[:nbytes // 2] == 7).all()) and bool((dst[nbytes // 2:] == 0).all())
    assert comm.async_error(clear=True) == hb.ERR_TIMEOUT
    assert comm.async_error() == hb.OK
    xs = W.rank_inputs("uniform", 31, R, n, dtype)
    want = oracle.ring_allreduce(xs)
    got = run_allreduce(comm, xs, dtype)
    for r in range(R):
        assert same_bits(got[r], want[r], dtype)
    assert comm.async_error() == hb.OK
    assert comm.destroy() == hb.OK
