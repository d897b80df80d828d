"""GPU parity for the direct all-gather ("ag_direct" = 1): the all-gather phase as the R-1 permutation stages r -> r+k of
its traffic matrix (the paper's stage decomposition, Sec. 3.4) instead of R-1 dependent ring hops.

The reduce-scatter half is untouched, a rank still sends only what it owns, and the bytes are the same, so every result
must carry the oracle's bits on every path and executor; on the SM path all stages of a piece must go out as one batched
launch (R (R-1) segments, cut only by the segment table)."""
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


CONFIGS = [
    (hb.PATH_CE, dict()),
    (hb.PATH_CE, dict(use_graph=0)),
    (hb.PATH_CE, dict(forward=1)),
    (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=8)),
    (hb.PATH_SM, dict(sum_ctas=148, copy_ctas=148)),
    (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=8, use_graph=0)),
    (hb.PATH_SM, dict(fused=1, sum_ctas=148, copy_ctas=148)),
    (hb.PATH_SM, dict(fused=1, sum_ctas=8, copy_ctas=8)),
    (hb.PATH_SM, dict(forward=1, sum_ctas=32, copy_ctas=32)),
    (hb.PATH_SM, dict(handshake=1, watchdog_ms=5000)),
]


@pytest.mark.parametrize("path,params", CONFIGS)
def test_allreduce_with_direct_allgather(oracle, path, params):
    for dtype in ("fp32", "bf16"):
        e = W.elem_size(dtype)
        for R, n in [(2, 1), (2, 100_003), (3, 5), (4, 262_144 + 9), (8, 8 * 70_000 + 3), (8, 7), (5, 99_999)]:
            xs = W.rank_inputs("uniform", 90 + R, R, n, dtype)
            want = oracle.ring_allreduce(xs)
            comm = make_comm(R, n, dtype, path, ag_direct=1, piece_bytes=65536, max_pieces=4, **params)
            for in_place in (False, True):
                offs = [(r % 4) * e for r in range(R)] if in_place else None
                got = run_allreduce(comm, xs, dtype, in_place=in_place, offs=offs)
                for r in range(R):
                    assert same_bits(got[r], want[r], dtype), (dtype, R, n, in_place, r)
            comm.destroy()


@pytest.mark.parametrize("path,params", [(hb.PATH_CE, dict()), (hb.PATH_CE, dict(use_graph=0)), (hb.PATH_SM, dict(copy_ctas=8)),
                                         (hb.PATH_SM, dict(copy_ctas=148)), (hb.PATH_SM, dict(fused=1, copy_ctas=148))])
def test_standalone_direct_allgather(path, params):
    for dtype in ("fp32", "bf16"):
        e = W.elem_size(dtype)
        for R, count in [(1, 9), (2, 1), (4, 1025), (8, 40_099), (3, 77), (8, 1)]:
            ys = W.rank_inputs("uniform", 45, R, count, dtype)
            cat = np.concatenate(ys)
            comm = make_comm(R, R * count, dtype, path, ag_direct=1, **params)
            gs = [DevBuf(count * e, (r % 3) * e).put(ys[r]) for r in range(R)]
            gr = [DevBuf(R * count * e) for _ in range(R)]
            comm.allgather(gs, gr, count, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert (gr[r].get(np_dtype(dtype)).view(np.uint8) == cat.view(np.uint8)).all(), (dtype, R, count, r)
                assert (gs[r].get(np_dtype(dtype)).view(np.uint8) == ys[r].view(np.uint8)).all()
                assert gr[r].guards_intact() and gs[r].guards_intact()
            gi = [DevBuf(R * count * e) for _ in range(R)]
            for r in range(R):
                gi[r].view[r * count * e:(r + 1) * count * e].copy_(torch.from_numpy(ys[r].view(np.uint8).copy()))
            comm.allgather([gi[r].ptr + r * count * e for r in range(R)], gi, count, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert (gi[r].get(np_dtype(dtype)).view(np.uint8) == cat.view(np.uint8)).all()
                assert gi[r].guards_intact()
            comm.destroy()


def test_sm_path_batches_all_stages_into_one_launch(oracle):
    """R = 8, one piece: the ring all-gather needs 7 copy launches behind each other, the direct one a single fan-out launch
    (8 sources, 7 destinations each); the reduce-scatter half keeps its 7 copy launches.  Same bits either way."""
    R, n, dtype = 8, 8 * 100_000, "bf16"
    xs = W.rank_inputs("normal", 91, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    launches = {}
    for direct in (0, 1):
        comm = make_comm(R, n, dtype, hb.PATH_SM, ag_direct=direct, sum_ctas=148, copy_ctas=148, piece_bytes=1 << 30, max_pieces=1)
        got = run_allreduce(comm, xs, dtype)
        for r in range(R):
            assert same_bits(got[r], want[r], dtype)
        st = comm.last_stats()
        launches[direct] = (st["n_move_launches"], st["n_moves"], st["n_sum_launches"])
        comm.destroy()
    assert launches[0] == (14, 112, 7), launches
    assert launches[1] == (7 + 1, 112, 7), launches


def test_host_allreduce_with_direct_allgather(oracle):
    R, n, dtype = 8, 8 * 200_000 + 5, "bf16"
    xs = W.rank_inputs("normal", 92, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    from test_gpu_host_allreduce import _pinned, _with_staging
    for path, params in [(hb.PATH_CE, dict()), (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=8))]:
        comm = make_comm(R, n, dtype, path, ag_direct=1, host_pieces=4, **params)
        _with_staging(comm, R, n, dtype)
        h_send = [_pinned(x) for x in xs]
        h_recv = [torch.zeros(n * 2, dtype=torch.uint8).pin_memory() for _ in range(R)]
        for rep in range(2):
            comm.host_allreduce(h_send, h_recv, n, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert same_bits(h_recv[r].numpy().view(np.uint16), want[r], dtype), (path, r, rep)
        assert comm.last_stats()["n_pieces"] > 1
        comm.destroy()


@pytest.mark.parametrize("ctas", [1, 8, 148])
def test_fanout_kernel_moves_exact_bytes(ctas):
    """One read, ndst stores: every destination gets the source's bytes, nothing else is touched, whatever the alignment
    (destinations out of phase with the source fall back to bytes, the others keep the vector path)."""
    rng = np.random.default_rng(5)
    for nbytes, ndst in [(1, 1), (15, 3), (16, 2), (4096 + 7, 7), (1_000_003, 7), (3 * 131_072, 31), (70_001, 64)]:
        data = rng.integers(0, 256, nbytes, dtype=np.uint8)
        for offs in ([0] * (ndst + 1), [3] * (ndst + 1), [(5 * k) % 16 for k in range(ndst + 1)]):
            src = DevBuf(nbytes, offs[0]).put(data)
            dsts = [DevBuf(nbytes, offs[1 + d]) for d in range(ndst)]
            assert hd.fanout_launch(src, dsts, nbytes, ctas) == hb.OK
            torch.cuda.synchronize()
            assert (src.get(np.uint8) == data).all() and src.guards_intact()
            for d in dsts:
                assert (d.get(np.uint8) == data).all(), (nbytes, ndst, offs[:3])
                assert d.guards_intact()
    # refused: overlapping destinations, destination over the source, too many destinations
    big = DevBuf(4096)
    assert hd.fanout_launch(big.ptr, [big.ptr + 1024, big.ptr + 1500], 1024, 8) == hb.ERR_INVALID_ARG
    assert hd.fanout_launch(big.ptr, [big.ptr + 512], 1024, 8) == hb.ERR_INVALID_ARG
    assert hd.fanout_launch(big.ptr, [big.ptr + 2048] * 257, 16, 8) == hb.ERR_INVALID_ARG


@pytest.mark.parametrize("use_graph", [0, 1])
def test_many_ranks_need_several_fan_out_launches(oracle, use_graph):
    """R = 20 and 40: R (R-1) = 380 and 1560 destinations, more than one launch carries (256), so chunks and even the
    destinations of one chunk are spread over several launches; odd send alignments put some destinations out of phase."""
    dtype, e = "fp32", 4
    for R, n in [(20, 20 * 300 + 7), (40, 40 * 64 + 1)]:
        xs = W.rank_inputs("uniform", 95, R, n, dtype)
        want = oracle.ring_allreduce(xs)
        comm = make_comm(R, n, dtype, hb.PATH_SM, ag_direct=1, sum_ctas=16, copy_ctas=16, use_graph=use_graph)
        got = run_allreduce(comm, xs, dtype, in_place=True, offs=[(r % 3) * e for r in range(R)])
        for r in range(R):
            assert same_bits(got[r], want[r], dtype), (R, r)
        st = comm.last_stats()
        assert st["n_moves"] == 2 * R * (R - 1)
        comm.destroy()


def test_automatic_choice(oracle):
    """ag_direct = 2: the SM path takes the direct form (one fan-out launch), the copy route takes it only while a ring
    chunk is at most 64 MiB; the bits are the oracle's on both sides of that switch."""
    R, dtype = 8, "bf16"
    n = 8 * 100_000
    xs = W.rank_inputs("normal", 96, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    comm = make_comm(R, n, dtype, hb.PATH_SM, ag_direct=2, sum_ctas=148, copy_ctas=148)
    got = run_allreduce(comm, xs, dtype)
    assert all(same_bits(got[r], want[r], dtype) for r in range(R))
    assert comm.last_stats()["n_move_launches"] == 7 + 1
    comm.destroy()
    R = 2
    for chunk_bytes in ((64 << 20), (64 << 20) + 4096):        # the last size at which the copy route goes direct, and the next
        n = R * chunk_bytes // 2
        xs = W.rank_inputs("normal", 97, R, n, dtype, 1e-3)
        want = oracle.ring_allreduce(xs, threads=oracle.max_threads())
        comm = make_comm(R, n, dtype, hb.PATH_CE, ag_direct=2)
        got = run_allreduce(comm, xs, dtype, in_place=True)
        assert all(same_bits(got[r], want[r], dtype) for r in range(R)), chunk_bytes
        comm.destroy()


def test_config2_bucket_full_size_every_timed_variant(oracle):
    """The gradient bucket at full size (R = 8, 25 MiB bf16 per rank), reduce-scatter then all-gather as the benchmark runs
    it, in every configuration its variant tables time with the direct all-gather (and the ring beside it): all bits
    equal the oracle's."""
    c = W.C2_DP_BUCKET
    R, n, e = c.R, c.count, 2
    xs = W.rank_inputs(c.dist, c.seed, R, n, c.dtype, c.sigma)
    want = oracle.ring_allreduce(xs, threads=oracle.max_threads())
    count = n // R
    send = [DevBuf(n * e).put(xs[r]) for r in range(R)]
    recv = [DevBuf(n * e) for _ in range(R)]
    host = torch.empty(400 << 20, dtype=torch.uint8).pin_memory()
    variants = [(hb.PATH_CE, dict(sum_ctas=8, ag_direct=1)), (hb.PATH_CE, dict(sum_ctas=148, ag_direct=1)),
                (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=8, ag_direct=1)), (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=48, ag_direct=1)),
                (hb.PATH_SM, dict(sum_ctas=148, copy_ctas=148, ag_direct=1)), (hb.PATH_SM, dict(sum_ctas=148, copy_ctas=148, ag_direct=1, forward=1)),
                (hb.PATH_SM, dict(sum_ctas=148, copy_ctas=148, ag_direct=0)), (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=48, ag_direct=2)),
                (hb.PATH_CE_HOST, dict(sum_ctas=8, ag_direct=1))]
    for path, params in variants:
        comm = make_comm(R, n, c.dtype, path, **params)
        if path == hb.PATH_CE_HOST:
            comm.set_host_staging(host)
        for two_calls in (True, False):
            for b in recv:
                b.view.fill_(0)
            if two_calls:
                rs_out = [recv[r].ptr + r * count * e for r in range(R)]
                comm.reduce_scatter(send, rs_out, count, c.dtype)
                comm.allgather(rs_out, recv, count, c.dtype)
            else:
                comm.allreduce(send, recv, n, c.dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert same_bits(recv[r].get(np.uint16), want[r], c.dtype), (path, params, two_calls, r)
                assert recv[r].guards_intact() and send[r].guards_intact()
        comm.destroy()


def test_ordering_kernels_are_counted_and_optional(oracle):
    """Copy route: the graphs carry empty one-warp kernels in front of their first copies and behind groups of copies that
    other copies (or the graph's end) wait for; "order_kernels" = 0 builds the plain graphs.  Same bits either way."""
    R, n, dtype = 8, 8 * 50_000 + 5, "bf16"
    count = n // R
    xs = W.rank_inputs("normal", 98, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    for order, direct in ((1, 0), (0, 0), (1, 1), (0, 1)):
        comm = make_comm(R, n, dtype, hb.PATH_CE, order_kernels=order, ag_direct=direct)
        got = run_allreduce(comm, xs, dtype)
        assert all(same_bits(got[r], want[r], dtype) for r in range(R)), (order, direct)
        st = comm.last_stats()
        # one all-reduce graph: a root in front of the 8 first copies; ring all-gather: a join behind each of the first 6 stages
        # (the next stage waits for it) and one at the end of the graph; direct all-gather: its 7 stages all end the graph and
        # share the one join there
        assert st["n_order_launches"] == ((1 + (1 if direct else 7)) if order else 0), (order, direct, st)
        assert st["n_sum_launches"] == 7 and st["n_move_launches"] == 0 and st["n_moves"] == 112
        comm.destroy()
    # the SM path and the stream executor have none
    for path, params in ((hb.PATH_SM, dict()), (hb.PATH_CE, dict(use_graph=0))):
        comm = make_comm(R, n, dtype, path, **params)
        got = run_allreduce(comm, xs, dtype)
        assert all(same_bits(got[r], want[r], dtype) for r in range(R))
        assert comm.last_stats()["n_order_launches"] == 0
        comm.destroy()
