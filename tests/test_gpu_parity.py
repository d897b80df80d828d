"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element.

Bar: bit-exact for moves, gathers and point-to-point; bit-exact for sums taken in the fixed ring
order (NaN matches NaN regardless of payload); and, as a sanity net, within (R-1)*2^-24 * sum|x| of
an fp64 sum for fp32 (looser stated tolerance: 2e-6 * R) and within gamma_{R-1}(2^-8) * sum|x| for bf16.
"""
import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import diag as hd
from paper_2609_34334_b200 import workloads as W
from gpu_util import DevBuf, np_dtype, same_bits

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    torch.cuda.set_device(0)
    yield
    torch.cuda.synchronize()


def make_comm(R, count, dtype, path=hb.PATH_CE, **params):
    """Communicator with guarded scratch for buffers of up to `count` elements (allreduce convention)."""
    comm = hb.Comm(R, 0)
    comm.set_path(path)
    # these tests are small: without this, every call on the copy route would take the small-message rule and run on the
    # copy kernel; the rule has tests of its own (test_small_messages_on_the_copy_route)
    params.setdefault("ce_small_bytes", 0)
    for k, v in params.items():
        comm.set_param(k, v)
    nb = hb.scratch_bytes_direct(R, count, dtype) if params.get("rs_direct") else hb.scratch_bytes(R, count, dtype)
    scratch = DevBuf(nb + 256)
    pad = (-scratch.ptr) % 256
    comm._scratch_keep = scratch
    if nb:
        assert hb.lib().hoccl_comm_set_scratch(comm._h, scratch.ptr + pad, nb) == hb.OK
    return comm


def run_allreduce(comm, xs, dtype, in_place=False, offs=None, stream=None):
    R, n = len(xs), xs[0].size
    e = W.elem_size(dtype)
    offs = offs or [0] * R
    send = [DevBuf(n * e, offs[r]).put(xs[r]) for r in range(R)]
    recv = send if in_place else [DevBuf(n * e, offs[r]) for r in range(R)]
    comm.allreduce(send, recv, n, dtype, stream)
    torch.cuda.synchronize()
    for b in send + recv + [comm._scratch_keep]:
        assert b.guards_intact()
    if not in_place:
        for r in range(R):
            assert (send[r].get(np_dtype(dtype)).view(np.uint8) == xs[r].view(np.uint8)).all(), "send buffer was written"
    return [b.get(np_dtype(dtype)) for b in recv]


# ------------------------------------------------------------------------------- kernels ----------
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("ctas", [1, 8, 148])
def test_sum_kernel_against_oracle(oracle, dtype, ctas):
    e = W.elem_size(dtype)
    sizes = [1, 3, 4, 7, 8, 9, 1023, 4096, 8 * 1024 * 16 // e + 5, 1_000_003]
    for n in sizes:
        a, b = W.rank_inputs("uniform", 31 + n % 7, 2, n, dtype)
        want = oracle.ring_allreduce([b, a])[0]       # R = 2: one add, inbox + local
        for offs in ((0, 0, 0), (e, e, e), (16 - e, 16 - e, 16 - e), (0, e, 0), (e, 0, 2 * e)):
            A = DevBuf(n * e, offs[0]).put(a)
            B = DevBuf(n * e, offs[1]).put(b)
            O = DevBuf(n * e, offs[2])
            assert hd.sum_launch(A, B, O, n, dtype, ctas) == hb.OK
            torch.cuda.synchronize()
            assert same_bits(O.get(np_dtype(dtype)), want, dtype), (n, offs)
            assert A.guards_intact() and B.guards_intact() and O.guards_intact()


@pytest.mark.parametrize("ctas", [1, 8, 32])
def test_copy_kernel_is_identity(ctas):
    rng = np.random.default_rng(3)
    for nbytes in [1, 15, 16, 17, 4095, 65536 + 3, 3_000_001]:
        src = rng.integers(0, 256, size=nbytes, dtype=np.uint8)
        for so, do in ((0, 0), (1, 1), (3, 3), (5, 2), (0, 9)):
            S = DevBuf(nbytes, so).put(src)
            D = DevBuf(nbytes, do)
            assert hd.copy_launch(S, D, nbytes, ctas) == hb.OK
            torch.cuda.synchronize()
            assert (D.get(np.uint8) == src).all() and D.guards_intact() and S.guards_intact()


def test_sum_kernel_special_values(oracle):
    inf, nan = np.float32(np.inf), np.float32(np.nan)
    tiny = np.float32(1e-45)
    a = np.array([inf, nan, -0.0, tiny, 1.0, -inf, 3e38, 1e-40, 1.17549435e-38] * 5, dtype=np.float32)
    b = np.array([1.0, 1.0, -0.0, tiny, -1.0, inf, 3e38, -3e-41, -1e-45] * 5, dtype=np.float32)
    want = oracle.ring_allreduce([b, a])[0]
    A, B, O = DevBuf(a.nbytes).put(a), DevBuf(b.nbytes).put(b), DevBuf(a.nbytes)
    assert hd.sum_launch(A, B, O, a.size, "fp32", 8) == hb.OK
    torch.cuda.synchronize()
    got = O.get(np.float32)
    assert same_bits(got, want, "fp32")
    assert got[3] != 0 and got[7] != 0            # subnormals are not flushed
    # bf16: subnormal and tie cases through the packed path and the scalar path
    hb16 = np.array([0x0001, 0x8001, 0x0080, 0x7F7F, 0x4380, 0x3F80, 0x7F80, 0x7FC0, 0x8000] * 3, dtype=np.uint16)
    gb16 = np.array([0x0001, 0x0001, 0x8001, 0x7F7F, 0x3F80, 0x3B80, 0xFF80, 0x3F80, 0x8000] * 3, dtype=np.uint16)
    want = oracle.ring_allreduce([gb16, hb16])[0]
    A, B, O = DevBuf(hb16.nbytes).put(hb16), DevBuf(gb16.nbytes).put(gb16), DevBuf(hb16.nbytes)
    assert hd.sum_launch(A, B, O, hb16.size, "bf16", 8) == hb.OK
    torch.cuda.synchronize()
    assert same_bits(O.get(np.uint16), want, "bf16")


# ------------------------------------------------------------------------------- collectives ------
SMALL = [(1, 5), (2, 1), (2, 4099), (3, 10), (4, 3), (4, 4 * 4096 + 3), (5, 12345), (8, 7), (8, 70001)]


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("path", [hb.PATH_CE, hb.PATH_SM])
@pytest.mark.parametrize("use_graph", [0, 1])
def test_allreduce_small_and_ragged(oracle, dtype, path, use_graph):
    for R, n in SMALL:
        xs = W.rank_inputs("uniform", 100 + n % 13, R, n, dtype)
        want = oracle.ring_allreduce(xs)
        comm = make_comm(R, n, dtype, path, use_graph=use_graph, piece_bytes=4096, max_pieces=3)
        for in_place in (False, True):
            got = run_allreduce(comm, xs, dtype, in_place)
            for r in range(R):
                assert same_bits(got[r], want[r], dtype), (R, n, r, in_place)
        assert comm.destroy() == hb.OK


@pytest.mark.parametrize("R", [16, 33, 64])
def test_many_ranks_split_a_step_over_several_launches(oracle, R):
    """More than 32 ranks: the segments of one ring step no longer fit one batched launch."""
    for dtype, n in (("bf16", R * 1000 + 5), ("fp32", R * 257)):
        xs = W.rank_inputs("uniform", 500 + R, R, n, dtype)
        want = oracle.ring_allreduce(xs)
        for path in (hb.PATH_CE, hb.PATH_SM):
            for use_graph in (1, 0):
                comm = make_comm(R, n, dtype, path, use_graph=use_graph, piece_bytes=2048, max_pieces=2)
                got = run_allreduce(comm, xs, dtype)
                for r in range(R):
                    assert same_bits(got[r], want[r], dtype), (R, dtype, path, use_graph, r)
                comm.destroy()
        comm = make_comm(R, n, dtype, hb.PATH_CE, onepass=1)
        got = run_allreduce(comm, xs, dtype)
        assert all(same_bits(got[r], want[r], dtype) for r in range(R))
        comm.destroy()
        count = 100
        ys = W.rank_inputs("uniform", 600 + R, R, R * count, dtype)
        wa = oracle.alltoall(ys)
        comm = hb.Comm(R, 0)
        e = W.elem_size(dtype)
        send = [DevBuf(R * count * e).put(ys[r]) for r in range(R)]
        recv = [DevBuf(R * count * e) for _ in range(R)]
        comm.alltoall(send, recv, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert (recv[r].get(np_dtype(dtype)).view(np.uint8) == wa[r].view(np.uint8)).all()
        comm.destroy()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_allreduce_unaligned_rank_buffers(oracle, dtype):
    e = W.elem_size(dtype)
    R, n = 4, 4 * 3000 + 2
    xs = W.rank_inputs("normal", 5, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    comm = make_comm(R, n, dtype, hb.PATH_CE, piece_bytes=2048, max_pieces=4)
    for offs in ([e, e, e, e], [0, e, 2 * e, 3 * e]):
        got = run_allreduce(comm, xs, dtype, False, offs)
        for r in range(R):
            assert same_bits(got[r], want[r], dtype)
    comm.destroy()


def test_config1_allreduce_r4_fp32(oracle):
    """R=4, 1,048,576 fp32 per rank, uniform[-1,1), seed 0: every path and executor, bit for bit."""
    c = W.C1_SMALL_ALLREDUCE
    xs = W.rank_inputs(c.dist, c.seed, c.R, c.count, c.dtype)
    want = oracle.ring_allreduce(xs)
    s64, a64 = oracle.sum_f64(xs)
    for path in (hb.PATH_CE, hb.PATH_SM):
        for use_graph in (1, 0):
            comm = make_comm(c.R, c.count, c.dtype, path, use_graph=use_graph)
            got = run_allreduce(comm, xs, c.dtype)
            for r in range(c.R):
                assert same_bits(got[r], want[r], c.dtype)
            err = np.abs(got[0].astype(np.float64) - s64)
            assert (err <= (c.R - 1) * 2.0 ** -24 * a64 * 1.0000001).all()
            assert (err <= 2e-6 * c.R * a64).all()
            st = comm.last_stats()
            assert st["n_sum_launches"] == (c.R - 1) * st["n_pieces"]
            assert st["max_sum_ctas"] <= 8
            comm.destroy()


def test_config2_bucket_rs_then_ag_equals_allreduce(oracle):
    """R=8, 25 MiB bf16 bucket per rank: reduce_scatter then allgather (two calls) == one allreduce == oracle."""
    c = W.C2_DP_BUCKET
    R, n, e = c.R, c.count, 2
    xs = W.rank_inputs(c.dist, c.seed, R, n, c.dtype, c.sigma)
    want = oracle.ring_allreduce(xs, threads=oracle.max_threads())
    s64, a64 = oracle.sum_f64([x[:1 << 16] for x in xs])
    count = n // R
    comm = make_comm(R, n, c.dtype, hb.PATH_CE)       # the benchmark's launch configuration (defaults)
    send = [DevBuf(n * e).put(xs[r]) for r in range(R)]
    recv = [DevBuf(n * e) for _ in range(R)]
    # two calls: reduce-scatter into chunk r of recv[r] (the NCCL in-place all-gather layout), then all-gather in place
    rs_out = [recv[r].ptr + r * count * e for r in range(R)]
    comm.reduce_scatter(send, rs_out, count, c.dtype)
    comm.allgather(rs_out, recv, count, c.dtype)
    torch.cuda.synchronize()
    two = [b.get(np.uint16) for b in recv]
    for r in range(R):
        assert same_bits(two[r], want[r], c.dtype), r
        assert recv[r].guards_intact() and send[r].guards_intact()
    for b in recv:
        b.view.fill_(0)
    comm.allreduce(send, recv, n, c.dtype)
    comm.allreduce(send, recv, n, c.dtype)            # replay of the cached graph
    torch.cuda.synchronize()
    assert comm.last_stats()["graph_hit"] == 1
    for r in range(R):
        assert same_bits(recv[r].get(np.uint16), want[r], c.dtype), r
    got = oracle.bf16_bits_to_f32(two[0][:1 << 16]).astype(np.float64)
    u = 2.0 ** -8
    assert (np.abs(got - s64) <= (R - 1) * u / (1 - (R - 1) * u) * a64).all()
    comm.destroy()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("path", [hb.PATH_CE, hb.PATH_SM])
def test_reduce_scatter_and_allgather(oracle, dtype, path):
    e = W.elem_size(dtype)
    for R, count in [(1, 9), (2, 1), (4, 1025), (8, 4099), (3, 77)]:
        xs = W.rank_inputs("uniform", 41, R, R * count, dtype)
        want = oracle.ring_reduce_scatter(xs)
        comm = make_comm(R, R * count, dtype, path, piece_bytes=2048, max_pieces=5)
        send = [DevBuf(R * count * e).put(xs[r]) for r in range(R)]
        recv = [DevBuf(count * e) for _ in range(R)]
        comm.reduce_scatter(send, recv, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert same_bits(recv[r].get(np_dtype(dtype)), want[r], dtype)
            assert recv[r].guards_intact() and send[r].guards_intact()
        # in place: recv[r] = send[r] + r*count
        comm.reduce_scatter(send, [send[r].ptr + r * count * e for r in range(R)], count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert same_bits(send[r].get(np_dtype(dtype))[r * count:(r + 1) * count], want[r], dtype)
        # all-gather, out of place and in place
        ys = W.rank_inputs("uniform", 43, R, count, dtype)
        cat = np.concatenate(ys)
        gs = [DevBuf(count * e).put(ys[r]) for r in range(R)]
        gr = [DevBuf(R * count * e) for _ in range(R)]
        comm.allgather(gs, gr, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert (gr[r].get(np_dtype(dtype)).view(np.uint8) == cat.view(np.uint8)).all()
            assert (gs[r].get(np_dtype(dtype)).view(np.uint8) == ys[r].view(np.uint8)).all()
            assert gr[r].guards_intact()
        gi = [DevBuf(R * count * e) for _ in range(R)]
        for r in range(R):
            gi[r].view[r * count * e:(r + 1) * count * e].copy_(torch.from_numpy(ys[r].view(np.uint8).copy()))
        comm.allgather([gi[r].ptr + r * count * e for r in range(R)], gi, count, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert (gi[r].get(np_dtype(dtype)).view(np.uint8) == cat.view(np.uint8)).all()
        comm.destroy()


@pytest.mark.parametrize("path", [hb.PATH_CE, hb.PATH_SM])
@pytest.mark.parametrize("use_graph", [0, 1])
def test_alltoall(oracle, path, use_graph):
    for dtype in ("fp32", "bf16"):
        e = W.elem_size(dtype)
        for R, count in [(1, 7), (2, 1), (4, 4099), (8, 100_003), (5, 33)]:
            xs = W.rank_inputs("uniform", 83, R, R * count, dtype)
            want = oracle.alltoall(xs)
            comm = hb.Comm(R, 0)
            comm.set_path(path)
            comm.set_param("use_graph", use_graph)
            send = [DevBuf(R * count * e, (r % 3) * e).put(xs[r]) for r in range(R)]
            recv = [DevBuf(R * count * e) for _ in range(R)]
            comm.alltoall(send, recv, count, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert (recv[r].get(np_dtype(dtype)).view(np.uint8) == want[r].view(np.uint8)).all(), (R, count, r)
                assert recv[r].guards_intact() and send[r].guards_intact()
                assert (send[r].get(np_dtype(dtype)).view(np.uint8) == xs[r].view(np.uint8)).all()
            assert comm.alltoall_rc(send, send, count, dtype) == hb.ERR_INVALID_ARG       # no in-place form
            assert comm.destroy() == hb.OK


@pytest.mark.parametrize("use_graph", [0, 1])
@pytest.mark.parametrize("path", [hb.PATH_CE, hb.PATH_SM])
def test_alltoallv_user_defined_pattern(oracle, path, use_graph):
    from test_oracle_pins import _random_pattern
    for dtype in ("fp32", "bf16"):
        e = W.elem_size(dtype)
        for R, max_count, piece in [(2, 100, 65536), (4, 200_000, 65536), (8, 60_000, 131072), (5, 3, 65536)]:
            rng = np.random.default_rng(R * 7 + max_count)
            counts, sd, rd, send_sizes, recv_sizes = _random_pattern(R, rng, max_count)
            xs = [W.uniform(56, u, send_sizes[u], dtype) for u in range(R)]
            fill = np.frombuffer(bytes([0xA5]) * e, dtype=np_dtype(dtype))[0]
            want = oracle.alltoallv(xs, counts.ravel(), sd.ravel(), rd.ravel(), recv_sizes, fill=fill)
            comm = hb.Comm(R, 0)
            comm.set_path(path)
            comm.set_param("piece_bytes", piece)
            comm.set_param("use_graph", use_graph)
            send = [DevBuf(send_sizes[u] * e).put(xs[u]) for u in range(R)]
            recv = [DevBuf(recv_sizes[v] * e) for v in range(R)]           # DevBuf pre-fills with 0xA5 bytes
            for rep in range(2):                                           # the second call replays the cached graph
                if rep:
                    for v in range(R):
                        recv[v].view.fill_(0xA5)
                comm.alltoallv(send, counts.ravel(), sd.ravel(), recv, rd.ravel(), dtype)
                torch.cuda.synchronize()
                if counts.sum() > 0:
                    assert comm.last_stats()["graph_hit"] == (1 if (rep and use_graph) else 0)
                for v in range(R):
                    assert (recv[v].get(np_dtype(dtype)).view(np.uint8) == want[v].view(np.uint8)).all(), (R, v, rep)
                    assert recv[v].guards_intact() and send[v].guards_intact()
            # overlapping receive regions are refused
            bad = rd.copy()
            if R >= 2 and counts[0, 1] > 0 and counts[1, 1] > 0:
                bad[1, 0] = bad[1, 1]
                assert comm.alltoallv_rc(send, counts.ravel(), sd.ravel(), recv, bad.ravel(), dtype) == hb.ERR_INVALID_ARG
            assert comm.destroy() == hb.OK


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_onepass_reduction_gives_the_ring_bits(oracle, dtype):
    """The one-kernel comparison variant reduces in the ring's order and rounding: same bits as the oracle."""
    e = W.elem_size(dtype)
    for R, n in SMALL + [(8, 8 * 65_536), (4, 4 * 100_000 + 8), (7, 7 * 4096)]:
        xs = W.rank_inputs("normal", 300 + n % 11, R, n, dtype, 1.0)
        want = oracle.ring_allreduce(xs)
        for ctas in (3, 148):
            comm = make_comm(R, n, dtype, hb.PATH_CE, onepass=1, sum_ctas=ctas)
            for in_place in (False, True):
                got = run_allreduce(comm, xs, dtype, in_place)
                for r in range(R):
                    assert same_bits(got[r], want[r], dtype), (R, n, r, in_place, ctas)
            offs = [e * (r % 3) for r in range(R)]              # unaligned buffers take the element-wise path
            got = run_allreduce(comm, xs, dtype, False, offs)
            for r in range(R):
                assert same_bits(got[r], want[r], dtype)
            assert comm.last_stats()["n_sum_launches"] == 1 and comm.last_stats()["n_moves"] == 0
            if n % R == 0:
                count = n // R
                wrs = oracle.ring_reduce_scatter(xs)
                send = [DevBuf(n * e).put(xs[r]) for r in range(R)]
                recv = [DevBuf(count * e) for _ in range(R)]
                comm.reduce_scatter(send, recv, count, dtype)
                torch.cuda.synchronize()
                for r in range(R):
                    assert same_bits(recv[r].get(np_dtype(dtype)), wrs[r], dtype) and recv[r].guards_intact()
            comm.destroy()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("path", [hb.PATH_CE, hb.PATH_SM])
def test_forward_variant_gives_the_ring_bits(oracle, dtype, path):
    """Fused sum-and-forward (a SUM stores into the next rank's inbox): same bits as the rank-local ring."""
    e = W.elem_size(dtype)
    for R, n in SMALL + [(8, 8 * 65_536)]:
        xs = W.rank_inputs("normal", 400 + n % 7, R, n, dtype, 1.0)
        want = oracle.ring_allreduce(xs)
        for use_graph in (1, 0):
            comm = make_comm(R, n, dtype, path, forward=1, use_graph=use_graph, piece_bytes=8192, max_pieces=3)
            for in_place in (False, True):
                got = run_allreduce(comm, xs, dtype, in_place)
                for r in range(R):
                    assert same_bits(got[r], want[r], dtype), (R, n, r, in_place, use_graph)
            if R > 1:
                st = comm.last_stats()
                assert st["n_moves"] <= 2 * R * st["n_pieces"] * (R - 1)      # fewer moves than the rank-local ring
            if n % R == 0 and R > 1:
                count = n // R
                wrs = oracle.ring_reduce_scatter(xs)
                send = [DevBuf(n * e).put(xs[r]) for r in range(R)]
                recv = [DevBuf(count * e) for _ in range(R)]
                comm.reduce_scatter(send, recv, count, dtype)
                torch.cuda.synchronize()
                for r in range(R):
                    assert same_bits(recv[r].get(np_dtype(dtype)), wrs[r], dtype) and recv[r].guards_intact()
            comm.destroy()


def test_settings_never_change_a_bit(oracle):
    """Piece size, lane count, CTA budgets, path and executor are pure scheduling choices."""
    R, n, dtype = 8, 8 * 40000 + 8, "bf16"
    xs = W.rank_inputs("normal", 77, R, n, dtype, 1.0)
    want = oracle.ring_allreduce(xs)
    settings = [
        dict(path=hb.PATH_CE, use_graph=1, piece_bytes=1024, max_pieces=64),
        dict(path=hb.PATH_CE, use_graph=0, piece_bytes=8192, max_pieces=8, lanes=1),
        dict(path=hb.PATH_CE, use_graph=0, piece_bytes=8192, max_pieces=8, lanes=8, sum_ctas=1),
        dict(path=hb.PATH_SM, use_graph=1, piece_bytes=1 << 20, max_pieces=1, sum_ctas=148, copy_ctas=148),
        dict(path=hb.PATH_SM, use_graph=0, piece_bytes=16384, max_pieces=3, sum_ctas=3, copy_ctas=5),
        dict(path=hb.PATH_CE, use_graph=1, profile=1),
        dict(path=hb.PATH_CE, use_graph=1, forward=1, piece_bytes=4096, max_pieces=16),
        dict(path=hb.PATH_SM, use_graph=0, forward=1, piece_bytes=65536, max_pieces=4, lanes=2),
        dict(path=hb.PATH_CE, onepass=1, sum_ctas=5),
    ]
    for s in settings:
        s = dict(s)
        comm = make_comm(R, n, dtype, s.pop("path"), **s)
        for _ in range(3):       # also: repeated runs give the same bits
            got = run_allreduce(comm, xs, dtype)
            for r in range(R):
                assert same_bits(got[r], want[r], dtype)
        comm.destroy()


def test_integer_inputs_are_order_free(oracle):
    R, n, dtype = 8, 8 * 5000, "bf16"
    xs = W.rank_inputs("int", 5, R, n, dtype)
    exact = np.sum([oracle.bf16_bits_to_f32(x).astype(np.float64) for x in xs], axis=0)
    comm = make_comm(R, n, dtype)
    got = run_allreduce(comm, xs, dtype)
    for r in range(R):
        assert (oracle.bf16_bits_to_f32(got[r]).astype(np.float64) == exact).all()
    comm.destroy()


def test_large_periodic_inputs_full_compare(oracle):
    """R=2 x 256 Mi fp32 (1 GiB per rank) and R=8 x 40 MiB bf16: inputs are a seeded block repeated on the
    device; the expectation is the oracle's chain result on that block, repeated, compared on the device."""
    cases = [(2, 1 << 28, "fp32", 1 << 20), (8, 20_971_520, "bf16", 1 << 16), (8, 4_194_304, "bf16", 1 << 16)]
    for R, n, dtype, period in cases:
        e = W.elem_size(dtype)
        assert (n // R) % period == 0
        base = W.rank_inputs("normal", 3, R, period, dtype, 1e-3)
        tdt = torch.float32 if dtype == "fp32" else torch.int16
        send = [torch.from_numpy(b.view(np.int16) if dtype == "bf16" else b).cuda().repeat(n // period) for b in base]
        recv = [torch.empty(n, dtype=tdt, device="cuda") for _ in range(R)]
        comm = make_comm(R, n, dtype)
        comm.allreduce(send, recv, n, dtype)
        torch.cuda.synchronize()
        # chunk c of the result follows the chain order that starts at rank c+1
        expect = torch.empty(n, dtype=tdt, device="cuda")
        q = n // R
        for c in range(R):
            blk = oracle.chain_sum(base, c, 0, period)
            t = torch.from_numpy(blk.view(np.int16) if dtype == "bf16" else blk).cuda()
            expect[c * q:(c + 1) * q] = t.repeat(q // period)
        for r in range(R):
            assert torch.equal(recv[r].view(torch.int32 if dtype == "fp32" else torch.int16),
                               expect.view(torch.int32 if dtype == "fp32" else torch.int16)), (R, n, r)
        comm.destroy()
        del send, recv, expect
        torch.cuda.empty_cache()


def test_small_messages_on_the_copy_route(oracle):
    """Default settings on HOCCL_PATH_CE: a message of at most ce_small_bytes (8 MiB) per rank moves through batched copy-kernel
    launches (the statistics show them), a larger one through driver copies; ce_small_bytes = 0 keeps driver copies at every
    size.  The bits are the oracle's either way, for every collective."""
    R, dtype = 4, "fp32"
    for n, small in ((4096, True), (2 * 1024 * 1024, True), (2 * 1024 * 1024 + 4, False)):     # 16 KiB, 8 MiB, just above
        xs = W.rank_inputs("uniform", 300, R, n, dtype)
        want = oracle.ring_allreduce(xs)
        for limit in (None, 0):
            comm = make_comm(R, n, dtype, hb.PATH_CE, **({"ce_small_bytes": 8 << 20} if limit is None else {"ce_small_bytes": 0}))
            got = run_allreduce(comm, xs, dtype)
            st = comm.last_stats()
            for r in range(R):
                assert same_bits(got[r], want[r], dtype), (n, limit, r)
            if small and limit is None:
                assert st["n_move_launches"] > 0 and st["max_copy_ctas"] == 148, st
            else:
                assert st["n_move_launches"] == 0 and st["n_moves"] > 0, st
            assert comm.get_param("copy_ctas") == 8       # the communicator's own settings are untouched by the rule
            comm.destroy()
    # the other collectives under the rule
    n = 4 * 3000
    xs = W.rank_inputs("uniform", 301, R, n, dtype)
    comm = make_comm(R, n, dtype, hb.PATH_CE, ce_small_bytes=8 << 20)
    send = [DevBuf(n * 4).put(x) for x in xs]
    rs = [DevBuf(n) for _ in range(R)]
    comm.reduce_scatter(send, rs, n // R, dtype)
    assert comm.last_stats()["n_move_launches"] > 0
    ag = [DevBuf(n * 4) for _ in range(R)]
    comm.allgather([s.ptr for s in send], ag, n // R, dtype)
    assert comm.last_stats()["n_move_launches"] > 0
    a2a = [DevBuf(n * 4) for _ in range(R)]
    comm.alltoall(send, a2a, n // R, dtype)
    assert comm.last_stats()["n_move_launches"] > 0
    torch.cuda.synchronize()
    wrs, wag, wa2a = oracle.ring_reduce_scatter(xs), oracle.allgather([x[:n // R] for x in xs]), oracle.alltoall(xs)
    for r in range(R):
        assert same_bits(rs[r].get(np.float32), wrs[r], dtype)
        assert (ag[r].get(np.float32).view(np.uint32) == wag[r].view(np.uint32)).all()
        assert (a2a[r].get(np.float32).view(np.uint32) == wa2a[r].view(np.uint32)).all()
        assert rs[r].guards_intact() and ag[r].guards_intact() and a2a[r].guards_intact()
    comm.destroy()


# ------------------------------------------------------------------------------- ordering ---------
def test_stream_ordering_with_neighbouring_kernels(oracle):
    """Work enqueued before the call on the same stream is seen by it; work enqueued after sees its result."""
    R, n, dtype = 4, 1 << 20, "fp32"
    xs = W.rank_inputs("uniform", 9, R, n, dtype)
    want = oracle.ring_allreduce([x * np.float32(2.0) for x in xs])
    for use_graph in (1, 0):
        comm = make_comm(R, n, dtype, use_graph=use_graph)
        st = torch.cuda.Stream()
        base = [torch.from_numpy(x).cuda() for x in xs]
        send = [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(R)]
        recv = [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(R)]
        after = [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(R)]
        torch.cuda.synchronize()
        with torch.cuda.stream(st):
            for r in range(R):
                torch.mul(base[r], 2.0, out=send[r])          # producer kernels
            comm.allreduce(send, recv, n, dtype, st)
            for r in range(R):
                after[r].copy_(recv[r])                        # consumer kernels
        st.synchronize()
        for r in range(R):
            assert same_bits(after[r].cpu().numpy(), want[r], dtype)
        comm.destroy()


# ------------------------------------------------------------------------------- point to point ---
def test_send_recv_matching(oracle):
    R = 4
    comm = hb.Comm(R, 0)
    dtype, n = "bf16", 300_001
    msgs = [W.uniform(50 + k, 0, n, dtype) for k in range(3)]
    for path in (hb.PATH_CE, hb.PATH_SM):
        comm.set_path(path)
        src = [DevBuf(n * 2).put(m) for m in msgs]
        dst = [DevBuf(n * 2) for _ in msgs]
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        # sender posts first (twice), receiver matches in FIFO order; third: receiver first
        comm.send(src[0], n, dtype, 0, 1, s1)
        comm.send(src[1], n, dtype, 0, 1, s1)
        assert comm.pending() == 2
        comm.recv(dst[0], n, dtype, 0, 1, s2)
        comm.recv(dst[1], n, dtype, 0, 1, s2)
        comm.recv(dst[2], n, dtype, 2, 3, s2)
        assert comm.pending() == 1
        comm.send(src[2], n, dtype, 2, 3, s2)                 # same stream on both sides
        assert comm.pending() == 0
        torch.cuda.synchronize()
        for k in range(3):
            assert (dst[k].get(np.uint16) == oracle.sendrecv(msgs[k])).all()
            assert dst[k].guards_intact() and src[k].guards_intact()
    # mismatch: the parked post is dropped, nothing is enqueued
    a, b = DevBuf(64), DevBuf(64, fill=0x11)
    comm.send(a, 16, "fp32", 1, 2)
    assert comm.recv_rc(b, 8, "fp32", 1, 2) == hb.ERR_MISMATCH
    assert comm.pending() == 0
    torch.cuda.synchronize()
    assert (b.get(np.uint8) == 0x11).all()
    # argument errors
    assert comm.send_rc(a, 16, "fp32", 1, 1) == hb.ERR_INVALID_ARG
    assert comm.send_rc(a, 16, "fp32", 0, 4) == hb.ERR_INVALID_ARG
    assert comm.send_rc(None, 16, "fp32", 0, 1) == hb.ERR_INVALID_ARG
    # an unmatched post blocks destroy and can never hang a stream
    comm.recv(b, 16, "fp32", 3, 0)
    assert comm.pending() == 1
    assert comm.destroy() == hb.ERR_PENDING
    comm.send(a, 16, "fp32", 3, 0)
    torch.cuda.synchronize()
    assert (b.get(np.uint8) == a.get(np.uint8)).all()
    assert comm.destroy() == hb.OK


@pytest.mark.parametrize("per_stage_streams", [False, True])
@pytest.mark.parametrize("path", [hb.PATH_CE, hb.PATH_SM])
def test_pipeline_wave_small(oracle, per_stage_streams, path):
    """Stage-to-stage forwarding: microbatch m travels 0 -> 1 -> ... -> S-1; hop s+1 depends on hop s.
    With one stream per stage the dependency runs through the matched posts only (send on stage s's stream,
    recv on stage s+1's stream); a 40 MiB message also exercises the sliced copy."""
    S, M, dtype = 8, 4, "bf16"
    for n, split in ((65_536 + 8, 1), (20 * 1024 * 1024 + 8, 2)):
        comm = hb.Comm(S, 0)
        comm.set_path(path)
        comm.set_param("p2p_split", split)
        acts = [W.normal(2, m, n, dtype) for m in range(M)]
        slots = [[DevBuf(n * 2) for _ in range(M)] for _ in range(S)]
        for m in range(M):
            slots[0][m].put(acts[m])
        torch.cuda.synchronize()
        streams = [torch.cuda.Stream() for _ in range(S)] if per_stage_streams else [torch.cuda.Stream()] * S
        for m in range(M):
            for s in range(S - 1):
                comm.send(slots[s][m], n, dtype, s, s + 1, streams[s])
                comm.recv(slots[s + 1][m], n, dtype, s, s + 1, streams[s + 1])
        torch.cuda.synchronize()
        for m in range(M):
            assert (slots[S - 1][m].get(np.uint16) == oracle.sendrecv(acts[m])).all()
            assert all(slots[s][m].guards_intact() for s in range(S))
        assert comm.destroy() == hb.OK


def test_config3_pipeline_full_size(oracle):
    """bf16 activations [4, 2048, 4096] (64 MiB per message) over 8 stages and 16 microbatches, one stream per stage,
    copy-route path: every microbatch arrives bit for bit.  Microbatch m is the seeded block rotated by m * 4099."""
    c = W.C3_PIPELINE
    n = c.count
    base = W.normal(c.seed, 0, n, c.dtype, 1.0)
    want = oracle.sendrecv(base)
    dev = torch.from_numpy(base.view(np.int16)).cuda()
    comm = hb.Comm(c.stages, 0)
    slots = [[torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(c.microbatches)] for _ in range(c.stages)]
    for m in range(c.microbatches):
        slots[0][m].copy_(torch.roll(dev, 4099 * m))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in range(c.stages)]
    for m in range(c.microbatches):
        for s in range(c.stages - 1):
            comm.send(slots[s][m], n, c.dtype, s, s + 1, streams[s])
            comm.recv(slots[s + 1][m], n, c.dtype, s, s + 1, streams[s + 1])
    torch.cuda.synchronize()
    assert comm.pending() == 0
    expect = torch.from_numpy(want.view(np.int16)).cuda()
    for m in range(c.microbatches):
        for s in range(1, c.stages):
            assert torch.equal(slots[s][m], torch.roll(expect, 4099 * m)), (m, s)
    assert comm.destroy() == hb.OK


# ------------------------------------------------------------------------------- errors, host path -
def test_argument_errors_enqueue_nothing():
    R, n = 4, 4096
    comm = hb.Comm(R, 0)
    bufs = [DevBuf(n * 4, fill=0x22) for _ in range(2 * R)]
    send, recv = bufs[:R], bufs[R:]
    assert comm.allreduce_rc(send, recv, n, "fp32") == hb.ERR_SCRATCH          # no scratch attached
    small = DevBuf(1024)
    pad = (-small.ptr) % 256
    assert hb.lib().hoccl_comm_set_scratch(comm._h, small.ptr + pad, 256) == hb.OK
    assert comm.allreduce_rc(send, recv, n, "fp32") == hb.ERR_SCRATCH
    assert hb.lib().hoccl_comm_set_scratch(comm._h, small.ptr + pad + 8, 256) == hb.ERR_INVALID_ARG
    comm2 = make_comm(R, n, "fp32")
    assert comm2.allreduce_rc(send, recv, n, "fp32", op=3) == hb.ERR_UNSUPPORTED
    assert comm2.allreduce_rc(send, recv, n, 5) == hb.ERR_UNSUPPORTED
    assert comm2.allreduce_rc([send[0], send[0], send[2], send[3]], recv, n, "fp32") == hb.ERR_INVALID_ARG   # two ranks share a buffer
    assert comm2.allreduce_rc([send[0].ptr + 2] + send[1:], recv, n, "fp32") == hb.ERR_INVALID_ARG          # misaligned
    assert comm2.allreduce_rc([0] + send[1:], recv, n, "fp32") == hb.ERR_INVALID_ARG
    assert comm2.allreduce_rc(send, [send[0].ptr + 64] + recv[1:], n, "fp32") == hb.ERR_INVALID_ARG         # partial overlap
    assert comm2.allreduce_rc([send[0]] + recv[1:], [send[0]] + send[1:], n, "fp32") == hb.ERR_INVALID_ARG  # mixed in-place
    assert comm2.allreduce_rc(send, recv, 0, "fp32") == hb.OK
    torch.cuda.synchronize()
    for b in bufs:
        assert (b.get(np.uint8) == 0x22).all()
    with pytest.raises(hb.HocclError):
        comm2.set_param("no_such_key", 1)
    with pytest.raises(hb.HocclError):
        comm2.set_param("sum_ctas", 0)
    comm.destroy()
    comm2.destroy()


def test_host_buffer_allreduce(oracle):
    R, n, dtype = 4, 262_144 + 16, "fp32"
    xs = W.rank_inputs("uniform", 12, R, n, dtype)
    want = oracle.ring_allreduce(xs)
    comm = make_comm(R, n, dtype)
    h_send = [torch.from_numpy(x).pin_memory() for x in xs]
    h_recv = [torch.zeros(n, dtype=torch.float32).pin_memory() for _ in range(R)]
    with pytest.raises(hb.HocclError):
        comm.host_allreduce(h_send, h_recv, n, dtype)          # staging missing
    per = (n * 4 + 255) // 256 * 256
    staging = torch.empty(2 * R * per + 256, dtype=torch.uint8, device="cuda")
    pad = (-staging.data_ptr()) % 256
    comm.set_staging(staging.data_ptr() + pad, 2 * R * per)
    comm.host_allreduce(h_send, h_recv, n, dtype)
    torch.cuda.synchronize()
    for r in range(R):
        assert same_bits(h_recv[r].numpy(), want[r], dtype)
    comm.destroy()


def test_probe_move_needs_sm_terminates():
    comm = hb.Comm(2, 0)
    comm.set_param("copy_ctas", 8)
    a = torch.ones(1 << 22, dtype=torch.uint8, device="cuda")
    b = torch.zeros(1 << 22, dtype=torch.uint8, device="cuda")
    needs_sm_kernel, end_us = hd.probe_move_needs_sm(comm, hb.PATH_SM, b, a, a.numel(), 1500)
    assert needs_sm_kernel is True and end_us >= 1300        # an SM copy cannot start while every SM is taken
    assert torch.equal(a, b)
    needs_ce, end_ce = hd.probe_move_needs_sm(comm, hb.PATH_CE, b, a, a.numel(), 1500)
    assert isinstance(needs_ce, bool) and end_ce > 0         # the answer is the driver's; it is reported, not asserted
    comm.destroy()


def test_probe_copy_routes_controls_and_copy_kernel():
    """Every same-device route is tried in turn; what the driver does with its own copies is reported, not asserted,
    but the controls are fixed: a stream memory write and pinned-host copies need no SM, copy_kernel needs one."""
    comm = hb.Comm(2, 0)
    comm.set_param("copy_ctas", 8)
    n = 1 << 20
    a = torch.full((n,), 3, dtype=torch.uint8, device="cuda")
    b = torch.zeros(n, dtype=torch.uint8, device="cuda")
    host = torch.empty(n, dtype=torch.uint8).pin_memory()
    comm.set_host_staging(host)
    rows = {name: (needs, end) for name, needs, end in hd.probe_copy_routes(comm, b, a, n, 3000)}
    assert len(rows) >= 9
    for name, (needs, end) in rows.items():
        assert end > 0, name
    assert rows["copy_kernel (this library, by construction)"][0] is True
    assert rows["control: cuStreamWriteValue32"][0] is False
    assert rows["control: device->pinned host"][0] is False
    assert rows["control: pinned host->device"][0] is False
    assert torch.equal(b, a)                                  # the last route copied host (= a) back into b
    comm.destroy()


@pytest.mark.parametrize("kind", ["sum", "copy"])
def test_kernels_occupy_as_many_sms_as_their_cta_budget(kind):
    """SMs used, counted: every CTA reports the SM it ran on.  Under a budget of up to 148 CTAs (one CTA per SM by
    registers and threads) the launch occupies exactly `ctas` distinct SMs; the result is still right."""
    n = 8 << 20
    a = torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
    b = torch.empty(n, dtype=torch.bfloat16, device="cuda").normal_(0, 1e-3)
    out = torch.empty(n, dtype=torch.bfloat16, device="cuda")
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    for ctas in (1, 8, 32, n_sm):
        ids = torch.full((ctas,), 0xFFFF, dtype=torch.int32, device="cuda")
        assert hd.kernel_sms(kind, a, b if kind == "sum" else None, out, n * 2, "bf16", ctas, ids) == hb.OK
        torch.cuda.synchronize()
        got = ids.cpu().numpy()
        assert (got >= 0).all() and (got < n_sm).all()
        assert len(set(got.tolist())) == ctas, (kind, ctas, sorted(got.tolist()))
        want = (a.float() + b.float()).to(torch.bfloat16) if kind == "sum" else a
        assert torch.equal(out, want)


def test_graph_cache_eviction_with_work_in_flight(oracle):
    """More distinct call signatures than the graph cache holds (48), issued back to back without host synchronisation:
    the least recently used graphs are evicted while earlier launches may still be running; every result stays right,
    and a signature that was evicted is simply rebuilt."""
    R, dtype = 4, "fp32"
    counts = [4096 + 4 * k for k in range(70)]
    n_max = max(counts)
    xs = W.rank_inputs("uniform", 77, R, n_max, dtype)
    comm = make_comm(R, n_max, dtype, hb.PATH_SM, sum_ctas=8, copy_ctas=8)
    send = [DevBuf(n_max * 4).put(xs[r]) for r in range(R)]
    recvs = [[DevBuf(n * 4) for _ in range(R)] for n in counts]
    stream = torch.cuda.Stream()
    for n, recv in zip(counts, recvs):
        comm.allreduce(send, recv, n, dtype, stream)
        assert comm.last_stats()["graph_hit"] == 0
    comm.allreduce(send, recvs[-1], counts[-1], dtype, stream)
    assert comm.last_stats()["graph_hit"] == 1              # the newest entry is still cached
    comm.allreduce(send, recvs[0], counts[0], dtype, stream)
    assert comm.last_stats()["graph_hit"] == 0              # the oldest was evicted and is rebuilt
    stream.synchronize()
    for n, recv in zip(counts, recvs):
        want = oracle.ring_allreduce([x[:n] for x in xs])
        for r in range(R):
            assert same_bits(recv[r].get(np.float32), want[r], dtype), (n, r)
            assert recv[r].guards_intact()
    assert comm.destroy() == hb.OK


@pytest.mark.parametrize("params", [dict(), dict(path=hb.PATH_SM, sum_ctas=8, copy_ctas=8), dict(path=hb.PATH_SM, fused=1, sum_ctas=148, copy_ctas=148)])
def test_two_communicators_on_two_streams_at_once(oracle, params):
    """Collectives that overlap in time must not share a communicator; two communicators on two streams may run at the same
    time and must not disturb each other (no state is shared between communicators)."""
    R, dtype = 4, "bf16"
    ns = (4 * 70_000 + 3, 4 * 90_000 + 1)
    p = dict(params)
    path = p.pop("path", hb.PATH_CE)
    comms, sends, recvs, wants, streams = [], [], [], [], []
    for k, n in enumerate(ns):
        xs = W.rank_inputs("normal", 300 + k, R, n, dtype, 1e-3)
        wants.append(oracle.ring_allreduce(xs))
        comms.append(make_comm(R, n, dtype, path, **p))
        sends.append([DevBuf(n * 2).put(x) for x in xs])
        recvs.append([DevBuf(n * 2) for _ in range(R)])
        streams.append(torch.cuda.Stream())
    for rep in range(6):                                   # interleaved issue, no host synchronisation in between
        for k in range(2):
            comms[k].allreduce(sends[k], recvs[k], ns[k], dtype, streams[k])
    torch.cuda.synchronize()
    for k in range(2):
        for r in range(R):
            assert same_bits(recvs[k][r].get(np.uint16), wants[k][r], dtype), (k, r)
            assert recvs[k][r].guards_intact() and sends[k][r].guards_intact()
        assert comms[k].async_error() == hb.OK
        assert comms[k].destroy() == hb.OK


def test_port_probe_reads_and_writes_what_it_says():
    """The memory-port probe behind the 8-SM ceiling: write mode stores a known pattern over whole 128 KiB tiles and
    nothing else; read mode leaves the buffer alone."""
    nbytes = (3 * 128 << 10) + 4096                     # three tiles and a remainder that must stay untouched
    buf = torch.full((nbytes // 4,), -1, dtype=torch.int32, device="cuda")
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    assert hd.port_probe("write", buf, nbytes, 2, sink) == hb.OK
    torch.cuda.synchronize()
    v = buf.cpu().numpy().reshape(-1, 4)
    tile_vecs = 8 * 1024
    for t, u, tid in ((0, 0, 0), (0, 1, 5), (1, 7, 1023), (2, 3, 77)):
        assert v[t * tile_vecs + u * 1024 + tid].tolist() == [t, u, tid, 0]
    assert (v[3 * tile_vecs:] == -1).all()
    before = buf.clone()
    assert hd.port_probe("read", buf, nbytes, 2, sink) == hb.OK
    torch.cuda.synchronize()
    assert torch.equal(buf, before)
    assert hd.port_probe("read", buf, 1024, 2, sink) == hb.ERR_INVALID_ARG
