"""GPU parity for the direct reduce-scatter ("rs_direct" = 1): the reduce-scatter as the R-1 permutation stages r -> r+k of its
traffic matrix (the paper's stage decomposition, Sec. 3.4) into R-1 inbox slots of the owner, then one chain sum per rank in
the ring's order with a rounding after every add.

The order of addition and every rounding are the ring's, so all results must carry the oracle's bits: on every path and
executor, for both dtypes, in place, with ragged sizes and misaligned buffers, alone and combined with the direct all-gather."""
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
    (hb.PATH_CE, dict(ag_direct=1)),
    (hb.PATH_CE, dict(use_graph=0)),
    (hb.PATH_CE, dict(order_kernels=0)),
    (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=8)),
    (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=8, ag_direct=1)),
    (hb.PATH_SM, dict(sum_ctas=148, copy_ctas=148, ag_direct=1)),
    (hb.PATH_SM, dict(sum_ctas=3, copy_ctas=5, use_graph=0)),
    (hb.PATH_SM, dict(handshake=1, watchdog_ms=5000)),
    (hb.PATH_CE_HOST, dict(ag_direct=1)),
]


@pytest.mark.parametrize("path,params", CONFIGS)
def test_allreduce_with_direct_reduce_scatter(oracle, path, params):
    for dtype in ("fp32", "bf16"):
        e = W.elem_size(dtype)
        for R, n in [(2, 1), (2, 100_003), (3, 5), (4, 262_144 + 9), (8, 8 * 70_000 + 3), (8, 7), (5, 99_999)]:
            xs = W.rank_inputs("uniform", 190 + R, R, n, dtype)
            want = oracle.ring_allreduce(xs)
            comm = make_comm(R, n, dtype, path, rs_direct=1, piece_bytes=65536, max_pieces=4, **params)
            if path == hb.PATH_CE_HOST:
                comm.set_host_staging(torch.empty(4 * R * (n * e + 4096), dtype=torch.uint8).pin_memory())
            for in_place in (False, True):
                offs = [(r % 4) * e for r in range(R)] if in_place else None
                got = run_allreduce(comm, xs, dtype, in_place=in_place, offs=offs)
                for r in range(R):
                    assert same_bits(got[r], want[r], dtype), (dtype, R, n, in_place, r)
            st = comm.last_stats()
            if R > 1 and n >= R:
                assert st["n_sum_launches"] == st["n_pieces"], st          # one chain launch per piece instead of R-1 sums
            comm.destroy()


def test_what_does_not_combine_with_the_direct_reduce_scatter_is_refused():
    """The one-kernel form has no chain phase and the direct form has no steps to forward between: asking for either together
    with rs_direct = 1 is an error, nothing is enqueued; with rs_direct = 2 (automatic) the option that was asked for wins."""
    R, n, dtype = 4, 4096, "fp32"
    send = [DevBuf(n * 4) for _ in range(R)]
    recv = [DevBuf(n * 4, fill=0x3C) for _ in range(R)]
    for extra in (dict(fused=1), dict(forward=1), dict(onepass=1)):
        comm = make_comm(R, n, dtype, hb.PATH_SM, rs_direct=1, **extra)
        assert comm.allreduce_rc(send, recv, n, dtype) == hb.ERR_UNSUPPORTED, extra
        assert comm.reduce_scatter_rc(send, [r.ptr for r in recv], n // R, dtype) == hb.ERR_UNSUPPORTED, extra
        torch.cuda.synchronize()
        assert all((b.get(np.uint8) == 0x3C).all() for b in recv)
        comm.set_param("rs_direct", 2)
        assert comm.allreduce_rc(send, recv, n, dtype) == hb.OK, extra
        torch.cuda.synchronize()
        assert comm.last_stats()["n_sum_launches"] != 1 or extra.get("onepass")       # not the one chain launch of the direct form
        for b in recv:
            b.view.fill_(0x3C)
        torch.cuda.synchronize()
        comm.destroy()


@pytest.mark.parametrize("path", [hb.PATH_CE, hb.PATH_SM])
def test_reduce_scatter_call_direct(oracle, path):
    for dtype in ("fp32", "bf16"):
        e = W.elem_size(dtype)
        for R, count in [(1, 9), (2, 1), (4, 1025), (8, 4099), (3, 77)]:
            xs = W.rank_inputs("uniform", 141, R, R * count, dtype)
            want = oracle.ring_reduce_scatter(xs)
            comm = make_comm(R, R * count, dtype, path, rs_direct=1, piece_bytes=2048, max_pieces=5)
            send = [DevBuf(R * count * e).put(xs[r]) for r in range(R)]
            recv = [DevBuf(count * e, (r % 2) * e) for r in range(R)]
            comm.reduce_scatter(send, recv, count, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert same_bits(recv[r].get(np_dtype(dtype)), want[r], dtype), (dtype, R, count, r)
                assert recv[r].guards_intact() and send[r].guards_intact()
                assert (send[r].get(np_dtype(dtype)).view(np.uint8) == xs[r].view(np.uint8)).all(), "send buffer was written"
            comm.reduce_scatter(send, [send[r].ptr + r * count * e for r in range(R)], count, dtype)      # in place
            torch.cuda.synchronize()
            for r in range(R):
                assert same_bits(send[r].get(np_dtype(dtype))[r * count:(r + 1) * count], want[r], dtype)
            comm.destroy()


def test_special_values_and_many_ranks(oracle):
    """NaN, infinities, signed zeros and subnormals go through the chain like through the ring; R = 20 and 40 need several
    operand batches per element (more than 8 operands) and several launches per group."""
    for dtype in ("fp32", "bf16"):
        for R, n in [(4, 4 * 2048 + 3), (20, 20 * 300 + 7), (40, 40 * 64 + 1)]:
            xs = W.rank_inputs("uniform", 195, R, n, dtype)
            special = np.array([np.nan, np.inf, -np.inf, 0.0, -0.0, 1e-40, -1e-40, 3.0e38, -3.0e38, 1.0], dtype=np.float32)
            for r in range(R):
                v = np.roll(special, r)
                if dtype == "fp32":
                    xs[r][:v.size] = v
                else:
                    xs[r][:v.size] = (v.view(np.uint32) >> 16).astype(np.uint16)
            want = oracle.ring_allreduce(xs)
            for path, params in ((hb.PATH_CE, dict()), (hb.PATH_SM, dict(sum_ctas=16, copy_ctas=16, ag_direct=1))):
                comm = make_comm(R, n, dtype, path, rs_direct=1, **params)
                got = run_allreduce(comm, xs, dtype, in_place=True, offs=[(r % 3) * W.elem_size(dtype) for r in range(R)])
                for r in range(R):
                    assert same_bits(got[r], want[r], dtype), (dtype, R, path, r)
                comm.destroy()


def test_scratch_bound_is_checked():
    R, n, dtype = 8, 8 * 10_000, "fp32"
    comm = make_comm(R, n, dtype, hb.PATH_CE)                       # scratch for the ring: two slots per rank
    a = [DevBuf(n * 4) for _ in range(R)]
    b = [DevBuf(n * 4) for _ in range(R)]
    assert comm.allreduce_rc(a, b, n, dtype) == hb.OK
    comm.set_param("rs_direct", 1)
    assert comm.allreduce_rc(a, b, n, dtype) == hb.ERR_SCRATCH      # R-1 slots per rank do not fit
    torch.cuda.synchronize()
    comm.destroy()
    assert hb.scratch_bytes_direct(R, n, dtype) >= (R - 1) * hb.scratch_bytes(R, n, dtype) // 2
    assert hb.scratch_bytes_direct(2, n, dtype) == hb.scratch_bytes(2, n, dtype)
    assert hb.scratch_bytes_direct(1, n, dtype) == 0


def test_config2_bucket_full_size(oracle):
    """The gradient bucket at full size, two calls and one call, copy route with 8-CTA sums and the SM path."""
    c = W.C2_DP_BUCKET
    R, n, e = c.R, c.count, 2
    xs = W.rank_inputs(c.dist, c.seed, R, n, c.dtype, c.sigma)
    want = oracle.ring_allreduce(xs, threads=oracle.max_threads())
    count = n // R
    send = [DevBuf(n * e).put(xs[r]) for r in range(R)]
    recv = [DevBuf(n * e) for _ in range(R)]
    for path, params in [(hb.PATH_CE, dict(sum_ctas=8)), (hb.PATH_CE, dict(sum_ctas=8, ag_direct=1)),
                         (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=48, ag_direct=1)), (hb.PATH_SM, dict(sum_ctas=148, copy_ctas=148, ag_direct=1))]:
        comm = make_comm(R, n, c.dtype, path, rs_direct=1, **params)
        for two_calls in (True, False):
            for b in recv:
                b.view.fill_(0)
            torch.cuda.synchronize()
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
        assert comm._scratch_keep.guards_intact()
        comm.destroy()


def test_native_bf16_add_equals_the_reference_add_for_all_operand_pairs():
    """The chain kernel adds bf16 with add.rn.bf16x2.  It must give the bits of every other SUM (binary32 add of the widened
    operands, rounded to nearest even) for all 2^32 pairs of bf16 bit patterns, NaN payloads included."""
    counts = torch.zeros(2, dtype=torch.int64, device="cuda")
    torch.cuda.synchronize()
    assert hd.selftest_bf16_add(counts) == hb.OK
    torch.cuda.synchronize()
    assert counts.tolist() == [0, 0]


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("ctas", [1, 3, 8, 148])
def test_chain_kernel_against_the_oracles_chain(oracle, dtype, ctas):
    """hoccl_chain_launch against the oracle's closed form of the ring order, ((x_{c+1} + x_{c+2}) + ...) + x_c with a rounding
    after every add: R = 2..12 operands (every operand count the software-pipelined kernel is compiled for, and beyond it the
    plain one), ragged lengths, operands off the 16-byte grid together (vector path) or not.  The lengths give a CTA fewer
    tiles than its pipeline is deep, exactly as many, many more with a ragged last tile, and an uneven split over 3 CTAs."""
    e = W.elem_size(dtype)
    vec = 16 // e
    tile = 512 * vec                      # elements of one tile of the pipelined kernel
    cases = [(2, 1), (3, 1023), (8, 4096 * 5 + 3), (8, 1_000_003), (12, 70_001),
             (4, 3 * tile), (5, 2 * tile + 7), (6, 9 * tile + vec), (7, 25 * tile - vec + 1), (8, 3 * ctas * tile),
             (8, (3 * ctas + 1) * tile + 5), (2, 40 * tile + 3), (3, 17 * tile)]
    for R, n in cases:
        xs = W.rank_inputs("uniform", 230 + R, R, n, dtype)
        c = R // 2
        want = oracle.chain_sum(xs, c, 0, n)
        stride = (n * e + 255) // 256 * 256 + 256
        for offs in ((0, 0, 0), (e, e, e), (0, e, 0)):
            inbox = DevBuf(stride * (R - 1), offs[0])
            for j in range(R - 1):                                   # slot j holds source c + 1 + j: the ring's order
                src = xs[(c + 1 + j) % R].view(np.uint8)
                inbox.view[j * stride:j * stride + n * e].copy_(torch.from_numpy(src.copy()))
            local = DevBuf(n * e, offs[1]).put(xs[c])
            out = DevBuf(n * e, offs[2])
            torch.cuda.synchronize()
            assert hd.chain_launch(inbox, stride, R - 1, local, out, n, dtype, ctas) == hb.OK
            torch.cuda.synchronize()
            assert same_bits(out.get(np_dtype(dtype)), want, dtype), (dtype, R, n, offs)
            assert out.guards_intact() and inbox.guards_intact() and local.guards_intact()
            # in place on the local operand
            assert hd.chain_launch(inbox, stride, R - 1, local, local, n, dtype, ctas) == hb.OK
            torch.cuda.synchronize()
            assert same_bits(local.get(np_dtype(dtype)), want, dtype), ("in place", dtype, R, n, offs)
    assert hd.chain_launch(inbox, 24, 1, local, out, 4, dtype, 8) == hb.ERR_INVALID_ARG      # stride not a multiple of 16
    assert hd.chain_launch(inbox, 32, 64, local, out, 4, dtype, 8) == hb.ERR_INVALID_ARG     # too many operands


def test_automatic_choice_follows_the_scratch(oracle):
    """rs_direct = 2: the direct form when the attached scratch holds R-1 inbox slots per rank, the ring otherwise."""
    R, n, dtype = 8, 8 * 60_000 + 1, "bf16"
    xs = W.rank_inputs("normal", 199, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    for big, sums in ((True, 1), (False, R - 1)):
        params = dict(rs_direct=1) if big else dict()            # make_comm sizes the scratch from this
        comm = make_comm(R, n, dtype, hb.PATH_CE, piece_bytes=1 << 30, max_pieces=1, **params)
        comm.set_param("rs_direct", 2)
        got = run_allreduce(comm, xs, dtype)
        assert all(same_bits(got[r], want[r], dtype) for r in range(R)), big
        assert comm.last_stats()["n_sum_launches"] == sums, (big, comm.last_stats())
        comm.destroy()


def test_host_allreduce_with_the_direct_schedule(oracle):
    """The pipelined host entry point cuts chunks into pieces; every piece runs its own direct reduce-scatter and all-gather."""
    from test_gpu_host_allreduce import _pinned, _with_staging
    R, n, dtype = 8, 8 * 200_000 + 5, "bf16"
    xs = W.rank_inputs("normal", 198, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    for path, params in [(hb.PATH_CE, dict()), (hb.PATH_SM, dict(sum_ctas=8, copy_ctas=8))]:
        comm = make_comm(R, n, dtype, path, rs_direct=1, ag_direct=1, host_pieces=4, **params)
        _with_staging(comm, R, n, dtype)
        h_send = [_pinned(x) for x in xs]
        h_recv = [torch.zeros(n * 2, dtype=torch.uint8).pin_memory() for _ in range(R)]
        for rep in range(2):
            comm.host_allreduce(h_send, h_recv, n, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert same_bits(h_recv[r].numpy().view(np.uint16), want[r], dtype), (path, r, rep)
        st = comm.last_stats()
        assert st["n_pieces"] > 1 and st["n_sum_launches"] == st["n_pieces"], st
        comm.destroy()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_overlapped_copy_route_and_pipelined_sm_path_give_the_oracle_bits(oracle, dtype):
    """The direct schedule cut into pieces: on the copy route the three parts of every piece run as graphs of their own on three
    internal streams ("ce_overlap"), on the SM path under CTA budgets the copy launches are issued as a software pipeline.
    Both are scheduling only: the bits are the oracle's, for ragged sizes and piece counts, in place, repeated, and for the
    reduce-scatter call alone; sums still run one launch at a time."""
    e = W.elem_size(dtype)
    cases = [(8, 8 * 70_000 + 3, dict(ce_overlap=5)), (4, 4 * 300_000, dict(ce_overlap=2)), (3, 100_001, dict(ce_overlap=16)),
             (2, (8 << 20) // e + 8, dict()),                         # 4 MiB ring chunks: the automatic choice (4 pieces)
             (8, 8 * 600_000 + 8, dict(path=hb.PATH_SM, sum_ctas=8, copy_ctas=40)),      # > 1 MiB chunks: pipelined pieces
             (5, 5 * 700_000 + 1, dict(path=hb.PATH_SM, sum_ctas=3, copy_ctas=5))]
    for R, n, params in cases:
        params = dict(params)
        path = params.pop("path", hb.PATH_CE)
        xs = W.rank_inputs("uniform", 400 + R, R, n, dtype)
        want = oracle.ring_allreduce(xs)
        comm = make_comm(R, n, dtype, path, rs_direct=1, **params)
        for in_place in (False, True, False):
            got = run_allreduce(comm, xs, dtype, in_place=in_place)
            for r in range(R):
                assert same_bits(got[r], want[r], dtype), (dtype, R, n, params, in_place, r)
        st = comm.last_stats()
        assert st["n_pieces"] > 1 and st["n_sum_launches"] == st["n_pieces"], st
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
    # ordering against the caller's stream: producers before, consumers after, on a side stream
    R, n = 4, (16 << 20) // e
    xs = W.rank_inputs("uniform", 410, R, n, dtype)
    want = oracle.ring_allreduce(xs)
    comm = make_comm(R, n, dtype, hb.PATH_CE, rs_direct=1)
    tdt = torch.float32 if dtype == "fp32" else torch.int16
    base = [torch.from_numpy(x if dtype == "fp32" else x.view(np.int16)).cuda() for x in xs]
    send = [torch.zeros(n, dtype=tdt, device="cuda") for _ in range(R)]
    recv = [torch.zeros(n, dtype=tdt, device="cuda") for _ in range(R)]
    after = [torch.zeros(n, dtype=tdt, device="cuda") for _ in range(R)]
    st = torch.cuda.Stream()
    torch.cuda.synchronize()
    for rep in range(3):
        with torch.cuda.stream(st):
            for r in range(R):
                send[r].copy_(base[r])
            comm.allreduce(send, recv, n, dtype, st)
            for r in range(R):
                after[r].copy_(recv[r])
                recv[r].zero_()
        st.synchronize()
        assert comm.last_stats()["n_pieces"] == 4
        for r in range(R):
            got = after[r].cpu().numpy()
            assert same_bits(got if dtype == "fp32" else got.view(np.uint16), want[r], dtype), (rep, r)
    comm.destroy()
