"""GPU parity for hoccl_host_allreduce: host buffers in, host buffers out, bits equal to the oracle.

The pipelined form runs, per piece of every ring chunk, the host-to-device copies on one internal stream, the ring on
that piece (its own cached graph) on the caller's stream and the device-to-host copies on a second internal stream; the
sequential form (host_pieces = 1 or use_graph = 0) copies everything in, runs the all-reduce and copies everything out.  Both must give the oracle's bits for every size class: ragged sizes where
trailing chunks are short or empty, sizes below one piece, in place on the host, and every path."""
import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import workloads as W
from gpu_util import np_dtype, same_bits
from test_gpu_parity import make_comm

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def _need_gpu():
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    torch.cuda.set_device(0)
    yield
    torch.cuda.synchronize()


def _with_staging(comm, R, n, dtype):
    per = (n * W.elem_size(dtype) + 255) // 256 * 256
    staging = torch.full((2 * R * per + 256,), 0x77, dtype=torch.uint8, device="cuda")
    pad = (-staging.data_ptr()) % 256
    comm.set_staging(staging.data_ptr() + pad, 2 * R * per)
    comm._staging_keep = staging
    torch.cuda.synchronize()          # filled on torch's current stream; the calls may run on another one


def _pinned(x):
    return torch.from_numpy(x.view(np.uint8).copy()).pin_memory()


CASES = [(1, 1000), (2, 1), (2, 300_001), (4, 262_144 + 16), (4, 7), (8, 8 * 131_072), (8, 1_000_003), (5, 9), (3, 200_000)]


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("host_pieces", [1, 3, 8])
def test_host_allreduce_pipelined_and_sequential(oracle, dtype, host_pieces):
    e = W.elem_size(dtype)
    for R, n in CASES:
        xs = W.rank_inputs("uniform", 70 + R, R, n, dtype)
        want = oracle.ring_allreduce(xs)
        comm = make_comm(R, n, dtype, hb.PATH_CE, host_pieces=host_pieces)
        _with_staging(comm, R, n, dtype)
        h_send = [_pinned(x) for x in xs]
        h_recv = [torch.full((n * e + 64,), 0x5A, dtype=torch.uint8).pin_memory() for _ in range(R)]
        for rep in range(2):                                  # the second call replays the cached graph
            comm.host_allreduce(h_send, h_recv, n, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                got = h_recv[r].numpy()
                assert same_bits(got[:n * e].view(np_dtype(dtype)), want[r], dtype), (R, n, r, rep)
                assert (got[n * e:] == 0x5A).all(), "wrote past the end of a host buffer"
                assert (h_send[r].numpy() == xs[r].view(np.uint8)).all(), "a host send buffer was written"
        st = comm.last_stats()
        if R > 1 and n * e >= 8 * 65536 * R and host_pieces > 1:
            assert st["n_pieces"] > 1, st                     # large enough to be cut: really pipelined
        comm.destroy()


@pytest.mark.parametrize("path,params", [(hb.PATH_SM, dict(sum_ctas=8, copy_ctas=8)), (hb.PATH_SM, dict(sum_ctas=148, copy_ctas=148)),
                                         (hb.PATH_CE, dict(use_graph=0)), (hb.PATH_CE, dict(forward=1)),
                                         (hb.PATH_SM, dict(fused=1)), (hb.PATH_CE, dict(onepass=1)),
                                         (hb.PATH_SM, dict(handshake=1, watchdog_ms=5000))])
def test_host_allreduce_every_path(oracle, path, params):
    R, n, dtype = 8, 8 * 200_000 + 5, "bf16"
    xs = W.rank_inputs("normal", 71, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    comm = make_comm(R, n, dtype, path, **params)
    _with_staging(comm, R, n, dtype)
    h_send = [_pinned(x) for x in xs]
    h_recv = [torch.zeros(n * 2, dtype=torch.uint8).pin_memory() for _ in range(R)]
    comm.host_allreduce(h_send, h_recv, n, dtype)
    torch.cuda.synchronize()
    for r in range(R):
        assert same_bits(h_recv[r].numpy().view(np.uint16), want[r], dtype), r
    comm.destroy()


def test_host_allreduce_in_place_and_stream_order(oracle):
    """h_recv[r] == h_send[r] is legal; two calls back to back on one stream see each other's results."""
    R, n, dtype = 4, 4 * 300_000 + 2, "fp32"
    xs = W.rank_inputs("uniform", 72, R, n, dtype)
    once = oracle.ring_allreduce(xs)
    twice = oracle.ring_allreduce([once[r].copy() for r in range(R)])
    comm = make_comm(R, n, dtype, hb.PATH_CE)
    _with_staging(comm, R, n, dtype)
    bufs = [_pinned(x) for x in xs]
    stream = torch.cuda.Stream()
    comm.host_allreduce(bufs, bufs, n, dtype, stream)
    comm.host_allreduce(bufs, bufs, n, dtype, stream)
    stream.synchronize()
    for r in range(R):
        assert same_bits(bufs[r].numpy().view(np.float32), twice[r], dtype), r
    # partially overlapping host buffers of two ranks are refused and nothing runs
    big = torch.zeros(2 * n * 4, dtype=torch.uint8).pin_memory()
    bad_recv = [big[0:n * 4], big[n * 2:n * 2 + n * 4]] + [torch.zeros(n * 4, dtype=torch.uint8).pin_memory() for _ in range(R - 2)]
    rc = hb.lib().hoccl_host_allreduce(hb._ptr_array(bufs), hb._ptr_array(bad_recv), n, hb._dtype(dtype), hb.SUM, comm._h, None)
    assert rc == hb.ERR_INVALID_ARG
    comm.destroy()
