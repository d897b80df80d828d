"""Parity over the message-size sweep (the fifth benchmark configuration), sampled: every operation, R in {2, 4, 8},
both dtypes, both paths, sizes from 4 KiB to 16 MiB per rank (uniform[-1,1), seed 4) against the oracle, bit for bit.
Larger sizes: the periodic-input test in test_gpu_parity.py, and the largest point of the sweep (R = 8, 1 GiB per rank) below."""
import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import workloads as W

pytestmark = pytest.mark.gpu

SIZES = [1 << 12, 1 << 16, 1 << 20, 1 << 24]


def _dev(x, dtype):
    return torch.from_numpy(x if dtype == "fp32" else x.view(np.int16)).cuda()


def _host(t, dtype):
    a = t.cpu().numpy()
    return a if dtype == "fp32" else a.view(np.uint16)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("R", [2, 4, 8])
def test_sweep_points_match_the_oracle(oracle, R, dtype):
    torch.cuda.set_device(0)
    e = W.elem_size(dtype)
    seed = W.C5_SWEEP.seed
    threads = oracle.max_threads()
    for S in SIZES:
        n = S // e
        xs = W.rank_inputs("uniform", seed, R, n, dtype)
        want_ar = oracle.ring_allreduce(xs, threads=threads)
        want_rs = oracle.ring_reduce_scatter(xs, threads=threads)
        want_ag = oracle.allgather([x[:n // R] for x in xs])
        want_a2a = oracle.alltoall(xs)
        tdt = torch.float32 if dtype == "fp32" else torch.int16
        send = [_dev(x, dtype) for x in xs]
        scratch = torch.empty(hb.scratch_bytes(R, n, dtype) + 256, dtype=torch.uint8, device="cuda")
        pad = (-scratch.data_ptr()) % 256
        # the copy route with its small-message rule (default: up to 8 MiB per rank the moves are copy-kernel launches), the
        # copy route with driver copies at every size, and the SM path
        for path, small in ((hb.PATH_CE, None), (hb.PATH_CE, 0), (hb.PATH_SM, None)):
            comm = hb.Comm(R, 0)
            comm.set_scratch(scratch.data_ptr() + pad, scratch.numel() - 256)
            comm.set_path(path)
            if small is not None:
                comm.set_param("ce_small_bytes", small)
            recv = [torch.zeros(n, dtype=tdt, device="cuda") for _ in range(R)]
            comm.allreduce(send, recv, n, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert (_host(recv[r], dtype).view(np.uint8) == want_ar[r].view(np.uint8)).all(), ("allreduce", S, path, r)
            rs = [torch.zeros(n // R, dtype=tdt, device="cuda") for _ in range(R)]
            comm.reduce_scatter(send, rs, n // R, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                assert (_host(rs[r], dtype).view(np.uint8) == want_rs[r].view(np.uint8)).all(), ("reduce_scatter", S, path, r)
            ag = [torch.zeros(n, dtype=tdt, device="cuda") for _ in range(R)]
            comm.allgather([s[:n // R] for s in send], ag, n // R, dtype)
            a2a = [torch.zeros(n, dtype=tdt, device="cuda") for _ in range(R)]
            comm.alltoall(send, a2a, n // R, dtype)
            p2p = torch.zeros(n, dtype=tdt, device="cuda")
            comm.send(send[1], n, dtype, 1, 0)
            comm.recv(p2p, n, dtype, 1, 0)
            torch.cuda.synchronize()
            for r in range(R):
                assert (_host(ag[r], dtype) == want_ag[r]).all(), ("allgather", S, path, r)
                assert (_host(a2a[r], dtype) == want_a2a[r]).all(), ("alltoall", S, path, r)
            assert (_host(p2p, dtype) == oracle.sendrecv(xs[1])).all(), ("sendrecv", S, path)
            assert comm.destroy() == hb.OK


def test_largest_sweep_point_r8_1GiB_per_rank(oracle):
    """The largest point of the sweep: R = 8, 1 GiB per rank, bf16 (16 GiB of rank buffers).  Inputs are a seeded
    block per rank repeated on the device, so the oracle's chain result on one block, repeated, is the expectation
    for every element; compared on the device.  All-reduce on the copy route, the SM path and the one-kernel form;
    all-gather, all-to-all and send/recv as identities on bytes."""
    torch.cuda.set_device(0)
    R, dtype, period = 8, "bf16", 1 << 16
    n = (1 << 30) // 2
    q = n // R
    assert q % period == 0
    base = W.rank_inputs("uniform", W.C5_SWEEP.seed, R, period, dtype)
    send = [torch.from_numpy(b.view(np.int16)).cuda().repeat(n // period) for b in base]
    recv = [torch.empty(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    expect = torch.empty(n, dtype=torch.int16, device="cuda")
    for c in range(R):
        blk = oracle.chain_sum(base, c, 0, period)
        expect[c * q:(c + 1) * q] = torch.from_numpy(blk.view(np.int16)).cuda().repeat(q // period)
    scratch = torch.empty(hb.scratch_bytes(R, n, dtype) + 256, dtype=torch.uint8, device="cuda")
    pad = (-scratch.data_ptr()) % 256
    for path, params in ((hb.PATH_CE, {}), (hb.PATH_SM, {"sum_ctas": 148, "copy_ctas": 148}),
                         (hb.PATH_SM, {"sum_ctas": 148, "copy_ctas": 148, "fused": 1})):
        comm = hb.Comm(R, 0)
        comm.set_scratch(scratch.data_ptr() + pad, scratch.numel() - 256)
        comm.set_path(path)
        for k, v in params.items():
            comm.set_param(k, v)
        for t in recv:
            t.zero_()
        comm.allreduce(send, recv, n, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert torch.equal(recv[r], expect), (path, params, r)
        assert comm.async_error() == hb.OK
        if path == hb.PATH_CE:
            # all-gather of the first 1/R of every send buffer; all-to-all of whole buffers; one 1 GiB message
            comm.allgather([s[:q] for s in send], recv, q, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                for c in range(R):
                    assert torch.equal(recv[r][c * q:(c + 1) * q], send[c][:q]), ("allgather", r, c)
            comm.alltoall(send, recv, q, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                for c in range(R):
                    assert torch.equal(recv[r][c * q:(c + 1) * q], send[c][r * q:(r + 1) * q]), ("alltoall", r, c)
            comm.send(send[3], n, dtype, 3, 5)
            comm.recv(recv[5], n, dtype, 3, 5)
            torch.cuda.synchronize()
            assert torch.equal(recv[5], send[3])
        assert comm.destroy() == hb.OK
    del send, recv, expect, scratch
    torch.cuda.empty_cache()
