"""HOCCL_PATH_CE_HOST: moves bounce through pinned host memory, so both legs run on the copy engines.  Checked:
every collective and send/recv give the oracle's bits, a move finishes while a kernel holds every SM (the paper's
zero-SM claim, measured), and missing or too small host staging is refused."""
import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import diag as hd
from paper_2609_34334_b200 import workloads as W
from gpu_util import DevBuf, np_dtype, same_bits

pytestmark = pytest.mark.gpu


def _comm(R, n, dtype, host_bytes):
    comm = hb.Comm(R, 0)
    nb = hb.scratch_bytes(R, n, dtype)
    scratch = torch.empty(nb + 256, dtype=torch.uint8, device="cuda")
    pad = (-scratch.data_ptr()) % 256
    if nb:
        comm.set_scratch(scratch.data_ptr() + pad, nb)
    comm._keep_scratch = scratch
    comm.set_path(hb.PATH_CE_HOST)
    if host_bytes:
        comm.set_host_staging(torch.empty(host_bytes, dtype=torch.uint8).pin_memory())
    return comm


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("use_graph", [0, 1])
@pytest.mark.parametrize("ag_direct", [0, 1])
def test_collectives_over_host_bounce(oracle, dtype, use_graph, ag_direct):
    """ag_direct = 1: the all-gather's moves that read the same chunk share one outbound copy into the host staging."""
    torch.cuda.set_device(0)
    e = W.elem_size(dtype)
    for R, n in [(2, 4099), (4, 4 * 30_000 + 4), (8, 8 * 8192), (3, 10)]:
        xs = W.rank_inputs("uniform", 700 + n % 9, R, n, dtype)
        want = oracle.ring_allreduce(xs)
        comm = _comm(R, n, dtype, 4 * R * (n * e + 4096))
        comm.set_param("use_graph", use_graph)
        comm.set_param("ag_direct", ag_direct)
        comm.set_param("piece_bytes", 16384)
        send = [DevBuf(n * e).put(xs[r]) for r in range(R)]
        recv = [DevBuf(n * e) for _ in range(R)]
        comm.allreduce(send, recv, n, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert same_bits(recv[r].get(np_dtype(dtype)), want[r], dtype), (R, n, r)
            assert recv[r].guards_intact() and send[r].guards_intact()
        if n % R == 0:
            count = n // R
            wa = oracle.alltoall(xs)
            a2a = [DevBuf(n * e) for _ in range(R)]
            comm.alltoall(send, a2a, count, dtype)
            ag = [DevBuf(n * e) for _ in range(R)]
            comm.allgather([send[r].ptr for r in range(R)], ag, count, dtype)
            torch.cuda.synchronize()
            wg = oracle.allgather([x[:count] for x in xs])
            for r in range(R):
                assert (a2a[r].get(np_dtype(dtype)).view(np.uint8) == wa[r].view(np.uint8)).all()
                assert (ag[r].get(np_dtype(dtype)).view(np.uint8) == wg[r].view(np.uint8)).all()
        dst = DevBuf(n * e)
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        comm.send(send[1], n, dtype, 1, 0, s1)
        comm.recv(dst, n, dtype, 1, 0, s2)
        torch.cuda.synchronize()
        assert (dst.get(np_dtype(dtype)).view(np.uint8) == oracle.sendrecv(xs[1]).view(np.uint8)).all()
        assert comm.destroy() == hb.OK


def test_host_bounce_moves_need_no_sm_and_staging_is_checked():
    torch.cuda.set_device(0)
    R, n = 4, 4 * 4096
    comm = _comm(R, n, "fp32", 0)
    a = [torch.ones(n, dtype=torch.float32, device="cuda") for _ in range(R)]
    b = [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(R)]
    assert comm.allreduce_rc(a, b, n, "fp32") == hb.ERR_SCRATCH            # no host staging attached
    assert comm.send_rc(a[0], n, "fp32", 0, 1) == hb.OK and comm.recv_rc(b[0], n, "fp32", 0, 1) == hb.ERR_SCRATCH
    pageable = torch.empty(1 << 20, dtype=torch.uint8)
    assert hb.lib().hoccl_comm_set_host_staging(comm._h, pageable.data_ptr(), pageable.numel()) == hb.ERR_INVALID_ARG
    comm.set_host_staging(torch.empty(1024, dtype=torch.uint8).pin_memory())
    assert comm.allreduce_rc(a, b, n, "fp32") == hb.ERR_SCRATCH            # too small
    comm.set_host_staging(torch.empty(32 << 20, dtype=torch.uint8).pin_memory())
    src = torch.ones(8 << 20, dtype=torch.uint8, device="cuda")
    dst = torch.zeros(8 << 20, dtype=torch.uint8, device="cuda")
    needs_sm, end_us = hd.probe_move_needs_sm(comm, hb.PATH_CE_HOST, dst, src, src.numel(), 3000)
    assert needs_sm is False and end_us < 2700            # finished while a kernel held every SM: copy engines only
    assert torch.equal(src, dst)
    comm.set_param("handshake", 1)
    assert comm.allreduce_rc(a, b, n, "fp32") == hb.ERR_UNSUPPORTED
    comm.set_param("handshake", 0)
    assert comm.allreduce_rc(a, b, n, "fp32") == hb.OK
    torch.cuda.synchronize()
    assert float(b[2][77]) == 4.0
    assert comm.destroy() == hb.OK


def test_large_messages_are_pipelined_through_the_staging_area():
    """send/recv of messages larger than one staging chunk: the two legs run chunk by chunk on two lanes.  Messages that
    follow one another reuse the staging area in order; every message arrives bit for bit."""
    import time
    torch.cuda.set_device(0)
    n = (48 << 20) + 12345 * 2                                   # bf16 elements x 2 B: 48 MiB and a ragged tail
    comm = hb.Comm(4, 0)
    comm.set_path(hb.PATH_CE_HOST)
    comm.set_host_staging(torch.empty(2 * n + 4096, dtype=torch.uint8).pin_memory())
    msgs = [torch.randint(-30000, 30000, (n,), dtype=torch.int16, device="cuda") for _ in range(3)]
    dsts = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(3)]
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()                                      # the tensors above were filled on torch's current stream
    for k in range(3):                                            # back to back, no host synchronisation
        comm.send(msgs[k], n, "bf16", k, k + 1, s1)
        comm.recv(dsts[k], n, "bf16", k, k + 1, s2)
    torch.cuda.synchronize()
    for k in range(3):
        assert torch.equal(msgs[k], dsts[k]), k
    # timing: the pipelined legs beat the same two copies issued one after the other, measured side by side (best of three
    # each: one slow PCIe transfer must not decide it)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    host = torch.empty(n, dtype=torch.int16).pin_memory()
    with torch.cuda.stream(s1):
        host.copy_(msgs[0], non_blocking=True)                    # touch the pages once
    torch.cuda.synchronize()
    t_pipe, t_seq = [], []
    for trial in range(3):
        e0.record(s1)
        comm.send(msgs[0], n, "bf16", 0, 1, s1)
        comm.recv(dsts[1], n, "bf16", 0, 1, s1)
        e1.record(s1)
        torch.cuda.synchronize()
        assert torch.equal(msgs[0], dsts[1])
        t_pipe.append(e0.elapsed_time(e1))
        with torch.cuda.stream(s1):
            e0.record(s1)
            host.copy_(msgs[0], non_blocking=True)
            dsts[2].copy_(host, non_blocking=True)
            e1.record(s1)
        torch.cuda.synchronize()
        t_seq.append(e0.elapsed_time(e1))
    assert min(t_pipe) < 0.85 * min(t_seq), (t_pipe, t_seq)
    assert comm.destroy() == hb.OK
