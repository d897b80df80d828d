"""Handshake mode: the paper's stream manager (CPU proxy + two flags moved by stream memory operations).

Checked: results equal the oracle bit for bit; the operation is ordered against neighbouring kernels of the
caller's stream; a send/recv post may wait for a partner that is posted later on another stream; the watchdog
releases a stream whose partner never comes and reports it (no wait on this library is unbounded).
"""
import time

import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import workloads as W
from gpu_util import DevBuf, np_dtype, same_bits

pytestmark = pytest.mark.gpu


def _wait(stream, seconds=60.0):
    """Polls instead of blocking, so that a parked stream fails the test instead of hanging the run."""
    t0 = time.time()
    while not stream.query():
        if time.time() - t0 > seconds:
            pytest.fail("stream still busy after %.0f s" % seconds)
        time.sleep(0.002)


def _comm(R, n, dtype, **params):
    comm = hb.Comm(R, 0)
    nb = hb.scratch_bytes(R, n, dtype)
    scratch = torch.empty(nb + 256, dtype=torch.uint8, device="cuda")
    pad = (-scratch.data_ptr()) % 256
    if nb:
        comm.set_scratch(scratch.data_ptr() + pad, nb)
    comm._keep_scratch = scratch
    for k, v in params.items():
        comm.set_param(k, v)
    return comm


def test_collectives_through_the_proxy_match_the_oracle(oracle):
    torch.cuda.set_device(0)
    path = hb.PATH_SM
    R, n, dtype = 8, 8 * 50_000 + 8, "bf16"
    xs = W.rank_inputs("normal", 91, R, n, dtype, 1e-3)
    want = oracle.ring_allreduce(xs)
    comm = _comm(R, n, dtype, handshake=1, watchdog_ms=5000)
    comm.set_path(path)
    st = torch.cuda.Stream()
    base = [torch.from_numpy(x.view(np.int16)).cuda() for x in xs]
    send = [torch.zeros_like(b) for b in base]
    recv = [torch.zeros_like(b) for b in base]
    after = [torch.zeros_like(b) for b in base]
    torch.cuda.synchronize()
    for rep in range(3):
        with torch.cuda.stream(st):
            for r in range(R):
                send[r].copy_(base[r])                 # producer kernels on the same stream
            comm.allreduce(send, recv, n, dtype, st)
            for r in range(R):
                after[r].copy_(recv[r])                # consumer kernels on the same stream
        _wait(st)
        for r in range(R):
            assert same_bits(after[r].cpu().numpy().view(np.uint16), want[r], dtype), (rep, r)
            recv[r].zero_()
        torch.cuda.synchronize()                       # zero_ ran on torch's current stream, the next repetition runs on st
    assert comm.handshakes() == 3
    assert comm.async_error() == hb.OK
    # all-gather and all-to-all go the same way
    ys = W.rank_inputs("uniform", 92, R, 4096, dtype)
    gs = [torch.from_numpy(y.view(np.int16)).cuda() for y in ys]
    gr = [torch.zeros(R * 4096, dtype=torch.int16, device="cuda") for _ in range(R)]
    torch.cuda.synchronize()
    comm.allgather(gs, gr, 4096, dtype, st)
    _wait(st)
    cat = np.concatenate(ys)
    for r in range(R):
        assert (gr[r].cpu().numpy().view(np.uint16) == cat).all()
    assert comm.destroy() == hb.OK


def test_send_recv_waits_for_a_partner_posted_later(oracle):
    torch.cuda.set_device(0)
    comm = hb.Comm(4, 0)
    comm.set_param("handshake", 1)
    comm.set_param("watchdog_ms", 5000)
    comm.set_path(hb.PATH_SM)
    n, dtype = 1_000_003, "fp32"
    msg = W.uniform(93, 0, n, dtype)
    src = DevBuf(n * 4).put(msg)
    dst = DevBuf(n * 4)
    seen = torch.zeros(n, dtype=torch.float32, device="cuda")
    s_recv, s_send = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    # the receiver posts first and keeps working on its stream: the consumer kernel must wait for the data
    comm.recv(dst, n, dtype, 1, 2, s_recv)
    with torch.cuda.stream(s_recv):
        seen.copy_(dst.view.view(torch.float32))
    time.sleep(0.05)                                   # the partner comes later
    assert comm.pending() == 1
    assert not s_recv.query()                          # the receiver's stream is parked in the hand-over
    comm.send(src, n, dtype, 1, 2, s_send)
    _wait(s_recv)
    _wait(s_send)
    assert (seen.cpu().numpy() == oracle.sendrecv(msg)).all()
    assert dst.guards_intact() and src.guards_intact()
    assert comm.pending() == 0 and comm.async_error() == hb.OK
    assert comm.destroy() == hb.OK


def test_watchdog_releases_an_unmatched_post_and_reports_it():
    torch.cuda.set_device(0)
    comm = hb.Comm(2, 0)
    comm.set_param("handshake", 1)
    comm.set_param("watchdog_ms", 300)
    # the copy route is refused in handshake mode (driver copies can queue behind the parked stream's own copies)
    probe = DevBuf(64)
    assert comm.recv_rc(probe, 16, "fp32", 0, 1) == hb.ERR_UNSUPPORTED and comm.pending() == 0
    comm.set_path(hb.PATH_SM)
    buf = DevBuf(4096, fill=0x33)
    st = torch.cuda.Stream()
    t0 = time.time()
    comm.recv(buf, 1024, "fp32", 0, 1, st)             # nobody ever sends
    _wait(st, 20)                                      # returns once the watchdog has released the stream
    dt = time.time() - t0
    assert 0.25 < dt < 5.0, dt
    assert comm.async_error(clear=True) == hb.ERR_TIMEOUT
    assert comm.async_error() == hb.OK
    assert comm.pending() == 0
    assert (buf.get(np.uint8) == 0x33).all()           # nothing was written
    # a count mismatch is reported the same way and both streams are released
    a, b = DevBuf(4096), DevBuf(4096, fill=0x44)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    comm.send(a, 1024, "fp32", 0, 1, s1)
    comm.recv(b, 512, "fp32", 0, 1, s2)
    _wait(s1, 20)
    _wait(s2, 20)
    assert comm.async_error(clear=True) == hb.ERR_MISMATCH
    assert (b.get(np.uint8) == 0x44).all()
    # the communicator still works afterwards
    comm.send(a, 1024, "fp32", 0, 1, s1)
    comm.recv(b, 1024, "fp32", 0, 1, s2)
    _wait(s1, 20)
    _wait(s2, 20)
    assert (b.get(np.uint8) == a.get(np.uint8)).all() and comm.async_error() == hb.OK
    assert comm.destroy() == hb.OK
