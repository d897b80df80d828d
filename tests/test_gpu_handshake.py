"""Handshake mode: the paper's stream manager (CPU proxy + counters moved by stream memory operations).

Checked: results equal the oracle bit for bit; the operation is ordered against neighbouring kernels of the
caller's stream; a send/recv post may wait for a partner that is posted later on another stream; the watchdog
releases a stream whose partner never comes and reports it (no wait on this library is unbounded); destroying a
communicator while a hand-over is still queued behind earlier work of its stream lets that stream go; the mode is
refused on the copy routes by every entry point with nothing enqueued; "p2p_strict" gives send/recv alone the same
ordering; the proxy reports how busy it was.  Every failure here is made on the host (a partner that is never posted, a
stream kept busy by a bounded delay kernel): no GPU fault is involved.
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


def test_destroy_releases_a_hand_over_that_its_stream_has_not_reached_yet(oracle):
    """A stream is kept busy by a bounded delay kernel (about 0.4 s), an all-reduce is enqueued behind it, and the
    communicator is destroyed at once.  The proxy cannot serve the hand-over in time (watchdog 20 ms): destroy releases it
    by force and says so (TIMEOUT), the stream ends by itself when the delay is over (it does not wait on counters that
    nobody will write), the output was not produced, and a new communicator works normally afterwards."""
    torch.cuda.set_device(0)
    R, n, dtype = 4, 4096, "fp32"
    xs = W.rank_inputs("uniform", 95, R, n, dtype)
    send = [torch.from_numpy(x).cuda() for x in xs]
    recv = [torch.full((n,), 7.0, dtype=torch.float32, device="cuda") for _ in range(R)]
    comm = _comm(R, n, dtype, handshake=1, watchdog_ms=20)
    comm.set_path(hb.PATH_SM)
    st = torch.cuda.Stream()
    comm.allreduce(send, recv, n, dtype, st)             # first use: creates the proxy, builds and uploads the graph
    _wait(st)
    for t in recv:
        t.fill_(7.0)
    torch.cuda.synchronize()
    clock_hz = torch.cuda.get_device_properties(0).clock_rate * 1000 if hasattr(torch.cuda.get_device_properties(0), "clock_rate") else 1.9e9
    with torch.cuda.stream(st):
        torch.cuda._sleep(int(0.4 * clock_hz))           # bounded: a fixed number of clock cycles
    comm.allreduce(send, recv, n, dtype, st)             # queued behind the delay: the stream has not arrived at it
    t0 = time.time()
    rc = comm.destroy()
    assert rc == hb.ERR_TIMEOUT, rc
    assert time.time() - t0 < 5.0
    _wait(st, 20)                                        # the stream is not held by anything once the delay is over
    assert all(bool((t == 7.0).all().item()) for t in recv)     # released without its result, as the return code said
    # a fresh communicator (and a fresh proxy) on the same device
    comm2 = _comm(R, n, dtype, handshake=1, watchdog_ms=5000)
    comm2.set_path(hb.PATH_SM)
    comm2.allreduce(send, recv, n, dtype, st)
    _wait(st)
    want = oracle.ring_allreduce(xs)
    for r in range(R):
        assert same_bits(recv[r].cpu().numpy(), want[r], dtype)
    assert comm2.destroy() == hb.OK


def test_handshake_is_refused_on_the_copy_routes_by_every_entry_point():
    """The proxy cannot drive driver copies behind a parked stream (they can queue up behind that stream's own copies), so
    on HOCCL_PATH_CE and HOCCL_PATH_CE_HOST every entry point returns UNSUPPORTED in handshake mode and enqueues nothing."""
    torch.cuda.set_device(0)
    R, n, dtype = 4, 4096, "fp32"
    for path in (hb.PATH_CE, hb.PATH_CE_HOST):
        for mode in ("handshake", "p2p_strict"):
            comm = _comm(R, n * R, dtype, **{mode: 1})
            comm.set_path(path)
            host = torch.empty(1 << 20, dtype=torch.uint8).pin_memory()
            comm.set_host_staging(host)
            send = [DevBuf(n * R * 4) for _ in range(R)]
            recv = [DevBuf(n * R * 4, fill=0x3C) for _ in range(R)]
            st = torch.cuda.Stream()
            if mode == "handshake":
                assert comm.allreduce_rc(send, recv, n * R, dtype, st) == hb.ERR_UNSUPPORTED
                assert comm.reduce_scatter_rc(send, recv, n, dtype, st) == hb.ERR_UNSUPPORTED
                assert comm.allgather_rc(send, recv, n, dtype, st) == hb.ERR_UNSUPPORTED
                assert comm.alltoall_rc(send, recv, n, dtype, st) == hb.ERR_UNSUPPORTED
                cnt = [n] * (R * R)
                dis = [(k % R) * n for k in range(R * R)]
                assert comm.alltoallv_rc(send, cnt, dis, recv, dis, dtype, st) == hb.ERR_UNSUPPORTED
                hs = [torch.zeros(n, dtype=torch.float32).pin_memory() for _ in range(R)]
                hr = [torch.zeros(n, dtype=torch.float32).pin_memory() for _ in range(R)]
                stage = torch.empty(2 * R * (n * 4 + 256) + 256, dtype=torch.uint8, device="cuda")
                comm.set_staging(stage.data_ptr() + (-stage.data_ptr()) % 256, 2 * R * (n * 4 + 256))
                assert hb.lib().hoccl_host_allreduce(hb._ptr_array(hs), hb._ptr_array(hr), n, hb.FLOAT32, hb.SUM, comm._h,
                                                     hb._stream(st)) == hb.ERR_UNSUPPORTED
            assert comm.send_rc(send[0], n, dtype, 0, 1, st) == hb.ERR_UNSUPPORTED
            assert comm.recv_rc(recv[1], n, dtype, 0, 1, st) == hb.ERR_UNSUPPORTED
            assert comm.pending() == 0 and comm.handshakes() == 0
            assert st.query()                                # nothing was enqueued
            torch.cuda.synchronize()
            assert all((b.get(np.uint8) == 0x3C).all() for b in recv)
            assert comm.destroy() == hb.OK


def test_strict_send_recv_orders_a_consumer_enqueued_between_the_two_posts(oracle):
    """The receiver posts first and enqueues a consumer of its buffer before the sender posts.  With the default matching
    on the host that consumer is not ordered against the transfer (stated in the header); with p2p_strict = 1 the post holds
    the receiver's stream until the data is there, so the consumer sees it.  Collectives on the same communicator are
    still launched directly (no hand-over)."""
    torch.cuda.set_device(0)
    R, n, dtype = 4, 500_003, "fp32"
    comm = _comm(R, n, dtype, p2p_strict=1, watchdog_ms=5000)
    comm.set_path(hb.PATH_SM)
    msg = W.uniform(96, 0, n, dtype)
    src = DevBuf(n * 4).put(msg)
    dst = DevBuf(n * 4)
    seen = torch.zeros(n, dtype=torch.float32, device="cuda")
    s_recv, s_send = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    comm.recv(dst, n, dtype, 2, 3, s_recv)
    with torch.cuda.stream(s_recv):
        seen.copy_(dst.view.view(torch.float32))            # the consumer, enqueued before the partner exists
    time.sleep(0.05)
    assert not s_recv.query() and comm.pending() == 1
    comm.send(src, n, dtype, 2, 3, s_send)
    _wait(s_recv)
    _wait(s_send)
    assert (seen.cpu().numpy() == oracle.sendrecv(msg)).all()
    served = comm.handshakes()
    assert served == 2
    xs = W.rank_inputs("uniform", 97, R, n, dtype)
    send = [torch.from_numpy(x).cuda() for x in xs]
    recv = [torch.zeros_like(t) for t in send]
    comm.allreduce(send, recv, n, dtype, s_send)
    _wait(s_send)
    assert comm.handshakes() == served                       # the collective did not go through the proxy
    want = oracle.ring_allreduce(xs)
    for r in range(R):
        assert same_bits(recv[r].cpu().numpy(), want[r], dtype)
    assert comm.async_error() == hb.OK and comm.destroy() == hb.OK


def test_proxy_reports_how_busy_it_was():
    torch.cuda.set_device(0)
    R, n, dtype = 8, 8 * 100_000, "bf16"
    comm = _comm(R, n, dtype, handshake=1, watchdog_ms=5000)
    comm.set_path(hb.PATH_SM)
    assert comm.proxy_stats() == (0.0, 0.0)                  # no proxy yet
    send = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    recv = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    st = torch.cuda.Stream()
    comm.allreduce(send, recv, n, dtype, st)
    _wait(st)
    comm.proxy_stats(reset=True)
    for _ in range(20):
        comm.allreduce(send, recv, n, dtype, st)
    _wait(st)
    busy, span = comm.proxy_stats(reset=True)
    assert 0.0 < busy < span, (busy, span)
    assert comm.proxy_stats() == (0.0, 0.0)
    assert comm.destroy() == hb.OK
