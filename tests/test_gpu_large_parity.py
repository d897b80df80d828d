"""Full-size parity on inputs WITHOUT a period: 64 MiB, 256 MiB and 1 GiB per rank.

The other large tests repeat a seeded block, so a piece, tile or chunk that lands a whole number of periods away from its
place would go unseen.  Here every element depends on (rank, position):

* integer-valued inputs in [-8, 8], hashed from (rank, index) and generated on the device.  Every partial sum of up to 8
  ranks is exact in bf16 and fp32, so the all-reduce result must be the exact integer sum of the element's R inputs,
  whatever the order: EVERY element of EVERY rank's result is compared with that sum (taken on the device with integer
  adds, no code of the library), and the oracle's ring all-reduce confirms the expectation on a one-Mi-element prefix
  and on windows that straddle every ring-chunk and pipeline-piece boundary;
* uniform[-1, 1) inputs, hashed the same way: the whole result against the oracle's step-by-step ring on the same bytes
  (order sensitive), at 64 MiB, 256 MiB and 1 GiB per rank.

The copy route (default schedule, which at these sizes runs its pieces on three overlapping streams; the ring step by
step; the direct schedule in one graph) and the SM path; R = 2 and R = 8; the ring at R = 2 and 1 GiB is the case that cuts a
ring chunk of more than 256 MiB into two pieces.
"""
import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import workloads as W

pytestmark = pytest.mark.gpu

MiB = 1 << 20
SEED = 4   # the size sweep's seed


def _bits(t):
    return t.view(torch.int32 if t.dtype == torch.float32 else torch.int16)


def _np(t):
    a = _bits(t).cpu().numpy()
    return a.view(np.float32) if t.dtype == torch.float32 else a.view(np.uint16)


def _comm(R, n, dtype, path, **params):
    comm = hb.Comm(R, 0)
    comm.set_path(path)
    for k, v in params.items():
        comm.set_param(k, v)
    direct = params.get("rs_direct", 0)
    nb = hb.scratch_bytes_direct(R, n, dtype) if direct else hb.scratch_bytes(R, n, dtype)
    scratch = torch.empty(nb + 256, dtype=torch.uint8, device="cuda")
    pad = (-scratch.data_ptr()) % 256
    comm.set_scratch(scratch.data_ptr() + pad, nb)
    comm._keep = scratch
    return comm


def _exact_integer_sum(send):
    """Exact per-element sum of integer-valued inputs, by integer adds on the device."""
    acc = torch.zeros(send[0].numel(), dtype=torch.int32, device=send[0].device)
    for s in send:
        acc += s.to(torch.int32)
    return acc.to(send[0].dtype)     # |sum| <= 64: exact in bf16 and fp32


def _boundaries(comm, R, n, e):
    """Element indices where a ring chunk or a pipeline piece of the last call starts: the planner's own piece offsets for the
    piece count the call reports, for equal and for graded pieces (the call may have used either)."""
    from paper_2609_34334_b200 import diag as hd
    q = -(-n // R)
    pieces = max(1, int(comm.last_stats()["n_pieces"]))
    dtype = "fp32" if e == 4 else "bf16"
    out = set(min(c * q, n) for c in range(R))
    if pieces > 1:
        for flags in (hd.PLAN_FLAG_RS_DIRECT, hd.PLAN_FLAG_RS_DIRECT | hd.PLAN_FLAG_GRADED):
            plan = hd.Plan(hd.PLAN_ALLREDUCE | flags, R, n, dtype, False, -(-(q * e) // pieces), pieces)
            out.update(op["local_off"] // e for op in plan.ops if op["kind"] == hd.OP_CHAIN)
    out.discard(0)
    out.discard(n)
    return sorted(out)


CONFIGS = [
    ("copy_route_sum8", hb.PATH_CE, {}),
    ("copy_route_ring", hb.PATH_CE, {"rs_direct": 0, "ag_direct": 0}),
    ("sm_path_whole_gpu", hb.PATH_SM, {"sum_ctas": 148, "copy_ctas": 148}),
    ("copy_route_direct_one_graph", hb.PATH_CE, {"rs_direct": 1, "ag_direct": 1, "ce_overlap": 0}),
    # with the scratch of the direct form attached (rs_direct = 2 is the default; naming it makes _comm attach that scratch):
    # the configurations bench.py times
    ("copy_route_default_overlapped", hb.PATH_CE, {"rs_direct": 2}),
    ("sm_path_sum8_copy40", hb.PATH_SM, {"rs_direct": 2, "sum_ctas": 8, "copy_ctas": 40}),
    ("sm_path_roles_sum8_copy40", hb.PATH_SM, {"rs_direct": 2, "sum_ctas": 8, "copy_ctas": 40, "roles": 1}),
]


@pytest.mark.parametrize("R,dtype,mib", [(2, "fp32", 64), (8, "bf16", 64), (2, "bf16", 256), (8, "bf16", 256),
                                         (8, "fp32", 256), (2, "fp32", 1024), (2, "bf16", 1024), (8, "bf16", 1024)])
def test_position_dependent_integer_inputs_give_the_exact_sum_everywhere(oracle, R, dtype, mib):
    torch.cuda.set_device(0)
    e = W.elem_size(dtype)
    n = mib * MiB // e
    send = [W.hashed_device("int", SEED, r, n, dtype) for r in range(R)]
    keep = [s.clone() for s in send[:1]]
    expect = _exact_integer_sum(send)
    recv = [torch.empty_like(s) for s in send]
    threads = oracle.max_threads()

    # the expectation itself, against the oracle's ring on the same values produced on the host: a prefix of 1 Mi
    # elements (order free, so the prefix's own chunking does not matter) ...
    m = 1 << 20
    pre = [W.hashed("int", SEED, r, 0, m, dtype) for r in range(R)]
    for r in range(R):
        assert (_np(send[r][:m]).view(np.uint8) == pre[r].view(np.uint8)).all(), "host and device generators differ"
    want = oracle.ring_allreduce(pre, threads=threads)[0]
    assert (_np(expect[:m]).view(np.uint8) == want.view(np.uint8)).all()

    for name, path, params in CONFIGS:
        if params.get("rs_direct") and hb.scratch_bytes_direct(R, n, dtype) > (40 << 30):
            continue
        comm = _comm(R, n, dtype, path, **params)
        for t in recv:
            t.fill_(3.0)
        comm.allreduce(send, recv, n, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert torch.equal(_bits(recv[r]), _bits(expect)), (name, R, dtype, mib, r)
        # ... and windows across every chunk and piece boundary of this call, through the oracle
        w = 4096
        for b in _boundaries(comm, R, n, e):
            lo, hi = max(0, b - w), min(n, b + w)
            win = [W.hashed("int", SEED, r, lo, hi - lo, dtype) for r in range(R)]
            ow = oracle.ring_allreduce(win)[0]
            assert (_np(recv[0][lo:hi]).view(np.uint8) == ow.view(np.uint8)).all(), (name, "boundary", b)
            assert (_np(recv[R - 1][lo:hi]).view(np.uint8) == ow.view(np.uint8)).all(), (name, "boundary", b)
        if R == 2 and mib == 1024 and name == "copy_route_ring":
            assert comm.last_stats()["n_pieces"] == 2      # the branch that cuts a 512 MiB ring chunk in two
        assert comm.destroy() == hb.OK
        del comm
    assert torch.equal(_bits(send[0]), _bits(keep[0])), "a send buffer was written"
    del send, recv, expect
    torch.cuda.empty_cache()


@pytest.mark.parametrize("R,dtype,mib", [(2, "fp32", 64), (8, "bf16", 64), (4, "fp32", 64), (8, "bf16", 256), (2, "fp32", 256),
                                         (2, "fp32", 1024), (8, "bf16", 1024)])
def test_position_dependent_uniform_inputs_against_the_whole_oracle_result(oracle, R, dtype, mib):
    """Order sensitive and without a period: every element against the step-by-step ring on the same bytes."""
    torch.cuda.set_device(0)
    e = W.elem_size(dtype)
    n = mib * MiB // e
    send = [W.hashed_device("uniform", SEED, r, n, dtype) for r in range(R)]
    xs = [_np(s) for s in send]
    # spot check of the device generator against the host one (the oracle must see what the device sees)
    for r in (0, R - 1):
        assert (W.hashed("uniform", SEED, r, n - 1000, 1000, dtype).view(np.uint8) == xs[r][n - 1000:].view(np.uint8)).all()
    want_all = oracle.ring_allreduce(xs, threads=oracle.max_threads())
    for r in range(1, R):
        assert (want_all[r] == want_all[0]).all()
    want = torch.from_numpy(want_all[0].view(np.int32 if dtype == "fp32" else np.int16)).cuda()
    del want_all, xs
    recv = [torch.empty_like(s) for s in send]
    for name, path, params in CONFIGS:
        comm = _comm(R, n, dtype, path, **params)
        for t in recv:
            t.zero_()
        comm.allreduce(send, recv, n, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert torch.equal(_bits(recv[r]), want), (name, R, dtype, mib, r)
        assert comm.destroy() == hb.OK
    # reduce-scatter and all-gather as two calls (the form the gradient bucket uses) give the same bits
    if n % R == 0:
        comm = _comm(R, n, dtype, hb.PATH_CE)
        part = [torch.empty(n // R, dtype=send[0].dtype, device="cuda") for _ in range(R)]
        comm.reduce_scatter(send, part, n // R, dtype)
        comm.allgather(part, recv, n // R, dtype)
        torch.cuda.synchronize()
        for r in range(R):
            assert torch.equal(_bits(recv[r]), want), ("rs+ag", r)
        assert comm.destroy() == hb.OK
    del send, recv, want
    torch.cuda.empty_cache()


def test_moves_at_full_size_on_position_dependent_bytes():
    """All-gather, all-to-all and send/recv at 256 MiB and 1 GiB per rank: identities on hashed bytes, both paths."""
    torch.cuda.set_device(0)
    R, dtype = 8, "bf16"
    for mib in (256, 1024):
        n = mib * MiB // 2
        q = n // R
        send = [W.hashed_device("uniform", SEED + 1, r, n, dtype) for r in range(R)]
        recv = [torch.empty_like(s) for s in send]
        for path, params in ((hb.PATH_CE, {}), (hb.PATH_SM, {"copy_ctas": 148}), (hb.PATH_SM, {"copy_ctas": 148, "ag_direct": 1})):
            comm = hb.Comm(R, 0)
            comm.set_path(path)
            for k, v in params.items():
                comm.set_param(k, v)
            comm.allgather([s[:q] for s in send], recv, q, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                for c in range(R):
                    assert torch.equal(_bits(recv[r][c * q:(c + 1) * q]), _bits(send[c][:q])), ("allgather", mib, path, r, c)
            comm.alltoall(send, recv, q, dtype)
            torch.cuda.synchronize()
            for r in range(R):
                for c in range(R):
                    assert torch.equal(_bits(recv[r][c * q:(c + 1) * q]), _bits(send[c][r * q:(r + 1) * q])), ("alltoall", mib, path, r, c)
            comm.send(send[2], n, dtype, 2, 6)
            comm.recv(recv[6], n, dtype, 2, 6)
            torch.cuda.synchronize()
            assert torch.equal(_bits(recv[6]), _bits(send[2]))
            assert comm.destroy() == hb.OK
        del send, recv
        torch.cuda.empty_cache()
