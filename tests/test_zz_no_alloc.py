"""hoccl_allreduce_static: the all-reduce for callers that cannot allocate device memory.

Such callers (a communication thread that must not trigger an allocation's device-wide synchronisation,
a process whose memory is owned by a static planner) have no scratch to attach, so the entry point uses
the fixed array inside the library.  The check: through the C ABI, two calls in a row give exactly the
bits of the regular hoccl_allreduce (whose scratch is caller-attached) AND of the CPU oracle's ring, the
second call is not disturbed by what the first left in the shared array, a warm call leaves the device's
free memory unchanged, and requests beyond the fixed maximum are refused.
Collected last on purpose (file name), so a run that stops at the first failure has run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _regular_allreduce(xs_dev, n, dtype, R):
    comm = hb.Comm(R, 0)
    scratch = torch.empty(hb.scratch_bytes(R, n, dtype) + 256, dtype=torch.uint8, device="cuda")
    pad = (-scratch.data_ptr()) % 256
    comm.set_scratch(scratch.data_ptr() + pad, scratch.numel() - 256)
    out = [torch.zeros_like(x) for x in xs_dev]
    comm.allreduce(xs_dev, out, n, dtype)
    torch.cuda.synchronize()
    assert comm.destroy() == hb.OK
    return out


@pytest.mark.parametrize("dtype,R,n", [("bf16", 8, 8 * 100_000 + 8), ("fp32", 4, 1_048_576), ("fp32", 3, 10_007)])
def test_static_scratch_allreduce_matches_regular_entry_point_twice(oracle, dtype, R, n):
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    tdt = torch.float32 if dtype == "fp32" else torch.int16
    first = W.rank_inputs("normal", 61, R, n, dtype, 1e-3)
    second = W.rank_inputs("uniform", 62, R, n, dtype)
    for xs in (first, second):          # two calls in a row on the shared array, different data
        dev = [torch.from_numpy(x if dtype == "fp32" else x.view(np.int16)).cuda() for x in xs]
        want = _regular_allreduce(dev, n, dtype, R)
        got = [torch.full((n,), 7, dtype=tdt, device="cuda") for _ in range(R)]
        assert hb.allreduce_static(dev, got, n, dtype, R) == hb.OK
        torch.cuda.synchronize()
        for r in range(R):
            # bit-exact: the tolerance of the parity tests for sums in the fixed ring order
            assert torch.equal(got[r].view(torch.int32 if dtype == "fp32" else torch.int16),
                               want[r].view(torch.int32 if dtype == "fp32" else torch.int16)), (dtype, R, r)
            assert torch.equal(dev[r].cpu(), torch.from_numpy(xs[r] if dtype == "fp32" else xs[r].view(np.int16)))
        # and the oracle's step-by-step ring on the same bytes
        ring = oracle.ring_allreduce(xs)
        for r in range(R):
            assert (got[r].cpu().numpy().view(np.uint8) == ring[r].view(np.uint8)).all(), ("oracle", dtype, R, r)
    # in place as well
    dev = [torch.from_numpy(x if dtype == "fp32" else x.view(np.int16)).cuda() for x in second]
    assert hb.allreduce_static(dev, dev, n, dtype, R) == hb.OK
    torch.cuda.synchronize()
    for r in range(R):
        assert torch.equal(dev[r], want[r])


def test_a_warm_call_allocates_no_device_memory(oracle):
    """After the first call on the device (which looks up the array and may load the library's module), further calls
    leave the device's free memory exactly as it was: nothing is allocated, cached or freed by the call."""
    torch.cuda.set_device(0)
    R, n, dtype = 4, 262_144, "fp32"
    xs = W.rank_inputs("uniform", 63, R, n, dtype)
    dev = [torch.from_numpy(x).cuda() for x in xs]
    got = [torch.empty_like(d) for d in dev]
    assert hb.allreduce_static(dev, got, n, dtype, R) == hb.OK       # first call: set-up happens here
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        assert hb.allreduce_static(dev, got, n, dtype, R) == hb.OK
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    want = oracle.ring_allreduce(xs)
    for r in range(R):
        assert (got[r].cpu().numpy().view(np.uint8) == want[r].view(np.uint8)).all()


def test_static_scratch_rejects_sizes_beyond_the_maximum():
    torch.cuda.set_device(0)
    R = 2
    n = (hb.STATIC_SCRATCH_BYTES // 4)          # needs 2*R*(n/R*4 + pad) > the fixed array
    a = [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(R)]
    b = [torch.full((n,), 3.0, dtype=torch.float32, device="cuda") for _ in range(R)]
    assert hb.allreduce_static(a, b, n, "fp32", R) == hb.ERR_SCRATCH
    torch.cuda.synchronize()
    assert float(b[0][0]) == 3.0 and float(b[1][-1]) == 3.0     # nothing was enqueued
    assert hb.allreduce_static(a, b, 0, "fp32", R) == hb.OK
    assert hb.allreduce_static(a, b, 16, "fp32", 0) == hb.ERR_INVALID_ARG
    assert hb.allreduce_static(a, b, 16, 9, R) == hb.ERR_UNSUPPORTED
    assert hb.allreduce_static([a[0], a[0]], b, 16, "fp32", R) == hb.ERR_INVALID_ARG
