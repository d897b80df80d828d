"""GPU parity for the gradient-stream workload: GPT-6.7B shaped bf16 gradients cut into 40 MiB buckets over
R = 8 ranks, one all-reduce per bucket issued back to back on one stream through a small pool of reusable
per-rank buffers (the launch configuration the `gradients` sweep times).  A sample of the 308 buckets is
compared with the oracle bit for bit: the first two buckets, the bucket that straddles the first layer
boundary, one from the middle, the last full one and the ragged 8 MiB tail."""
import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import workloads as W
from gpu_util import DevBuf, same_bits
from test_gpu_parity import make_comm

pytestmark = pytest.mark.gpu

POOL = 3


def _bucket_inputs(g, sizes, b):
    per = sizes[0]
    from concurrent.futures import ThreadPoolExecutor

    with ThreadPoolExecutor(max_workers=8) as pool:
        return list(pool.map(lambda r: W.normal(g.seed, r, sizes[b], g.dtype, g.sigma, start=b * per), range(g.R)))


def test_config4_gradient_buckets_sampled(oracle):
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    torch.cuda.set_device(0)
    g = W.C4_GRADIENTS
    sizes = g.buckets()
    per, R = sizes[0], g.R
    assert len(sizes) == 308 and sizes[-1] * 2 == 8 << 20 and per * 2 == 40 << 20
    boundary = g.elements_per_layer // per                  # the bucket holding the end of layer 0
    sample = [0, 1, boundary, 160, len(sizes) - 2, len(sizes) - 1]
    comm = make_comm(R, per, g.dtype, hb.PATH_CE)
    send = [[DevBuf(per * 2) for _ in range(R)] for _ in range(POOL)]
    recv = [[DevBuf(per * 2) for _ in range(R)] for _ in range(POOL)]
    stream = torch.cuda.Stream()
    for first in range(0, len(sample), POOL):
        group = sample[first:first + POOL]
        xs = [_bucket_inputs(g, sizes, b) for b in group]
        for k, b in enumerate(group):
            for r in range(R):
                send[k][r].view[:sizes[b] * 2].copy_(torch.from_numpy(xs[k][r].view(np.uint8)))
                recv[k][r].view.fill_(0x5A)
        torch.cuda.synchronize()
        for k, b in enumerate(group):                       # back to back, no host synchronisation between buckets
            comm.allreduce(send[k], recv[k], sizes[b], g.dtype, stream)
        torch.cuda.synchronize()
        for k, b in enumerate(group):
            want = oracle.ring_allreduce(xs[k], threads=oracle.max_threads())
            for r in range(R):
                got = recv[k][r].get(np.uint16)
                assert same_bits(got[:sizes[b]], want[r], g.dtype), (b, r)
                assert (got[sizes[b]:] == 0x5A5A).all(), "wrote past the end of a short bucket"
                assert recv[k][r].guards_intact() and send[k][r].guards_intact()
    assert comm._scratch_keep.guards_intact()
    comm.destroy()
