"""A modelled two-node topology run as real copies (paper Sec. 3.4: traffic-matrix expansion Eq. 2-4 and Algorithm 1).

With "model_gpus_per_node" set below the rank count, hoccl_alltoallv treats the logical ranks as GPUs of several nodes: a
flow between two nodes is carried, portion by portion as Algorithm 1 stages it, by the sender-side forwarding copy into a
staging slot at the sender's symmetric peer, the "RDMA" leg into a staging slot at the receiver's symmetric peer, and the
receiver-side forwarding copy into the receive buffer; native flows fill the NVLink slack of the stages.  The result must
be what the definition of all-to-allv says (the oracle), bit for bit, on both routes, whatever the chunk size and whether
or not the RDMA leg is cut into sub-copies; the call reports as many stages as the host-side scheduler produces for the
same traffic matrix.
"""
import numpy as np
import pytest
import torch

from paper_2609_34334_b200 import binding as hb
from paper_2609_34334_b200 import workloads as W
from gpu_util import DevBuf, np_dtype
from test_oracle_pins import _random_pattern

pytestmark = pytest.mark.gpu


def _staging_need(counts, e, gpn):
    R = counts.shape[0]
    need = 0
    for u in range(R):
        for v in range(R):
            if u != v and u // gpn != v // gpn and counts[u, v]:
                need += (int(counts[u, v]) * e + 255) // 256 * 256
    return 2 * need


@pytest.mark.parametrize("path", [hb.PATH_CE, hb.PATH_SM])
@pytest.mark.parametrize("R,gpn", [(8, 4), (8, 2), (6, 3), (4, 1), (5, 4)])
def test_two_node_schedule_moves_the_bytes_the_definition_says(oracle, path, R, gpn):
    torch.cuda.set_device(0)
    for dtype, max_count, piece, sub in (("bf16", 150_000, 65536, 0), ("fp32", 40_000, 131072, 16384), ("bf16", 5, 65536, 0)):
        e = W.elem_size(dtype)
        rng = np.random.default_rng(R * 100 + gpn * 10 + max_count % 7)
        counts, sd, rd, send_sizes, recv_sizes = _random_pattern(R, rng, max_count)
        xs = [W.uniform(57, u, send_sizes[u], dtype) for u in range(R)]
        fill = np.frombuffer(bytes([0xA5]) * e, dtype=np_dtype(dtype))[0]
        want = oracle.alltoallv(xs, counts.ravel(), sd.ravel(), rd.ravel(), recv_sizes, fill=fill)
        comm = hb.Comm(R, 0)
        comm.set_path(path)
        comm.set_param("piece_bytes", piece)
        comm.set_param("copy_ctas", 16)
        comm.set_param("model_gpus_per_node", gpn)
        comm.set_param("model_rdma_sub_bytes", sub)
        send = [DevBuf(send_sizes[u] * e).put(xs[u]) for u in range(R)]
        recv = [DevBuf(recv_sizes[v] * e) for v in range(R)]               # pre-filled with 0xA5 bytes
        need = _staging_need(counts, e, gpn)
        if need:
            assert comm.alltoallv_rc(send, counts.ravel(), sd.ravel(), recv, rd.ravel(), dtype) == hb.ERR_SCRATCH     # no staging attached yet
        stage = DevBuf(need + 256)
        pad = (-stage.ptr) % 256
        comm.set_staging(stage.ptr + pad, need)
        for rep in range(2):                                               # the second call replays the cached graph
            if rep:
                for v in range(R):
                    recv[v].view.fill_(0xA5)
                torch.cuda.synchronize()
            comm.alltoallv(send, counts.ravel(), sd.ravel(), recv, rd.ravel(), dtype)
            torch.cuda.synchronize()
            st = comm.last_stats()
            if counts.sum() > 0:
                assert st["graph_hit"] == rep
            for v in range(R):
                assert (recv[v].get(np_dtype(dtype)).view(np.uint8) == want[v].view(np.uint8)).all(), (R, gpn, dtype, v, rep)
                assert recv[v].guards_intact() and send[v].guards_intact()
            assert stage.guards_intact()
        # the stage count is the host-side scheduler's for the same traffic matrix, topology and chunk size
        sched = hb.Schedule(counts.astype(np.uint64) * e, gpn, chunk_bytes=max(piece, 65536))
        assert st["n_pieces"] == len(sched.stages)
        inter = sum(1 for u in range(R) for v in range(R) if u // gpn != v // gpn and counts[u, v])
        if inter:
            # every inter-node flow is moved at least twice (RDMA leg + at least one forwarding copy when a peer exists)
            assert st["n_moves"] >= int((counts > 0).sum())
            assert any(f["cls"] == hb.FLOW_RDMA for s in sched.stages for f in s["flows"])
        # the stream executor has no modelled form
        comm.set_param("use_graph", 0)
        assert comm.alltoallv_rc(send, counts.ravel(), sd.ravel(), recv, rd.ravel(), dtype) == hb.ERR_UNSUPPORTED
        assert comm.destroy() == hb.OK


def test_one_node_is_the_plain_schedule():
    """model_gpus_per_node = 0 (default) or >= R: one NVLink domain, no staging needed, T = C."""
    torch.cuda.set_device(0)
    R, dtype, e = 4, "fp32", 4
    rng = np.random.default_rng(3)
    counts, sd, rd, send_sizes, recv_sizes = _random_pattern(R, rng, 1000)
    for gpn in (0, 4, 9):
        comm = hb.Comm(R, 0)
        comm.set_param("model_gpus_per_node", gpn)
        send = [DevBuf(send_sizes[u] * e) for u in range(R)]
        recv = [DevBuf(recv_sizes[v] * e) for v in range(R)]
        assert comm.alltoallv_rc(send, counts.ravel(), sd.ravel(), recv, rd.ravel(), dtype) == hb.OK
        torch.cuda.synchronize()
        assert comm.destroy() == hb.OK
