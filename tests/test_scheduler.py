"""Host-only checks of the collective scheduler (traffic matrix, Algorithm 1, chunk interleaving) through the C ABI.

Pins: the paper's own worked expansion F1 = f1 + f2' + f3' + f8'' + f11'' (tests/golden/traffic_matrix_eq4.txt),
completeness (the stages add up to T), the per-stage RDMA degree bound, the stage-time formula recomputed here from
the stage matrices, a lower bound no staging can beat (met with equality where the optimum is known), and the
proportional-service property of the chunk interleaving.
"""
import os

import numpy as np
import pytest

from paper_2609_34334_b200 import binding as hb

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _golden():
    d = {}
    for line in open(os.path.join(GOLD, "traffic_matrix_eq4.txt")):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split(":")
            d[k.strip()] = [int(t) for t in v.split()]
    return d


def test_expansion_matches_the_papers_worked_example():
    g = _golden()
    G, per = g["gpus"][0], g["gpus_per_node"][0]
    C = np.zeros((G, G), dtype=np.uint64)
    idx = 0
    flow = {}
    for u in range(G):
        for v in range(G):
            if u != v:
                idx += 1
                C[u, v] = 1 << idx           # distinct powers of two: a sum shows exactly which flows are in it
                flow[idx] = (u, v)
    s = hb.Schedule(C, per, chunk_bytes=1 << 30)
    u, v = g["edge"]
    assert int(s.T[u, v]) == sum(1 << k for k in g["terms_of_T_on_edge"])
    # by symmetry the other three peer edges, written out from the same rule
    assert int(s.T[1, 0]) == sum(1 << k for k in (4, 5, 6, 7, 10))
    assert int(s.T[2, 3]) == sum(1 << k for k in (9, 7, 8, 3, 6))
    assert int(s.T[3, 2]) == sum(1 << k for k in (12, 10, 11, 2, 5))
    for a in range(G):
        for b in range(G):
            if a // per != b // per:
                assert s.T[a, b] == C[a, b]                    # RDMA entries carry the logical flow only


def _check_schedule(C, per, bw_nv, bw_rd, chunk):
    G = C.shape[0]
    s = hb.Schedule(C, per, bw_nv, bw_rd, chunk)
    node = lambda g: g // per
    # completeness (Eq. 5-6)
    total = np.zeros((G, G), dtype=np.uint64)
    for st in s.stages:
        total += st["matrix"]
    assert (total == s.T).all()
    logical = {}
    for st in s.stages:
        m = st["matrix"]
        # degree bound (Eq. 7): at most one RDMA flow out of and into every GPU
        out_deg, in_deg = [0] * G, [0] * G
        for f in st["flows"]:
            if f["cls"] == hb.FLOW_RDMA:
                assert node(f["src"]) != node(f["dst"])
                out_deg[f["src"]] += 1
                in_deg[f["dst"]] += 1
            elif f["src"] != f["dst"]:
                assert node(f["src"]) == node(f["dst"])
        assert max(out_deg) <= 1 and max(in_deg) <= 1
        # stage time (Eq. 8-9) recomputed from the stage matrix
        l_rdma = max([int(m[a, b]) for a in range(G) for b in range(G) if node(a) != node(b)] + [0])
        l_nv = max([int(m[a, b]) for a in range(G) for b in range(G) if node(a) == node(b) and a != b] + [0])
        tau = max(l_rdma / bw_rd, l_nv / bw_nv)
        assert abs(tau - st["tau"]) <= 1e-9 * max(tau, 1e-30) + 1e-18
        # every forwarding copy accompanies an RDMA transfer of the same logical flow and size in the same stage
        rd = {(f["origin_src"], f["origin_dst"]): f["bytes"] for f in st["flows"] if f["cls"] == hb.FLOW_RDMA}
        for f in st["flows"]:
            if f["cls"] in (hb.FLOW_FWD_SEND, hb.FLOW_FWD_RECV):
                assert rd[(f["origin_src"], f["origin_dst"])] == f["bytes"]
                if f["cls"] == hb.FLOW_FWD_SEND:
                    assert f["src"] == f["origin_src"] and f["dst"] == (f["src"] ^ 1)
                else:
                    assert f["dst"] == f["origin_dst"] and f["src"] == (f["dst"] ^ 1)
            if f["cls"] in (hb.FLOW_NATIVE, hb.FLOW_RDMA):
                key = (f["origin_src"], f["origin_dst"])
                logical.setdefault(key, []).append((f["origin_offset"], f["bytes"]))
        # chunk queues: the chunks of every DMA-served flow tile it exactly, in order
        for gq, q in enumerate(st["queues"]):
            seen = {}
            for fl, off, nb in q:
                f = st["flows"][fl]
                assert f["src"] == gq and f["cls"] != hb.FLOW_RDMA
                assert off == seen.get(fl, 0) and 0 < nb <= chunk
                seen[fl] = off + nb
            for fl, f in enumerate(st["flows"]):
                if f["src"] == gq and f["cls"] != hb.FLOW_RDMA:
                    assert seen.get(fl, 0) == f["bytes"]
    # every logical flow is delivered exactly once, in contiguous portions
    for (u, v), parts in logical.items():
        pos = 0
        for off, nb in sorted(parts):
            assert off == pos
            pos += nb
        assert pos == int(C[u, v])
    assert len(logical) == int((C > 0).sum())
    assert abs(s.total_tau - sum(st["tau"] for st in s.stages)) <= 1e-12 * max(s.total_tau, 1e-30)
    assert s.total_tau >= s.lower_bound * (1 - 1e-12)
    return s


@pytest.mark.parametrize("G,per", [(4, 2), (8, 4), (8, 2), (6, 3), (16, 8), (5, 1)])
def test_random_matrices_meet_the_three_requirements(G, per):
    rng = np.random.default_rng(G * 10 + per)
    for trial in range(6):
        C = rng.integers(0, 1 << 22, size=(G, G)).astype(np.uint64)
        C[rng.random((G, G)) < 0.3] = 0
        if trial == 0:
            np.fill_diagonal(C, 0)
        _check_schedule(C, per, 400e9, 50e9, 1 << 18)


def test_known_optima():
    # uniform all-to-all over single-GPU nodes: G-1 permutation stages, total = row sum / NIC bandwidth (optimal)
    G, f = 8, 1 << 24
    C = np.full((G, G), f, dtype=np.uint64)
    np.fill_diagonal(C, 0)
    s = _check_schedule(C, 1, 400e9, 50e9, 1 << 20)
    assert len(s.stages) == G - 1
    assert abs(s.total_tau - (G - 1) * f / 50e9) < 1e-12
    assert abs(s.total_tau - s.lower_bound) < 1e-12
    # one NVLink domain (the single-device build): T == C and every stage is a matching
    s = _check_schedule(C, G, 400e9, 50e9, 1 << 20)
    assert (s.T == C).all() and len(s.stages) == G - 1
    for st in s.stages:
        srcs = [f["src"] for f in st["flows"]]
        dsts = [f["dst"] for f in st["flows"]]
        assert len(set(srcs)) == len(srcs) and len(set(dsts)) == len(dsts)
    # a permutation needs exactly one stage
    P = np.zeros((G, G), dtype=np.uint64)
    for u in range(G):
        P[u, (u + 3) % G] = 1000 + u
    s = _check_schedule(P, 1, 400e9, 50e9, 512)
    assert max(len(st["flows"]) for st in s.stages) <= G and sum(int(st["matrix"].sum()) for st in s.stages) == int(P.sum())
    # two nodes of two GPUs, one inter-node flow: three copies in one stage (f', f, f'')
    C = np.zeros((4, 4), dtype=np.uint64)
    C[0, 2] = 1 << 20
    s = _check_schedule(C, 2, 400e9, 50e9, 1 << 18)
    assert len(s.stages) == 1
    kinds = sorted((f["cls"], f["src"], f["dst"]) for f in s.stages[0]["flows"])
    assert kinds == [(hb.FLOW_RDMA, 0, 2), (hb.FLOW_FWD_SEND, 0, 1), (hb.FLOW_FWD_RECV, 3, 2)]
    assert abs(s.stages[0]["tau"] - (1 << 20) / 50e9) < 1e-15


def test_chunk_interleaving_serves_flows_in_proportion_to_their_size():
    # one DMA queue with three native flows of very different sizes (one source GPU sending to three peers in one
    # stage cannot happen inside a matching, so build the case with local + forwarding + native traffic of GPU 0)
    C = np.zeros((4, 4), dtype=np.uint64)
    C[0, 0] = 10 << 20          # local copy, served by GPU 0's engine
    C[0, 1] = 3 << 20           # native flow 0 -> 1
    C[0, 2] = 40 << 20          # inter-node flow: its sender-side copy 0 -> 1 is served by GPU 0's engine too
    chunk = 1 << 20
    s = hb.Schedule(C, 2, 400e9, 50e9, chunk)
    st = s.stages[0]
    q = st["queues"][0]
    sizes = {}
    for fl, off, nb in q:
        sizes[fl] = sizes.get(fl, 0) + nb
    assert sorted(sizes.values()) == sorted([10 << 20, 3 << 20, 40 << 20]) or len(s.stages) > 1
    W = len(q)
    weights = {fl: -(-b // chunk) for fl, b in sizes.items()}
    served = {fl: 0 for fl in sizes}
    worst = 0.0
    for t, (fl, off, nb) in enumerate(q, 1):
        served[fl] += 1
        for k in served:
            worst = max(worst, abs(served[k] - t * weights[k] / W))
    assert worst <= 1.0 + 1e-9            # service never drifts more than one chunk from the proportional share
    finish = {fl: max(t for t, item in enumerate(q, 1) if item[0] == fl) for fl in sizes}
    for fl in sizes:                      # every flow finishes in the last turn of its own period: no early finisher
        assert finish[fl] > W - W / weights[fl] - 1
