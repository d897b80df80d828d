"""CPU checks of the flattened segment view that the host hands to the batched kernels (hoccl_flatten_inspect, no device).

The kernels form every address from this view: a segment is an element-wise head, a body of 16-byte vectors cut into
CTA tiles, and an element-wise tail; running totals put all tiles (and all element-wise items) of a batch into one index
space.  Here the kernels' index arithmetic is replayed on the host for random segment addresses and lengths and every
touched byte offset is recorded: each byte of each segment must be touched exactly once, nothing outside it, and vector
accesses must be 16-byte aligned on all operands."""
import numpy as np
from hypothesis import HealthCheck, given, settings
from hypothesis import strategies as st

from paper_2609_34334_b200 import binding as hb


def _replay(kind, dtype, ctas, addrs_a, addrs_b, addrs_o, lens):
    """Returns per segment a byte-coverage count array, replaying the device loops for every CTA and thread."""
    e = 1 if kind == "copy" else (4 if dtype == "fp32" else 2)
    ve = 16 // e
    view, tile_v = hb.flatten_inspect(kind, dtype, ctas, addrs_a, addrs_b, addrs_o, lens)
    cover = [np.zeros(n * e, dtype=np.int32) for n in lens]
    tiles_prev, scal_prev = 0, 0
    for k, (head, nvec, tiles_end, scal_end) in enumerate(view):
        n = lens[k]
        ops = [addrs_a[k], addrs_o[k]] + ([addrs_b[k]] if kind == "sum" else [])
        congruent = len({a % 16 for a in ops}) == 1 and (ops[0] % 16) % e == 0
        if nvec:
            assert congruent, "vector body on operands without a common 16-byte phase"
            for a in ops:
                assert (a + head * e) % 16 == 0, "vector body not 16-byte aligned"
        # tiles of this segment: first vector (t - tiles_prev) * tile_v, up to tile_v vectors each
        assert tiles_end - tiles_prev == -(-nvec // tile_v)
        for t in range(tiles_prev, tiles_end):
            first = (t - tiles_prev) * tile_v
            n_here = min(tile_v, nvec - first)
            assert n_here > 0
            lo = (head + first * ve) * e
            cover[k][lo:lo + n_here * 16] += 1
        # element-wise items: i < head before the body, the rest after it
        n_scalar = scal_end - scal_prev
        assert n_scalar == n - nvec * ve
        for j in range(n_scalar):
            i = j if j < head else j + nvec * ve
            assert 0 <= i < n
            cover[k][i * e:(i + 1) * e] += 1
        tiles_prev, scal_prev = tiles_end, scal_end
    return cover


segment = st.tuples(st.integers(0, 15), st.integers(0, 15), st.integers(0, 15), st.one_of(st.integers(0, 70), st.integers(71, 70_000)))


@settings(max_examples=200, deadline=None, suppress_health_check=list(HealthCheck), derandomize=True)
@given(kind=st.sampled_from(["sum", "copy"]), dtype=st.sampled_from(["fp32", "bf16"]), ctas=st.sampled_from([1, 8, 127, 128, 148, 592]),
       segs=st.lists(segment, min_size=1, max_size=32), same_phase=st.booleans())
def test_every_byte_of_every_segment_is_touched_exactly_once(kind, dtype, ctas, segs, same_phase):
    e = 1 if kind == "copy" else (4 if dtype == "fp32" else 2)
    base = 1 << 30
    a, b, o, lens = [], [], [], []
    for k, (pa, pb, po, n) in enumerate(segs):
        if same_phase:
            pb = po = pa
        a.append(base + k * (1 << 22) + pa // e * e)
        b.append(base + (64 + k) * (1 << 22) + pb // e * e)
        o.append(base + (128 + k) * (1 << 22) + po // e * e)
        lens.append(n)
    cover = _replay(kind, dtype, ctas, a, b, o, lens)
    for k, c in enumerate(cover):
        assert (c == 1).all(), (k, lens[k], int(c.min()) if c.size else None, int(c.max()) if c.size else None)


def test_aligned_segments_take_the_vector_path():
    view, tile_v = hb.flatten_inspect("sum", "bf16", 8, [4096, 8192 + 6], [1 << 20, (1 << 20) + 6], [2 << 20, (2 << 20) + 6], [8000, 8003])
    assert tile_v == 4 * 1024
    (h0, v0, t0, s0), (h1, v1, t1, s1) = view
    assert (h0, v0, s0) == (0, 1000, 0) and t0 == 1
    assert h1 == 5 and v1 == (8003 - 5) // 8 and s1 == 8003 - v1 * 8       # 6 bytes off: 5 bf16 elements up to the next 16-byte line
    view, tile_v = hb.flatten_inspect("copy", "bf16", 148, [4096 + 3], None, [8192 + 3], [100_000])
    assert tile_v == 4 * 512 and view[0][0] == 13 and view[0][1] == (100_000 - 13) // 16
    view, _ = hb.flatten_inspect("copy", "bf16", 8, [4096 + 3], None, [8192 + 4], [100_000])
    assert view[0][1] == 0 and view[0][3] == 100_000                         # no common phase: element-wise fallback
