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
from paper_2609_34334_b200 import diag as hd


def _replay(kind, dtype, ctas, addrs_a, addrs_b, addrs_o, lens):
    """Returns per segment a byte-coverage count array, replaying the device loops for every CTA and thread."""
    e = 1 if kind == "copy" else (4 if dtype == "fp32" else 2)
    ve = 16 // e
    view, tile_v = hd.flatten_inspect(kind, dtype, ctas, addrs_a, addrs_b, addrs_o, lens)
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
    view, tile_v = hd.flatten_inspect("sum", "bf16", 8, [4096, 8192 + 6], [1 << 20, (1 << 20) + 6], [2 << 20, (2 << 20) + 6], [8000, 8003])
    assert tile_v == 4 * 1024
    (h0, v0, t0, s0), (h1, v1, t1, s1) = view
    assert (h0, v0, s0) == (0, 1000, 0) and t0 == 1
    assert h1 == 5 and v1 == (8003 - 5) // 8 and s1 == 8003 - v1 * 8       # 6 bytes off: 5 bf16 elements up to the next 16-byte line
    view, tile_v = hd.flatten_inspect("copy", "bf16", 148, [4096 + 3], None, [8192 + 3], [100_000])
    assert tile_v == 4 * 512 and view[0][0] == 13 and view[0][1] == (100_000 - 13) // 16
    view, _ = hd.flatten_inspect("copy", "bf16", 8, [4096 + 3], None, [8192 + 4], [100_000])
    assert view[0][1] == 0 and view[0][3] == 100_000                         # no common phase: element-wise fallback


# ---- fan-out packing (hoccl_fanout_inspect): the moves of a direct all-gather that read the same bytes share one segment
move_set = st.lists(st.tuples(st.integers(0, 5), st.integers(0, 15), st.sampled_from([0, 0, 0, 3, 8]), st.integers(1, 40)),
                    min_size=1, max_size=700)


@settings(max_examples=150, deadline=None, suppress_health_check=list(HealthCheck), derandomize=True)
@given(moves=move_set, n_len=st.integers(1, 3), ctas=st.sampled_from([8, 148]))
def test_fan_out_packing_serves_every_move_exactly_once(moves, n_len, ctas):
    """Random groups of moves (few sources, few lengths, many destinations with a few 16-byte phases).  Every move must
    appear exactly once, a segment's destinations share their phase, its split follows that phase, and a launch carries
    at most 32 segments and 256 destinations."""
    base, lens = 1 << 32, [4096 + 16 * 7, 100_000, 17][:n_len]
    src_phase = {}
    flat = []
    for k, (s, sp, dp, l) in enumerate(moves):
        src = base + s * (1 << 24) + src_phase.setdefault(s, sp)      # one address per source
        dst = base + (64 + k) * (1 << 24) + (src % 16 + dp) % 16      # mostly in phase with the source
        flat.append((src, dst, lens[l % n_len]))
    segs, launches = hd.fanout_inspect(flat, ctas)
    repeats = len({(m[0], m[2], m[1] % 16) for m in flat}) < len(flat)
    if not repeats:
        assert segs == [] and launches == 0
        return
    served = sorted((src, d, ln) for (_, src, ln, dsts, _, _) in segs for d in dsts)
    assert served == sorted(flat)
    per_launch = {}
    for launch, src, ln, dsts, head, nvec in segs:
        assert 1 <= len(dsts) <= 256
        assert len({d % 16 for d in dsts}) == 1
        in_phase = dsts[0] % 16 == src % 16
        if in_phase:
            assert head == min((16 - src % 16) % 16, ln) and nvec == (ln - head) // 16
        else:
            assert nvec == 0                                         # element-wise: no vector access on a misaligned pair
        acc = per_launch.setdefault(launch, [0, 0])
        acc[0] += 1
        acc[1] += len(dsts)
    assert sorted(per_launch) == list(range(launches))
    for nseg, nd in per_launch.values():
        assert nseg <= 32 and nd <= 256


def test_fan_out_packing_of_a_direct_all_gather():
    """R = 8 ranks, chunk of 3,276,800 bytes: 56 moves become 8 segments of 7 destinations in one launch."""
    R, chunk = 8, 3_276_800
    recv = [(1 << 33) + r * (1 << 28) for r in range(R)]
    moves = [(recv[r] + r * chunk, recv[(r + k) % R] + r * chunk, chunk) for k in range(1, R) for r in range(R)]
    segs, launches = hd.fanout_inspect(moves, 148)
    assert launches == 1 and len(segs) == R
    for launch, src, ln, dsts, head, nvec in segs:
        r = (src - recv[0]) // (1 << 28)
        assert ln == chunk and head == 0 and nvec == chunk // 16 and len(dsts) == R - 1
        assert sorted(dsts) == sorted(recv[d] + r * chunk for d in range(R) if d != r)
    # R = 40: 1560 destinations need 7 launches of at most 256
    R = 40
    recv = [(1 << 33) + r * (1 << 26) for r in range(R)]
    moves = [(recv[r] + r * 4096, recv[(r + k) % R] + r * 4096, 4096) for k in range(1, R) for r in range(R)]
    segs, launches = hd.fanout_inspect(moves, 16)
    assert launches == -(-R * (R - 1) // 256) and sum(len(s[3]) for s in segs) == R * (R - 1)
