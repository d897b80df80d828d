"""Pins for the CPU oracle: everything here checks oracle/ against something other than itself.

* two hand-worked order fingerprints (tests/golden/ring_order_w*.txt);
* exact integer sums (any order gives the same, so this isolates the arithmetic from the order);
* R = 2 (one commutative add) against numpy's float32 add;
* the chain closed form evaluated with numpy float32 scalars and an exact-rational bf16 rounding
  written with `fractions.Fraction`;
* allgather == concatenation, send/recv == identity, all ranks identical after allreduce;
* reduce_scatter == chunk r of allreduce, allreduce == reduce_scatter followed by allgather;
* the recursive-summation error bound against an fp64 sum.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from paper_2609_34334_b200 import workloads as W

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(":")
            out[k.strip()] = [float(t) for t in v.split()]
    return out


def _f32_to_bf16_bits_exact(x: float) -> int:
    """Round a finite real to bf16 (8-bit significand, RNE) with exact rational arithmetic."""
    if x == 0:
        return 0x8000 if np.signbit(np.float64(x)) else 0
    fx = Fraction(x)
    sign = 0x8000 if fx < 0 else 0
    fx = abs(fx)
    e = 0
    while fx >= 2 ** (e + 1):
        e += 1
    while fx < 2 ** e:
        e -= 1
    e = max(e, -126)                      # subnormal range shares the exponent of 2^-126
    ulp = Fraction(2) ** (e - 7)
    q = fx / ulp
    lo = q.numerator // q.denominator
    rem = q - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    val = lo * ulp                        # exact value of the rounded result
    if val == 0:
        return sign
    f = np.float32(float(val))
    assert Fraction(float(f)) == val
    return sign | (int(f.view(np.uint32)) >> 16)


def _bf16_val(bits: int) -> float:
    return float(np.array([bits << 16], dtype=np.uint32).view(np.float32)[0])


def _python_chain(vals, c, dtype):
    """((x_{c+1} + x_{c+2}) + ... ) + x_c with one rounding per add, independent of the C code."""
    R = len(vals)
    if R == 1:
        return vals[0]
    acc = vals[(c + 1) % R]
    for k in range(2, R + 1):
        b = vals[(c + k) % R]
        if dtype == "fp32":
            acc = np.float32(np.float32(acc) + np.float32(b))
        else:
            s = np.float32(np.float32(_bf16_val(acc)) + np.float32(_bf16_val(b)))   # exact-or-RN binary32 add
            acc = _f32_to_bf16_bits_exact(float(s))
    return acc


def _literal_chunk(n, R, c):
    """Ring chunk c of n elements over R ranks: q = ceil(n / R) elements per chunk, clipped to n."""
    q = -(-n // R)
    return min(c * q, n), min((c + 1) * q, n)


# (n, R) -> the R chunk ranges, typed out by hand from q = ceil(n / R): trailing chunks are short or empty
CHUNK_TABLE = {
    (10, 4): [(0, 3), (3, 6), (6, 9), (9, 10)],
    (7, 3): [(0, 3), (3, 6), (6, 7)],
    (5, 4): [(0, 2), (2, 4), (4, 5), (5, 5)],
    (9, 8): [(0, 2), (2, 4), (4, 6), (6, 8), (8, 9), (9, 9), (9, 9), (9, 9)],
    (3, 8): [(0, 1), (1, 2), (2, 3), (3, 3), (3, 3), (3, 3), (3, 3), (3, 3)],
    (1, 4): [(0, 1), (1, 1), (1, 1), (1, 1)],
    (0, 3): [(0, 0), (0, 0), (0, 0)],
    (12, 4): [(0, 3), (3, 6), (6, 9), (9, 12)],
    (13, 1): [(0, 13)],
    (1_000_001, 8): [(0, 125001), (125001, 250002), (250002, 375003), (375003, 500004), (500004, 625005), (625005, 750006),
                     (750006, 875007), (875007, 1000001)],
}


@pytest.mark.parametrize("n,R", sorted(CHUNK_TABLE))
def test_chunk_partition_against_literal_values(oracle, n, R):
    """The partition for counts that R does not divide (and n < R, where trailing chunks are empty)."""
    for c, want in enumerate(CHUNK_TABLE[(n, R)]):
        assert oracle.chunk_range(n, R, c) == want, (n, R, c)
        assert _literal_chunk(n, R, c) == want


def test_a_wrong_chunk_owner_changes_the_bits(oracle):
    """The order fingerprint depends on which chunk an element is in, so a wrong partition for R that does not divide n
    cannot hide: with x = (1e8, 1, -1e8, 1) on ranks 0..3 the chain of chunk c gives (0, 1, 0, 1)[c]."""
    R, n = 4, 10
    xs = [np.full(n, v, dtype=np.float32) for v in (1e8, 1.0, -1e8, 1.0)]
    y = oracle.ring_allreduce(xs)[0]
    want = np.empty(n, dtype=np.float32)
    for c, (lo, hi) in enumerate(CHUNK_TABLE[(n, R)]):
        want[lo:hi] = (0.0, 1.0, 0.0, 1.0)[c]
    assert (y == want).all()


@pytest.mark.parametrize("name,dtype", [("ring_order_w1_fp32.txt", "fp32"), ("ring_order_w2_bf16.txt", "bf16")])
def test_worked_order_fingerprints(oracle, name, dtype):
    g = _read_golden(name)
    R = len(g["rank_values"])
    n = R                                  # one element per ring chunk
    if dtype == "fp32":
        xs = [np.full(n, v, dtype=np.float32) for v in g["rank_values"]]
        expect = np.array(g["expected_by_chunk"], dtype=np.float32)
    else:
        xs = [np.full(n, _f32_to_bf16_bits_exact(v), dtype=np.uint16) for v in g["rank_values"]]
        expect = np.array([_f32_to_bf16_bits_exact(v) for v in g["expected_by_chunk"]], dtype=np.uint16)
    ys = oracle.ring_allreduce(xs)
    for y in ys:
        assert (y == expect).all(), (y, expect)
    # the order matters in these examples: the exact sum differs from at least one chunk's result
    got = ys[0] if dtype == "fp32" else oracle.bf16_bits_to_f32(ys[0])
    assert (got != np.float32(g["exact_sum"][0])).any()
    # reduce_scatter with count = 1 must hand chunk r to rank r
    rs = oracle.ring_reduce_scatter(xs)
    for r in range(R):
        assert rs[r][0] == expect[r]


def test_bf16_rounding_against_exact_rational(oracle):
    """rn_bf16 of the oracle (through R=2 sums with a zero operand) equals exact-rational RNE."""
    rng = np.random.default_rng(7)
    # values a + b whose binary32 sum is exact but needs rounding to bf16: a, b bf16 with close exponents
    a = (rng.integers(0, 1 << 16, size=4096, dtype=np.uint32)).astype(np.uint16)
    b = (rng.integers(0, 1 << 16, size=4096, dtype=np.uint32)).astype(np.uint16)
    fa, fb = oracle.bf16_bits_to_f32(a), oracle.bf16_bits_to_f32(b)
    with np.errstate(invalid="ignore", over="ignore"):
        ok = np.isfinite(fa) & np.isfinite(fb) & np.isfinite(fa + fb)
    a, b = a[ok], b[ok]
    ys = oracle.ring_allreduce([a, b])
    fa, fb = oracle.bf16_bits_to_f32(a), oracle.bf16_bits_to_f32(b)
    for i in range(a.size):
        s32 = np.float32(fa[i] + fb[i])                      # one binary32 add (numpy)
        expect = _f32_to_bf16_bits_exact(float(s32))
        got = int(ys[0][i])
        if s32 == 0:
            assert oracle.bf16_bits_to_f32(np.array([got], dtype=np.uint16))[0] == 0
        else:
            assert got == expect, (i, hex(int(a[i])), hex(int(b[i])), hex(got), hex(expect))


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("R", [1, 2, 3, 4, 5, 8])
def test_chain_closed_form_bruteforce(oracle, dtype, R):
    """Step-by-step ring == chain closed form, the latter evaluated in pure Python per element."""
    for n in [0, 1, R - 1, R, R + 1, 2 * R + 1, 3 * R + 1, 37]:
        if n < 0:
            continue
        xs = W.rank_inputs("uniform", 11 + n, R, n, dtype)
        ys = oracle.ring_allreduce(xs)
        for r in range(1, R):
            assert (ys[r] == ys[0]).all()
        for c in range(R):
            lo, hi = _literal_chunk(n, R, c)      # the partition written out here, not taken from the oracle
            assert oracle.chunk_range(n, R, c) == (lo, hi)
            for i in range(lo, hi):
                vals = [x[i] if dtype == "fp32" else int(x[i]) for x in xs]
                expect = _python_chain(vals, c, dtype)
                assert ys[0][i] == expect, (R, n, c, i)
            if hi > lo:
                cf = oracle.chain_sum(xs, c, lo, hi)
                assert (cf == ys[0][lo:hi]).all()
        # every element is in exactly one chunk
        cover = np.zeros(n, dtype=np.int32)
        for c in range(R):
            lo, hi = oracle.chunk_range(n, R, c)
            cover[lo:hi] += 1
        assert (cover == 1).all()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("R", [2, 4, 7, 8])
def test_integer_inputs_sum_exactly(oracle, dtype, R):
    n = 1000 + R
    xs = W.rank_inputs("int", 5, R, n, dtype)
    vals = [x.astype(np.float64) if dtype == "fp32" else oracle.bf16_bits_to_f32(x).astype(np.float64) for x in xs]
    exact = np.sum(vals, axis=0)
    assert np.abs(exact).max() <= 64 and np.abs(exact).max() > 0
    ys = oracle.ring_allreduce(xs)
    got = ys[0].astype(np.float64) if dtype == "fp32" else oracle.bf16_bits_to_f32(ys[0]).astype(np.float64)
    assert (got == exact).all()
    for y in ys:
        assert (y == ys[0]).all()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_r2_is_one_commutative_add(oracle, dtype):
    n = 4099
    xs = W.rank_inputs("uniform", 9, 2, n, dtype)
    ys = oracle.ring_allreduce(xs)
    sw = oracle.ring_allreduce(xs[::-1])
    assert (ys[0] == sw[0]).all() and (ys[0] == ys[1]).all()
    if dtype == "fp32":
        assert (ys[0] == xs[0] + xs[1]).all()        # numpy float32 add is the IEEE add
    else:
        import torch
        a = torch.from_numpy(xs[0].view(np.int16)).view(torch.bfloat16)
        b = torch.from_numpy(xs[1].view(np.int16)).view(torch.bfloat16)
        ref = (a.float() + b.float()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        assert (ys[0] == ref).all()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("R", [1, 2, 3, 8])
def test_allgather_is_concatenation_and_sendrecv_identity(oracle, dtype, R):
    for count in [0, 1, 5, 1024 + 3]:
        xs = W.rank_inputs("uniform", 3, R, count, dtype)
        ys = oracle.allgather(xs)
        cat = np.concatenate(xs) if count else np.empty(0, dtype=xs[0].dtype)
        for y in ys:
            assert y.shape == cat.shape and (y == cat).all()
    x = W.uniform(1, 0, 777, dtype)
    assert (oracle.sendrecv(x) == x).all()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("R", [2, 4, 8])
def test_reduce_scatter_allgather_compose_to_allreduce(oracle, dtype, R):
    count = 515
    xs = W.rank_inputs("normal", 21, R, R * count, dtype, 1e-3)
    ar = oracle.ring_allreduce(xs)
    rs = oracle.ring_reduce_scatter(xs)
    for r in range(R):
        assert (rs[r] == ar[0][r * count:(r + 1) * count]).all()
    ag = oracle.allgather(rs)
    for r in range(R):
        assert (ag[r] == ar[r]).all()
    ip = oracle.ring_allreduce(xs, in_place=True)
    for r in range(R):
        assert (ip[r] == ar[r]).all()
    th = oracle.ring_allreduce(xs, threads=4)
    for r in range(R):
        assert (th[r] == ar[r]).all()


@pytest.mark.parametrize("R", [2, 4, 8])
def test_fp64_error_bound(oracle, R):
    n = 1 << 14
    xs = W.rank_inputs("uniform", 0, R, n, "fp32")
    ys = oracle.ring_allreduce(xs)
    s, a = oracle.sum_f64(xs)
    np_s = np.sum([x.astype(np.float64) for x in xs], axis=0)
    assert np.allclose(s, np_s, rtol=0, atol=1e-12)
    err = np.abs(ys[0].astype(np.float64) - s)
    assert (err <= (R - 1) * 2.0 ** -24 * a * 1.0000001 + 1e-300).all()     # textbook recursive-summation bound
    assert (err <= 2e-6 * R * a).all()                                      # the stated tolerance is looser
    xb = W.rank_inputs("normal", 1, R, n, "bf16", 1e-3)
    yb = oracle.ring_allreduce(xb)
    sb, ab = oracle.sum_f64(xb)
    errb = np.abs(oracle.bf16_bits_to_f32(yb[0]).astype(np.float64) - sb)
    u = 2.0 ** -8                                    # bf16 unit roundoff (8 significant bits)
    gamma = (R - 1) * u / (1 - (R - 1) * u)          # Higham's gamma_{R-1} for R-1 rounded adds
    assert (errb <= gamma * ab).all()
    assert errb.max() > 0       # bf16 re-rounding at every hop is visible


def test_special_values(oracle):
    inf, nan = np.float32(np.inf), np.float32(np.nan)
    tiny = np.float32(1e-45)                       # smallest subnormal
    xs = [np.array([inf, nan, -0.0, tiny, 1.0, -inf], dtype=np.float32),
          np.array([1.0, 1.0, -0.0, tiny, -1.0, inf], dtype=np.float32)]
    y = oracle.ring_allreduce(xs)[0]
    assert y[0] == inf and np.isnan(y[1]) and np.isnan(y[5])
    assert y[2] == 0 and np.signbit(y[2])          # -0 + -0 = -0
    assert y[3] == np.float32(2) * tiny and y[3] != 0      # no flush to zero
    assert y[4] == 0 and not np.signbit(y[4])      # 1 + -1 = +0 in round-to-nearest


def test_generator_checksum():
    """The generator is position independent and stable (recorded checksums)."""
    import zlib
    a = W.uniform(0, 0, 1000, "fp32")
    b = W.uniform(0, 0, 400, "fp32", start=600)
    assert (a[600:] == b).all()
    assert a.min() >= -1 and a.max() < 1
    z = W.normal(1, 3, 200000, "fp32", 1e-3)
    assert abs(z.mean()) < 2e-5 and abs(z.std() - 1e-3) < 2e-5
    path = os.path.join(GOLD, "generator_crc.txt")
    want = {}
    with open(path) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                want[k] = int(v, 16)
    got = {
        "uniform_fp32_seed0_rank0_n4096": zlib.crc32(W.uniform(0, 0, 4096, "fp32").tobytes()),
        "normal_bf16_seed1_rank7_n4096": zlib.crc32(W.normal(1, 7, 4096, "bf16", 1e-3).tobytes()),
        "int_bf16_seed5_rank2_n4096": zlib.crc32(W.small_integers(5, 2, 4096, "bf16").tobytes()),
    }
    assert got == want


def test_stored_oracle_results_unchanged(oracle):
    """The oracle's results on the two small benchmark configurations match the recorded checksums."""
    import zlib
    want = {}
    with open(os.path.join(GOLD, "oracle_result_crc.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                want[k] = int(v, 16)
    c1 = W.C1_SMALL_ALLREDUCE
    ys = oracle.ring_allreduce(W.rank_inputs(c1.dist, c1.seed, c1.R, c1.count, c1.dtype))
    assert zlib.crc32(ys[0].tobytes()) == want[c1.name]
    c2 = W.C2_DP_BUCKET
    xs = W.rank_inputs(c2.dist, c2.seed, c2.R, c2.count, c2.dtype, c2.sigma)
    ys = oracle.ring_allreduce(xs, threads=oracle.max_threads())
    assert zlib.crc32(ys[0].tobytes()) == want[c2.name]
    # the two-call form (reduce_scatter then allgather) gives the same bits
    rs = oracle.ring_reduce_scatter(xs, threads=oracle.max_threads())
    ag = oracle.allgather(rs)
    assert (ag[3] == ys[3]).all()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("R", [1, 2, 3, 8])
def test_alltoall_is_block_transpose(oracle, dtype, R):
    for count in [1, 5, 1000]:
        xs = W.rank_inputs("uniform", 71, R, R * count, dtype)
        ys = oracle.alltoall(xs)
        cube = np.stack(xs).reshape(R, R, count)              # [source rank, block, element]
        want = cube.transpose(1, 0, 2)                         # [destination rank, source rank, element]
        for r in range(R):
            assert (ys[r].reshape(R, count) == want[r]).all()
        back = oracle.alltoall(ys)                             # an all-to-all is its own inverse
        for r in range(R):
            assert (back[r] == xs[r]).all()


def _random_pattern(R, rng, max_count=500):
    """Counts and displacements of a random user-defined pattern (elements), with gaps between regions."""
    counts = rng.integers(0, max_count, size=(R, R))
    counts[rng.random((R, R)) < 0.25] = 0
    sd = np.zeros((R, R), dtype=np.int64)
    rd = np.zeros((R, R), dtype=np.int64)
    send_sizes, recv_sizes = [], []
    for u in range(R):
        pos = 3
        for v in rng.permutation(R):
            sd[u, v] = pos
            pos += counts[u, v] + int(rng.integers(0, 5))
        send_sizes.append(pos + 2)
    for v in range(R):
        pos = 1
        for u in rng.permutation(R):
            rd[v, u] = pos
            pos += counts[u, v] + int(rng.integers(0, 5))
        recv_sizes.append(pos + 4)
    return counts, sd, rd, send_sizes, recv_sizes


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("R", [1, 2, 5, 8])
def test_alltoallv_is_the_definition(oracle, dtype, R):
    rng = np.random.default_rng(R + 100)
    counts, sd, rd, send_sizes, recv_sizes = _random_pattern(R, rng)
    xs = [W.uniform(55, u, send_sizes[u], dtype) for u in range(R)]
    ys = oracle.alltoallv(xs, counts.ravel(), sd.ravel(), rd.ravel(), recv_sizes, fill=7)
    for v in range(R):
        want = np.full(recv_sizes[v], 7, dtype=xs[0].dtype)
        for u in range(R):
            want[rd[v, u]:rd[v, u] + counts[u, v]] = xs[u][sd[u, v]:sd[u, v] + counts[u, v]]
        assert (ys[v] == want).all()
