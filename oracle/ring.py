"""ctypes front end of the CPU oracle (oracle/ring_oracle.c).

TEST INFRASTRUCTURE ONLY.  Importable from tests/, the smoke check and the CPU-baseline leg of the
benchmark; the product package never imports it and it never imports the product package.

Arrays are numpy: float32 for fp32, uint16 (raw bit patterns) for bf16.  Every function takes a list
of R per-rank arrays and returns new per-rank arrays; the C code does all arithmetic.

The operations follow the paper's workloads (AllGather and send/recv as byte moves, Sec. 3.3 and
Sec. 5) and, for the reduction the paper leaves out (Sec. 4 "Limitations"), the textbook ring in the
fixed order described at the top of ring_oracle.c.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ring_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None

F32 = 0
BF16 = 1


def build(force: bool = False) -> str:
    """Compile ring_oracle.c into liboracle.so next to it (gcc, strict IEEE flags)."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fno-fast-math", "-fopenmp", "-fPIC", "-shared",
                   "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        build()
        L = ctypes.CDLL(_LIB)
        vpp = ctypes.POINTER(ctypes.c_void_p)
        L.oracle_ring_allreduce.argtypes = [ctypes.c_int, ctypes.c_size_t, ctypes.c_int, vpp, vpp, ctypes.c_int]
        L.oracle_ring_reduce_scatter.argtypes = [ctypes.c_int, ctypes.c_size_t, ctypes.c_int, vpp, vpp, ctypes.c_int]
        L.oracle_allgather.argtypes = [ctypes.c_int, ctypes.c_size_t, ctypes.c_int, vpp, vpp, ctypes.c_int]
        L.oracle_alltoall.argtypes = [ctypes.c_int, ctypes.c_size_t, ctypes.c_int, vpp, vpp]
        szp = ctypes.POINTER(ctypes.c_size_t)
        L.oracle_alltoallv.argtypes = [ctypes.c_int, ctypes.c_int, vpp, szp, szp, vpp, szp]
        L.oracle_sendrecv.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int]
        L.oracle_chain_sum.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_size_t, ctypes.c_size_t, ctypes.c_int, vpp,
                                       ctypes.c_void_p]
        L.oracle_sum_f64.argtypes = [ctypes.c_int, ctypes.c_size_t, ctypes.c_int, vpp, ctypes.c_void_p, ctypes.c_void_p]
        L.oracle_chunk_range.argtypes = [ctypes.c_size_t, ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_size_t),
                                         ctypes.POINTER(ctypes.c_size_t)]
        L.oracle_max_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def dtype_code(arr: np.ndarray) -> int:
    if arr.dtype == np.float32:
        return F32
    if arr.dtype == np.uint16:
        return BF16
    raise TypeError("oracle arrays are float32 (fp32) or uint16 (bf16 bit patterns), got %s" % arr.dtype)


def _ptrs(arrs):
    p = (ctypes.c_void_p * len(arrs))()
    for i, a in enumerate(arrs):
        assert a.flags["C_CONTIGUOUS"]
        p[i] = a.ctypes.data
    return p


def _check(xs):
    assert len(xs) >= 1
    dt = dtype_code(xs[0])
    n = xs[0].size
    for x in xs:
        assert dtype_code(x) == dt and x.size == n and x.ndim == 1
    return dt, n


def max_threads() -> int:
    return int(lib().oracle_max_threads())


def chunk_range(n: int, R: int, c: int):
    lo, hi = ctypes.c_size_t(), ctypes.c_size_t()
    lib().oracle_chunk_range(n, R, c, ctypes.byref(lo), ctypes.byref(hi))
    return lo.value, hi.value


def ring_allreduce(xs, threads: int = 1, in_place: bool = False):
    """xs: R arrays of n elements.  Returns R arrays of n elements (all identical)."""
    dt, n = _check(xs)
    R = len(xs)
    if in_place:
        ys = [x.copy() for x in xs]
        src = ys
    else:
        ys = [np.empty_like(x) for x in xs]
        src = xs
    rc = lib().oracle_ring_allreduce(R, n, dt, _ptrs(src), _ptrs(ys), max(1, threads))
    assert rc == 0, rc
    return ys


def ring_reduce_scatter(xs, threads: int = 1):
    """xs: R arrays of R*count elements.  Returns R arrays of count elements (rank r gets chunk r)."""
    dt, n = _check(xs)
    R = len(xs)
    assert n % R == 0
    count = n // R
    ys = [np.empty(count, dtype=xs[0].dtype) for _ in range(R)]
    rc = lib().oracle_ring_reduce_scatter(R, count, dt, _ptrs(xs), _ptrs(ys), max(1, threads))
    assert rc == 0, rc
    return ys


def allgather(xs, threads: int = 1):
    """xs: R arrays of count elements.  Returns R arrays of R*count elements."""
    dt, count = _check(xs)
    R = len(xs)
    ys = [np.empty(R * count, dtype=xs[0].dtype) for _ in range(R)]
    rc = lib().oracle_allgather(R, count, dt, _ptrs(xs), _ptrs(ys), max(1, threads))
    assert rc == 0, rc
    return ys


def alltoall(xs):
    """xs: R arrays of R*count elements.  Returns R arrays: block j of result r is block r of xs[j]."""
    dt, n = _check(xs)
    R = len(xs)
    assert n % R == 0
    ys = [np.empty_like(x) for x in xs]
    rc = lib().oracle_alltoall(R, n // R, dt, _ptrs(xs), _ptrs(ys))
    assert rc == 0, rc
    return ys


def alltoallv(xs, sendcounts, sdispls, rdispls, recv_sizes, fill=0):
    """xs: R send arrays; counts/displacements: R*R sequences in elements.  Returns R receive arrays of recv_sizes[v]
    elements, pre-filled with `fill` where nothing is received."""
    R = len(xs)
    dt = dtype_code(xs[0])
    ys = [np.full(int(recv_sizes[v]), fill, dtype=xs[0].dtype) for v in range(R)]
    arr = lambda v: (ctypes.c_size_t * (R * R))(*[int(t) for t in v])
    rc = lib().oracle_alltoallv(R, dt, _ptrs(xs), arr(sendcounts), arr(sdispls), _ptrs(ys), arr(rdispls))
    assert rc == 0, rc
    return ys


def sendrecv(x):
    y = np.empty_like(x)
    lib().oracle_sendrecv(x.ctypes.data, y.ctypes.data, x.size, dtype_code(x))
    return y


def chain_sum(xs, c: int, lo: int, hi: int):
    """Closed-form ring order for elements [lo, hi) treated as members of chunk c."""
    dt, n = _check(xs)
    assert 0 <= lo <= hi <= n
    out = np.empty(hi - lo, dtype=xs[0].dtype)
    rc = lib().oracle_chain_sum(len(xs), c, lo, hi, dt, _ptrs(xs), out.ctypes.data)
    assert rc == 0, rc
    return out


def sum_f64(xs):
    """Returns (sum, sum of magnitudes) per element, accumulated in float64."""
    dt, n = _check(xs)
    s = np.empty(n, dtype=np.float64)
    a = np.empty(n, dtype=np.float64)
    lib().oracle_sum_f64(len(xs), n, dt, _ptrs(xs), s.ctypes.data, a.ctypes.data)
    return s, a


def bf16_bits_to_f32(u16: np.ndarray) -> np.ndarray:
    """View helper for tests: bf16 bit patterns -> float32 values (exact)."""
    return (u16.astype(np.uint32) << 16).view(np.float32)
