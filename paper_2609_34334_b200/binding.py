"""Thin ctypes binding of libhoccl.so: same names as include/hoccl.h, argument marshalling only (the diagnostics of
include/hoccl_diag.h are bound in diag.py).

Buffers are given as objects with a `data_ptr()` method (torch tensors) or as integer device
addresses; streams as `torch.cuda.Stream`, raw integer handles or None (the current torch stream).
Nothing here computes: every step of a collective runs inside the library.  If the library cannot
be built or loaded the import of `lib()` raises; there is no fallback.
"""
from __future__ import annotations

import ctypes
from typing import Optional, Sequence

from . import build as _build

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_CUDA, ERR_MISMATCH, ERR_PENDING, ERR_SCRATCH, ERR_INTERNAL, ERR_TIMEOUT = range(9)
FLOAT32, BFLOAT16 = 0, 1
SUM = 0
PATH_CE, PATH_SM, PATH_CE_HOST = 0, 1, 2

DTYPES = {"fp32": FLOAT32, "bf16": BFLOAT16}

EXPORTS = [   # every function include/hoccl.h declares
    "hoccl_comm_init", "hoccl_comm_destroy", "hoccl_scratch_bytes", "hoccl_scratch_bytes_direct",
    "hoccl_comm_set_scratch", "hoccl_comm_set_staging", "hoccl_comm_set_host_staging", "hoccl_comm_set_path",
    "hoccl_comm_set_param", "hoccl_comm_get_param", "hoccl_allreduce", "hoccl_reduce_scatter", "hoccl_allgather",
    "hoccl_alltoall", "hoccl_alltoallv", "hoccl_send", "hoccl_recv", "hoccl_comm_pending", "hoccl_comm_async_error",
    "hoccl_comm_handshakes", "hoccl_comm_proxy_stats", "hoccl_host_allreduce", "hoccl_error_string", "hoccl_last_cuda_error", "hoccl_last_stats",
    "hoccl_profile_reset", "hoccl_allreduce_static", "hoccl_sched_build", "hoccl_sched_destroy",
    "hoccl_sched_num_stages", "hoccl_sched_stage_tau", "hoccl_sched_total_tau", "hoccl_sched_lower_bound",
    "hoccl_sched_matrix", "hoccl_sched_num_flows", "hoccl_sched_get_flow", "hoccl_sched_queue_len",
    "hoccl_sched_queue_get",
]


class Stats(ctypes.Structure):
    _fields_ = [
        ("host_launch_us", ctypes.c_double), ("n_moves", ctypes.c_long), ("n_move_launches", ctypes.c_long),
        ("n_sum_launches", ctypes.c_long), ("max_sum_ctas", ctypes.c_long), ("max_copy_ctas", ctypes.c_long),
        ("n_pieces", ctypes.c_long), ("graph_hit", ctypes.c_long), ("sum_kernel_ms", ctypes.c_double),
        ("sum_kernel_launches_timed", ctypes.c_long), ("sum_kernel_bytes", ctypes.c_double),
        ("copy_kernel_ms", ctypes.c_double), ("copy_kernel_launches_timed", ctypes.c_long), ("copy_kernel_bytes", ctypes.c_double),
        ("n_order_launches", ctypes.c_long),
    ]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class SchedFlow(ctypes.Structure):
    _fields_ = [("src", ctypes.c_int), ("dst", ctypes.c_int), ("cls", ctypes.c_int), ("origin_src", ctypes.c_int),
                ("origin_dst", ctypes.c_int), ("bytes", ctypes.c_uint64), ("origin_offset", ctypes.c_uint64)]


FLOW_NATIVE, FLOW_RDMA, FLOW_FWD_SEND, FLOW_FWD_RECV = 0, 1, 2, 3


class HocclError(RuntimeError):
    def __init__(self, code: int, what: str, detail: str = ""):
        self.code = code
        super().__init__("%s failed: %s (code %d)%s" % (what, error_string(code), code, (": " + detail) if detail else ""))


_lib = None


def library_path() -> str:
    """Path of libhoccl.so (built first if it is missing or stale)."""
    return _build.build()


def lib() -> ctypes.CDLL:
    """Builds (if stale) and loads libhoccl.so.  Raises if that is not possible."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    L = ctypes.CDLL(path)
    vp, vpp, sz, i, l = ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.c_size_t, ctypes.c_int, ctypes.c_long
    sigs = {
        "hoccl_comm_init": (i, [vpp, i, i]),
        "hoccl_comm_destroy": (i, [vp]),
        "hoccl_scratch_bytes": (sz, [i, sz, i]),
        "hoccl_scratch_bytes_direct": (sz, [i, sz, i]),
        "hoccl_comm_set_scratch": (i, [vp, vp, sz]),
        "hoccl_comm_set_staging": (i, [vp, vp, sz]),
        "hoccl_comm_set_host_staging": (i, [vp, vp, sz]),
        "hoccl_comm_set_path": (i, [vp, i]),
        "hoccl_comm_set_param": (i, [vp, ctypes.c_char_p, l]),
        "hoccl_comm_get_param": (i, [vp, ctypes.c_char_p, ctypes.POINTER(l)]),
        "hoccl_allreduce": (i, [vpp, vpp, sz, i, i, vp, vp]),
        "hoccl_reduce_scatter": (i, [vpp, vpp, sz, i, i, vp, vp]),
        "hoccl_allgather": (i, [vpp, vpp, sz, i, vp, vp]),
        "hoccl_alltoall": (i, [vpp, vpp, sz, i, vp, vp]),
        "hoccl_alltoallv": (i, [vpp, ctypes.POINTER(sz), ctypes.POINTER(sz), vpp, ctypes.POINTER(sz), i, vp, vp]),
        "hoccl_sched_build": (i, [vpp, i, i, ctypes.c_double, ctypes.c_double, ctypes.POINTER(ctypes.c_uint64), ctypes.c_uint64]),
        "hoccl_sched_destroy": (None, [vp]),
        "hoccl_sched_num_stages": (i, [vp]),
        "hoccl_sched_stage_tau": (ctypes.c_double, [vp, i]),
        "hoccl_sched_total_tau": (ctypes.c_double, [vp]),
        "hoccl_sched_lower_bound": (ctypes.c_double, [vp]),
        "hoccl_sched_matrix": (i, [vp, i, ctypes.POINTER(ctypes.c_uint64)]),
        "hoccl_sched_num_flows": (i, [vp, i]),
        "hoccl_sched_get_flow": (i, [vp, i, i, ctypes.POINTER(SchedFlow)]),
        "hoccl_sched_queue_len": (i, [vp, i, i]),
        "hoccl_sched_queue_get": (i, [vp, i, i, i, ctypes.POINTER(i), ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_uint64)]),
        "hoccl_send": (i, [vp, sz, i, i, i, vp, vp]),
        "hoccl_recv": (i, [vp, sz, i, i, i, vp, vp]),
        "hoccl_comm_pending": (i, [vp]),
        "hoccl_comm_async_error": (i, [vp, i]),
        "hoccl_comm_handshakes": (l, [vp]),
        "hoccl_comm_proxy_stats": (i, [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), i]),
        "hoccl_host_allreduce": (i, [vpp, vpp, sz, i, i, vp, vp]),
        "hoccl_allreduce_static": (i, [vpp, vpp, sz, i, i, i, vp]),
        "hoccl_error_string": (ctypes.c_char_p, [i]),
        "hoccl_last_cuda_error": (ctypes.c_char_p, [vp]),
        "hoccl_last_stats": (i, [vp, ctypes.POINTER(Stats)]),
        "hoccl_profile_reset": (i, [vp]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(L, name)
        fn.restype = res
        fn.argtypes = args
    _lib = L
    return L


def error_string(code: int) -> str:
    return lib().hoccl_error_string(code).decode()


def _ptr(x) -> int:
    if x is None:
        return 0
    if hasattr(x, "data_ptr"):
        return int(x.data_ptr())
    return int(x)


def _ptr_array(xs: Sequence):
    arr = (ctypes.c_void_p * len(xs))()
    for k, x in enumerate(xs):
        arr[k] = _ptr(x)
    return arr


def _stream(s) -> int:
    if s is None:
        import torch

        return int(torch.cuda.current_stream().cuda_stream)
    if hasattr(s, "cuda_stream"):
        return int(s.cuda_stream)
    return int(s)


def _dtype(d) -> int:
    if isinstance(d, str):
        return DTYPES[d]
    return int(d)


class Comm:
    """Owner of one hoccl_comm_t.  Methods carry the C names without the prefix."""

    def __init__(self, R: int, device: int = 0):
        self._h = ctypes.c_void_p()
        self.R = R
        rc = lib().hoccl_comm_init(ctypes.byref(self._h), R, device)
        if rc != OK:
            self._h = ctypes.c_void_p()
            raise HocclError(rc, "hoccl_comm_init")
        self._keep = []

    # -- helpers
    def _check(self, rc: int, what: str):
        if rc != OK:
            raise HocclError(rc, what, self.last_cuda_error() if rc == ERR_CUDA else "")

    def last_cuda_error(self) -> str:
        return lib().hoccl_last_cuda_error(self._h).decode()

    def destroy(self):
        if self._h:
            rc = lib().hoccl_comm_destroy(self._h)
            if rc != ERR_PENDING:      # PENDING is the one case in which nothing was freed
                self._h = ctypes.c_void_p()
            return rc
        return OK

    def __del__(self):
        try:
            if self._h:
                lib().hoccl_comm_destroy(self._h)
        except Exception:
            pass

    # -- configuration
    def set_scratch(self, buf, nbytes: Optional[int] = None):
        if nbytes is None:
            nbytes = buf.numel() * buf.element_size() if buf is not None else 0
        self._keep = [b for b in self._keep if b[0] != "scratch"] + [("scratch", buf)]
        self._check(lib().hoccl_comm_set_scratch(self._h, _ptr(buf), nbytes), "hoccl_comm_set_scratch")

    def set_staging(self, buf, nbytes: Optional[int] = None):
        if nbytes is None:
            nbytes = buf.numel() * buf.element_size() if buf is not None else 0
        self._keep = [b for b in self._keep if b[0] != "staging"] + [("staging", buf)]
        self._check(lib().hoccl_comm_set_staging(self._h, _ptr(buf), nbytes), "hoccl_comm_set_staging")

    def set_host_staging(self, pinned, nbytes: Optional[int] = None):
        """Pinned host memory (e.g. a torch tensor created with pin_memory()) for the CE_HOST path."""
        if nbytes is None:
            nbytes = pinned.numel() * pinned.element_size() if pinned is not None else 0
        self._keep = [b for b in self._keep if b[0] != "host_staging"] + [("host_staging", pinned)]
        self._check(lib().hoccl_comm_set_host_staging(self._h, _ptr(pinned), nbytes), "hoccl_comm_set_host_staging")

    def set_path(self, path: int):
        self._check(lib().hoccl_comm_set_path(self._h, path), "hoccl_comm_set_path")

    def set_param(self, key: str, value: int):
        self._check(lib().hoccl_comm_set_param(self._h, key.encode(), value), "hoccl_comm_set_param(%s)" % key)

    def get_param(self, key: str) -> int:
        v = ctypes.c_long()
        self._check(lib().hoccl_comm_get_param(self._h, key.encode(), ctypes.byref(v)), "hoccl_comm_get_param(%s)" % key)
        return v.value

    # -- collectives (raise on error; the *_rc variants return the code)
    def allreduce_rc(self, send, recv, count, dtype, stream=None, op=SUM) -> int:
        return lib().hoccl_allreduce(_ptr_array(send), _ptr_array(recv), count, _dtype(dtype), op, self._h, _stream(stream))

    def reduce_scatter_rc(self, send, recv, count, dtype, stream=None, op=SUM) -> int:
        return lib().hoccl_reduce_scatter(_ptr_array(send), _ptr_array(recv), count, _dtype(dtype), op, self._h, _stream(stream))

    def allgather_rc(self, send, recv, count, dtype, stream=None) -> int:
        return lib().hoccl_allgather(_ptr_array(send), _ptr_array(recv), count, _dtype(dtype), self._h, _stream(stream))

    def alltoall_rc(self, send, recv, count, dtype, stream=None) -> int:
        return lib().hoccl_alltoall(_ptr_array(send), _ptr_array(recv), count, _dtype(dtype), self._h, _stream(stream))

    def alltoall(self, send, recv, count, dtype, stream=None):
        self._check(self.alltoall_rc(send, recv, count, dtype, stream), "hoccl_alltoall")

    def alltoallv_rc(self, send, sendcounts, sdispls, recv, rdispls, dtype, stream=None) -> int:
        R = self.R
        arr = lambda xs: (ctypes.c_size_t * (R * R))(*[int(x) for x in xs])
        return lib().hoccl_alltoallv(_ptr_array(send), arr(sendcounts), arr(sdispls), _ptr_array(recv), arr(rdispls), _dtype(dtype),
                                     self._h, _stream(stream))

    def alltoallv(self, send, sendcounts, sdispls, recv, rdispls, dtype, stream=None):
        self._check(self.alltoallv_rc(send, sendcounts, sdispls, recv, rdispls, dtype, stream), "hoccl_alltoallv")

    def allreduce(self, send, recv, count, dtype, stream=None, op=SUM):
        self._check(self.allreduce_rc(send, recv, count, dtype, stream, op), "hoccl_allreduce")

    def reduce_scatter(self, send, recv, count, dtype, stream=None, op=SUM):
        self._check(self.reduce_scatter_rc(send, recv, count, dtype, stream, op), "hoccl_reduce_scatter")

    def allgather(self, send, recv, count, dtype, stream=None):
        self._check(self.allgather_rc(send, recv, count, dtype, stream), "hoccl_allgather")

    def host_allreduce(self, h_send, h_recv, count, dtype, stream=None, op=SUM):
        self._check(lib().hoccl_host_allreduce(_ptr_array(h_send), _ptr_array(h_recv), count, _dtype(dtype), op, self._h,
                                               _stream(stream)), "hoccl_host_allreduce")

    # -- point to point
    def send_rc(self, buf, count, dtype, src, dst, stream=None) -> int:
        return lib().hoccl_send(_ptr(buf), count, _dtype(dtype), src, dst, self._h, _stream(stream))

    def recv_rc(self, buf, count, dtype, src, dst, stream=None) -> int:
        return lib().hoccl_recv(_ptr(buf), count, _dtype(dtype), src, dst, self._h, _stream(stream))

    def send(self, buf, count, dtype, src, dst, stream=None):
        self._check(self.send_rc(buf, count, dtype, src, dst, stream), "hoccl_send")

    def recv(self, buf, count, dtype, src, dst, stream=None):
        self._check(self.recv_rc(buf, count, dtype, src, dst, stream), "hoccl_recv")

    def pending(self) -> int:
        return lib().hoccl_comm_pending(self._h)

    def async_error(self, clear: bool = False) -> int:
        return lib().hoccl_comm_async_error(self._h, int(clear))

    def handshakes(self) -> int:
        return int(lib().hoccl_comm_handshakes(self._h))

    def proxy_stats(self, reset: bool = False):
        """(busy_us, span_us) of the proxy thread: see hoccl_comm_proxy_stats."""
        b, s = ctypes.c_double(), ctypes.c_double()
        self._check(lib().hoccl_comm_proxy_stats(self._h, ctypes.byref(b), ctypes.byref(s), int(reset)), "hoccl_comm_proxy_stats")
        return b.value, s.value

    # -- diagnostics
    def last_stats(self) -> dict:
        st = Stats()
        self._check(lib().hoccl_last_stats(self._h, ctypes.byref(st)), "hoccl_last_stats")
        return st.as_dict()

    def profile_reset(self):
        self._check(lib().hoccl_profile_reset(self._h), "hoccl_profile_reset")

STATIC_SCRATCH_BYTES = 32 << 20


def allreduce_static(send, recv, count, dtype, R, stream=None, op=SUM) -> int:
    """hoccl_allreduce_static: all-reduce that allocates nothing and uses the library's fixed scratch array.
    Returns the result code (OK, or ERR_SCRATCH when the buffers are too large for the fixed array)."""
    return lib().hoccl_allreduce_static(_ptr_array(send), _ptr_array(recv), count, _dtype(dtype), op, R, _stream(stream))


def scratch_bytes(R: int, max_count: int, dtype) -> int:
    return int(lib().hoccl_scratch_bytes(R, max_count, _dtype(dtype)))


def scratch_bytes_direct(R: int, max_count: int, dtype) -> int:
    """Scratch bound with "rs_direct" set (R-1 inbox slots per rank)."""
    return int(lib().hoccl_scratch_bytes_direct(R, max_count, _dtype(dtype)))


class Schedule:
    """Host-only view of the collective scheduler's output for a traffic matrix C (G x G bytes, row = source)."""

    def __init__(self, C, gpus_per_node, bw_nvlink=400e9, bw_rdma=50e9, chunk_bytes=1 << 20):
        import numpy as np

        C = np.ascontiguousarray(C, dtype=np.uint64)
        G = C.shape[0]
        assert C.shape == (G, G)
        L = lib()
        h = ctypes.c_void_p()
        rc = L.hoccl_sched_build(ctypes.byref(h), G, gpus_per_node, bw_nvlink, bw_rdma, C.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64)),
                                 chunk_bytes)
        if rc != OK:
            raise HocclError(rc, "hoccl_sched_build")
        self.G = G

        def mat(which):
            out = np.zeros((G, G), dtype=np.uint64)
            assert L.hoccl_sched_matrix(h, which, out.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64))) == OK
            return out

        self.C, self.T = mat(-2), mat(-1)
        self.total_tau = L.hoccl_sched_total_tau(h)
        self.lower_bound = L.hoccl_sched_lower_bound(h)
        self.stages = []
        for s in range(L.hoccl_sched_num_stages(h)):
            flows = []
            for k in range(L.hoccl_sched_num_flows(h, s)):
                f = SchedFlow()
                assert L.hoccl_sched_get_flow(h, s, k, ctypes.byref(f)) == OK
                flows.append({name: getattr(f, name) for name, _ in SchedFlow._fields_})
            queues = []
            for g in range(G):
                q = []
                for k in range(L.hoccl_sched_queue_len(h, s, g)):
                    fl, off, nb = ctypes.c_int(), ctypes.c_uint64(), ctypes.c_uint64()
                    assert L.hoccl_sched_queue_get(h, s, g, k, ctypes.byref(fl), ctypes.byref(off), ctypes.byref(nb)) == OK
                    q.append((fl.value, off.value, nb.value))
                queues.append(q)
            self.stages.append({"matrix": mat(s), "tau": L.hoccl_sched_stage_tau(h, s), "flows": flows, "queues": queues})
        L.hoccl_sched_destroy(h)
