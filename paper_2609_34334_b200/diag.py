"""ctypes binding of the diagnostics declared in include/hoccl_diag.h: measurements, self-tests, direct kernel launches,
and host-only inspection of plans and option rules.  Argument marshalling only; the product calls are in binding.py."""
from __future__ import annotations

import ctypes

from . import binding as _b
from .binding import OK, HocclError, _dtype, _ptr, _ptr_array, _stream

PLAN_ALLREDUCE, PLAN_REDUCE_SCATTER, PLAN_ALLGATHER, PLAN_ALLTOALL, PLAN_ALLREDUCE_FWD, PLAN_REDUCE_SCATTER_FWD = range(6)
PLAN_ALLREDUCE_AGD, PLAN_ALLGATHER_DIRECT, PLAN_ALLREDUCE_FWD_AGD = 6, 7, 8
OP_MOVE, OP_SUM, OP_CHAIN = 0, 1, 2
PLAN_FLAG_FORWARD, PLAN_FLAG_AG_DIRECT, PLAN_FLAG_RS_DIRECT, PLAN_FLAG_GRADED = 16, 32, 64, 128
BUF_SEND, BUF_RECV, BUF_INBOX, BUF_PARTIAL = 0, 1, 2, 3
EXEC_GRAPH, EXEC_STREAMS, EXEC_ONE_KERNEL, EXEC_ONEPASS, EXEC_PROXY, EXEC_ROLES = range(6)

EXPORTS = [   # every function include/hoccl_diag.h declares
    "hoccl_chain_launch", "hoccl_copy_launch", "hoccl_fanout_inspect", "hoccl_fanout_launch", "hoccl_flatten_inspect",
    "hoccl_kernel_sms", "hoccl_options_resolve", "hoccl_plan_build", "hoccl_plan_destroy", "hoccl_plan_get_op",
    "hoccl_plan_group_deps", "hoccl_plan_inbox_slots", "hoccl_plan_num_groups", "hoccl_plan_num_ops",
    "hoccl_plan_scratch_bytes", "hoccl_plan_slot_bytes", "hoccl_port_probe", "hoccl_probe_copy_routes",
    "hoccl_probe_move_needs_sm", "hoccl_selftest_barrier_timeout", "hoccl_selftest_roles_timeout", "hoccl_selftest_bf16_add", "hoccl_sum_launch",
]


class RouteProbe(ctypes.Structure):
    _fields_ = [("name", ctypes.c_char * 56), ("needs_sm", ctypes.c_int), ("end_us", ctypes.c_double)]


class PlanOp(ctypes.Structure):
    _fields_ = [
        ("kind", ctypes.c_int), ("phase", ctypes.c_int), ("step", ctypes.c_int), ("piece", ctypes.c_int),
        ("rank", ctypes.c_int), ("dst_rank", ctypes.c_int), ("chunk", ctypes.c_int), ("src_buf", ctypes.c_int),
        ("dst_buf", ctypes.c_int), ("local_buf", ctypes.c_int), ("src_off", ctypes.c_uint64), ("dst_off", ctypes.c_uint64),
        ("local_off", ctypes.c_uint64), ("bytes", ctypes.c_uint64), ("group", ctypes.c_int),
        ("nsrc", ctypes.c_int), ("src_stride", ctypes.c_uint64),
    ]


class Options(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("R", ctypes.c_int), ("count", ctypes.c_size_t), ("dtype", ctypes.c_int), ("path", ctypes.c_int),
                ("onepass", ctypes.c_long), ("forward", ctypes.c_long), ("fused", ctypes.c_long), ("rs_direct", ctypes.c_long),
                ("ag_direct", ctypes.c_long), ("handshake", ctypes.c_long), ("use_graph", ctypes.c_long),
                ("ce_small_bytes", ctypes.c_long), ("ce_small_ctas", ctypes.c_long), ("copy_ctas", ctypes.c_long),
                ("scratch_bytes", ctypes.c_size_t), ("host_call", ctypes.c_int), ("roles", ctypes.c_long)]


class Resolved(ctypes.Structure):
    _fields_ = [("plan_kind", ctypes.c_int), ("executor", ctypes.c_int), ("path", ctypes.c_int), ("copy_ctas", ctypes.c_long),
                ("small_switch", ctypes.c_int)]


_ready = False


def lib() -> ctypes.CDLL:
    """The library of binding.lib() with the argument types of the diagnostic entry points set."""
    global _ready
    L = _b.lib()
    if _ready:
        return L
    vp, vpp, sz, i = ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.c_size_t, ctypes.c_int
    sigs = {
        "hoccl_plan_inbox_slots": (i, [vp]),
        "hoccl_plan_scratch_bytes": (sz, [vp]),
        "hoccl_probe_move_needs_sm": (i, [vp, i, vp, vp, sz, i, ctypes.POINTER(i), ctypes.POINTER(ctypes.c_double)]),
        "hoccl_probe_copy_routes": (i, [vp, vp, vp, sz, i, ctypes.POINTER(RouteProbe), i, ctypes.POINTER(i)]),
        "hoccl_sum_launch": (i, [vp, vp, vp, sz, i, i, vp]),
        "hoccl_copy_launch": (i, [vp, vp, sz, i, vp]),
        "hoccl_fanout_launch": (i, [vp, vp, i, sz, i, vp]),
        "hoccl_selftest_bf16_add": (i, [vp, vp]),
        "hoccl_chain_launch": (i, [vp, sz, i, vp, vp, sz, i, i, vp]),
        "hoccl_fanout_inspect": (i, [i, vp, vp, vp, i, i, vp, vp, vp, vp, vp, vp, vp, ctypes.POINTER(i), ctypes.POINTER(i)]),
        "hoccl_kernel_sms": (i, [i, vp, vp, vp, sz, i, i, vp, vp]),
        "hoccl_selftest_barrier_timeout": (i, [vp, vp, vp, sz, vp]),
        "hoccl_selftest_roles_timeout": (i, [vpp, vpp, sz, i, vp, vp]),
        "hoccl_port_probe": (i, [i, vp, sz, i, vp, vp]),
        "hoccl_flatten_inspect": (i, [i, i, i, i, vp, vp, vp, vp, vp, vp, vp, vp, vp]),
        "hoccl_plan_build": (i, [vpp, i, i, sz, i, i, sz, i, ctypes.c_char_p]),
        "hoccl_plan_slot_bytes": (sz, [vp]),
        "hoccl_plan_destroy": (None, [vp]),
        "hoccl_plan_num_ops": (i, [vp]),
        "hoccl_plan_num_groups": (i, [vp]),
        "hoccl_plan_get_op": (i, [vp, i, ctypes.POINTER(PlanOp)]),
        "hoccl_plan_group_deps": (i, [vp, i, ctypes.POINTER(i), i]),
        "hoccl_options_resolve": (i, [ctypes.POINTER(Options), ctypes.POINTER(Resolved)]),
    }
    for name, (res, args) in sigs.items():
        fn = getattr(L, name)
        fn.restype = res
        fn.argtypes = args
    _ready = True
    return L


def options_resolve(kind, R, count, dtype, path=_b.PATH_CE, scratch_bytes=0, host_call=0, **params):
    """hoccl_options_resolve (host only): the schedule, executor and move route a call with these settings would get.
    params: the communicator parameters of the same names (defaults as a new communicator has them).
    Returns (code, dict or None)."""
    vals = dict(onepass=0, forward=0, fused=0, rs_direct=2, ag_direct=2, handshake=0, use_graph=1, ce_small_bytes=8 << 20, ce_small_ctas=148,
                copy_ctas=8, roles=0)
    vals.update(params)
    o = Options(kind, R, count, _dtype(dtype), path, vals["onepass"], vals["forward"], vals["fused"], vals["rs_direct"], vals["ag_direct"],
                vals["handshake"], vals["use_graph"], vals["ce_small_bytes"], vals["ce_small_ctas"], vals["copy_ctas"], scratch_bytes,
                host_call, vals["roles"])
    r = Resolved()
    rc = lib().hoccl_options_resolve(ctypes.byref(o), ctypes.byref(r))
    if rc != OK:
        return rc, None
    return rc, {f: getattr(r, f) for f, _ in Resolved._fields_}


def selftest_barrier_timeout(comm, dst, src, nbytes, stream=None) -> int:
    return lib().hoccl_selftest_barrier_timeout(comm._h, _ptr(dst), _ptr(src), nbytes, _stream(stream))


def selftest_roles_timeout(comm, send, recv, count, dtype, stream=None) -> int:
    return lib().hoccl_selftest_roles_timeout(_b._ptr_array(send), _b._ptr_array(recv), count, _dtype(dtype), comm._h, _stream(stream))



def probe_move_needs_sm(comm, path, dst, src, nbytes, spin_us=3000):
    needs = ctypes.c_int()
    end_us = ctypes.c_double()
    comm._check(lib().hoccl_probe_move_needs_sm(comm._h, path, _ptr(dst), _ptr(src), nbytes, spin_us, ctypes.byref(needs),
                                                ctypes.byref(end_us)), "hoccl_probe_move_needs_sm")
    return bool(needs.value), end_us.value

def probe_copy_routes(comm, dst, src, nbytes, spin_us=3000):
    """[(route name, needs an SM, completion time in us)] for every same-device way of moving bytes."""
    out = (RouteProbe * 16)()
    n = ctypes.c_int()
    comm._check(lib().hoccl_probe_copy_routes(comm._h, _ptr(dst), _ptr(src), nbytes, spin_us, out, 16, ctypes.byref(n)),
                "hoccl_probe_copy_routes")
    return [(out[k].name.decode(), bool(out[k].needs_sm), out[k].end_us) for k in range(n.value)]



def sum_launch(inbox, local, out, count, dtype, ctas, stream=None) -> int:
    return lib().hoccl_sum_launch(_ptr(inbox), _ptr(local), _ptr(out), count, _dtype(dtype), ctas, _stream(stream))


def copy_launch(src, dst, nbytes, ctas, stream=None) -> int:
    return lib().hoccl_copy_launch(_ptr(src), _ptr(dst), nbytes, ctas, _stream(stream))


def fanout_launch(src, dsts, nbytes, ctas, stream=None) -> int:
    """hoccl_fanout_launch: every dsts[d] <- src, the source read once.  Returns the result code."""
    return lib().hoccl_fanout_launch(_ptr(src), _ptr_array(dsts), len(dsts), nbytes, ctas, _stream(stream))


def chain_launch(first, stride_bytes, nsrc, local, out, count, dtype, ctas, stream=None) -> int:
    """hoccl_chain_launch: out = (((s_0 + s_1) + ...) + s_{nsrc-1}) + local with s_j = first + j * stride_bytes."""
    return lib().hoccl_chain_launch(_ptr(first), stride_bytes, nsrc, _ptr(local), _ptr(out), count, _dtype(dtype), ctas, _stream(stream))


def selftest_bf16_add(counts, stream=None) -> int:
    """hoccl_selftest_bf16_add: counts = device array of two zeroed 64-bit words.  Returns the result code."""
    return lib().hoccl_selftest_bf16_add(_ptr(counts), _stream(stream))


def fanout_inspect(moves, ctas: int = 8):
    """hoccl_fanout_inspect (host only): moves = [(src_addr, dst_addr, nbytes), ...] -> (segments, launches) where a segment is
    (launch, src_addr, nbytes, [dst_addr, ...], head, nvec); no segments means the moves go as plain copies."""
    n = len(moves)
    u64 = ctypes.c_uint64 * n
    src, dst, ln = u64(*[m[0] for m in moves]), u64(*[m[1] for m in moves]), u64(*[m[2] for m in moves])
    cap = n
    seg_launch, seg_nd = (ctypes.c_int * cap)(), (ctypes.c_int * cap)()
    seg_src, seg_len, seg_nvec, dst_out = (ctypes.c_uint64 * cap)(), (ctypes.c_uint64 * cap)(), (ctypes.c_uint64 * cap)(), u64()
    seg_head = (ctypes.c_uint32 * cap)()
    n_seg, n_launch = ctypes.c_int(0), ctypes.c_int(0)
    rc = lib().hoccl_fanout_inspect(n, src, dst, ln, ctas, cap, seg_launch, seg_src, seg_len, seg_nd, seg_head, seg_nvec, dst_out,
                                    ctypes.byref(n_seg), ctypes.byref(n_launch))
    if rc != OK:
        raise HocclError(rc, "hoccl_fanout_inspect", "")
    segs, at = [], 0
    for k in range(n_seg.value):
        segs.append((seg_launch[k], seg_src[k], seg_len[k], [dst_out[at + d] for d in range(seg_nd[k])], seg_head[k], seg_nvec[k]))
        at += seg_nd[k]
    return segs, n_launch.value


def kernel_sms(kind: str, a, b, out, nbytes: int, dtype, ctas: int, smid_out, stream=None) -> int:
    """hoccl_kernel_sms: run the SUM ("sum") or copy ("copy") kernel with `ctas` CTAs; every CTA writes its SM id to
    smid_out (a device array of `ctas` 32-bit words).  Returns the result code."""
    return lib().hoccl_kernel_sms(0 if kind == "sum" else 1, _ptr(a), _ptr(b) if b is not None else None, _ptr(out), nbytes,
                                  _dtype(dtype), ctas, _ptr(smid_out), _stream(stream))


def port_probe(mode: str, buf, nbytes: int, ctas: int, sink, stream=None) -> int:
    """hoccl_port_probe: `ctas` CTAs only read ("read") or only write ("write") the buffer."""
    return lib().hoccl_port_probe(0 if mode == "read" else 1, _ptr(buf), nbytes, ctas, _ptr(sink), _stream(stream))


def flatten_inspect(kind: str, dtype, ctas: int, a_addr, b_addr, out_addr, lens):
    """hoccl_flatten_inspect (host only): per segment (head, nvec, tiles_end, scalars_end) and the tile size in vectors."""
    n = len(lens)
    U64 = ctypes.c_uint64 * n
    a, o, ln = U64(*a_addr), U64(*out_addr), U64(*lens)
    b = U64(*(b_addr if b_addr is not None else [0] * n))
    tiles, scal, nvec = U64(), U64(), U64()
    head = (ctypes.c_uint32 * n)()
    tv = ctypes.c_uint64()
    rc = lib().hoccl_flatten_inspect(0 if kind == "sum" else 1, _dtype(dtype), ctas, n, a, b, o, ln, tiles, scal, nvec, head, ctypes.byref(tv))
    if rc != OK:
        raise HocclError(rc, "hoccl_flatten_inspect", "")
    return [(int(head[k]), int(nvec[k]), int(tiles[k]), int(scal[k])) for k in range(n)], int(tv.value)


class Plan:
    """Host-only view of the planner's output."""

    def __init__(self, kind, R, count, dtype, in_place=False, piece_bytes=4 << 20, max_pieces=8, send_align=None):
        self._h = ctypes.c_void_p()
        align = bytes(send_align) if send_align is not None else None
        rc = lib().hoccl_plan_build(ctypes.byref(self._h), kind, R, count, _dtype(dtype), int(in_place), piece_bytes, max_pieces,
                                    align)
        if rc != OK:
            raise HocclError(rc, "hoccl_plan_build")
        L = lib()
        self.slot_bytes = int(L.hoccl_plan_slot_bytes(self._h))
        self.inbox_slots = int(L.hoccl_plan_inbox_slots(self._h))
        self.scratch_bytes = int(L.hoccl_plan_scratch_bytes(self._h))
        self.ops = []
        for k in range(L.hoccl_plan_num_ops(self._h)):
            op = PlanOp()
            assert L.hoccl_plan_get_op(self._h, k, ctypes.byref(op)) == OK
            self.ops.append({f: getattr(op, f) for f, _ in PlanOp._fields_})
        self.num_groups = L.hoccl_plan_num_groups(self._h)
        self.deps = []
        for g in range(self.num_groups):
            buf = (ctypes.c_int * 64)()
            n = L.hoccl_plan_group_deps(self._h, g, buf, 64)
            self.deps.append([buf[k] for k in range(n)])
        L.hoccl_plan_destroy(self._h)
        self._h = None


