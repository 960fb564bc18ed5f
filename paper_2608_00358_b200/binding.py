"""Thin ctypes binding of the C ABI in include/hccl.h: same names, argument marshalling only.

Every step of a collective runs inside the CUDA library; nothing here computes. Device memory and
streams come from the caller (torch tensors' ``data_ptr()`` and ``torch.cuda.Stream.cuda_stream``
work, as do raw integers). Importing this module fails loudly if the library cannot be built/loaded.
"""
from __future__ import annotations

import ctypes as C
from typing import Optional, Sequence

from . import _build

# ---- enums (mirrors of hccl.h)
OK, ERR_INVALID_ARG, ERR_DTYPE, ERR_COUNT_MISMATCH, ERR_OVERLAP, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_BUSY, \
    ERR_CUDA, ERR_TIMEOUT, ERR_BAD_DESCRIPTOR, ERR_NOT_BOUND, ERR_HAZARD = range(13)
FP32, BF16, FP16 = 0, 1, 2
ALGO_RING, ALGO_ONESHOT, ALGO_RING_FUSED, ALGO_RING_2LEVEL, ALGO_FANOUT, ALGO_TREE, ALGO_AUTO = 0, 1, 2, 3, 4, 5, 6
ENGINE_AUTO, ENGINE_LSU, ENGINE_BULK = 0, 1, 2
FLAG_LEVEL_MAJOR, FLAG_CHECK_HAZARDS, FLAG_STAGED_RING, FLAG_BIDIRECTIONAL = 1, 2, 4, 8
FLAG_STATIC_CHAINS, FLAG_DYNAMIC_TICKETS, FLAG_DEVICE_TABLES = 16, 32, 64
OP_COPY, OP_REDUCE, OP_REDUCE_N, OP_WAIT, OP_SET, OP_NOOP = range(6)
BUF_SEND, BUF_RECV, BUF_SCRATCH, BUF_SIGNAL, BUF_USER_SIGNAL = range(5)
DEP_FENCE, DEP_SYNC, DEP_WQE_SYNC, DEP_RECV_SYNC, DEP_SEND_SYNC, DEP_ELEMENTWISE, DEP_ELEMENTWISE2 = 1, 2, 4, 8, 16, 32, 64
CMP_EQ, CMP_NE, CMP_GE, CMP_GT, CMP_LE, CMP_LT = range(6)
HINT_READ_ONCE, HINT_LAST_READ_A = 1, 2
MAX_RANKS = 256
NOALLOC_WORKSPACE_BYTES = 8 << 20
ELEM_BYTES = {FP32: 4, BF16: 2, FP16: 2}


class Opts(C.Structure):
    _fields_ = [("sm_budget", C.c_int32), ("engine", C.c_int32), ("chunk_bytes", C.c_uint64),
                ("tile_bytes", C.c_uint64), ("timeout_ns", C.c_uint64), ("flags", C.c_uint32),
                ("chain_group", C.c_int32), ("threads", C.c_int32), ("stages", C.c_int32), ("cluster", C.c_int32), ("light", C.c_int32),
                ("copy_by_warps", C.c_int32), ("rack_size", C.c_int32), ("stage_kib", C.c_int32), ("quantum", C.c_int32)]


class Ref(C.Structure):
    _fields_ = [("kind", C.c_int32), ("rank", C.c_int32), ("offset", C.c_int64)]


class Wqe(C.Structure):
    _fields_ = [("op", C.c_int32), ("dtype_dst", C.c_int32), ("dtype_a", C.c_int32), ("dtype_b", C.c_int32),
                ("dst", Ref), ("a", Ref), ("b", Ref), ("count", C.c_int64), ("nsrc", C.c_int32),
                ("dep_flags", C.c_uint32), ("dep_wqe", C.c_int64), ("dep_wqe2", C.c_int64), ("cmp", C.c_int32),
                ("hints", C.c_int32), ("ndst", C.c_int32), ("reserved", C.c_int32), ("tile_count", C.c_int64), ("value", C.c_uint64),
                ("value_per_epoch", C.c_uint64)]


class PlanInfo(C.Structure):
    _fields_ = [("n_wqe", C.c_int64), ("n_tiles", C.c_int64), ("n_syncs", C.c_int64), ("chain_depth", C.c_int64),
                ("schedule_bytes", C.c_int64), ("compulsory_bytes", C.c_int64), ("scratch_bytes", C.c_int64),
                ("send_bytes_total", C.c_int64), ("recv_bytes_total", C.c_int64), ("R", C.c_int32),
                ("sm_budget", C.c_int32), ("threads", C.c_int32), ("engine", C.c_int32), ("tile_bytes", C.c_int64),
                ("epoch", C.c_int64), ("crossrack_bytes", C.c_int64), ("static_chains", C.c_int64)]


class HcclError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        msg = "%s: %s" % (what, status_string(status))
        if status == ERR_CUDA:
            msg += " (%s)" % _lib.hccl_last_cuda_error().decode()
        super().__init__(msg)


def _load() -> C.CDLL:
    path = _build.build()
    lib = C.CDLL(path)
    P, I64P = C.c_void_p, C.POINTER(C.c_int64)
    sigs = {
        "hccl_plan_allreduce": [C.c_int, C.c_int64, C.c_int, C.c_int, C.POINTER(Opts), C.POINTER(P)],
        "hccl_plan_reducescatter": [C.c_int, I64P, C.c_int64, C.c_int, C.c_int, C.POINTER(Opts), C.POINTER(P)],
        "hccl_plan_allgather": [C.c_int, I64P, C.c_int64, C.c_int, C.c_int, C.POINTER(Opts), C.POINTER(P)],
        "hccl_plan_alltoallv": [C.c_int, I64P, I64P, I64P, I64P, C.c_int, C.c_int64, C.POINTER(Opts), C.POINTER(P)],
        "hccl_plan_alltoallv_dynamic": [C.c_int, I64P, I64P, C.c_int, C.c_int64, C.POINTER(Opts), C.POINTER(P)],
        "hccl_plan_set_dynamic_metadata": [P, P, P, P],
        "hccl_graph_create": [C.c_int, I64P, I64P, C.c_int64, C.c_int32, C.POINTER(P)],
        "hccl_graph_add_subgraph": [P, C.c_int, C.POINTER(C.c_int32)],
        "hccl_graph_add_wqe": [P, C.c_int32, C.POINTER(Wqe), I64P],
        "hccl_graph_compile": [P, C.POINTER(Opts), C.POINTER(P)],
        "hccl_plan_workspace_bytes": [P, C.POINTER(C.c_size_t)],
        "hccl_plan_bind": [P, P, C.c_size_t, P],
        "hccl_execute": [P, C.POINTER(P), C.POINTER(P), P],
        "hccl_execute_host": [P, C.POINTER(P), C.POINTER(P), C.POINTER(P), C.POINTER(P), P],
        "hccl_execute_noalloc": [P, C.POINTER(P), C.POINTER(P), P],
        "hccl_server_start": [P, C.POINTER(P), C.POINTER(P), P, C.c_uint64, P],
        "hccl_server_ring": [P],
        "hccl_server_wait": [P, C.c_uint64],
        "hccl_server_stop": [P],
        "hccl_plan_set_user_signals": [P, P, C.c_int64],
        "hccl_plan_set_trace": [P, P, C.c_int64],
        "hccl_plan_set_trigger": [P, C.c_int64, C.c_int32, C.c_uint64, C.c_uint64, C.c_int64, C.c_uint64, C.c_uint64],
        "hccl_plan_status": [P, C.POINTER(C.c_int), I64P],
        "hccl_plan_info": [P, C.POINTER(PlanInfo)],
        "hccl_plan_extents": [P, C.c_int, I64P, I64P],
        "hccl_plan_layout": [P, I64P],
        "hccl_plan_check_hazards": [P, I64P],
        "hccl_plan_interpret_host": [P, C.POINTER(P), C.POINTER(P), P, C.POINTER(C.c_uint64), C.c_uint64],
        "hccl_hostpipe_alltoallv_create": [C.c_int, I64P, C.c_int, C.c_int64, C.c_int, C.POINTER(Opts), C.POINTER(P)],
        "hccl_hostpipe_windows": [P, C.POINTER(C.c_int32), C.POINTER(C.c_int32)],
        "hccl_hostpipe_workspace_bytes": [P, C.POINTER(C.c_size_t)],
        "hccl_hostpipe_bind": [P, P, C.c_size_t, P],
        "hccl_hostpipe_execute": [P, C.POINTER(P), C.POINTER(P), C.POINTER(P), C.POINTER(P), P, P, P],
        "hccl_hostpipe_status": [P, C.POINTER(C.c_int), I64P],
    }
    for name, args in sigs.items():
        fn = getattr(lib, name)
        fn.argtypes = args
        fn.restype = C.c_int
    lib.hccl_graph_destroy.argtypes = [P]
    lib.hccl_graph_destroy.restype = None
    lib.hccl_plan_destroy.argtypes = [P]
    lib.hccl_plan_destroy.restype = None
    lib.hccl_hostpipe_destroy.argtypes = [P]
    lib.hccl_hostpipe_destroy.restype = None
    lib.hccl_status_string.argtypes = [C.c_int]
    lib.hccl_status_string.restype = C.c_char_p
    lib.hccl_last_cuda_error.argtypes = []
    lib.hccl_last_cuda_error.restype = C.c_char_p
    lib.hccl_version.argtypes = []
    lib.hccl_version.restype = C.c_int
    lib.hccl_opts_for_overlap.argtypes = [C.POINTER(Opts)]
    lib.hccl_opts_for_overlap.restype = None
    return lib


_lib = _load()
LIBRARY_PATH = _build.LIB
EXPORTS = ["hccl_plan_allreduce", "hccl_plan_reducescatter", "hccl_plan_allgather", "hccl_plan_alltoallv",
           "hccl_plan_alltoallv_dynamic", "hccl_plan_set_dynamic_metadata",
           "hccl_graph_create", "hccl_graph_add_subgraph", "hccl_graph_add_wqe", "hccl_graph_compile",
           "hccl_graph_destroy", "hccl_plan_workspace_bytes", "hccl_plan_bind", "hccl_execute", "hccl_execute_host",
           "hccl_execute_noalloc", "hccl_server_start", "hccl_server_ring", "hccl_server_wait", "hccl_server_stop",
           "hccl_plan_set_user_signals", "hccl_plan_set_trace", "hccl_plan_set_trigger", "hccl_plan_status", "hccl_plan_info",
           "hccl_plan_extents", "hccl_plan_layout", "hccl_plan_destroy", "hccl_status_string", "hccl_last_cuda_error", "hccl_version",
           "hccl_plan_check_hazards", "hccl_plan_interpret_host",
           "hccl_hostpipe_alltoallv_create", "hccl_hostpipe_windows", "hccl_hostpipe_workspace_bytes", "hccl_hostpipe_bind",
           "hccl_hostpipe_execute", "hccl_hostpipe_status", "hccl_hostpipe_destroy", "hccl_opts_for_overlap"]


def status_string(status: int) -> str:
    return _lib.hccl_status_string(status).decode()


def _chk(rc: int, what: str):
    if rc != OK:
        raise HcclError(rc, what)


def _i64(a) -> Optional[C.Array]:
    if a is None:
        return None
    flat = [int(v) for row in a for v in (row if hasattr(row, "__len__") else [row])]
    return (C.c_int64 * len(flat))(*flat)


def _ptr_array(ptrs: Sequence[int]):
    return (C.c_void_p * len(ptrs))(*[int(p) if p else None for p in ptrs])


def hccl_opts_for_overlap() -> dict:
    """The library's operating point for running beside a saturating compute kernel, as a dict of options."""
    o = Opts()
    _lib.hccl_opts_for_overlap(C.byref(o))
    return {name: getattr(o, name) for name, _ in Opts._fields_ if getattr(o, name)}


def make_opts(opts=None, **kw) -> Opts:
    o = Opts()
    if isinstance(opts, Opts):
        C.memmove(C.byref(o), C.byref(opts), C.sizeof(Opts))
    elif isinstance(opts, dict):
        kw = {**opts, **kw}
    for k, v in kw.items():
        setattr(o, k, v)
    return o


class Plan:
    """Owner of one hccl_plan_t*. Methods carry the names of the C calls they wrap."""

    def __init__(self, handle: int):
        self._h = C.c_void_p(handle)

    def __del__(self):
        self.destroy()

    def destroy(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.hccl_plan_destroy(self._h)
        self._h = None

    def workspace_bytes(self) -> int:
        n = C.c_size_t()
        _chk(_lib.hccl_plan_workspace_bytes(self._h, C.byref(n)), "hccl_plan_workspace_bytes")
        return n.value

    def info(self) -> PlanInfo:
        i = PlanInfo()
        _chk(_lib.hccl_plan_info(self._h, C.byref(i)), "hccl_plan_info")
        return i

    def extents(self, rank: int):
        s, r = C.c_int64(), C.c_int64()
        _chk(_lib.hccl_plan_extents(self._h, rank, C.byref(s), C.byref(r)), "hccl_plan_extents")
        return s.value, r.value

    def layout(self) -> dict:
        o = (C.c_int64 * 8)()
        _chk(_lib.hccl_plan_layout(self._h, o), "hccl_plan_layout")
        return dict(zip(["control", "counters", "signals", "descs", "tiles", "waits", "scratch", "total"], list(o)))

    def bind(self, dev_workspace: int, nbytes: int, stream: int = 0):
        _chk(_lib.hccl_plan_bind(self._h, C.c_void_p(dev_workspace), nbytes, C.c_void_p(stream)), "hccl_plan_bind")

    def execute(self, sendbufs: Sequence[int], recvbufs: Sequence[int], stream: int = 0):
        _chk(_lib.hccl_execute(self._h, _ptr_array(sendbufs), _ptr_array(recvbufs), C.c_void_p(stream)), "hccl_execute")

    def execute_ptrs(self, send_arr, recv_arr, stream: int = 0) -> int:
        """Same as execute() with pre-marshalled pointer arrays; returns the status instead of raising."""
        return _lib.hccl_execute(self._h, send_arr, recv_arr, C.c_void_p(stream))

    def execute_host(self, host_send, host_recv, dev_send, dev_recv, stream: int = 0):
        _chk(_lib.hccl_execute_host(self._h, _ptr_array(host_send), _ptr_array(host_recv), _ptr_array(dev_send),
                                    _ptr_array(dev_recv), C.c_void_p(stream)), "hccl_execute_host")

    def execute_noalloc(self, sendbufs: Sequence[int], recvbufs: Sequence[int], stream: int = 0):
        """One blocking execution on the library's built-in 8 MiB workspace (for callers that cannot
        allocate device memory). Raises HcclError with the device-side verdict if it failed."""
        _chk(_lib.hccl_execute_noalloc(self._h, _ptr_array(sendbufs), _ptr_array(recvbufs), C.c_void_p(stream)),
             "hccl_execute_noalloc")

    def server_start(self, sendbufs: Sequence[int], recvbufs: Sequence[int], host_doorbell: int, idle_timeout_ns: int = 0,
                     stream: int = 0):
        _chk(_lib.hccl_server_start(self._h, _ptr_array(sendbufs), _ptr_array(recvbufs), C.c_void_p(host_doorbell),
                                    idle_timeout_ns, C.c_void_p(stream)), "hccl_server_start")

    def server_ring(self) -> int:
        return _lib.hccl_server_ring(self._h)

    def server_wait(self, timeout_ns: int = 0) -> int:
        return _lib.hccl_server_wait(self._h, timeout_ns)

    def server_stop(self):
        _chk(_lib.hccl_server_stop(self._h), "hccl_server_stop")

    def set_dynamic_metadata(self, dev_sendcounts: int, dev_recvcounts_out: int = 0, dev_rdispls_out: int = 0):
        _chk(_lib.hccl_plan_set_dynamic_metadata(self._h, C.c_void_p(dev_sendcounts), C.c_void_p(dev_recvcounts_out or None),
                                                 C.c_void_p(dev_rdispls_out or None)), "hccl_plan_set_dynamic_metadata")

    def set_trace(self, dev_trace: int, capacity_items: int):
        _chk(_lib.hccl_plan_set_trace(self._h, C.c_void_p(dev_trace or None), capacity_items), "hccl_plan_set_trace")

    def set_user_signals(self, dev_signals: int, n_slots: int):
        _chk(_lib.hccl_plan_set_user_signals(self._h, C.c_void_p(dev_signals), n_slots), "hccl_plan_set_user_signals")

    def set_trigger(self, wait_slot=-1, cmp=CMP_GE, wait_value=0, wait_per_epoch=0, set_slot=-1, set_value=0,
                    set_per_epoch=0):
        _chk(_lib.hccl_plan_set_trigger(self._h, wait_slot, cmp, wait_value, wait_per_epoch, set_slot, set_value,
                                        set_per_epoch), "hccl_plan_set_trigger")

    def status(self):
        st, detail = C.c_int(), C.c_int64()
        _chk(_lib.hccl_plan_status(self._h, C.byref(st), C.byref(detail)), "hccl_plan_status")
        return st.value, detail.value

    def check_hazards(self) -> int:
        n = C.c_int64()
        _chk(_lib.hccl_plan_check_hazards(self._h, C.byref(n)), "hccl_plan_check_hazards")
        return n.value

    def interpret_host(self, host_send: Sequence[int], host_recv: Sequence[int], host_scratch: int = 0,
                       host_signals: int = 0, seed: int = 0) -> int:
        return _lib.hccl_plan_interpret_host(self._h, _ptr_array(host_send), _ptr_array(host_recv),
                                             C.c_void_p(host_scratch),
                                             C.cast(C.c_void_p(host_signals), C.POINTER(C.c_uint64)), seed)


def _new_plan(rc: int, h: C.c_void_p, what: str) -> Plan:
    _chk(rc, what)
    return Plan(h.value)


def hccl_plan_allreduce(R: int, count: int, dt: int, algo: int = ALGO_RING, opts=None) -> Plan:
    h = C.c_void_p()
    return _new_plan(_lib.hccl_plan_allreduce(R, count, dt, algo, C.byref(make_opts(opts)), C.byref(h)), h,
                     "hccl_plan_allreduce")


def hccl_plan_reducescatter(R: int, recvcounts, count: int, dt: int, algo: int = ALGO_RING, opts=None) -> Plan:
    h = C.c_void_p()
    return _new_plan(_lib.hccl_plan_reducescatter(R, _i64(recvcounts), count, dt, algo, C.byref(make_opts(opts)),
                                                  C.byref(h)), h, "hccl_plan_reducescatter")


def hccl_plan_allgather(R: int, sendcounts, count: int, dt: int, algo: int = ALGO_RING, opts=None) -> Plan:
    h = C.c_void_p()
    return _new_plan(_lib.hccl_plan_allgather(R, _i64(sendcounts), count, dt, algo, C.byref(make_opts(opts)),
                                              C.byref(h)), h, "hccl_plan_allgather")


def hccl_plan_alltoallv(R: int, sendcounts, sdispls=None, recvcounts=None, rdispls=None, dt: int = BF16,
                        row_elems: int = 1, opts=None) -> Plan:
    h = C.c_void_p()
    return _new_plan(_lib.hccl_plan_alltoallv(R, _i64(sendcounts), _i64(sdispls), _i64(recvcounts), _i64(rdispls), dt,
                                              row_elems, C.byref(make_opts(opts)), C.byref(h)), h,
                     "hccl_plan_alltoallv")


def hccl_plan_alltoallv_dynamic(R: int, max_send_rows, max_recv_rows, dt: int = BF16, row_elems: int = 1, opts=None) -> Plan:
    h = C.c_void_p()
    return _new_plan(_lib.hccl_plan_alltoallv_dynamic(R, _i64(max_send_rows), _i64(max_recv_rows), dt, row_elems,
                                                      C.byref(make_opts(opts)), C.byref(h)), h, "hccl_plan_alltoallv_dynamic")


class HostPipe:
    """Owner of one hccl_hostpipe_t*: AllToAllv through host buffers, pipelined by destination windows."""

    def __init__(self, handle: int):
        self._h = C.c_void_p(handle)

    def __del__(self):
        self.destroy()

    def destroy(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.hccl_hostpipe_destroy(self._h)
        self._h = None

    def windows(self):
        n = C.c_int32()
        first = (C.c_int32 * (MAX_RANKS + 1))()
        _chk(_lib.hccl_hostpipe_windows(self._h, C.byref(n), first), "hccl_hostpipe_windows")
        return list(first[: n.value + 1])

    def workspace_bytes(self) -> int:
        n = C.c_size_t()
        _chk(_lib.hccl_hostpipe_workspace_bytes(self._h, C.byref(n)), "hccl_hostpipe_workspace_bytes")
        return n.value

    def bind(self, dev_workspace: int, nbytes: int, stream: int = 0):
        _chk(_lib.hccl_hostpipe_bind(self._h, C.c_void_p(dev_workspace), nbytes, C.c_void_p(stream)), "hccl_hostpipe_bind")

    def execute(self, host_send, host_recv, dev_send, dev_recv, stream_in: int, stream_exec: int, stream_out: int):
        _chk(_lib.hccl_hostpipe_execute(self._h, _ptr_array(host_send), _ptr_array(host_recv), _ptr_array(dev_send),
                                        _ptr_array(dev_recv), C.c_void_p(stream_in), C.c_void_p(stream_exec),
                                        C.c_void_p(stream_out)), "hccl_hostpipe_execute")

    def status(self):
        st, detail = C.c_int(), C.c_int64()
        _chk(_lib.hccl_hostpipe_status(self._h, C.byref(st), C.byref(detail)), "hccl_hostpipe_status")
        return st.value, detail.value


def hccl_hostpipe_alltoallv_create(R: int, sendcounts, dt: int = BF16, row_elems: int = 1, n_windows: int = 8, opts=None) -> HostPipe:
    h = C.c_void_p()
    _chk(_lib.hccl_hostpipe_alltoallv_create(R, _i64(sendcounts), dt, row_elems, n_windows, C.byref(make_opts(opts)), C.byref(h)),
         "hccl_hostpipe_alltoallv_create")
    return HostPipe(h.value)


class Graph:
    """Owner of one hccl_graph_t* (a work packet under construction)."""

    def __init__(self, R: int, send_bytes, recv_bytes, scratch_bytes: int = 0, n_signals: int = 0):
        h = C.c_void_p()
        _chk(_lib.hccl_graph_create(R, _i64(send_bytes), _i64(recv_bytes), scratch_bytes, n_signals, C.byref(h)),
             "hccl_graph_create")
        self._h = h

    def __del__(self):
        if getattr(self, "_h", None) and _lib is not None:
            _lib.hccl_graph_destroy(self._h)
        self._h = None

    def add_subgraph(self, rank: int = 0) -> int:
        sg = C.c_int32()
        _chk(_lib.hccl_graph_add_subgraph(self._h, rank, C.byref(sg)), "hccl_graph_add_subgraph")
        return sg.value

    def add_wqe(self, subgraph: int, op: int, dst=None, a=None, b=None, count: int = 0, dtypes=(FP32, FP32, FP32),
                nsrc: int = 0, dep_flags: int = 0, dep_wqe: int = -1, dep_wqe2: int = -1, cmp: int = 0,
                value: int = 0, value_per_epoch: int = 0, tile_count: int = 0, hints: int = 0, ndst: int = 0) -> int:
        w = Wqe()
        w.op = op
        w.dtype_dst, w.dtype_a, w.dtype_b = dtypes
        for name, r in (("dst", dst), ("a", a), ("b", b)):
            if r is not None:
                setattr(w, name, Ref(*r))
        w.count, w.nsrc, w.dep_flags, w.dep_wqe, w.dep_wqe2 = count, nsrc, dep_flags, dep_wqe, dep_wqe2
        w.cmp, w.value, w.value_per_epoch, w.tile_count, w.hints = cmp, value, value_per_epoch, tile_count, hints
        w.ndst = ndst
        wid = C.c_int64()
        _chk(_lib.hccl_graph_add_wqe(self._h, subgraph, C.byref(w), C.byref(wid)), "hccl_graph_add_wqe")
        return wid.value

    def compile(self, opts=None) -> Plan:
        h = C.c_void_p()
        return _new_plan(_lib.hccl_graph_compile(self._h, C.byref(make_opts(opts)), C.byref(h)), h,
                         "hccl_graph_compile")
