"""Device-side plumbing around the C ABI: torch supplies memory and streams, nothing more.

``DeviceCollective`` owns the workspace tensor of one bound plan and the pointer arrays of one set of
rank buffers, so that re-running a cached plan is a single C call (the cached re-enqueue of Sec. V-B).
"""
from __future__ import annotations

import ctypes as C
from typing import List, Optional, Sequence

import torch

from . import binding as hb


def require_cuda():
    if not torch.cuda.is_available():
        raise RuntimeError("paper_2608_00358_b200: a CUDA device is required; there is no CPU fallback")


def alloc_rank_buffers(nbytes: Sequence[int], device="cuda", guard: int = 0, fill: Optional[int] = None) -> List[torch.Tensor]:
    """One uint8 tensor per rank (at least 16 bytes so that every rank has a valid pointer)."""
    out = []
    for n in nbytes:
        t = torch.empty(max(int(n), 16) + 2 * guard, dtype=torch.uint8, device=device)
        if fill is not None:
            t.fill_(fill)
        out.append(t)
    return out


class DeviceCollective:
    def __init__(self, plan: hb.Plan, stream: Optional[torch.cuda.Stream] = None, device="cuda"):
        require_cuda()
        self.plan = plan
        self.stream = stream
        self.info = plan.info()
        self.R = self.info.R
        nbytes = plan.workspace_bytes()
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=device)
        base = self.workspace.data_ptr()
        self._ws_ptr = (base + 255) // 256 * 256
        plan.bind(self._ws_ptr, nbytes, self._stream_handle())
        self._send_arr = None
        self._recv_arr = None
        self._keep = None

    def _stream_handle(self) -> int:
        s = self.stream if self.stream is not None else torch.cuda.current_stream()
        return s.cuda_stream

    def set_buffers(self, send_ptrs: Sequence[int], recv_ptrs: Sequence[int], keep=None):
        self._send_arr = (C.c_void_p * self.R)(*[int(p) for p in send_ptrs])
        self._recv_arr = (C.c_void_p * self.R)(*[int(p) for p in recv_ptrs])
        self._keep = keep

    def execute(self, stream: Optional[torch.cuda.Stream] = None):
        s = stream.cuda_stream if stream is not None else self._stream_handle()
        rc = self.plan.execute_ptrs(self._send_arr, self._recv_arr, s)
        if rc != hb.OK:
            raise hb.HcclError(rc, "hccl_execute")

    def check(self):
        """Synchronise and raise if the last execution failed on the device."""
        torch.cuda.synchronize()
        st, detail = self.plan.status()
        if st != hb.OK:
            raise hb.HcclError(st, "device status (tile %d)" % detail)


def enable_trace(plan: hb.Plan, device="cuda") -> torch.Tensor:
    """Allocates a trace array for every work item of `plan` and switches tracing on. Returns the tensor
    ([n_tiles, 4] int64: item | block << 32, claimed, released, stored; nanoseconds of %globaltimer)."""
    n = max(int(plan.info().n_tiles), 1)
    t = torch.zeros((n, 4), dtype=torch.int64, device=device)
    plan.set_trace(t.data_ptr(), n)
    return t


def chrome_trace(trace: torch.Tensor, name: str = "hccl") -> dict:
    """Trace array -> Chrome trace-event JSON (one row per thread block, one slice per work item from the
    moment its data movement was released to its last store, with the wait before it as a separate slice)."""
    rows = trace.cpu().numpy()
    rows = rows[rows[:, 1] != 0]
    if rows.shape[0] == 0:
        return {"traceEvents": []}
    t0 = int(rows[:, 1].min())
    ev = []
    for item_block, claimed, released, stored in rows.tolist():
        item, block = item_block & 0xFFFFFFFF, item_block >> 32
        if released and released > claimed:
            ev.append({"name": "wait", "cat": "dependency", "ph": "X", "pid": name, "tid": block,
                       "ts": (claimed - t0) / 1e3, "dur": (released - claimed) / 1e3, "args": {"item": item}})
        if stored and released:
            ev.append({"name": "item %d" % item, "cat": "data", "ph": "X", "pid": name, "tid": block,
                       "ts": (released - t0) / 1e3, "dur": max(stored - released, 0) / 1e3, "args": {"item": item}})
    return {"traceEvents": ev, "displayTimeUnit": "ns"}


class PlanCache:
    """Work-packet cache (paper Sec. V-B): a collective that was compiled and bound once is found again by its
    arguments and only re-enqueued, so neither generation nor upload is repeated. Keys are the planner's
    arguments; AllToAllv keys include the count matrix."""

    def __init__(self, device="cuda"):
        self.device = device
        self._entries = {}
        self.hits = 0
        self.misses = 0

    @staticmethod
    def _freeze(x):
        if x is None:
            return None
        if isinstance(x, dict):
            return tuple(sorted(x.items()))
        if hasattr(x, "tobytes"):
            return (getattr(x, "shape", None), x.tobytes())
        if isinstance(x, (list, tuple)):
            return tuple(PlanCache._freeze(v) for v in x)
        return x

    def _get(self, key, make):
        ent = self._entries.get(key)
        if ent is None:
            self.misses += 1
            ent = DeviceCollective(make(), device=self.device)
            self._entries[key] = ent
        else:
            self.hits += 1
        return ent

    def allreduce(self, R, count, dt, algo=hb.ALGO_RING, opts=None) -> DeviceCollective:
        return self._get(("allreduce", R, count, dt, algo, self._freeze(opts)), lambda: hb.hccl_plan_allreduce(R, count, dt, algo, opts))

    def reducescatter(self, R, recvcounts, count, dt, algo=hb.ALGO_RING, opts=None) -> DeviceCollective:
        return self._get(("reducescatter", R, self._freeze(recvcounts), count, dt, algo, self._freeze(opts)),
                         lambda: hb.hccl_plan_reducescatter(R, recvcounts, count, dt, algo, opts))

    def allgather(self, R, sendcounts, count, dt, algo=hb.ALGO_RING, opts=None) -> DeviceCollective:
        return self._get(("allgather", R, self._freeze(sendcounts), count, dt, algo, self._freeze(opts)),
                         lambda: hb.hccl_plan_allgather(R, sendcounts, count, dt, algo, opts))

    def alltoallv(self, R, sendcounts, sdispls=None, rdispls=None, dt=hb.BF16, row_elems=1, opts=None) -> DeviceCollective:
        key = ("alltoallv", R, self._freeze(sendcounts), self._freeze(sdispls), self._freeze(rdispls), dt, row_elems, self._freeze(opts))
        return self._get(key, lambda: hb.hccl_plan_alltoallv(R, sendcounts, sdispls, None, rdispls, dt, row_elems, opts))

    def __len__(self):
        return len(self._entries)
