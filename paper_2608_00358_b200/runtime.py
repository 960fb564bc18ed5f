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
