"""Interference harness: a saturating bf16 GEMM on one stream, back-to-back collectives on a second one.

The paper's overlap experiment (Sec. V-E) runs a large GEMM that fills the compute grid while 100
collectives of one size run back to back on a parallel stream, and reports the GEMM's loss (about 0.5 %
on its hardware, attributed to HBM contention). Here the GEMM is cuBLAS through torch.matmul and the
collective is one bound plan re-enqueued on a high-priority stream; the benchmark suite the paper used
is not available and is not reproduced.

Run as a module for the SM-budget sweep and for the other ways of sharing the GPU with the GEMM:
    python -m paper_2608_00358_b200.interference --budgets 4,8,16,32,64,148 --cap 32768
    python -m paper_2608_00358_b200.interference --method idle_sms --quanta 1,2,4 --opts tile_bytes=122880

OVERLAP_OPTS is the operating point measured to cost a saturating 8192^3 GEMM less than 5 % in every run: twelve persistent
blocks of the register engine's 64-register build with 128 threads each, which are small enough to run on SMs
that GEMM blocks occupy (they hold no SM against the GEMM). IDLE_SM_OPTS is the other way of holding no SM:
short-lived blocks (one work item of 120 KiB each) on a stream of lower priority than the GEMM's.
"""
from __future__ import annotations

import argparse
import json
import time
from typing import Optional

import numpy as np
import torch

from . import workloads as wk


OVERLAP_OPTS = wk.hb.hccl_opts_for_overlap()      # engine = register, light = 1, threads = 128, sm_budget = 12
IDLE_SM_OPTS = dict(quantum=1, tile_bytes=122880)


class Gemm:
    def __init__(self, n: int = 8192):
        self.n = n
        g = torch.Generator(device="cuda")
        g.manual_seed(1)
        self.a = torch.randn(n, n, device="cuda", dtype=torch.float32, generator=g).to(torch.bfloat16)
        self.b = torch.randn(n, n, device="cuda", dtype=torch.float32, generator=g).to(torch.bfloat16)
        self.c = torch.empty(n, n, device="cuda", dtype=torch.bfloat16)
        self.flops = 2.0 * n ** 3

    def run(self):
        torch.matmul(self.a, self.b, out=self.c)


def overlap(gemm: Gemm, wl: Optional[wk.Workload], seconds: float = 3.0, discard: float = 1.0, gemm_batch: int = 10,
            collective_first: bool = True, streams=None) -> dict:
    """GEMM loop on one stream, collective loop on another; rates are computed only inside the window in which
    events show both loops running. `collective_first`: the collective's stream has the higher priority (its
    blocks take SMs as soon as GEMM blocks retire); otherwise the GEMM's has, and the collective gets the SMs the
    GEMM leaves idle. `streams`: (gemm stream, collective stream) made by the caller, e.g. in green contexts."""
    if streams is not None:
        sg, sc = streams
    elif collective_first:
        sg, sc = torch.cuda.Stream(), torch.cuda.Stream(priority=-1)
    else:
        sg, sc = torch.cuda.Stream(priority=-1), torch.cuda.Stream()
    base = torch.cuda.Event(enable_timing=True)
    eg, ec = [], []
    torch.cuda.synchronize()
    base.record(torch.cuda.current_stream())
    sg.wait_event(base)
    sc.wait_event(base)
    # Both queues are kept a few batches deep independently of each other, so neither loop is ever
    # starved by the other's enqueue rate.
    depth, done_g, done_c = 3, 0, 0
    t0 = time.time()
    while time.time() - t0 < seconds:
        while done_g < len(eg) and eg[done_g].query():
            done_g += 1
        while done_c < len(ec) and ec[done_c].query():
            done_c += 1
        busy = True
        if len(eg) - done_g < depth:
            with torch.cuda.stream(sg):
                for _ in range(gemm_batch):
                    gemm.run()
                e = torch.cuda.Event(enable_timing=True)
                e.record(sg)
                eg.append(e)
            busy = False
        if wl is not None and len(ec) - done_c < depth:
            wl.dc.execute(sc)
            e = torch.cuda.Event(enable_timing=True)
            e.record(sc)
            ec.append(e)
            busy = False
        if busy:
            time.sleep(0.0002)
    torch.cuda.synchronize()
    tg = np.array([base.elapsed_time(e) for e in eg])
    if wl is None:      # same enqueue loop with no collective: the GEMM-alone figure, measured the same way
        kg = tg[tg >= discard * 1e3]
        return dict(window_s=float((kg[-1] - kg[0]) * 1e-3), gemm_batches=int(len(kg) - 1),
                    gemm_tflops=float(gemm.flops * gemm_batch * (len(kg) - 1) / ((kg[-1] - kg[0]) * 1e-3) / 1e12))
    wl.dc.check()
    tc = np.array([base.elapsed_time(e) for e in ec])
    lo = max(discard * 1e3, min(tg[0], tc[0]))
    hi = min(tg[-1], tc[-1])
    kg = tg[(tg >= lo) & (tg <= hi)]
    kc = tc[(tc >= lo) & (tc <= hi)]
    out = dict(window_s=float((hi - lo) * 1e-3), gemm_batches=int(max(len(kg) - 1, 0)), collectives=int(max(len(kc) - 1, 0)))
    if len(kg) >= 2:
        out["gemm_tflops"] = float(gemm.flops * gemm_batch * (len(kg) - 1) / ((kg[-1] - kg[0]) * 1e-3) / 1e12)
    if len(kc) >= 2:
        ms = (kc[-1] - kc[0]) / (len(kc) - 1)
        out["collective_ms"] = float(ms)
        out["collective_gbs"] = float(wl.info.schedule_bytes / ms / 1e6)
    return out


# ---- the two remedies for a GEMM that was tiled for more SMs than it gets (process-local, nothing outlives the process)
def _cublas():
    """The cuBLAS library torch has loaded (found in this process's memory map), for cublasSetSmCountTarget."""
    import ctypes
    for line in open("/proc/self/maps"):
        if "libcublas.so" in line:
            lib = ctypes.CDLL(line.split()[-1])
            lib.cublasSetSmCountTarget.argtypes = [ctypes.c_void_p, ctypes.c_int]
            lib.cublasGetSmCountTarget.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_int)]
            return lib
    raise RuntimeError("cuBLAS is not loaded yet: run a matmul first")


def set_sm_count_target(n: int, stream: Optional[torch.cuda.Stream] = None) -> int:
    """Tells cuBLAS (torch's handle for `stream`) to plan its kernels for n SMs (0 = all). Returns the value
    cuBLAS reports back."""
    import ctypes
    lib = _cublas()
    with torch.cuda.stream(stream or torch.cuda.current_stream()):
        h = ctypes.c_void_p(torch.cuda.current_blas_handle())
        rc = lib.cublasSetSmCountTarget(h, ctypes.c_int(n))
        if rc != 0:
            raise RuntimeError("cublasSetSmCountTarget failed: %d" % rc)
        got = ctypes.c_int(-1)
        lib.cublasGetSmCountTarget(h, ctypes.byref(got))
    return got.value


class GreenPartition:
    """Two green contexts that split the device's SMs into `small` SMs (rounded up to what the device allows)
    for the collective and the rest for the GEMM, with one stream in each. Released by close()."""

    def __init__(self, small: int):
        from cuda.bindings import driver as drv
        self.drv = drv

        def ck(res):
            if int(res[0]) != 0:
                raise RuntimeError("CUDA driver error %s" % res[0])
            return None if len(res) == 1 else (res[1] if len(res) == 2 else res[1:])
        self.ck = ck
        dev = ck(drv.cuDeviceGet(torch.cuda.current_device()))
        sm = ck(drv.cuDeviceGetDevResource(dev, drv.CUdevResourceType.CU_DEV_RESOURCE_TYPE_SM))
        groups, _, rest = ck(drv.cuDevSmResourceSplitByCount(1, sm, 0, small))
        self.small_sms, self.rest_sms = int(groups[0].sm.smCount), int(rest.sm.smCount)
        self.ctx = [ck(drv.cuGreenCtxCreate(ck(drv.cuDevResourceGenerateDesc([r], 1)), dev, drv.CUgreenCtxCreate_flags.CU_GREEN_CTX_DEFAULT_STREAM))
                    for r in (groups[0], rest)]
        self.raw = [ck(drv.cuGreenCtxStreamCreate(self.ctx[0], drv.CUstream_flags.CU_STREAM_NON_BLOCKING, -1)),
                    ck(drv.cuGreenCtxStreamCreate(self.ctx[1], drv.CUstream_flags.CU_STREAM_NON_BLOCKING, 0))]
        self.collective_stream = torch.cuda.ExternalStream(int(self.raw[0]))
        self.gemm_stream = torch.cuda.ExternalStream(int(self.raw[1]))

    def close(self):
        torch.cuda.synchronize()
        for s_ in self.raw:
            self.ck(self.drv.cuStreamDestroy(s_))
        for c in self.ctx:
            self.ck(self.drv.cuGreenCtxDestroy(c))


def measure(wl: wk.Workload, seconds: float = 3.0, gemm: Optional[Gemm] = None, collective_first: bool = True, streams=None,
            alone_tflops: Optional[float] = None, discard: float = 1.0) -> dict:
    """GEMM slowdown = 1 - (GEMM rate beside the collective) / (rate of the UNRESTRICTED GEMM alone: default streams,
    all SMs, no SM-count target). Pass `alone_tflops` when that figure was taken before a restriction was applied.
    Otherwise the GEMM alone is timed before AND after the overlapped run and the two are averaged: a GEMM at the
    power limit drifts by a few per cent over seconds, which is the size of the effect that is measured here."""
    gemm = gemm or Gemm()
    before = alone_tflops if alone_tflops is not None else overlap(gemm, None, seconds, discard)["gemm_tflops"]
    coll_alone_ms = wk.time_back_to_back(wl, 5, 2)
    both = overlap(gemm, wl, seconds, discard, collective_first=collective_first, streams=streams)
    after = alone_tflops if alone_tflops is not None else overlap(gemm, None, seconds, discard)["gemm_tflops"]
    alone = dict(tflops=0.5 * (before + after))
    res = dict(gemm_alone_tflops=alone["tflops"], gemm_alone_before_after=[float(before), float(after)],
               collective_alone_ms=float(coll_alone_ms),
               collective_alone_gbs=float(wl.info.schedule_bytes / coll_alone_ms / 1e6), overlap=both,
               sm_budget=int(wl.info.sm_budget))
    if "gemm_tflops" in both:
        res["gemm_slowdown"] = float(1.0 - both["gemm_tflops"] / alone["tflops"])
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--budgets", default="2,4,8,16,32,64,128,148")
    ap.add_argument("--cap", type=int, default=32768)
    ap.add_argument("--seconds", type=float, default=3.0)
    ap.add_argument("--engine", type=int, default=0)
    ap.add_argument("--gemm-n", type=int, default=8192, help="the GEMM is n x n x n, bf16")
    ap.add_argument("--opts", default="", help="extra plan options, e.g. threads=256,light=1,cluster=2")
    ap.add_argument("--method", default="plain", choices=["plain", "sm_target", "green", "green_sm_target", "idle_sms"],
                    help="plain: collective on a high-priority stream; sm_target: cuBLAS plans for 148 - budget SMs; green: GEMM and "
                         "collective in two green contexts that split the SMs; idle_sms: short-lived blocks (--quanta) on a stream of "
                         "LOWER priority than the GEMM's, so they only take SMs the GEMM leaves idle")
    ap.add_argument("--quanta", default="4,8,16", help="items per block for --method idle_sms")
    ap.add_argument("--gemm-first", action="store_true", help="--method plain with the GEMM's stream at the higher priority")
    args = ap.parse_args()
    extra = {k: int(v) for k, v in (kv.split("=") for kv in args.opts.split(",") if kv)}
    gemm = Gemm(args.gemm_n)
    gemm.run()
    torch.cuda.synchronize()
    unrestricted = overlap(gemm, None, args.seconds)["gemm_tflops"]     # the reference for every slowdown below
    base = wk.config4(dict(sm_budget=148, engine=args.engine), cap=args.cap)

    def plan_for(**o):
        plan = wk.hb.hccl_plan_alltoallv(base.meta["R"], base.meta["counts"], None, None, None, wk.hb.FP16,
                                         base.meta["row_elems"], {"engine": args.engine, **extra, **o})
        return wk._bind(base.name, plan, base.send, base.recv, base.meta)

    if args.method == "idle_sms":
        for q in [int(x) for x in args.quanta.split(",")]:
            wl = plan_for(quantum=q)
            res = measure(wl, args.seconds, gemm, collective_first=False)   # GEMM alone timed before and after
            res.update(method=args.method, quantum=q, opts=extra, gemm_n=args.gemm_n)
            print(json.dumps(res), flush=True)
        return
    for b in [int(x) for x in args.budgets.split(",")]:
        part, streams, target = None, None, 0
        try:
            if args.method in ("green", "green_sm_target"):
                part = GreenPartition(b)
                streams = (part.gemm_stream, part.collective_stream)
                b = part.small_sms
            wl = plan_for(sm_budget=b)
            if args.method in ("sm_target", "green_sm_target"):
                target = set_sm_count_target(148 - b, streams[0] if streams else None)
            # (a restricted GEMM is compared with the unrestricted one timed at the start; otherwise alone = before and after)
            res = measure(wl, args.seconds, gemm, streams=streams, alone_tflops=None if args.method == "plain" else unrestricted,
                          collective_first=not args.gemm_first)
            res.update(method=args.method, sm_count_target=target, opts=extra, gemm_n=args.gemm_n, gemm_first=bool(args.gemm_first))
            print(json.dumps(res), flush=True)
        finally:
            if target:
                set_sm_count_target(0, streams[0] if streams else None)
            if part is not None:
                part.close()


if __name__ == "__main__":
    main()
