"""Interference harness: a saturating bf16 GEMM on one stream, back-to-back collectives on a second one.

The paper's overlap experiment (Sec. V-E) runs a large GEMM that fills the compute grid while 100
collectives of one size run back to back on a parallel stream, and reports the GEMM's loss (about 0.5 %
on its hardware, attributed to HBM contention). Here the GEMM is cuBLAS through torch.matmul and the
collective is one bound plan re-enqueued on a high-priority stream; the benchmark suite the paper used
is not available and is not reproduced.

Run as a module for the SM-budget sweep:
    python -m paper_2608_00358_b200.interference --budgets 4,8,16,32,64,148 --cap 32768
"""
from __future__ import annotations

import argparse
import json
import time
from typing import Optional

import numpy as np
import torch

from . import workloads as wk


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


def overlap(gemm: Gemm, wl: Optional[wk.Workload], seconds: float = 3.0, discard: float = 1.0, gemm_batch: int = 10) -> dict:
    """GEMM loop on one stream, collective loop on a high-priority stream; rates are computed only inside
    the window in which events show both loops running."""
    sg = torch.cuda.Stream()
    sc = torch.cuda.Stream(priority=-1)
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


def measure(wl: wk.Workload, seconds: float = 3.0, gemm: Optional[Gemm] = None) -> dict:
    gemm = gemm or Gemm()
    alone = overlap(gemm, None, seconds)      # identical loop, no collective
    alone = dict(tflops=alone["gemm_tflops"])
    coll_alone_ms = wk.time_back_to_back(wl, 5, 2)
    both = overlap(gemm, wl, seconds)
    res = dict(gemm_alone_tflops=alone["tflops"], collective_alone_ms=float(coll_alone_ms),
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
    args = ap.parse_args()
    extra = {k: int(v) for k, v in (kv.split("=") for kv in args.opts.split(",") if kv)}
    gemm = Gemm(args.gemm_n)
    base = wk.config4(dict(sm_budget=148, engine=args.engine), cap=args.cap)
    for b in [int(x) for x in args.budgets.split(",")]:
        plan = wk.hb.hccl_plan_alltoallv(base.meta["R"], base.meta["counts"], None, None, None, wk.hb.FP16,
                                         base.meta["row_elems"], dict(sm_budget=b, engine=args.engine, **extra))
        wl = wk._bind(base.name, plan, base.send, base.recv, base.meta)
        res = measure(wl, args.seconds, gemm)
        res["opts"] = extra
        res["gemm_n"] = args.gemm_n
        print(json.dumps(res), flush=True)


if __name__ == "__main__":
    main()
