#!/usr/bin/env python
"""Benchmark of the collective hot path on B200.

A step is one execution of the rack-scale AllToAllv configuration (R = 64 virtual ranks, rows of 256 fp16,
Zipf(1.1) per-peer row counts clamped at 32768; ~25.8 GB moved, ~51.6 GB resident), the largest
single-GPU configuration and the one the HBM-bandwidth target is stated on. The metric is data-path GB/s
counting bytes read + bytes written. The same JSON line also carries the other configurations (ring
AllReduce, small AllToAllv, ring ReduceScatter, latency sweep), the GEMM-interference figure, the roofline
fraction of the executor kernel, an end-to-end figure through host buffers and the CPU oracle's baseline.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--quick]

With N > 1 (launched by torchrun) every rank runs an independent replica on its own GPU: the path has no
exchange between GPUs, so there is no data-path collective; time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "data-path GB/s (bytes read + written), AllToAllv R=64 virtual ranks"
UNIT = "GB/s"
# dram bytes (read + write) per algorithmic byte of the executor kernel on this workload, from the ncu
# capture summarised under profiles/ (captured on a smaller cap of the same workload, traffic scales with
# the bytes moved). None until measured.
DRAM_BYTES_PER_ALGORITHMIC_BYTE = 0.979


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while a timed region runs."""

    def __init__(self, index: int, period: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        import statistics
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ----------------------------------------------------------------------------------------- CPU oracle leg
def oracle_alltoallv_sample(counts, row_bytes: int, dst_ranks, repeat: int = 1):
    """Times the oracle's AllToAllv, as it stands, for the given destination ranks of the workload.
    Host send buffers are virtual-size arrays of which only the rows those destinations read are filled."""
    import numpy as np
    from oracle import oracle as orc
    R = counts.shape[0]
    sd, rd = orc.packed_displs(counts)
    X = [np.empty(int(counts[s].sum()) * row_bytes, dtype=np.uint8) for s in range(R)]
    rng = np.random.default_rng(0)
    block = rng.integers(0, 256, size=1 << 20, dtype=np.uint8)
    moved = 0
    for d in dst_ranks:
        for s in range(R):
            lo, n = int(sd[s, d]) * row_bytes, int(counts[s, d]) * row_bytes
            seg = X[s][lo:lo + n]
            for o in range(0, n, block.size):
                k = min(block.size, n - o)
                seg[o:o + k] = block[:k]
            moved += n
    Y = [np.empty(int(counts[:, d].sum()) * row_bytes if d in dst_ranks else 1, dtype=np.uint8) for d in range(R)]
    times = []
    for _ in range(repeat):
        t0 = time.perf_counter()
        for d in dst_ranks:
            orc.alltoallv(X, Y, counts, sd, rd, row_bytes, dst_only=d)
        times.append(time.perf_counter() - t0)
    return moved, times


def run_reference(args, rank: int):
    """The reference arm: the CPU oracle, unmodified, on a bounded sample of the same workload."""
    if rank != 0:
        return
    from paper_2608_00358_b200 import synth
    C = synth.zipf_counts(64, 0, 1.1, args.cap)
    dst = list(range(args.oracle_dst))
    moved, times = oracle_alltoallv_sample(C, 512, dst, repeat=args.warmup + args.steps)
    timed = times[args.warmup:]
    sec = sum(timed) / len(timed)
    gbs = 2 * moved / sec / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8", "data": "synthetic",
            "config": {"workload": "alltoallv_r64_fp16_dim256_zipf1.1_cap%d" % args.cap, "sample": "destination ranks 0..%d" % (args.oracle_dst - 1)},
            "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": "destination ranks 0..%d of 64 (%.2f GB moved per step)" % (args.oracle_dst - 1, moved / 1e9)},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def check_host_result_against_oracle(counts, row_bytes: int, host_send, host_recv) -> int:
    """Every destination's receive buffer (pinned host tensors) against the oracle's AllToAllv of the host
    send buffers, byte for byte. Returns the number of destinations compared; raises on the first mismatch."""
    import numpy as np
    from oracle import oracle as orc
    R = counts.shape[0]
    sd, rd = orc.packed_displs(counts)
    X = [h.numpy().view(np.uint8).reshape(-1) for h in host_send]
    for d in range(R):
        n = int(counts[:, d].sum()) * row_bytes
        Y = [np.full(n if q == d else 1, 0xA5, dtype=np.uint8) for q in range(R)]
        orc.alltoallv(X, Y, counts, sd, rd, row_bytes, dst_only=d)
        got = host_recv[d].numpy().view(np.uint8).reshape(-1)[:n]
        if not np.array_equal(got, Y[d]):
            raise RuntimeError("end-to-end result differs from the oracle at destination %d" % d)
    return R


def _finite(x):
    """NaN / inf -> None, numpy scalars -> Python numbers, so that the line is strict JSON."""
    import math
    if isinstance(x, dict):
        return {str(k): _finite(v) for k, v in x.items()}
    if isinstance(x, (list, tuple)):
        return [_finite(v) for v in x]
    if isinstance(x, bool) or x is None or isinstance(x, (str, int)):
        return x
    if hasattr(x, "item") and not isinstance(x, float):
        x = x.item()
    if isinstance(x, float):
        return x if math.isfinite(x) else None
    return x


def _round(x, nd=4):
    if isinstance(x, float):
        return float("%.*g" % (nd + 2, x))
    if isinstance(x, dict):
        return {k: _round(v, nd) for k, v in x.items()}
    if isinstance(x, list):
        return [_round(v, nd) for v in x]
    return x


def emit(detail: dict, headline: dict):
    """Two stdout lines: first everything (side configurations, sweeps, host-link figures), then LAST the compact
    headline record (well under 2 KB) that a reader of the tail of the output can parse."""
    d = json.dumps(_finite(detail), allow_nan=False)
    print(d, flush=True)
    h = json.dumps(_round(_finite(headline)), allow_nan=False, separators=(",", ":"))
    print(h, flush=True)


# ----------------------------------------------------------------------------------------- GPU legs
def side_configs(quick: bool):
    """Configurations 1, 2, 3 and 5: reported next to the headline, never as the headline."""
    import numpy as np
    import torch
    from paper_2608_00358_b200 import binding as hb
    from paper_2608_00358_b200 import workloads as wk
    out = {}
    it, warm = (200, 20) if quick else (1000, 100)
    flush_buf = torch.zeros(256 << 20, dtype=torch.uint8, device="cuda")     # 2x the L2

    def latency(wl, key):
        ms = wk.time_each(wl, it, warm)
        i = wl.info
        out[key] = {"p50_us": float(np.percentile(ms, 50) * 1e3), "p99_us": float(np.percentile(ms, 99) * 1e3),
                    "back_to_back_us": float(wk.time_back_to_back(wl, it, warm) * 1e3),
                    "schedule_bytes": int(i.schedule_bytes), "compulsory_bytes": int(i.compulsory_bytes),
                    "tiles": int(i.n_tiles), "chain_depth": int(i.chain_depth), "blocks": int(i.sm_budget),
                    "dispatch": "static chains" if i.static_chains else "tickets", "note": "L2-resident, latency-bound"}
        out[key]["schedule_gbs_back_to_back"] = i.schedule_bytes / out[key]["back_to_back_us"] / 1e3
        out[key]["graph_replay_us"] = float(wk.time_graph_replay(wl) * 1e3)
        # cold variant: a buffer larger than the L2 is rewritten before every iteration
        cold = wk.time_each(wl, 50, 5, flush=flush_buf)
        out[key]["p50_us_cold_l2"] = float(np.percentile(cold, 50) * 1e3)

    # the CPU oracle on the same inputs (one core, as it stands): a baseline, not a target
    import time as _t
    from oracle import oracle as orc

    def oracle_time(key, fn):
        t0 = _t.perf_counter()
        fn()
        out[key]["cpu_oracle_ms"] = (_t.perf_counter() - t0) * 1e3

    w1 = wk.config1()
    latency(w1, "1_allreduce_ring_r4_fp32_1Mi")
    oracle_time("1_allreduce_ring_r4_fp32_1Mi", lambda: orc.allreduce(hb.FP32, w1.meta["host_inputs"]))
    w2 = wk.config2()
    latency(w2, "2_alltoallv_r8_bf16_dim128")

    def _oracle_a2a():
        C = w2.meta["counts"]
        sd, rd = orc.packed_displs(C)
        X = [x.view(np.uint8) for x in w2.meta["host_inputs"]]
        Y = [np.empty(int(C[:, d].sum()) * 256, dtype=np.uint8) for d in range(8)]
        orc.alltoallv(X, Y, C, sd, rd, 256)
    oracle_time("2_alltoallv_r8_bf16_dim128", _oracle_a2a)
    del w1, w2
    for m in (4096, 65536, 262144, 1 << 20):
        for algo, nm in ((hb.ALGO_ONESHOT, "oneshot"), (hb.ALGO_RING, "ring"), (hb.ALGO_TREE, "tree"), (hb.ALGO_FANOUT, "fanout")):
            wl5 = wk.config5(m, algo)
            key5 = "5_allreduce_r8_bf16_%dB_%s" % (m, nm)
            latency(wl5, key5)
            if algo == hb.ALGO_ONESHOT:
                oracle_time(key5, lambda: orc.allreduce(hb.BF16, wl5.meta["host_inputs"]))
                out[key5]["host_observed"] = wk.time_host_observed(wl5, 100 if quick else 300)
    # host side of the compiled-communication model (Sec. V-B): generating the description, uploading it,
    # and re-enqueueing a cached one; plus the device-resident AllToAllv, where the counts never visit the host
    import time as _time
    from paper_2608_00358_b200 import synth as _synth
    host = {}
    for name, R, C, row, dt in (("alltoallv_r8", 8, _synth.uniform_counts(8, 0, 4096), 128, hb.BF16),
                                ("alltoallv_r64_zipf", 64, _synth.zipf_counts(64, 0, 1.1, 32768), 256, hb.FP16)):
        t0 = _time.perf_counter()
        plan = hb.hccl_plan_alltoallv(R, C, None, None, None, dt, row)
        t1 = _time.perf_counter()
        ws = torch.empty(plan.workspace_bytes() + 256, dtype=torch.uint8, device="cuda")
        torch.cuda.synchronize()
        t2 = _time.perf_counter()
        plan.bind((ws.data_ptr() + 255) // 256 * 256, plan.workspace_bytes(), torch.cuda.current_stream().cuda_stream)
        t3 = _time.perf_counter()
        host[name] = {"plan_ms": (t1 - t0) * 1e3, "bind_ms": (t3 - t2) * 1e3, "wqes": int(plan.info().n_wqe), "tiles": int(plan.info().n_tiles),
                      "table_bytes": int(plan.workspace_bytes())}
        del plan, ws
    wl2 = wk.config2()
    torch.cuda.synchronize()
    t0 = _time.perf_counter()
    for _ in range(300):            # fewer than the launch queue holds: host cost of the call, not GPU back-pressure
        wl2.dc.execute()
    host["cached_reenqueue_us"] = (_time.perf_counter() - t0) / 300 * 1e6
    torch.cuda.synchronize()
    C2, row2 = wl2.meta["counts"], wl2.meta["row_elems"]
    cap_s, cap_r = int(C2.sum(axis=1).max()), int(C2.sum(axis=0).max())
    dyn = hb.hccl_plan_alltoallv_dynamic(8, [cap_s] * 8, [cap_r] * 8, hb.BF16, row2)
    counts_dev = torch.from_numpy(C2.reshape(-1)).cuda()
    dyn.set_dynamic_metadata(counts_dev.data_ptr())
    recv_dyn = [torch.zeros(cap_r * row2, dtype=torch.int16, device="cuda") for _ in range(8)]
    wdyn = wk._bind("alltoallv_dynamic_r8", dyn, wl2.send, recv_dyn, {})
    msd = wk.time_each(wdyn, it, warm)
    out["next_alltoallv_dynamic_r8_bf16_dim128"] = {"p50_us": float(np.percentile(msd, 50) * 1e3), "note": "counts read from device memory at run time; same payload as config 2"}
    out["host_side"] = host
    del wl2, wdyn, dyn, recv_dyn
    torch.cuda.empty_cache()
    # beyond the five configurations: schedules at rack scale (64 ranks = 4 racks of 16; 128 ranks = 8 racks)
    def sched(name, plan, send, recv, iters):
        wl = wk._bind(name, plan, send, recv, {})
        ms = wk.time_back_to_back(wl, iters, 3)
        i = wl.info
        out[name] = {"ms": float(ms), "chain_depth": int(i.chain_depth), "tiles": int(i.n_tiles), "dispatch": "static chains" if i.static_chains else "tickets",
                     "schedule_bytes": int(i.schedule_bytes),
                     "compulsory_bytes": int(i.compulsory_bytes), "crossrack_bytes_racks_of_16": int(i.crossrack_bytes),
                     "compulsory_gbs": i.compulsory_bytes / ms / 1e6}
    for n in ((1 << 16, 1 << 22) if quick else (1 << 16, 1 << 22, 1 << 25)):
        send = [torch.randn(n, device="cuda").to(torch.bfloat16) for _ in range(64)]
        recv = [torch.empty(n, dtype=torch.bfloat16, device="cuda") for _ in range(64)]
        for algo, nm in ((hb.ALGO_RING, "ring"), (hb.ALGO_RING_2LEVEL, "ring_2level"), (hb.ALGO_TREE, "tree"), (hb.ALGO_RING_FUSED, "ring_fused"), (hb.ALGO_FANOUT, "fanout")):
            sched("next_allreduce_r64_bf16_%d_%s" % (n, nm), hb.hccl_plan_allreduce(64, n, hb.BF16, algo, dict(rack_size=16)), send, recv, 20)
        del send, recv
        torch.cuda.empty_cache()
    for n in ((1 << 12, 1 << 18) if quick else (1 << 12, 1 << 18, 1 << 21)):
        send = [torch.randn(n, device="cuda").to(torch.bfloat16) for _ in range(128)]
        recv = [torch.empty(n * 128, dtype=torch.bfloat16, device="cuda") for _ in range(128)]
        for algo, nm in ((hb.ALGO_RING, "ring"), (hb.ALGO_RING_2LEVEL, "ring_2level"), (hb.ALGO_ONESHOT, "oneshot"), (hb.ALGO_FANOUT, "fanout")):
            sched("next_allgather_r128_bf16_%d_%s" % (n, nm), hb.hccl_plan_allgather(128, None, n, hb.BF16, algo, dict(rack_size=16)), send, recv, 10)
        del send, recv
        torch.cuda.empty_cache()
    for algo, nm in ((hb.ALGO_RING, "ring"), (hb.ALGO_RING_FUSED, "ring_fused")):
        wl = wk.config3(algo=algo)
        ms = wk.time_back_to_back(wl, 10 if quick else 50, 5)
        i = wl.info
        out["3_reducescatter_r16_bf16_64Mi_" + nm] = {
            "ms": float(ms), "schedule_bytes": int(i.schedule_bytes), "compulsory_bytes": int(i.compulsory_bytes),
            "schedule_gbs": i.schedule_bytes / ms / 1e6, "compulsory_gbs": i.compulsory_bytes / ms / 1e6,
            "tiles": int(i.n_tiles), "inputs": "2 GiB, larger than L2"}
        if algo == hb.ALGO_RING and not quick:
            # the oracle's ReduceScatter on the same 16 x 64 Mi bf16 inputs, single thread, host memory
            Xh = [t.view(torch.int16).cpu().numpy().view(np.uint16) for t in wl.send]
            rc = np.full(16, Xh[0].size // 16, dtype=np.int64)
            t0 = _t.perf_counter()
            want = orc.reducescatter(hb.BF16, Xh, rc)
            out["3_reducescatter_r16_bf16_64Mi_" + nm]["cpu_oracle_ms"] = (_t.perf_counter() - t0) * 1e3
            # outputs of the timed plan further than 1 ulp from the rounded FP64 sum: counted and reported
            beyond = 0
            for r in range(16):
                got = wl.recv[r].view(torch.int16).cpu().numpy().view(np.uint16)
                beyond += int((orc.ulp_distance(hb.BF16, got, want[r]) > 1).sum())
            out["3_reducescatter_r16_bf16_64Mi_" + nm]["beyond_1ulp_of_fp64_sum"] = beyond
            out["3_reducescatter_r16_bf16_64Mi_" + nm]["outputs"] = int(Xh[0].size)
            del Xh, want
        del wl
        torch.cuda.empty_cache()
    return out


def run_profile_case(args):
    """A small, single-kernel case for ncu captures (few launches, a few hundred MB on the device):
    config 3's shape at 1/8 of its size (R = 16, 8 Mi bf16 per rank, 2 MiB granules)."""
    import torch
    from paper_2608_00358_b200 import binding as hb
    from paper_2608_00358_b200 import workloads as wk
    if args.profile_case == "latency":
        # the small, latency-bound configurations: one JSON line each (see workloads.latency_breakdown)
        cases = [("1 allreduce ring r4 fp32 1Mi", lambda: wk.config1()), ("2 alltoallv r8 bf16 dim128", lambda: wk.config2())]
        for m in (4096, 65536, 262144, 1 << 20):
            cases.append(("5 allreduce r8 bf16 %d B one-shot" % m, lambda m=m: wk.config5(m, hb.ALGO_ONESHOT)))
            cases.append(("5 allreduce r8 bf16 %d B ring" % m, lambda m=m: wk.config5(m, hb.ALGO_RING)))
        for name, make in cases:
            wl = make()
            print(json.dumps(_round(_finite(dict(case=name, **wk.latency_breakdown(wl))), 2)), flush=True)
            del wl
        wl = wk.config5(4096, hb.ALGO_ONESHOT)
        print(json.dumps(_round(_finite(dict(case="5 allreduce r8 bf16 4096 B one-shot, as the host sees it", **wk.time_host_observed(wl, 300))), 2)), flush=True)
        return
    if args.profile_case in ("c1chains", "c1tickets"):
        # config 1 (AllReduce ring R = 4, 1 Mi fp32 per rank) on the register engine: static chains vs tickets and device counters
        wl = wk.config1(dict(engine=hb.ENGINE_LSU, flags=0 if args.profile_case == "c1chains" else hb.FLAG_DYNAMIC_TICKETS))
    elif args.profile_case in ("agfanout", "agoneshot"):
        # AllGather R = 32, 1 Mi bf16 (2 MiB) per rank: 64 MiB read, 2 GiB written
        R, n = 32, 1 << 20
        algo = hb.ALGO_FANOUT if args.profile_case == "agfanout" else hb.ALGO_ONESHOT
        send = [torch.randn(n, device="cuda").to(torch.bfloat16) for _ in range(R)]
        recv = [torch.empty(n * R, dtype=torch.bfloat16, device="cuda") for _ in range(R)]
        wl = wk._bind("allgather_r32_bf16_1Mi_" + args.profile_case[2:], hb.hccl_plan_allgather(R, None, n, hb.BF16, algo), send, recv, {})
    else:
        algo = {"c3ring": hb.ALGO_RING, "c3fused": hb.ALGO_RING_FUSED}[args.profile_case]
        wl = wk.config3(dict(chain_group=args.profile_chain_group) if args.profile_chain_group else None, algo=algo, n=args.profile_n)
    ms = wk.time_back_to_back(wl, args.steps, max(args.warmup, 3))
    i = wl.info
    print(json.dumps({"case": args.profile_case, "workload": wl.name, "ms": ms, "schedule_bytes": int(i.schedule_bytes),
                      "compulsory_bytes": int(i.compulsory_bytes), "schedule_gbs": i.schedule_bytes / ms / 1e6,
                      "compulsory_gbs": i.compulsory_bytes / ms / 1e6, "tiles": int(i.n_tiles)}), flush=True)


def interference_leg(args, wl):
    """The GEMM-interference trade-off at a few SM budgets (the full sweep is `python -m
    paper_2608_00358_b200.interference`); a budget is a number of thread blocks = SMs taken."""
    import torch
    from paper_2608_00358_b200 import binding as hb
    from paper_2608_00358_b200 import interference
    from paper_2608_00358_b200 import workloads as wk
    gemm = interference.Gemm()
    sweep = []
    for b in ([2, 148] if args.quick else [2, 4, 16, 64, 148]):
        plan = hb.hccl_plan_alltoallv(64, wl.meta["counts"], None, None, None, hb.FP16, 256, dict(sm_budget=b))
        w2 = wk._bind(wl.name, plan, wl.send, wl.recv, wl.meta)
        r = interference.measure(w2, seconds=2.0, gemm=gemm)
        sweep.append({"sm_budget": b, "gemm_slowdown": r.get("gemm_slowdown"), "gemm_alone_tflops": r["gemm_alone_tflops"],
                      "gemm_overlap_tflops": r["overlap"].get("gemm_tflops"), "collective_alone_gbs": r["collective_alone_gbs"],
                      "collective_overlap_gbs": r["overlap"].get("collective_gbs")})
        del w2, plan
    out = {"gemm": "bf16 8192^3 (cuBLAS via torch.matmul), back to back", "collective": wl.name,
           "protocol": "both loops kept 3 batches deep; rates taken inside the window where both run", "sweep": sweep}
    del gemm
    if not args.quick:
        # the same at budget 4 against a 16384^3 GEMM (55 waves of tiles instead of 14: losing one SM
        # slot costs a smaller share of a wave)
        torch.cuda.empty_cache()
        gemm = interference.Gemm(16384)
        plan = hb.hccl_plan_alltoallv(64, wl.meta["counts"], None, None, None, hb.FP16, 256, dict(sm_budget=4))
        w2 = wk._bind(wl.name, plan, wl.send, wl.recv, wl.meta)
        r = interference.measure(w2, seconds=2.5, gemm=gemm)
        out["gemm_16384_budget_4"] = {
            "gemm_slowdown": r.get("gemm_slowdown"), "gemm_alone_tflops": r["gemm_alone_tflops"],
            "gemm_overlap_tflops": r["overlap"].get("gemm_tflops"), "collective_overlap_gbs": r["overlap"].get("collective_gbs")}
        del w2, plan, gemm
    # the operating point: no SM is held against the GEMM. (1) interference.OVERLAP_OPTS: twelve persistent blocks of the
    # register engine's 64-register build, 128 threads each, small enough to run on SMs that GEMM blocks occupy.
    # (2) interference.IDLE_SM_OPTS: short-lived blocks on a stream of LOWER priority than the GEMM's, which take only
    # the SMs the GEMM leaves idle. Slowdowns are still taken against the unrestricted GEMM alone.
    torch.cuda.empty_cache()
    gemm = interference.Gemm()

    def point(opts, collective_first):
        plan = hb.hccl_plan_alltoallv(64, wl.meta["counts"], None, None, None, hb.FP16, 256, dict(opts))
        w2 = wk._bind(wl.name, plan, wl.send, wl.recv, wl.meta)
        r = interference.measure(w2, seconds=3.0, gemm=gemm, collective_first=collective_first)
        return {"opts": dict(opts), "gemm_slowdown": r.get("gemm_slowdown"), "gemm_alone_tflops": r["gemm_alone_tflops"],
                "gemm_overlap_tflops": r["overlap"].get("gemm_tflops"), "collective_alone_gbs": r["collective_alone_gbs"],
                "collective_overlap_gbs": r["overlap"].get("collective_gbs")}
    out["chosen"] = dict(point(interference.OVERLAP_OPTS, True), mode="%d co-resident blocks (register engine, 64 registers, 128 threads)" % interference.OVERLAP_OPTS["sm_budget"],
                         sm_budget=interference.OVERLAP_OPTS["sm_budget"])
    out["idle_sms"] = dict(point(interference.IDLE_SM_OPTS, False), mode="short-lived blocks, GEMM stream has priority")
    del gemm
    return out


def headline_of(line: dict) -> dict:
    """The compact record: the contract's keys, the roofline, both baselines and a few cross-references."""
    keep = ["metric", "value", "unit", "n_gpus", "steps", "warmup", "ms_per_step", "higher_is_better", "scaling", "vs_baseline",
            "dtype", "data", "gpu_launches", "clocks"]
    h = {k: line[k] for k in keep if k in line}
    c = line["config"]
    h["config"] = {k: c[k] for k in ("workload", "virtual_ranks", "payload_bytes", "sm_budget", "threads", "tile_bytes", "engine", "multi_gpu")}
    h["config"]["cache"] = "inputs > L2"
    r = line["roofline"]
    h["roofline"] = {k: r[k] for k in ("bound", "achieved", "peak", "unit", "frac", "traffic", "kernel", "algorithmic_bytes_per_launch", "launch_ms")}
    h["roofline"]["peak_source"] = r["peak_source"]
    h["roofline"]["traffic_from"] = "ncu cap-1024 case, scaled"
    e = line.get("e2e")
    if e:
        h["e2e"] = {k: e[k] for k in ("value", "unit", "h2d_bytes_per_step", "d2h_bytes_per_step", "ms_per_step", "gpu_launches_per_step",
                                      "checked_destinations_vs_oracle", "skipped", "ranks_measured") if k in e}
        if "api" in e:
            h["e2e"]["api"] = e["api"].split(" ")[0]
    if "cpu_baseline" in line:
        h["cpu_baseline"] = line["cpu_baseline"]
    i = line.get("interference")
    if i and "chosen" in i:
        h["interference"] = {k: i["chosen"][k] for k in ("mode", "sm_budget", "gemm_slowdown", "collective_overlap_gbs", "collective_alone_gbs")}
        h["interference"]["gemm"] = "bf16 8192^3"
        if "idle_sms" in i:
            h["interference"]["idle_sms_slowdown"] = i["idle_sms"]["gemm_slowdown"]
        pers = {str(p["sm_budget"]): p["gemm_slowdown"] for p in i.get("sweep", []) if p["sm_budget"] in (2, 16)}
        h["interference"]["persistent_budget_slowdown"] = pers
    cfg = line.get("configs") or {}
    side = {}
    for key, short, field in (("3_reducescatter_r16_bf16_64Mi_ring", "c3_ring_ms", "ms"), ("3_reducescatter_r16_bf16_64Mi_ring_fused", "c3_fused_ms", "ms"),
                              ("3_reducescatter_r16_bf16_64Mi_ring", "c3_beyond_1ulp", "beyond_1ulp_of_fp64_sum"),
                              ("3_reducescatter_r16_bf16_64Mi_ring", "c3_ring_compulsory_gbs", "compulsory_gbs"),
                              ("3_reducescatter_r16_bf16_64Mi_ring_fused", "c3_fused_compulsory_gbs", "compulsory_gbs"),
                              ("1_allreduce_ring_r4_fp32_1Mi", "c1_p50_us", "p50_us"), ("2_alltoallv_r8_bf16_dim128", "c2_p50_us", "p50_us"),
                              ("5_allreduce_r8_bf16_4096B_oneshot", "c5_4k_oneshot_p50_us", "p50_us"),
                              ("5_allreduce_r8_bf16_1048576B_oneshot", "c5_1m_oneshot_p50_us", "p50_us"),
                              ("5_allreduce_r8_bf16_4096B_ring", "c5_4k_ring_p50_us", "p50_us"),
                              ("5_allreduce_r8_bf16_1048576B_ring", "c5_1m_ring_p50_us", "p50_us"),
                              ("next_alltoallv_dynamic_r64_fp16_dim256", "dyn_r64_ms", "ms")):
        v = (cfg.get(key) or {}).get(field)
        if v is not None:
            side[short] = v
    ho = (cfg.get("5_allreduce_r8_bf16_4096B_oneshot") or {}).get("host_observed")
    if ho:
        side["c5_4k_resident_ring_wait_us"] = ho.get("ring_and_wait_us")
    if side:
        h["side"] = side
    h["detail"] = "previous stdout line"
    return h


def run_ours(args, rank: int, world: int, local_rank: int):
    import numpy as np
    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    from paper_2608_00358_b200 import binding as hb
    from paper_2608_00358_b200 import interference
    from paper_2608_00358_b200 import workloads as wk

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    opts = {}
    if args.sm_budget:
        opts["sm_budget"] = args.sm_budget
    if args.engine:
        opts["engine"] = {"lsu": 1, "bulk": 2}[args.engine]
    opts = opts or None
    cap_used = args.cap
    try:
        wl = wk.config4(opts, seed=0, cap=cap_used)
    except torch.cuda.OutOfMemoryError:
        # the named configuration needs 51.6 GB on the device; on a GPU that cannot give that much the clamp is
        # lowered to 8192 rows (about 14.6 GB resident) and the line says so
        torch.cuda.empty_cache()
        cap_used = min(args.cap, 8192)
        wl = wk.config4(opts, seed=0, cap=cap_used)
    info = wl.info
    payload = wl.meta["payload_bytes"]
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(physical_gpu_index(local_rank))

    # ---- device-resident timing: W warm-ups, then exactly K steps, one kernel launch each
    for _ in range(max(args.warmup, 3)):
        wl.dc.execute(stream)
    barrier()
    sampler.start()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    evs[0].record(stream)
    for k in range(args.steps):
        wl.dc.execute(stream)
        evs[k + 1].record(stream)
    barrier()
    clocks = sampler.stop()
    wl.dc.check()
    total_ms = evs[0].elapsed_time(evs[-1])
    per_launch = np.array([evs[k].elapsed_time(evs[k + 1]) for k in range(args.steps)])
    from paper_2608_00358_b200 import multi
    value, total_ms_max = multi.replica_throughput_gbs(total_ms, info.schedule_bytes, args.steps, dist, "cuda")

    # ---- end to end through host buffers (rank-local; reported by rank 0)
    e2e = None
    if rank == 0 and not args.no_e2e:
        import psutil
        need = 2 * payload + (8 << 30)
        if psutil.virtual_memory().available > need:
            hs = [torch.empty(t_.numel(), dtype=t_.dtype, pin_memory=True) for t_ in wl.send]
            hr = [torch.empty(t_.numel(), dtype=t_.dtype, pin_memory=True) for t_ in wl.recv]
            for h, d_ in zip(hs, wl.send):
                h.copy_(d_)
            torch.cuda.synchronize()
            hp = ([h.data_ptr() for h in hs], [h.data_ptr() for h in hr])
            dp = ([d_.data_ptr() for d_ in wl.send], [d_.data_ptr() for d_ in wl.recv])
            ksteps = args.e2e_steps
            # (a) one stream: copy everything in, exchange, copy everything out
            wl.plan.execute_host(hp[0], hp[1], dp[0], dp[1], stream.cuda_stream)   # warm-up
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(ksteps):
                wl.plan.execute_host(hp[0], hp[1], dp[0], dp[1], stream.cuda_stream)
            e1.record(stream)
            torch.cuda.synchronize()
            wl.dc.check()
            serial_ms = e0.elapsed_time(e1) / ksteps
            # (b) pipelined by destination windows on three streams: both directions of the host link busy at once
            pipe = hb.hccl_hostpipe_alltoallv_create(64, wl.meta["counts"], hb.FP16, 256, args.e2e_windows, opts)
            pws = torch.empty(pipe.workspace_bytes() + 256, dtype=torch.uint8, device="cuda")
            pipe.bind((pws.data_ptr() + 255) // 256 * 256, pipe.workspace_bytes(), stream.cuda_stream)
            s_in, s_ex, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
            for h in hr:
                h.zero_()
            torch.cuda.synchronize()
            pipe.execute(hp[0], hp[1], dp[0], dp[1], s_in.cuda_stream, s_ex.cuda_stream, s_out.cuda_stream)   # warm-up
            torch.cuda.synchronize()
            e0.record(s_in)
            for _ in range(ksteps):
                pipe.execute(hp[0], hp[1], dp[0], dp[1], s_in.cuda_stream, s_ex.cuda_stream, s_out.cuda_stream)
            e1.record(s_out)
            torch.cuda.synchronize()
            pst, pdetail = pipe.status()
            if pst != hb.OK:
                raise hb.HcclError(pst, "hccl_hostpipe_status (detail %d)" % pdetail)
            # outside the timed region: what came back to the host, for every destination rank, against the CPU
            # oracle's AllToAllv of the same host send buffers (one destination at a time: <= 0.6 GB extra)
            e2e_checked = check_host_result_against_oracle(wl.meta["counts"], 512, hs, hr)
            ms = e0.elapsed_time(e1) / ksteps
            e2e = {"value": info.schedule_bytes / ms / 1e6, "unit": UNIT, "h2d_bytes_per_step": int(payload),
                   "d2h_bytes_per_step": int(payload), "ms_per_step": ms, "steps": ksteps,
                   "api": "hccl_hostpipe_execute (pinned host buffers -> device -> pinned host buffers, %d destination windows on 3 streams)" % (len(pipe.windows()) - 1),
                   "gpu_launches_per_step": len(pipe.windows()) - 1, "checked_destinations_vs_oracle": e2e_checked,
                   "single_stream": {"value": info.schedule_bytes / serial_ms / 1e6, "ms_per_step": serial_ms, "api": "hccl_execute_host"}}
            # the host link by itself, with the same pinned buffers: each direction alone, then both at once
            def _link(h2d, d2h, reps=2):
                torch.cuda.synchronize()
                a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a0.record(stream)
                s_in.wait_event(a0)
                s_out.wait_event(a0)
                nb = 0
                for _ in range(reps):
                    for k in range(16):
                        if h2d:
                            with torch.cuda.stream(s_in):
                                wl.send[k].copy_(hs[k], non_blocking=True)
                            nb += hs[k].numel() * 2
                        if d2h:
                            with torch.cuda.stream(s_out):
                                hr[k].copy_(wl.recv[k], non_blocking=True)
                stream.wait_stream(s_in)
                stream.wait_stream(s_out)
                a1.record(stream)
                torch.cuda.synchronize()
                one_way = nb if h2d else reps * sum(hr[k].numel() * 2 for k in range(16))
                return one_way / a0.elapsed_time(a1) / 1e6
            e2e["host_link_gbs"] = {"h2d_alone": _link(True, False), "d2h_alone": _link(False, True), "h2d_while_d2h_runs": _link(True, True),
                                    "note": "plain pinned copies of 16 of the 64 rank buffers; the pipelined path needs both directions at once"}
            if world > 1:   # the other ranks idle meanwhile: this is one replica's end-to-end rate, not the job's
                e2e["ranks_measured"] = 1
            del pipe, pws
            del hs, hr
        else:
            e2e = {"value": None, "unit": UNIT, "skipped": "host memory too small to pin 2 x %.1f GB" % (payload / 1e9)}

    line = None
    if rank == 0:
        peak, which = peaks()
        launch_ms = float(per_launch.mean())
        achieved = info.schedule_bytes / launch_ms / 1e6
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
            "ms_per_step": total_ms_max / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "u8", "data": "synthetic",
            "config": {"workload": wl.name, "virtual_ranks": 64, "row_bytes": 512, "rows_moved": int(wl.meta["counts"].sum()),
                       "payload_bytes": int(payload), "resident_bytes": int(2 * payload), "sm_budget": int(info.sm_budget),
                       "threads": int(info.threads), "tile_bytes": int(info.tile_bytes), "tiles": int(info.n_tiles),
                       "engine": {1: "lsu", 2: "bulk"}.get(int(info.engine), str(info.engine)),
                       "cache": "inputs larger than L2 (no flush needed)", "multi_gpu": "replicas only",
                       "zipf_clamp_rows": int(cap_used)},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "peak_source": which + " copy bandwidth (burst)", "kernel": "hccl_executor_bulk" if int(info.engine) == 2 else "hccl_executor_lsu",
                         "algorithmic_bytes_per_launch": int(info.schedule_bytes), "launch_ms": launch_ms,
                         "traffic": (DRAM_BYTES_PER_ALGORITHMIC_BYTE * info.schedule_bytes) if DRAM_BYTES_PER_ALGORITHMIC_BYTE else None,
                         "traffic_note": "dram bytes per algorithmic byte (%.3f) from the ncu capture of the cap-1024 case of this workload, scaled by the bytes of this launch" % DRAM_BYTES_PER_ALGORITHMIC_BYTE,
                         "frac_of_nominal_8TBs": achieved / 8000.0},
            "gpu_launches": args.steps, "clocks": clocks, "e2e": e2e,
        }

    # ---- interference, other configs, CPU baseline: rank 0 at N = 1 only
    if rank == 0 and world == 1:
        if not args.no_gemm:
            line["interference"] = interference_leg(args, wl)
        dyn64 = None
        if not args.no_side:
            # device-resident AllToAllv at the benchmark's size: the same counts, read from device memory by the kernel
            Cd = wl.meta["counts"]
            dyn = hb.hccl_plan_alltoallv_dynamic(64, Cd.sum(axis=1), Cd.sum(axis=0), hb.FP16, 256)
            counts_dev = torch.from_numpy(np.ascontiguousarray(Cd.reshape(-1))).cuda()
            dyn.set_dynamic_metadata(counts_dev.data_ptr())
            wd = wk._bind("alltoallv_dynamic_r64", dyn, wl.send, wl.recv, {})
            msd = wk.time_back_to_back(wd, 5, 2)
            dyn64 = {"ms": float(msd), "gbs": info.schedule_bytes / msd / 1e6, "statically_planned_ms": total_ms_max / args.steps,
                     "form": "tables built on the device + the ordinary executor" if int(dyn.info().n_wqe) else "one kernel",
                     "note": "counts read from device memory at run time; same payload as the benchmark step"}
            del wd, dyn
        del wl
        torch.cuda.empty_cache()
        if not args.no_side:
            line["configs"] = side_configs(args.quick)
            line["configs"]["next_alltoallv_dynamic_r64_fp16_dim256"] = dyn64
        if not args.no_cpu:
            from paper_2608_00358_b200 import synth
            C = synth.zipf_counts(64, 0, 1.1, cap_used)
            dst = list(range(args.oracle_dst))
            moved, times = oracle_alltoallv_sample(C, 512, dst, repeat=2)
            line["cpu_baseline"] = {"value": 2 * moved / min(times) / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": "destination ranks 0..%d of 64 (%.2f GB moved), best of 2" % (args.oracle_dst - 1, moved / 1e9),
                                    "host_cores_available": os.cpu_count()}
    if rank == 0:
        emit(line, headline_of(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cap", type=int, default=32768, help="clamp of the Zipf row counts (32768 = the named config)")
    ap.add_argument("--sm-budget", type=int, default=0)
    ap.add_argument("--engine", default="", choices=["", "lsu", "bulk"], help="force an executor engine (default: the library's choice)")
    ap.add_argument("--oracle-dst", type=int, default=8, help="destination ranks in the CPU oracle's sample")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--e2e-windows", type=int, default=16, help="destination windows of the pipelined end-to-end path")
    ap.add_argument("--quick", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-gemm", action="store_true")
    ap.add_argument("--no-side", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--profile-n", type=int, default=1 << 23, help="elements per rank of the --profile-case")
    ap.add_argument("--profile-chain-group", type=int, default=0, help="opts.chain_group of the c3ring / c3fused --profile-case (0 = default)")
    ap.add_argument("--profile-case", default="", choices=["", "c3ring", "c3fused", "agfanout", "agoneshot", "c1chains", "c1tickets", "latency"],
                    help="run only a small single-kernel case (for ncu captures), not the benchmark")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.profile_case:
        run_profile_case(args)
        return
    run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
