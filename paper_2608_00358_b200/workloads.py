"""The five benchmark configurations, built on the device: seeded synthetic inputs, plans, bound executors.

Shapes follow the paper's description of its workloads (large AllToAllv of embedding rows with skewed
per-peer splits and gradient AllReduce/ReduceScatter in training, Sec. I and V-A; rack of 16 and jobs of
64 ranks, Sec. V-D; small latency-bound AllReduce for inference, Sec. IV-B and V-F). The production
traces and the PARAM suite the paper measured with are not available; these inputs stand in for them.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch

from . import binding as hb
from . import synth
from .runtime import DeviceCollective


@dataclass
class Workload:
    name: str
    plan: hb.Plan
    dc: DeviceCollective
    send: List[torch.Tensor]
    recv: List[torch.Tensor]
    meta: dict = field(default_factory=dict)

    @property
    def info(self):
        return self.plan.info()


def _bind(name, plan, send, recv, meta=None, stream=None) -> Workload:
    dc = DeviceCollective(plan, stream=stream)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv], keep=(send, recv))
    return Workload(name, plan, dc, send, recv, meta or {})


def config1(opts=None, seed=0) -> Workload:
    """AllReduce ring, R=4, 1 Mi fp32 per rank, uniform(-1,1)."""
    R, n = 4, 1 << 20
    X = synth.uniform_ranks(R, n, hb.FP32, seed)
    send = [torch.from_numpy(x).cuda() for x in X]
    recv = [torch.zeros(n, dtype=torch.float32, device="cuda") for _ in range(R)]
    plan = hb.hccl_plan_allreduce(R, n, hb.FP32, hb.ALGO_RING, opts)
    return _bind("allreduce_ring_r4_fp32_1Mi", plan, send, recv, dict(host_inputs=X, dt=hb.FP32, n=n, R=R))


def config2(opts=None, seed=0) -> Workload:
    """AllToAllv, R=8, rows of 128 bf16 ~ N(0,1), counts uniform in [0, 4096], packed."""
    R, row = 8, 128
    C = synth.uniform_counts(R, seed, hi=4096)
    X = [synth.normal_ranks(1, int(C[s].sum()) * row, hb.BF16, seed=1000 + s)[0] for s in range(R)]
    send = [torch.from_numpy(x.view(np.int16)).cuda() for x in X]
    recv = [torch.zeros(max(int(C[:, d].sum()) * row, 8), dtype=torch.int16, device="cuda") for d in range(R)]
    plan = hb.hccl_plan_alltoallv(R, C, None, None, None, hb.BF16, row, opts)
    return _bind("alltoallv_r8_bf16_dim128", plan, send, recv, dict(host_inputs=X, counts=C, row_elems=row, dt=hb.BF16, R=R))


def config3(opts=None, seed=0, n: int = 1 << 26, algo=hb.ALGO_RING) -> Workload:
    """ReduceScatter ring, R=16, n bf16 per rank ~ N(0, 0.02), fp32 partials, 2 MiB granules."""
    R = 16
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    send = []
    for _ in range(R):
        x = torch.empty(n, dtype=torch.float32, device="cuda")
        x.normal_(0.0, 0.02, generator=g)
        send.append(x.to(torch.bfloat16))
        del x
    recv = [torch.zeros(n // R, dtype=torch.bfloat16, device="cuda") for _ in range(R)]
    plan = hb.hccl_plan_reducescatter(R, None, n, hb.BF16, algo, opts)
    return _bind("reducescatter_ring_r16_bf16_%dMi" % (n >> 20), plan, send, recv, dict(dt=hb.BF16, n=n, R=R))


def config4(opts=None, seed=0, cap: int = 32768, R: int = 64, row: int = 256) -> Workload:
    """AllToAllv, R=64, rows of 256 fp16, counts Zipf(1.1) clamped at `cap`; payload regenerable row by row."""
    C = synth.zipf_counts(R, seed, s=1.1, cap=cap)
    send_rows = C.sum(axis=1)
    recv_rows = C.sum(axis=0)
    send = []
    for s in range(R):
        t = torch.empty(int(send_rows[s]) * row, dtype=torch.int16, device="cuda")
        synth.fill_hashed_rows_torch(t, s, row)
        send.append(t)
    recv = [torch.zeros(int(recv_rows[d]) * row, dtype=torch.int16, device="cuda") for d in range(R)]
    plan = hb.hccl_plan_alltoallv(R, C, None, None, None, hb.FP16, row, opts)
    payload = int(C.sum()) * row * 2
    return _bind("alltoallv_r64_fp16_dim256_zipf1.1_cap%d" % cap, plan, send, recv,
                 dict(counts=C, row_elems=row, dt=hb.FP16, R=R, payload_bytes=payload, seed=seed))


def config5(m_bytes: int, algo: int, opts=None, seed=0) -> Workload:
    """AllReduce, R=8, bf16 messages of m_bytes per rank ~ N(0,1), one-shot, ring or one of the fused forms."""
    R, n = 8, m_bytes // 2
    X = synth.normal_ranks(R, n, hb.BF16, seed=seed + m_bytes)
    send = [torch.from_numpy(x.view(np.int16)).cuda() for x in X]
    recv = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    plan = hb.hccl_plan_allreduce(R, n, hb.BF16, algo, opts)
    name = "allreduce_%s_r8_bf16_%dB" % ({hb.ALGO_RING: "ring", hb.ALGO_ONESHOT: "oneshot", hb.ALGO_RING_FUSED: "ringfused", hb.ALGO_FANOUT: "fanout", hb.ALGO_TREE: "tree"}[algo], m_bytes)
    return _bind(name, plan, send, recv, dict(host_inputs=X, dt=hb.BF16, n=n, R=R))


def time_back_to_back(wl: Workload, iters: int, warmup: int, stream: Optional[torch.cuda.Stream] = None) -> float:
    """Mean milliseconds per execution, enqueued back to back, CUDA events on the launching stream."""
    s = stream or torch.cuda.current_stream()
    with torch.cuda.stream(s):
        for _ in range(warmup):
            wl.dc.execute(s)
        s.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(s)
        for _ in range(iters):
            wl.dc.execute(s)
        e1.record(s)
        s.synchronize()
    wl.dc.check()
    return e0.elapsed_time(e1) / iters


def time_each(wl: Workload, iters: int, warmup: int, flush: Optional[torch.Tensor] = None) -> np.ndarray:
    """Per-execution milliseconds from one event pair per iteration (for percentiles). With `flush`, a buffer
    larger than the L2 is rewritten before every iteration so that each one starts cold."""
    s = torch.cuda.current_stream()
    for _ in range(warmup):
        wl.dc.execute(s)
    s.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
    for a, b in ev:
        if flush is not None:
            flush.add_(1)
        a.record(s)
        wl.dc.execute(s)
        b.record(s)
    s.synchronize()
    wl.dc.check()
    return np.array([a.elapsed_time(b) for a, b in ev])


def time_graph_replay(wl: Workload, per_graph: int = 50, replays: int = 10) -> float:
    """Mean milliseconds per execution when `per_graph` executions are captured in one CUDA graph and the
    graph is replayed: what is left when the per-launch host cost is taken out."""
    s = torch.cuda.Stream()
    wl.dc.execute(s)
    s.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        for _ in range(per_graph):
            wl.dc.execute(s)
    g.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        g.replay()
    e1.record()
    torch.cuda.synchronize()
    wl.dc.check()
    return e0.elapsed_time(e1) / (replays * per_graph)


def time_host_observed(wl: Workload, iters: int = 200) -> dict:
    """Wall-clock microseconds per collective as the host sees it, two ways: a launch followed by a stream
    synchronisation, and a ring + wait on the resident executor (kernel launched once, no CUDA call per
    collective). Register engine only."""
    import time
    s = torch.cuda.Stream()
    for _ in range(10):
        wl.dc.execute(s)
    s.synchronize()
    t0 = time.perf_counter()
    for _ in range(iters):
        wl.dc.execute(s)
        s.synchronize()
    launch_us = (time.perf_counter() - t0) / iters * 1e6
    bell = torch.zeros(8, dtype=torch.int64).pin_memory()
    wl.plan.server_start([t.data_ptr() for t in wl.send], [t.data_ptr() for t in wl.recv], bell.data_ptr(), 200_000_000, s.cuda_stream)
    try:
        for _ in range(10):
            wl.plan.server_ring()
            wl.plan.server_wait(2_000_000_000)
        t0 = time.perf_counter()
        for _ in range(iters):
            wl.plan.server_ring()
            rc = wl.plan.server_wait(2_000_000_000)
        ring_us = (time.perf_counter() - t0) / iters * 1e6
        on_device_us = (int(bell[7]) - int(bell[6])) / 1e3      # last execution: ring seen -> last block out, device clock
    finally:
        wl.plan.server_stop()
        s.synchronize()
    if rc != hb.OK:
        raise hb.HcclError(rc, "hccl_server_wait")
    return {"launch_and_sync_us": launch_us, "ring_and_wait_us": ring_us, "ring_seen_to_done_on_device_us": on_device_us}


def latency_breakdown(wl: Workload, iters: int = 1000, warmup: int = 100, traced_runs: int = 20) -> dict:
    """Where the microseconds of one execution go (the nesting T(engine) within T(control core) within T(event) that
    the paper uses to attribute its overheads, Sec. V-C): event-pair p50, back-to-back and graph-replay time per
    execution without tracing; then, from the per-item trace and the control block of the fastest of
    `traced_runs` traced executions, the span from the first claim to the last block's exit, its parts, and
    what is left of the event-pair time outside the kernel's own span (launch, kernel start, event records)."""
    from .runtime import enable_trace
    ms = time_each(wl, iters, warmup)
    out = {"p50_event_us": float(np.percentile(ms, 50) * 1e3), "back_to_back_us": float(time_back_to_back(wl, iters, warmup) * 1e3),
           "graph_replay_us": float(time_graph_replay(wl) * 1e3)}
    tr = enable_trace(wl.plan)
    base = wl.dc._ws_ptr - wl.dc.workspace.data_ptr()
    best = None
    for _ in range(traced_runs):
        tr.zero_()
        torch.cuda.synchronize()
        wl.dc.execute()
        torch.cuda.synchronize()
        rows = tr.cpu().numpy()
        rows = rows[rows[:, 1] != 0]
        ctl = wl.dc.workspace[base:base + 48].cpu().numpy().view(np.uint64)   # control block: [5] = last exit (ns)
        claimed, released, stored, blk = rows[:, 1], rows[:, 2], rows[:, 3], rows[:, 0] >> 32
        first = int(claimed.min())
        depth = max(int((blk == b).sum()) for b in np.unique(blk))
        d = {"in_kernel_span_us": (int(ctl[5]) - first) / 1e3,
             "first_item_records_and_dependencies_us": (int(released[np.argmin(claimed)]) - first) / 1e3,
             "first_claim_to_last_store_us": (int(stored.max()) - first) / 1e3,
             "last_store_to_last_exit_us": (int(ctl[5]) - int(stored.max())) / 1e3,
             "item_data_movement_median_us": float(np.median(stored - released)) / 1e3,
             "items": int(rows.shape[0]), "blocks": int(np.unique(blk).size), "items_in_a_row_per_block": depth}
        d["per_item_in_a_row_us"] = d["first_claim_to_last_store_us"] / depth
        if best is None or d["in_kernel_span_us"] < best["in_kernel_span_us"]:
            best = d
    wl.plan.set_trace(0, 0)
    out.update(best)
    out["outside_the_kernel_span_us"] = out["p50_event_us"] - out["in_kernel_span_us"]
    return out
