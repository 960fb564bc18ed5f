"""hccl_execute inside a CUDA graph: the launch is captured once and replayed; because the executor takes its
execution number from the device-side control block, dependency counters and epoch-relative signal values
stay consistent across replays (cached re-enqueue, paper Sec. V-B, taken one step further)."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("engine", [hb.ENGINE_LSU, hb.ENGINE_BULK], ids=["lsu", "bulk"])
def test_ring_allreduce_replayed_from_a_cuda_graph(engine):
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    R, n, dt = 6, 70001, hb.BF16
    plan = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(engine=engine, sm_budget=24, tile_bytes=8192, chunk_bytes=32768))
    send = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    recv = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    s = torch.cuda.Stream()
    dc.execute(s)                         # one plain execution first (epoch 1)
    s.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        dc.execute(s)                     # captured twice: two executions per replay
        dc.execute(s)
    for it in range(4):
        X = synth.normal_ranks(R, n, dt, seed=100 + it)
        for t, x in zip(send, X):
            t.copy_(torch.from_numpy(x.view(np.int16)))
        for t in recv:
            t.zero_()
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        st, done = plan.status()
        assert st == hb.OK and done == 1 + 2 * (it + 1)          # the device counted every execution
        want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
        for r in range(R):
            assert np.array_equal(recv[r].cpu().numpy().view(np.uint16), want[r]), (it, r)


def test_graph_replay_latency_is_reported():
    """Not a performance assertion: replays of a captured one-shot AllReduce must simply work back to back."""
    import torch
    from paper_2608_00358_b200 import workloads as wk
    wl = wk.config5(4096, hb.ALGO_ONESHOT)
    s = torch.cuda.Stream()
    wl.dc.execute(s)
    s.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        for _ in range(10):
            wl.dc.execute(s)
    for _ in range(5):
        g.replay()
    torch.cuda.synchronize()
    wl.dc.check()
    X = wl.meta["host_inputs"]
    want = orc.allreduce_oneshot_f32(hb.BF16, X)
    for r in range(8):
        assert np.array_equal(wl.recv[r].cpu().numpy().view(np.uint16), want[r])


def test_device_resident_alltoallv_over_128_ranks_replayed_from_a_cuda_graph():
    """The device-resident AllToAllv with tables built on the device is two launches (table builder, executor); both
    are captured, and every replay reads the counts that are in device memory at that moment."""
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    R, row, hi = 128, 32, 6
    cap, rb = hi * R + 1, row * 2
    plan = hb.hccl_plan_alltoallv_dynamic(R, [cap] * R, [cap] * R, hb.BF16, row, dict(sm_budget=32, tile_bytes=2048))
    X = [synth.hashed_rows_np(s, 0, cap, row).reshape(-1).view(np.uint8) for s in range(R)]
    send = [torch.from_numpy(x.copy()).cuda() for x in X]
    recv = [torch.full((cap * rb,), 0x5A, dtype=torch.uint8, device="cuda") for _ in range(R)]
    counts = torch.zeros(R * R, dtype=torch.int64, device="cuda")
    plan.set_dynamic_metadata(counts.data_ptr())
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    s = torch.cuda.Stream()
    dc.execute(s)                         # with all counts zero: nothing moves
    s.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=s):
        dc.execute(s)
    for it in range(3):
        C = synth.uniform_counts(R, 40 + it, hi=hi)
        counts.copy_(torch.from_numpy(C.reshape(-1)))
        for t in recv:
            t.fill_(0x5A)
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        st, done = plan.status()
        assert st == hb.OK and done == 2 + it
        SD, RD = orc.packed_displs(C)
        want = [np.full(cap * rb, 0x5A, dtype=np.uint8) for _ in range(R)]
        orc.alltoallv(X, want, C, SD, RD, rb)
        for d in range(R):
            assert np.array_equal(recv[d].cpu().numpy(), want[d]), (it, d)
