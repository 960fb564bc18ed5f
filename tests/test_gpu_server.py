"""Resident, doorbell-fed executor: the kernel is launched once, every collective after that is a store into
a pinned host record. Every test stops the server and waits for the kernel to leave, also on failure; the
kernel would leave by itself after its idle bound anyway."""
import time

import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

pytestmark = pytest.mark.gpu


def _setup(plan, X, R, nbytes_out):
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    send = [torch.from_numpy(np.ascontiguousarray(x).view(np.uint8).reshape(-1).copy()).cuda() for x in X]
    recv = [torch.zeros(nbytes_out, dtype=torch.uint8, device="cuda") for _ in range(R)]
    dc = DeviceCollective(plan)                    # binds the workspace
    bell = torch.zeros(8, dtype=torch.int64).pin_memory()
    return send, recv, dc, bell


@pytest.mark.parametrize("algo", [hb.ALGO_ONESHOT, hb.ALGO_RING])
def test_server_executes_once_per_ring(algo):
    import torch
    R, n, dt = 8, 2048, hb.BF16
    plan = hb.hccl_plan_allreduce(R, n, dt, algo, dict(engine=hb.ENGINE_LSU, sm_budget=16))
    X = synth.normal_ranks(R, n, dt, seed=1)
    send, recv, dc, bell = _setup(plan, X, R, n * 2)
    srv, side = torch.cuda.Stream(), torch.cuda.Stream()
    plan.server_start([t.data_ptr() for t in send], [t.data_ptr() for t in recv], bell.data_ptr(), 300_000_000, srv.cuda_stream)
    try:
        for it in range(4):
            X = synth.normal_ranks(R, n, dt, seed=10 + it)
            with torch.cuda.stream(side):
                for t, x in zip(send, X):
                    t.copy_(torch.from_numpy(x.view(np.uint8)), non_blocking=False)
                for t in recv:
                    t.zero_()
            side.synchronize()
            assert plan.server_ring() == hb.OK
            assert plan.server_wait(2_000_000_000) == hb.OK
            want = orc.allreduce_oneshot_f32(dt, X) if algo == hb.ALGO_ONESHOT else orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
            with torch.cuda.stream(side):
                got = [t.cpu().numpy().view(np.uint16) for t in recv]
            for r in range(R):
                assert np.array_equal(got[r], want[r]), (it, r)
        # host-observed latency of ring + wait, back to back
        t0 = time.perf_counter()
        for _ in range(200):
            plan.server_ring()
            assert plan.server_wait(2_000_000_000) == hb.OK
        print("resident executor, %s R=8 4 KiB: %.2f us per ring+wait (host clock)" % ("one-shot" if algo == hb.ALGO_ONESHOT else "ring", (time.perf_counter() - t0) / 200 * 1e6))
    finally:
        plan.server_stop()
        srv.synchronize()
    assert int(bell[3]) == 1                        # left because it was told to
    st, done = plan.status()
    assert st == hb.OK and done == 204


def test_server_leaves_by_itself_when_idle():
    import torch
    R, n, dt = 4, 1024, hb.FP32
    plan = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_ONESHOT, dict(engine=hb.ENGINE_LSU, sm_budget=4))
    X = synth.normal_ranks(R, n, dt, seed=2)
    send, recv, dc, bell = _setup(plan, X, R, n * 4)
    srv = torch.cuda.Stream()
    plan.server_start([t.data_ptr() for t in send], [t.data_ptr() for t in recv], bell.data_ptr(), 50_000_000, srv.cuda_stream)
    try:
        assert plan.server_ring() == hb.OK and plan.server_wait(2_000_000_000) == hb.OK
        time.sleep(0.3)                             # longer than the idle bound
        srv.synchronize()                           # returns: the kernel has already left
        assert int(bell[3]) == 2
        assert plan.server_ring() == hb.ERR_TIMEOUT
    finally:
        plan.server_stop()
        srv.synchronize()
    # and it can be started again on the same bound plan
    bell.zero_()
    plan.server_start([t.data_ptr() for t in send], [t.data_ptr() for t in recv], bell.data_ptr(), 200_000_000, srv.cuda_stream)
    try:
        assert plan.server_ring() == hb.OK and plan.server_wait(2_000_000_000) == hb.OK
    finally:
        plan.server_stop()
        srv.synchronize()
    want = orc.allreduce_oneshot_f32(dt, X)
    assert np.array_equal(recv[0].cpu().numpy().view(np.float32), want[0])


def test_server_refuses_more_blocks_than_fit():
    import torch
    R, n = 2, 1 << 20
    plan = hb.hccl_plan_allreduce(R, n, hb.FP32, hb.ALGO_ONESHOT, dict(engine=hb.ENGINE_LSU, sm_budget=400, tile_bytes=4096))
    X = synth.normal_ranks(R, n, hb.FP32, seed=3)
    send, recv, dc, bell = _setup(plan, X, R, n * 4)
    with pytest.raises(hb.HcclError) as e:
        plan.server_start([t.data_ptr() for t in send], [t.data_ptr() for t in recv], bell.data_ptr(), 50_000_000, 0)
    assert e.value.status == hb.ERR_INVALID_ARG


def test_server_reports_a_failed_execution_and_leaves():
    """A WAIT that nothing satisfies, bounded at 0.1 s: the ring is accepted, the wait returns the device's verdict
    (never HCCL_OK), the completion count is not advanced, the kernel leaves by itself and the GPU stays usable."""
    import torch
    N = 1024
    g = hb.Graph(2, [N * 4, N * 4], [N * 4, N * 4], n_signals=1)
    a = g.add_subgraph(0)
    g.add_wqe(a, hb.OP_COPY, dst=(hb.BUF_RECV, 0, 0), a=(hb.BUF_SEND, 0, 0), count=N * 4)
    g.add_wqe(a, hb.OP_WAIT, a=(hb.BUF_SIGNAL, 0, 0), cmp=hb.CMP_GE, value=5, dep_flags=hb.DEP_FENCE)
    g.add_wqe(a, hb.OP_COPY, dst=(hb.BUF_RECV, 1, 0), a=(hb.BUF_SEND, 1, 0), count=N * 4)
    plan = g.compile(dict(engine=hb.ENGINE_LSU, sm_budget=2, timeout_ns=100_000_000))
    X = [np.arange(N, dtype=np.float32) + r for r in range(2)]
    send, recv, dc, bell = _setup(plan, X, 2, N * 4)
    srv = torch.cuda.Stream()
    plan.server_start([t.data_ptr() for t in send], [t.data_ptr() for t in recv], bell.data_ptr(), 500_000_000, srv.cuda_stream)
    try:
        assert plan.server_ring() == hb.OK
        assert plan.server_wait(3_000_000_000) == hb.ERR_TIMEOUT
        srv.synchronize()                           # the kernel has left after the failed execution
        assert int(bell[3]) == 3 and int(bell[1]) == 0 and int(bell[4]) == hb.ERR_TIMEOUT
        assert plan.server_ring() == hb.ERR_TIMEOUT     # the verdict again: nothing is served any more
    finally:
        plan.server_stop()
        srv.synchronize()
    assert bool((recv[1] == 0).all())              # what was fenced behind the WAIT never ran
    assert float(torch.ones(8, device="cuda").sum()) == 8.0
