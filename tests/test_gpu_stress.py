"""Repetition: the same bound plan executed hundreds of times back to back must give the same bits every time
(dependency counters are never reset between executions; publication and acquisition of completions are
only as strong as they need to be, so any ordering mistake shows up as a rare wrong element)."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

pytestmark = pytest.mark.gpu
VARIANTS = {"lsu": dict(engine=hb.ENGINE_LSU), "bulk": dict(engine=hb.ENGINE_BULK),
            "bulk_warpstore": dict(engine=hb.ENGINE_BULK, copy_by_warps=1), "lsu_light": dict(engine=hb.ENGINE_LSU, light=1, threads=256)}


@pytest.mark.parametrize("variant", sorted(VARIANTS))
@pytest.mark.parametrize("budget", [3, 37, 148])
def test_ring_allreduce_repeated(variant, budget):
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    R, n, dt = 8, 120007, hb.BF16
    X = synth.normal_ranks(R, n, dt, seed=budget)
    plan = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(VARIANTS[variant], sm_budget=budget, tile_bytes=4096, chunk_bytes=16384, chain_group=3))
    send = [torch.from_numpy(x.view(np.int16)).cuda() for x in X]
    recv = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    want = [torch.from_numpy(w.view(np.int16)).cuda() for w in orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))]
    bad = torch.zeros((), dtype=torch.int64, device="cuda")
    for it in range(150):
        dc.execute()
        for r in (it % R, (it + 3) % R):
            bad += (recv[r] != want[r]).sum()
        if it % 10 == 0:
            for t in recv:
                t.zero_()
    dc.check()
    assert int(bad) == 0


@pytest.mark.parametrize("variant", ["bulk", "bulk_warpstore", "lsu"])
def test_ring_allgather_repeated(variant):
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    R, n = 6, 50001
    rng = np.random.default_rng(1)
    X = [rng.integers(0, 65536, size=n, dtype=np.uint16) for _ in range(R)]
    plan = hb.hccl_plan_allgather(R, None, n, hb.BF16, hb.ALGO_RING, dict(VARIANTS[variant], sm_budget=20, tile_bytes=4096, chunk_bytes=16384))
    send = [torch.from_numpy(x.view(np.int16)).cuda() for x in X]
    recv = [torch.zeros(n * R, dtype=torch.int16, device="cuda") for _ in range(R)]
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    want = torch.cat(send)
    bad = torch.zeros((), dtype=torch.int64, device="cuda")
    for it in range(150):
        for t in recv:
            t.zero_()
        dc.execute()
        bad += (recv[it % R] != want).sum()
    dc.check()
    assert int(bad) == 0


@pytest.mark.parametrize("variant", ["lsu", "bulk"])
def test_ring_makes_progress_while_a_gemm_owns_the_sms(variant):
    """Dependencies only point backwards in ticket order, so blocks that are not resident (a GEMM holds the
    SMs) cannot be waited for: the ring must finish, correctly, without timeouts."""
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    R, n, dt = 8, 400003, hb.BF16
    X = synth.normal_ranks(R, n, dt, seed=5)
    plan = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(VARIANTS[variant], sm_budget=148, tile_bytes=8192, chunk_bytes=65536))
    send = [torch.from_numpy(x.view(np.int16)).cuda() for x in X]
    recv = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    want = [torch.from_numpy(w.view(np.int16)).cuda() for w in orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))]
    a = torch.randn(4096, 4096, device="cuda", dtype=torch.bfloat16)
    b = torch.randn(4096, 4096, device="cuda", dtype=torch.bfloat16)
    c = torch.empty_like(a)
    sg, sc = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    bad = torch.zeros((), dtype=torch.int64, device="cuda")
    for it in range(20):
        with torch.cuda.stream(sg):
            for _ in range(10):
                torch.matmul(a, b, out=c)
        with torch.cuda.stream(sc):
            dc.execute(sc)
            bad += (recv[it % R] != want[it % R]).sum()
    torch.cuda.synchronize()
    st, _ = plan.status()
    assert st == hb.OK and int(bad) == 0
