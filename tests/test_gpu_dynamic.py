"""Device-resident and device-triggered AllToAllv: counts live in device memory, may change between
executions of one bound plan, and a producer on another stream releases a pre-launched collective."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

SENT = 0x5A


def test_dynamic_plan_validation():
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_alltoallv_dynamic(257, [1] * 257, [1] * 257, hb.BF16, 8)
    assert e.value.status == hb.ERR_INVALID_ARG
    # beyond 64 ranks (or on request) the tables are built on the device: the plan holds room for the largest
    # table the capacities allow (rows * row bytes / tile per source, plus one partial tile per pair, plus the
    # END markers) and names the ordinary executor
    big = hb.hccl_plan_alltoallv_dynamic(65, [100] * 65, [100] * 65, hb.BF16, 8, dict(tile_bytes=512))
    i = big.info()
    assert i.n_wqe == 65 * 65 and i.engine == hb.ENGINE_BULK and i.tile_bytes == 512
    assert i.n_tiles == 65 * (100 * 16 // 512) + 65 * 65 + 2 * 148 + 2
    same = hb.hccl_plan_alltoallv_dynamic(4, [10] * 4, [12] * 4, hb.FP16, 8, dict(flags=hb.FLAG_DEVICE_TABLES, engine=hb.ENGINE_LSU))
    assert same.info().n_wqe == 16 and same.info().engine == hb.ENGINE_LSU and same.extents(0) == (160, 192)
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_alltoallv_dynamic(2, [1, -1], [1, 1], hb.BF16, 8)
    assert e.value.status == hb.ERR_INVALID_ARG
    p = hb.hccl_plan_alltoallv_dynamic(4, [10] * 4, [12] * 4, hb.FP16, 8)
    assert p.extents(0) == (160, 192) and p.info().n_tiles == 0


def _setup(R, row_elems, cap_rows, dt=hb.BF16, opts=None):
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    rb = row_elems * hb.ELEM_BYTES[dt]
    plan = hb.hccl_plan_alltoallv_dynamic(R, [cap_rows] * R, [cap_rows] * R, dt, row_elems, opts)
    X = [synth.hashed_rows_np(s, 0, cap_rows, row_elems).reshape(-1).view(np.uint8) for s in range(R)]
    send = [torch.from_numpy(x.copy()).cuda() for x in X]
    recv = [torch.full((cap_rows * rb,), SENT, dtype=torch.uint8, device="cuda") for _ in range(R)]
    counts = torch.zeros(R * R, dtype=torch.int64, device="cuda")
    rc_out = torch.full((R * R,), -1, dtype=torch.int64, device="cuda")
    rd_out = torch.full((R * R,), -1, dtype=torch.int64, device="cuda")
    plan.set_dynamic_metadata(counts.data_ptr(), rc_out.data_ptr(), rd_out.data_ptr())
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    return plan, dc, X, send, recv, counts, rc_out, rd_out, rb


def _expect(X, C, rb, cap_rows):
    R = C.shape[0]
    SD, RD = orc.packed_displs(C)
    Y = [np.full(cap_rows * rb, SENT, dtype=np.uint8) for _ in range(R)]
    orc.alltoallv(X, Y, C, SD, RD, rb)
    return Y, RD


@pytest.mark.gpu
@pytest.mark.parametrize("R,row_elems,hi", [(2, 8, 5), (8, 128, 300), (8, 7, 50), (33, 64, 40), (64, 256, 24)])
def test_dynamic_alltoallv_counts_change_between_executions(R, row_elems, hi):
    import torch
    cap = hi * R + 3
    plan, dc, X, send, recv, counts, rc_out, rd_out, rb = _setup(R, row_elems, cap, opts=dict(sm_budget=24, tile_bytes=4096))
    for seed in (1, 2, 3):
        C = synth.uniform_counts(R, seed, hi=hi)
        if seed == 2:
            C[:, R // 2] = 0                       # a destination that receives nothing
            C[0, :] = 0                            # a source that sends nothing
        counts.copy_(torch.from_numpy(C.reshape(-1)))    # the "routing kernel": sizes written on the device
        for t in recv:
            t.fill_(SENT)
        dc.execute()
        dc.check()
        want, RD = _expect(X, C, rb, cap)
        for d in range(R):
            assert np.array_equal(recv[d].cpu().numpy(), want[d]), (seed, d)
        assert np.array_equal(rc_out.cpu().numpy().reshape(R, R), C.T)
        assert np.array_equal(rd_out.cpu().numpy().reshape(R, R), RD)


@pytest.mark.gpu
@pytest.mark.parametrize("R,row_elems,hi,opts", [
    (8, 16, 50, dict(flags=hb.FLAG_DEVICE_TABLES, engine=hb.ENGINE_LSU, sm_budget=24, tile_bytes=2048)),
    (8, 128, 300, dict(flags=hb.FLAG_DEVICE_TABLES, sm_budget=24, tile_bytes=4096)),
    (8, 7, 50, dict(flags=hb.FLAG_DEVICE_TABLES, sm_budget=16, tile_bytes=1024)),          # rows of 14 bytes: unaligned segments
    (64, 64, 24, dict(flags=hb.FLAG_DEVICE_TABLES, tile_bytes=4096)),
    (65, 32, 12, dict(sm_budget=32, tile_bytes=2048)),
    (128, 32, 12, dict(tile_bytes=4096)),
    (128, 64, 10, dict(engine=hb.ENGINE_LSU, sm_budget=64, tile_bytes=8192)),
    (256, 16, 6, None),
], ids=["r8_lsu", "r8_bulk", "r8_rows_of_14_bytes", "r64", "r65", "r128_bulk", "r128_lsu", "r256_defaults"])
def test_dynamic_alltoallv_tables_built_on_the_device(R, row_elems, hi, opts):
    """Beyond 64 ranks (and, with HCCL_FLAG_DEVICE_TABLES, below) a kernel writes descriptors and tiles into the
    workspace from the counts in device memory and the ordinary executor runs them. Counts change between
    executions of one bound plan, including a shrinking table (stale tiles behind the END markers)."""
    import torch
    cap = hi * R + 3
    plan, dc, X, send, recv, counts, rc_out, rd_out, rb = _setup(R, row_elems, cap, opts=opts)
    assert plan.info().n_wqe == R * R
    for seed in (1, 2, 3, 4):
        C = synth.uniform_counts(R, seed, hi=hi)
        if seed == 2:
            C[:, R // 2] = 0                       # a destination that receives nothing
            C[0, :] = 0                            # a source that sends nothing
            C[R - 1, :] = 0                        # ... the last one too (it writes the END markers)
        if seed == 3:
            C[:] = 0
            C[1, 0] = cap                          # one segment fills a whole send and a whole receive buffer
        if seed == 4:
            C[:] = 0                               # nothing at all
        counts.copy_(torch.from_numpy(C.reshape(-1)))
        for t in recv:
            t.fill_(SENT)
        rc_out.fill_(-1)
        rd_out.fill_(-1)
        dc.execute()
        dc.check()
        want, RD = _expect(X, C, rb, cap)
        for d in range(R):
            assert np.array_equal(recv[d].cpu().numpy(), want[d]), (seed, d)
        assert np.array_equal(rc_out.cpu().numpy().reshape(R, R), C.T)
        assert np.array_equal(rd_out.cpu().numpy().reshape(R, R), RD)
    for s_ in range(R):
        assert np.array_equal(send[s_].cpu().numpy(), X[s_])


@pytest.mark.gpu
@pytest.mark.parametrize("R", [8, 128])
def test_device_built_tables_reject_counts_beyond_capacity_without_writing(R):
    import torch
    row_elems, cap = 16, 3 * R
    opts = dict(flags=hb.FLAG_DEVICE_TABLES, tile_bytes=1024)
    plan, dc, X, send, recv, counts, rc_out, rd_out, rb = _setup(R, row_elems, cap, opts=opts)
    for bad in ("overflow_recv", "overflow_send", "negative", "overflow_recv_last_source"):
        C = np.full((R, R), 2, dtype=np.int64)
        if bad == "overflow_recv":
            C[: R // 2 + 1, 1] = 7                 # more than 3R rows into destination 1
        elif bad == "overflow_send":
            C[R // 2, :] = 4                       # source R/2 would send 4R rows
        elif bad == "negative":
            C[R - 2, 3] = -1
        else:
            C[R - 1, :] = 1
            C[R - 1, 0] = R + 3                    # only the last source's row tips destination 0 over (3R + 1 rows)
        counts.copy_(torch.from_numpy(C.reshape(-1)))
        dc.execute()
        torch.cuda.synchronize()
        st, _ = plan.status()
        assert st == hb.ERR_BAD_DESCRIPTOR, bad
        for t in recv:
            assert bool((t == SENT).all()), bad
        assert float(torch.ones(4, device="cuda").sum()) == 4.0
        # a good matrix straight afterwards, on the same bound plan
        C = synth.uniform_counts(R, 5, hi=2)
        counts.copy_(torch.from_numpy(C.reshape(-1)))
        dc.execute()
        dc.check()
        want, _ = _expect(X, C, rb, cap)
        for d in range(R):
            assert np.array_equal(recv[d].cpu().numpy(), want[d]), (bad, d)
        for t in recv:
            t.fill_(SENT)


@pytest.mark.gpu
def test_device_triggered_alltoallv_over_128_ranks():
    """Pre-launched on its own stream, held at the start gate by the table builder, released by a producer
    that writes the counts first; the completion value is stored by the executor behind the builder."""
    import torch
    R, row_elems, cap = 128, 32, 700
    plan, dc, X, send, recv, counts, rc_out, rd_out, rb = _setup(R, row_elems, cap, opts=dict(sm_budget=16))
    signals = torch.zeros(2, dtype=torch.int64, device="cuda")
    plan.set_user_signals(signals.data_ptr(), 2)
    plan.set_trigger(wait_slot=0, cmp=hb.CMP_GE, wait_value=0, wait_per_epoch=1, set_slot=1, set_value=100, set_per_epoch=1)
    coll, prod = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for epoch in (1, 2):
        C = synth.uniform_counts(R, 20 + epoch, hi=5)
        host_counts = torch.from_numpy(C.reshape(-1)).pin_memory()
        for t in recv:
            t.fill_(SENT)
        torch.cuda.synchronize()
        dc.execute(coll)
        with torch.cuda.stream(prod):
            counts.copy_(host_counts, non_blocking=True)
            signals[0:1].fill_(epoch)
        torch.cuda.synchronize()
        assert plan.status()[0] == hb.OK
        assert int(signals[1]) == 100 + epoch
        want, _ = _expect(X, C, rb, cap)
        for d in range(R):
            assert np.array_equal(recv[d].cpu().numpy(), want[d]), (epoch, d)


@pytest.mark.gpu
def test_dynamic_alltoallv_rejects_counts_beyond_capacity_without_writing():
    import torch
    R, row_elems, cap = 4, 16, 20
    plan, dc, X, send, recv, counts, rc_out, rd_out, rb = _setup(R, row_elems, cap)
    for bad in ("overflow_recv", "negative"):
        C = np.full((R, R), 2, dtype=np.int64)
        if bad == "overflow_recv":
            C[:, 1] = 6                        # 24 rows into a 20-row receive buffer
        else:
            C[2, 3] = -1
        counts.copy_(torch.from_numpy(C.reshape(-1)))
        dc.execute()
        torch.cuda.synchronize()
        st, _ = plan.status()
        assert st == hb.ERR_BAD_DESCRIPTOR
        for t in recv:
            assert bool((t == SENT).all())
    # the plan works again after being bound again, and the GPU is healthy
    from paper_2608_00358_b200.runtime import DeviceCollective
    dc2 = DeviceCollective(plan)
    dc2.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    C = np.full((R, R), 3, dtype=np.int64)
    counts.copy_(torch.from_numpy(C.reshape(-1)))
    dc2.execute()
    dc2.check()
    want, _ = _expect(X, C, rb, cap)
    for d in range(R):
        assert np.array_equal(recv[d].cpu().numpy(), want[d])


@pytest.mark.gpu
def test_device_triggered_dynamic_alltoallv_is_released_by_the_producer():
    """The collective is enqueued first, on its own stream, and holds at its start gate. The producer stream
    then writes the counts and raises the signal; when the collective is done it stores the completion value."""
    import torch
    R, row_elems, cap = 8, 64, 400
    plan, dc, X, send, recv, counts, rc_out, rd_out, rb = _setup(R, row_elems, cap, opts=dict(sm_budget=8))
    signals = torch.zeros(2, dtype=torch.int64, device="cuda")
    plan.set_user_signals(signals.data_ptr(), 2)
    # gate: slot 0 >= epoch; completion: slot 1 = 100 + epoch
    plan.set_trigger(wait_slot=0, cmp=hb.CMP_GE, wait_value=0, wait_per_epoch=1, set_slot=1, set_value=100, set_per_epoch=1)
    coll, prod = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for epoch in (1, 2):
        C = synth.uniform_counts(R, 10 + epoch, hi=40)
        host_counts = torch.from_numpy(C.reshape(-1)).pin_memory()
        for t in recv:
            t.fill_(SENT)
        torch.cuda.synchronize()
        dc.execute(coll)                                   # pre-launched: spins (bounded) on the gate
        with torch.cuda.stream(prod):
            counts.copy_(host_counts, non_blocking=True)   # stands in for the routing kernel's output
            signals[0:1].fill_(epoch)                      # the producer's release
        torch.cuda.synchronize()
        st, _ = plan.status()
        assert st == hb.OK
        assert int(signals[1]) == 100 + epoch
        want, _ = _expect(X, C, rb, cap)
        for d in range(R):
            assert np.array_equal(recv[d].cpu().numpy(), want[d]), (epoch, d)


@pytest.mark.gpu
def test_start_gate_that_never_opens_times_out_cleanly():
    """A wait that cannot come true ends in HCCL_ERR_TIMEOUT after the plan's bound, the kernel returns
    normally and the device stays usable."""
    import torch
    R, row_elems, cap = 2, 8, 8
    plan, dc, X, send, recv, counts, rc_out, rd_out, rb = _setup(R, row_elems, cap, opts=dict(sm_budget=2, timeout_ns=200_000_000))
    signals = torch.zeros(1, dtype=torch.int64, device="cuda")
    plan.set_user_signals(signals.data_ptr(), 1)
    plan.set_trigger(wait_slot=0, cmp=hb.CMP_EQ, wait_value=12345)
    counts.fill_(1)
    dc.execute()
    torch.cuda.synchronize()
    st, _ = plan.status()
    assert st == hb.ERR_TIMEOUT
    for t in recv:
        assert bool((t == SENT).all())
    assert float(torch.ones(4, device="cuda").sum()) == 4.0


@pytest.mark.gpu
@pytest.mark.parametrize("kind", ["ring_chains", "ring_tickets", "ring_forwarded", "alltoallv_bulk"])
def test_device_triggered_static_plans(kind):
    """The start gate and the completion value on statically planned collectives: the register engine with static
    chains and with tickets, the forwarding kernel, and the bulk engine. The collective is enqueued first and holds (bounded) at its
    gate on a few SMs; a fill on another stream releases it."""
    import torch
    from gpu_helpers import SENTINEL
    from oracle import oracle as orc
    R = 4
    if kind == "alltoallv_bulk":
        C = synth.uniform_counts(R, 3, hi=50)
        X = [synth.hashed_rows_np(s, 0, max(int(C[s].sum()), 1), 32).reshape(-1).view(np.uint8) for s in range(R)]
        plan = hb.hccl_plan_alltoallv(R, C, None, None, None, hb.FP16, 32, dict(sm_budget=8, engine=hb.ENGINE_BULK))
        want = [np.full(int(C[:, d].sum()) * 64, 0, dtype=np.uint8) for d in range(R)]
        SD, RD = orc.packed_displs(C)
        orc.alltoallv(X, want, C, SD, RD, 64)
    else:
        n = 30011
        X = synth.normal_ranks(R, n, hb.BF16, seed=9)
        flags = hb.FLAG_DYNAMIC_TICKETS if kind == "ring_tickets" else 0
        engine = hb.ENGINE_BULK if kind == "ring_forwarded" else hb.ENGINE_LSU
        plan = hb.hccl_plan_allreduce(R, n, hb.BF16, hb.ALGO_RING, dict(sm_budget=8, tile_bytes=4096, chunk_bytes=16384, flags=flags, engine=engine))
        assert (plan.info().static_chains > 0) == (kind != "ring_tickets") and plan.info().engine == engine
        want = [w.view(np.uint8) for w in orc.allreduce_ring_f32(hb.BF16, X, orc.floor_chunk_offsets(n, R))]
    send = [torch.from_numpy(x.view(np.uint8).copy()).cuda() for x in X]
    recv = [torch.full((max(plan.extents(r)[1], 16),), SENTINEL, dtype=torch.uint8, device="cuda") for r in range(R)]
    from paper_2608_00358_b200.runtime import DeviceCollective
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv], keep=(send, recv))
    signals = torch.zeros(2, dtype=torch.int64, device="cuda")
    plan.set_user_signals(signals.data_ptr(), 2)
    plan.set_trigger(wait_slot=0, cmp=hb.CMP_GE, wait_value=0, wait_per_epoch=1, set_slot=1, set_value=500, set_per_epoch=1)
    coll, prod = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for epoch in (1, 2):
        for t in recv:
            t.fill_(SENTINEL)
        torch.cuda.synchronize()
        dc.execute(coll)
        with torch.cuda.stream(prod):
            signals[0:1].fill_(epoch)
        torch.cuda.synchronize()
        assert plan.status()[0] == hb.OK
        assert int(signals[1]) == 500 + epoch
        for r in range(R):
            assert np.array_equal(recv[r].cpu().numpy()[:want[r].size], want[r]), (kind, epoch, r)


@pytest.mark.gpu
@pytest.mark.parametrize("engine,R,flags", [(hb.ENGINE_LSU, 2, 0), (hb.ENGINE_BULK, 2, hb.FLAG_DYNAMIC_TICKETS), (hb.ENGINE_BULK, 4, 0)],
                         ids=["lsu", "bulk", "forwarding"])
def test_static_plan_gate_that_never_opens_times_out_cleanly(engine, R, flags):
    import torch
    n = 4096
    X = synth.normal_ranks(R, n, hb.FP32, seed=1)
    plan = hb.hccl_plan_allreduce(R, n, hb.FP32, hb.ALGO_RING, dict(sm_budget=2, timeout_ns=200_000_000, engine=engine, flags=flags))
    assert (plan.info().static_chains > 0) == (flags == 0)     # static chains on the bulk engine: the forwarding kernel
    send = [torch.from_numpy(x).cuda() for x in X]
    recv = [torch.full((n,), 7.0, dtype=torch.float32, device="cuda") for _ in range(R)]
    from paper_2608_00358_b200.runtime import DeviceCollective
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv], keep=(send, recv))
    signals = torch.zeros(1, dtype=torch.int64, device="cuda")
    plan.set_user_signals(signals.data_ptr(), 1)
    plan.set_trigger(wait_slot=0, cmp=hb.CMP_EQ, wait_value=12345)
    dc.execute()
    torch.cuda.synchronize()
    assert plan.status()[0] == hb.ERR_TIMEOUT
    for t in recv:
        assert bool((t == 7.0).all())
    assert float(torch.ones(4, device="cuda").sum()) == 4.0


@pytest.mark.gpu
@pytest.mark.parametrize("seed", range(16))
def test_random_device_resident_alltoallv(seed):
    """Random rank counts on both sides of the 64-rank boundary (one kernel with the count matrix in shared memory up to
    64 ranks, device-built tables beyond), row sizes, engines, tiles and block counts; counts redrawn for each of three
    executions of one bound plan (dense, sparse, skewed onto one destination), always within the buffers' capacity."""
    import torch
    rng = np.random.default_rng(7000 + seed)
    R = int(rng.choice([1, 2, 5, 17, 40, 63, 64, 65, 90, 130, 200]))
    row_elems = int(rng.choice([4, 7, 16, 64, 128]))
    hi = int(rng.integers(2, max(3, 2400 // R)))
    cap = hi * R + int(rng.integers(0, 4))
    o = dict(sm_budget=int(rng.choice([1, 8, 24, 148])), tile_bytes=int(rng.choice([512, 2048, 4096, 16384])))
    if rng.random() < 0.5:
        o["engine"] = int(rng.choice([hb.ENGINE_LSU, hb.ENGINE_BULK]))
    if R <= 64 and rng.random() < 0.5:
        o["flags"] = hb.FLAG_DEVICE_TABLES
    plan, dc, X, send, recv, counts, rc_out, rd_out, rb = _setup(R, row_elems, cap, opts=o)
    for it in range(3):
        C = rng.integers(0, hi + 1, size=(R, R)).astype(np.int64)
        if it == 1:
            C *= (rng.random((R, R)) < 0.15)
        if it == 2:
            d = int(rng.integers(0, R))
            C[:] = 0
            C[:, d] = rng.integers(0, hi + 1, size=R)      # everything goes to one destination
        assert C.sum(axis=0).max() <= cap and C.sum(axis=1).max() <= cap
        counts.copy_(torch.from_numpy(C.reshape(-1)))
        for t in recv:
            t.fill_(SENT)
        dc.execute()
        dc.check()
        want, RD = _expect(X, C, rb, cap)
        for d in range(R):
            assert np.array_equal(recv[d].cpu().numpy(), want[d]), (seed, it, R, row_elems, o, d)
        assert np.array_equal(rc_out.cpu().numpy().reshape(R, R), C.T)
        assert np.array_equal(rd_out.cpu().numpy().reshape(R, R), RD)
    for s_ in range(R):
        assert np.array_equal(send[s_].cpu().numpy(), X[s_])
