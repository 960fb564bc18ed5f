"""hccl_execute_noalloc: execution on the library's built-in workspace, for callers that cannot allocate
device memory (they run under an allocator's lock or in its out-of-memory hooks, have no free device memory
left to ask for, or cannot afford cudaMalloc's synchronisation). Collected last on purpose, so that a run
that stops at the first failure has already run every other test.

The output must be bit-identical to what hccl_execute produces for the same plan and inputs, and to the
oracle's sums taken in the ring's order, on calls in a row that share the built-in array. Further cases:
a plan compiled for the other engine, a failed call (a wait that cannot come true) followed by a good
one on the same array, and the refusals."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth


def _device_buffers(plan, X):
    import torch
    R = plan.info().R
    send = [torch.from_numpy(np.ascontiguousarray(x).view(np.uint8).reshape(-1).copy()).cuda() for x in X]
    recv = [torch.full((max(plan.extents(r)[1], 16),), 0xA5, dtype=torch.uint8, device="cuda") for r in range(R)]
    return send, recv


def _reference(plan, X):
    """The existing entry point: bound workspace + hccl_execute."""
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    send, recv = _device_buffers(plan, X)
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    dc.execute()
    dc.check()
    return [t.cpu().numpy() for t in recv]


def _noalloc(plan, X):
    import torch
    send, recv = _device_buffers(plan, X)
    torch.cuda.synchronize()
    plan.execute_noalloc([t.data_ptr() for t in send], [t.data_ptr() for t in recv], torch.cuda.current_stream().cuda_stream)
    return [t.cpu().numpy() for t in recv]


@pytest.mark.gpu
def test_noalloc_matches_execute_on_two_calls_in_a_row():
    opts = dict(chunk_bytes=32 << 10, tile_bytes=8 << 10, chain_group=4, sm_budget=32)
    # call 1: ring ReduceScatter on bf16, which keeps FP32 partials in workspace scratch
    R, n = 8, 200003
    X1 = synth.normal_ranks(R, n, hb.BF16, seed=11, std=0.02)
    p1 = hb.hccl_plan_reducescatter(R, None, n, hb.BF16, hb.ALGO_RING, opts)
    assert p1.info().scratch_bytes > 0 and p1.workspace_bytes() <= hb.NOALLOC_WORKSPACE_BYTES
    want1 = _reference(p1, X1)
    got1 = _noalloc(p1, X1)
    rc1 = np.diff(orc.floor_chunk_offsets(n, R))                  # shard r = the floor split of n over R
    ring1 = orc.reducescatter_ring_f32(hb.BF16, X1, rc1)          # the oracle: FP32 adds in ring order, one rounding
    for r in range(R):
        assert p1.extents(r)[1] == 2 * int(rc1[r])
        assert np.array_equal(got1[r], want1[r]), "call 1, rank %d" % r
        assert np.array_equal(got1[r][:2 * int(rc1[r])].view(np.uint16), ring1[r]), "call 1, rank %d against the oracle" % r
    # call 2, straight after, different plan and data on the same built-in array: ring AllReduce on fp16
    R2, n2 = 5, 77777
    X2 = synth.normal_ranks(R2, n2, hb.FP16, seed=12)
    p2 = hb.hccl_plan_allreduce(R2, n2, hb.FP16, hb.ALGO_RING, opts)
    assert p2.info().scratch_bytes > 0
    got2 = _noalloc(p2, X2)
    want2 = _reference(p2, X2)
    ring2 = orc.allreduce_ring_f32(hb.FP16, X2, orc.floor_chunk_offsets(n2, R2))
    for r in range(R2):
        assert np.array_equal(got2[r], want2[r]), "call 2, rank %d" % r
        assert np.array_equal(got2[r][:2 * n2].view(np.uint16), ring2[r]), "call 2, rank %d against the oracle" % r
    # and the first plan once more: stale tables and counters from call 2 must not matter
    got3 = _noalloc(p1, X1)
    for r in range(R):
        assert np.array_equal(got3[r], want1[r]), "call 3, rank %d" % r
        assert np.array_equal(got3[r][:2 * int(rc1[r])].view(np.uint16), ring1[r]), "call 3, rank %d against the oracle" % r


@pytest.mark.gpu
def test_noalloc_runs_a_plan_compiled_for_the_bulk_engine():
    """Default options give an AllToAllv plan for the bulk engine (its thread count, its tile size); the
    no-allocation call runs it on the register path all the same, bit-exact against the oracle."""
    R, row = 8, 64
    C = synth.uniform_counts(R, 21, hi=300)
    C[2, 5] = 0
    plan = hb.hccl_plan_alltoallv(R, C, None, None, None, hb.BF16, row)
    assert plan.info().engine == hb.ENGINE_BULK and plan.workspace_bytes() <= hb.NOALLOC_WORKSPACE_BYTES
    X = [synth.hashed_rows_np(s, 0, max(int(C[s].sum()), 1), row).reshape(-1) for s in range(R)]
    SD, RD = orc.packed_displs(C)
    want = [np.full(max(plan.extents(d)[1], 16), 0xA5, dtype=np.uint8) for d in range(R)]
    orc.alltoallv([x.view(np.uint8) for x in X], want, C, SD, RD, row * 2)
    for call in range(2):
        got = _noalloc(plan, X)
        for d in range(R):
            assert np.array_equal(got[d], want[d]), "call %d, destination %d" % (call, d)
    ref = _reference(plan, X)
    for d in range(R):
        assert np.array_equal(ref[d], want[d])


@pytest.mark.gpu
def test_noalloc_returns_a_timeout_and_the_array_is_usable_afterwards():
    """A WAIT whose condition nothing satisfies, with a 0.1 s limit: the call itself returns the device's
    verdict, the GPU stays healthy, and the next call on the shared array is correct."""
    import torch
    N = 1024
    g = hb.Graph(2, [N * 4, N * 4], [N * 4, N * 4], n_signals=1)
    a = g.add_subgraph(0)
    g.add_wqe(a, hb.OP_COPY, dst=(hb.BUF_RECV, 0, 0), a=(hb.BUF_SEND, 0, 0), count=N * 4)
    g.add_wqe(a, hb.OP_WAIT, a=(hb.BUF_SIGNAL, 0, 0), cmp=hb.CMP_GE, value=5, dep_flags=hb.DEP_FENCE)
    g.add_wqe(a, hb.OP_COPY, dst=(hb.BUF_RECV, 1, 0), a=(hb.BUF_SEND, 1, 0), count=N * 4)
    bad = g.compile(dict(engine=hb.ENGINE_LSU, sm_budget=4, timeout_ns=100_000_000))
    send = [torch.arange(N, dtype=torch.float32, device="cuda") + r for r in range(2)]
    recv = [torch.full((N,), -1.0, device="cuda") for _ in range(2)]
    torch.cuda.synchronize()
    with pytest.raises(hb.HcclError) as e:
        bad.execute_noalloc([t.data_ptr() for t in send], [t.data_ptr() for t in recv], torch.cuda.current_stream().cuda_stream)
    assert e.value.status == hb.ERR_TIMEOUT
    assert bool((recv[1] == -1.0).all())                   # what was fenced behind the WAIT never ran
    assert float(torch.ones(8, device="cuda").sum()) == 8.0
    R, n = 4, 50001
    X = synth.normal_ranks(R, n, hb.BF16, seed=31)
    p = hb.hccl_plan_allreduce(R, n, hb.BF16, hb.ALGO_RING, dict(chunk_bytes=32 << 10, tile_bytes=8 << 10, chain_group=4, sm_budget=16))
    got = _noalloc(p, X)
    ring = orc.allreduce_ring_f32(hb.BF16, X, orc.floor_chunk_offsets(n, R))
    for r in range(R):
        assert np.array_equal(got[r][:2 * n].view(np.uint16), ring[r]), "rank %d after the failed call" % r


@pytest.mark.gpu
def test_noalloc_refuses_device_resident_plans():
    import torch
    dyn = hb.hccl_plan_alltoallv_dynamic(4, [8] * 4, [8] * 4, hb.BF16, 16)
    buf = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(hb.HcclError) as e:
        dyn.execute_noalloc([buf.data_ptr()] * 4, [buf.data_ptr()] * 4)
    assert e.value.status == hb.ERR_INVALID_ARG


@pytest.mark.gpu
def test_noalloc_rejects_plans_beyond_the_builtin_workspace():
    import torch
    big = hb.hccl_plan_reducescatter(16, None, 1 << 24, hb.BF16, hb.ALGO_RING)      # 2 MiB granules: 64 MiB of scratch
    assert big.workspace_bytes() > hb.NOALLOC_WORKSPACE_BYTES
    buf = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(hb.HcclError) as e:
        big.execute_noalloc([buf.data_ptr()] * 16, [buf.data_ptr()] * 16)
    assert e.value.status == hb.ERR_WORKSPACE
