"""hccl_execute_noalloc: execution on the library's built-in workspace, for callers that cannot allocate
device memory (they run under an allocator's lock or in its out-of-memory hooks, have no free device memory
left to ask for, or cannot afford cudaMalloc's synchronisation). Collected last on purpose, so that a run
that stops at the first failure has already run every other test.

The output must be bit-identical to what hccl_execute produces for the same plan and inputs (the tests of
the executor compare that one with the oracle), on two calls in a row that share the built-in array."""
import numpy as np
import pytest

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
    for r in range(R):
        assert np.array_equal(got1[r], want1[r]), "call 1, rank %d" % r
    # call 2, straight after, different plan and data on the same built-in array: ring AllReduce on fp16
    R2, n2 = 5, 77777
    X2 = synth.normal_ranks(R2, n2, hb.FP16, seed=12)
    p2 = hb.hccl_plan_allreduce(R2, n2, hb.FP16, hb.ALGO_RING, opts)
    assert p2.info().scratch_bytes > 0
    got2 = _noalloc(p2, X2)
    want2 = _reference(p2, X2)
    for r in range(R2):
        assert np.array_equal(got2[r], want2[r]), "call 2, rank %d" % r
    # and the first plan once more: stale tables and counters from call 2 must not matter
    got3 = _noalloc(p1, X1)
    for r in range(R):
        assert np.array_equal(got3[r], want1[r]), "call 3, rank %d" % r


@pytest.mark.gpu
def test_noalloc_rejects_plans_beyond_the_builtin_workspace():
    import torch
    big = hb.hccl_plan_reducescatter(16, None, 1 << 24, hb.BF16, hb.ALGO_RING)      # 2 MiB granules: 64 MiB of scratch
    assert big.workspace_bytes() > hb.NOALLOC_WORKSPACE_BYTES
    buf = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(hb.HcclError) as e:
        big.execute_noalloc([buf.data_ptr()] * 16, [buf.data_ptr()] * 16)
    assert e.value.status == hb.ERR_WORKSPACE
