"""Failure detection without faulting a GPU: every failure is made on the host (an unsatisfiable WAIT, a
damaged table entry, a workspace that is too small or misaligned) and must come back as a status code with
the device healthy. Nothing here traps, hangs or reads out of bounds."""
import pytest

from paper_2608_00358_b200 import binding as hb

N = 1024
NB = N * 4


def test_bind_rejects_small_or_misaligned_workspace_before_touching_the_device():
    p = hb.hccl_plan_allreduce(4, 1 << 16, hb.BF16)
    need = p.workspace_bytes()
    with pytest.raises(hb.HcclError) as e:
        p.bind(0x7F0000000000, need - 1)
    assert e.value.status == hb.ERR_WORKSPACE
    with pytest.raises(hb.HcclError) as e:
        p.bind(0x7F0000000010, need)
    assert e.value.status == hb.ERR_ALIGNMENT
    with pytest.raises(hb.HcclError) as e:
        p.execute([0] * 4, [0] * 4)
    assert e.value.status == hb.ERR_NOT_BOUND
    lay = p.layout()
    assert lay["total"] == need and lay["control"] == 0 and lay["tiles"] > lay["descs"] > lay["counters"]


def _graph_with_wait(never=True):
    g = hb.Graph(2, [NB, NB], [NB, NB], n_signals=1)
    a = g.add_subgraph(0)
    g.add_wqe(a, hb.OP_COPY, dst=(hb.BUF_RECV, 0, 0), a=(hb.BUF_SEND, 0, 0), count=NB)
    g.add_wqe(a, hb.OP_WAIT, a=(hb.BUF_SIGNAL, 0, 0), cmp=hb.CMP_GE, value=5 if never else 0, dep_flags=hb.DEP_FENCE)
    g.add_wqe(a, hb.OP_COPY, dst=(hb.BUF_RECV, 1, 0), a=(hb.BUF_SEND, 1, 0), count=NB)
    return g


@pytest.mark.gpu
@pytest.mark.parametrize("engine", [hb.ENGINE_LSU, hb.ENGINE_BULK], ids=["lsu", "bulk"])
def test_wait_that_never_comes_true_times_out(engine):
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    plan = _graph_with_wait().compile(dict(engine=engine, sm_budget=4, timeout_ns=150_000_000))
    send = [torch.arange(N, dtype=torch.float32, device="cuda") + r for r in range(2)]
    recv = [torch.full((N,), -1.0, device="cuda") for _ in range(2)]
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    dc.execute()
    torch.cuda.synchronize()
    st, detail = plan.status()
    assert st == hb.ERR_TIMEOUT and detail in (1, 2)       # the WAIT (tile 1) or the copy fenced behind it (tile 2)
    assert bool((recv[1] == -1.0).all())                   # what was fenced behind the WAIT never ran
    with pytest.raises(hb.HcclError):
        dc.check()
    assert float(torch.ones(8, device="cuda").sum()) == 8.0
    # the same graph with a satisfiable condition runs to completion
    ok = _graph_with_wait(never=False).compile(dict(engine=engine, sm_budget=4))
    dc2 = DeviceCollective(ok)
    dc2.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    dc2.execute()
    dc2.check()
    assert torch.equal(recv[1], send[1])


@pytest.mark.gpu
@pytest.mark.parametrize("engine,flags", [(hb.ENGINE_LSU, 0), (hb.ENGINE_BULK, hb.FLAG_DYNAMIC_TICKETS), (hb.ENGINE_BULK, 0)], ids=["lsu", "bulk", "forwarding"])
@pytest.mark.parametrize("damage", ["desc_index", "wait_range", "op_code", "rank"])
def test_damaged_table_entry_is_reported_not_dereferenced(engine, flags, damage):
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    plan = hb.hccl_plan_allreduce(4, 4096, hb.FP32, hb.ALGO_RING, dict(engine=engine, flags=flags, sm_budget=4, tile_bytes=4096, timeout_ns=150_000_000))
    assert (plan.info().static_chains > 0) == (flags == 0)     # static chains on the bulk engine: the forwarding kernel
    send = [torch.randn(4096, device="cuda") for _ in range(4)]
    recv = [torch.zeros(4096, device="cuda") for _ in range(4)]
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    lay = plan.layout()
    base = dc._ws_ptr - dc.workspace.data_ptr()
    ws32 = dc.workspace[base:base + (lay["scratch"] // 4) * 4].view(torch.int32)
    ws8 = dc.workspace[base:]
    if damage == "desc_index":
        ws32[lay["tiles"] // 4 + 8 * 3] = 0x7FFFFFF0           # tile 3: descriptor index far out of range
    elif damage == "wait_range":
        ws32[lay["tiles"] // 4 + 8 * 5 + 6] = 0x7FFFFFF0       # tile 5: wait list offset out of range
    elif damage == "op_code":
        ws8[lay["descs"] + 64 * 2] = 77                        # descriptor 2: unknown operation
    else:
        ws8[lay["descs"] + 64 * 1 + 8] = 200                   # descriptor 1: destination rank 200 of 4
    torch.cuda.synchronize()
    dc.execute()
    torch.cuda.synchronize()
    st, _ = plan.status()
    assert st == hb.ERR_BAD_DESCRIPTOR
    assert float(torch.ones(8, device="cuda").sum()) == 8.0
