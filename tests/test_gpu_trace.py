"""Optional per-item timestamps: every work item records who ran it and when it was claimed, released and
finished; the trace converts to Chrome trace-event JSON."""
import json

import numpy as np
import pytest

from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("engine", [hb.ENGINE_LSU, hb.ENGINE_BULK], ids=["lsu", "bulk"])
def test_trace_covers_every_item_in_order(engine, tmp_path):
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective, chrome_trace, enable_trace
    R, n, dt = 4, 200000, hb.BF16
    budget = 12
    plan = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(engine=engine, sm_budget=budget, tile_bytes=16384, chunk_bytes=65536))
    X = synth.normal_ranks(R, n, dt, seed=4)
    send = [torch.from_numpy(x.view(np.int16)).cuda() for x in X]
    recv = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    trace = enable_trace(plan)
    dc = DeviceCollective(plan)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    dc.execute()
    dc.check()
    rows = trace.cpu().numpy()
    nt = plan.info().n_tiles
    assert rows.shape == (nt, 4)
    assert np.array_equal(rows[:, 0] & 0xFFFFFFFF, np.arange(nt))            # every item, in its own slot
    assert np.all((rows[:, 0] >> 32) < budget)
    assert np.all(rows[:, 1] > 0) and np.all(rows[:, 1] <= rows[:, 2]) and np.all(rows[:, 2] <= rows[:, 3])
    assert np.all(np.diff(rows[:, 1]) > -50_000_000)                          # claims follow ticket order (loosely)
    doc = chrome_trace(trace, "allreduce")
    path = tmp_path / "trace.json"
    path.write_text(json.dumps(doc))
    assert len(json.loads(path.read_text())["traceEvents"]) >= nt
    # switching it off again leaves the array alone
    plan.set_trace(0, 0)
    trace.zero_()
    dc.execute()
    dc.check()
    assert int(trace.abs().sum()) == 0
