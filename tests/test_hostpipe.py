"""AllToAllv through host buffers, pipelined by destination windows (hccl_hostpipe_*), against the oracle."""
import numpy as np
import pytest

from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

ROW = 24  # fp16 elements per row: 48-byte rows, so slices start off the 16-byte grid as well as on it


def _case(R, seed, hi=40, zero_dest=None):
    rng = np.random.default_rng(seed)
    C = rng.integers(0, hi, size=(R, R)).astype(np.int64)
    C[rng.random((R, R)) < 0.2] = 0
    if zero_dest is not None:
        C[:, zero_dest] = 0
    X = [synth.hashed_rows_np(s + 100 * seed, 0, max(int(C[s].sum()), 1), ROW).reshape(-1).view(np.uint8) for s in range(R)]
    return C, X


def _want(C, X):
    R = C.shape[0]
    SD, RD = orc.packed_displs(C)
    Y = [np.full(int(C[:, d].sum()) * ROW * 2, 0xA5, dtype=np.uint8) for d in range(R)]
    orc.alltoallv(X, Y, C, SD, RD, ROW * 2)
    return Y


@pytest.mark.parametrize("R,windows", [(1, 1), (5, 1), (5, 2), (5, 3), (5, 9), (16, 4), (16, 16)])
def test_windows_partition_the_destinations(R, windows):
    C, _ = _case(R, seed=R + windows, zero_dest=R // 2 if R > 2 else None)
    first = hb.hccl_hostpipe_alltoallv_create(R, C, hb.FP16, ROW, windows).windows()
    assert first[0] == 0 and first[-1] == R and all(a < b for a, b in zip(first, first[1:]))
    assert len(first) - 1 <= min(windows, R)
    rows = C.sum(axis=0)
    if rows.sum() > 0:
        assert all(rows[a:b].sum() > 0 for a, b in zip(first, first[1:]))


def test_create_rejects_bad_arguments():
    C = np.ones((3, 3), dtype=np.int64)
    for kw in (dict(R=0), dict(n_windows=0), dict(row_elems=0), dict(dt=7)):
        a = dict(R=3, sendcounts=C, dt=hb.FP16, row_elems=4, n_windows=2)
        a.update(kw)
        with pytest.raises(hb.HcclError):
            hb.hccl_hostpipe_alltoallv_create(**a)
    C[1, 2] = -1
    with pytest.raises(hb.HcclError):
        hb.hccl_hostpipe_alltoallv_create(3, C, hb.FP16, 4, 2)
    z = hb.hccl_hostpipe_alltoallv_create(3, np.zeros((3, 3), dtype=np.int64), hb.FP16, 4, 3)
    assert z.windows() == [0, 3]
    # nothing runs, and no verdict exists, before the pipeline has a workspace
    with pytest.raises(hb.HcclError) as e:
        z.status()
    assert e.value.status == hb.ERR_NOT_BOUND
    with pytest.raises(hb.HcclError) as e:
        z.execute([0] * 3, [0] * 3, [0] * 3, [0] * 3, 0, 0, 0)
    assert e.value.status == hb.ERR_NOT_BOUND
    assert z.workspace_bytes() % 256 == 0 and z.workspace_bytes() > 0


@pytest.mark.gpu
@pytest.mark.parametrize("engine", [hb.ENGINE_LSU, hb.ENGINE_BULK], ids=["lsu", "bulk"])
@pytest.mark.parametrize("R,windows", [(1, 1), (5, 1), (5, 2), (5, 5), (9, 4), (16, 7)])
def test_pipelined_alltoallv_matches_oracle(R, windows, engine):
    import torch
    C, X1 = _case(R, seed=R * 10 + windows, zero_dest=(R // 2 if R > 2 else None))
    _, X2 = _case(R, seed=R * 10 + windows + 1)
    X2 = [synth.hashed_rows_np(s + 777, 0, max(int(C[s].sum()), 1), ROW).reshape(-1).view(np.uint8) for s in range(R)]
    pipe = hb.hccl_hostpipe_alltoallv_create(R, C, hb.FP16, ROW, windows, dict(engine=engine, sm_budget=8, tile_bytes=1024))
    ws = torch.empty(pipe.workspace_bytes() + 256, dtype=torch.uint8, device="cuda")
    pipe.bind((ws.data_ptr() + 255) // 256 * 256, pipe.workspace_bytes(), torch.cuda.current_stream().cuda_stream)
    sb = [max(int(C[s].sum()), 1) * ROW * 2 for s in range(R)]
    rb = [int(C[:, d].sum()) * ROW * 2 for d in range(R)]
    dev_send = [torch.full((sb[s] + 64,), 0x5A, dtype=torch.uint8, device="cuda") for s in range(R)]
    dev_recv = [torch.full((rb[d] + 64,), 0xA5, dtype=torch.uint8, device="cuda") for d in range(R)]
    streams = [torch.cuda.Stream() for _ in range(3)]
    torch.cuda.synchronize()
    outs = []
    for X in (X1, X2):   # two calls enqueued back to back: the second must not start before the first has finished
        hs = [torch.from_numpy(x.copy()).pin_memory() for x in X]
        hr = [torch.full((rb[d] + 32,), 0xA5, dtype=torch.uint8).pin_memory() for d in range(R)]
        pipe.execute([h.data_ptr() for h in hs], [h.data_ptr() for h in hr], [t.data_ptr() for t in dev_send],
                     [t.data_ptr() for t in dev_recv], *[s.cuda_stream for s in streams])
        outs.append((hs, hr))
    torch.cuda.synchronize()
    assert pipe.status() == (hb.OK, 0)
    for X, (hs, hr) in zip((X1, X2), outs):
        want = _want(C, X)
        for d in range(R):
            got = hr[d].numpy()
            assert np.array_equal(got[:rb[d]], want[d]), d
            assert np.all(got[rb[d]:] == 0xA5), "bytes past the receive extent of rank %d were written" % d
    for d in range(R):   # staging buffers: nothing beyond the extents
        assert bool((dev_recv[d][rb[d]:] == 0xA5).all())


@pytest.mark.gpu
def test_execute_host_single_stream():
    """hccl_execute_host: host buffers in, one stream (copy in, execute, copy out), host buffers out."""
    import torch
    R, n, dt = 4, 5001, hb.BF16
    X = synth.normal_ranks(R, n, dt, seed=4)
    plan = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(sm_budget=8))
    ws = torch.empty(plan.workspace_bytes() + 256, dtype=torch.uint8, device="cuda")
    s = torch.cuda.Stream()
    plan.bind((ws.data_ptr() + 255) // 256 * 256, plan.workspace_bytes(), s.cuda_stream)
    hs = [torch.from_numpy(x.view(np.int16).copy()).pin_memory() for x in X]
    hr = [torch.full((n + 8,), 0x5A5A, dtype=torch.int16).pin_memory() for _ in range(R)]
    ds = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    dr = [torch.zeros(n, dtype=torch.int16, device="cuda") for _ in range(R)]
    for _ in range(2):
        plan.execute_host([t.data_ptr() for t in hs], [t.data_ptr() for t in hr], [t.data_ptr() for t in ds],
                          [t.data_ptr() for t in dr], s.cuda_stream)
    s.synchronize()
    assert plan.status()[0] == hb.OK
    want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for r in range(R):
        got = hr[r].numpy().view(np.uint16)
        assert np.array_equal(got[:n], want[r]) and np.all(got[n:] == 0x5A5A)
