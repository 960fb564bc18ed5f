"""The interference harness itself (A10): a short run of every way of sharing the GPU with a GEMM must complete,
report both rates inside the overlap window, and leave the results of the collective intact. Sizes are small (a
2048^3 GEMM, a 75 MB exchange), windows short: this checks the plumbing, not the numbers."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import interference as itf
from paper_2608_00358_b200 import workloads as wk

pytestmark = pytest.mark.gpu


def _check_result(wl):
    C, row = wl.meta["counts"], wl.meta["row_elems"]
    R, rb = C.shape[0], row * 2
    SD, RD = orc.packed_displs(C)
    X = [t.cpu().numpy().view(np.uint8) for t in wl.send]
    Y = [np.full(int(C[:, d].sum()) * rb, 0xA5, dtype=np.uint8) for d in range(R)]
    orc.alltoallv(X, Y, C, SD, RD, rb)
    for d in range(R):
        assert np.array_equal(wl.recv[d].cpu().numpy().view(np.uint8), Y[d]), d


@pytest.mark.parametrize("mode", ["persistent", "co_resident", "idle_sms"])
def test_overlap_modes_run_and_keep_the_result(mode):
    gemm = itf.Gemm(2048)
    opts = {"persistent": dict(sm_budget=4), "co_resident": itf.OVERLAP_OPTS, "idle_sms": itf.IDLE_SM_OPTS}[mode]
    wl = wk.config4(dict(opts), cap=48, R=16)
    for t in wl.recv:
        t.zero_()
    r = itf.measure(wl, seconds=0.6, gemm=gemm, collective_first=mode != "idle_sms", discard=0.1)
    assert r["gemm_alone_tflops"] > 0 and r["collective_alone_gbs"] > 0
    assert r["overlap"].get("gemm_tflops", 0) > 0 and r["overlap"].get("collective_gbs", 0) > 0 and "gemm_slowdown" in r
    _check_result(wl)


def test_sm_count_target_round_trip_and_green_partition():
    gemm = itf.Gemm(1024)
    gemm.run()
    torch.cuda.synchronize()
    assert itf.set_sm_count_target(140) == 140
    gemm.run()
    assert itf.set_sm_count_target(0) == 0
    part = itf.GreenPartition(8)
    try:
        assert part.small_sms >= 8 and part.small_sms + part.rest_sms <= 148
        wl = wk.config4(dict(sm_budget=part.small_sms), cap=48, R=16)
        r = itf.measure(wl, seconds=0.5, gemm=gemm, streams=(part.gemm_stream, part.collective_stream), discard=0.1)
        assert r["overlap"].get("gemm_tflops", 0) > 0 and r["overlap"].get("collective_gbs", 0) > 0
        _check_result(wl)
    finally:
        part.close()
    assert float(torch.ones(8, device="cuda").sum()) == 8.0
