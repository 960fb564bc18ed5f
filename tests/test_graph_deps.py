"""The dependency kinds of the work-packet model (Fence, Sync, WQE Sync, Receive Sync, Send Sync, NOOP join,
WAIT/SET signal pairs), each on a tiny graph whose result is wrong if the dependency is not honoured.
CPU: host interpreter in random orders + hazard checker. GPU: the same graphs through the executor."""
import numpy as np
import pytest

from helpers import interpret
from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb

N = 4096            # fp32 elements per piece
NB = N * 4
S, Rv, SC, SIG = hb.BUF_SEND, hb.BUF_RECV, hb.BUF_SCRATCH, hb.BUF_SIGNAL
OPTS = dict(tile_bytes=1024, sm_budget=8)
F3 = (hb.FP32, hb.FP32, hb.FP32)


def _x(R, seed=0):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal(N).astype(np.float32) for _ in range(R)]


def _sum(a, b):
    return orc.nmc(hb.FP32, hb.FP32, a, hb.FP32, b)


def g_fence(with_dep=True):
    g = hb.Graph(2, [NB, NB], [NB, NB])
    sg = g.add_subgraph(0)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB, dep_flags=hb.DEP_FENCE if with_dep else 0)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, 0), a=(Rv, 0, 0), count=NB)
    return g, lambda X: [X[0], X[0]]


def g_sync(with_dep=True):
    g = hb.Graph(2, [NB, NB], [2 * NB, NB])
    sg = g.add_subgraph(0)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, NB), a=(S, 1, 0), count=NB)
    g.add_wqe(sg, hb.OP_REDUCE, dst=(Rv, 1, 0), a=(Rv, 0, 0), b=(Rv, 0, NB), count=N, dtypes=F3,
              dep_flags=hb.DEP_SYNC if with_dep else 0)
    return g, lambda X: [np.concatenate([X[0], X[1]]), _sum(X[0], X[1])]


def g_wqe_sync(with_dep=True):
    g = hb.Graph(2, [NB, NB], [NB, NB])
    a, b = g.add_subgraph(0), g.add_subgraph(1)
    w0 = g.add_wqe(a, hb.OP_REDUCE, dst=(Rv, 0, 0), a=(S, 0, 0), b=(S, 1, 0), count=N, dtypes=F3)
    g.add_wqe(b, hb.OP_REDUCE, dst=(Rv, 1, 0), a=(Rv, 0, 0), b=(S, 1, 0), count=N, dtypes=F3,
              dep_flags=hb.DEP_WQE_SYNC if with_dep else 0, dep_wqe=w0)
    return g, lambda X: [_sum(X[0], X[1]), _sum(_sum(X[0], X[1]), X[1])]


def g_recv_sync(with_dep=True, read_local=False):
    # subgraph of rank 1 receives from ranks 0 and 2, copies its own data locally, then sums what it received
    g = hb.Graph(3, [NB] * 3, [0, 4 * NB, 0])
    sg = g.add_subgraph(1)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, 0), a=(S, 0, 0), count=NB)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, NB), a=(S, 2, 0), count=NB)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, 2 * NB), a=(S, 1, 0), count=NB)          # local: not a receive
    second = (Rv, 1, 2 * NB) if read_local else (Rv, 1, NB)
    g.add_wqe(sg, hb.OP_REDUCE, dst=(Rv, 1, 3 * NB), a=(Rv, 1, 0), b=second, count=N, dtypes=F3,
              dep_flags=hb.DEP_RECV_SYNC if with_dep else 0)
    return g, lambda X: [np.zeros(0, np.float32), np.concatenate([X[0], X[2], X[1], _sum(X[0], X[1] if read_local else X[2])]),
                         np.zeros(0, np.float32)]


def g_send_sync(with_dep=True):
    # rank 0 first stages data in its receive buffer, rank 1 pulls it ("send"), then rank 0 reuses the buffer
    g = hb.Graph(2, [NB, NB], [NB, NB])
    sg = g.add_subgraph(0)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB, dep_flags=hb.DEP_FENCE)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, 0), a=(Rv, 0, 0), count=NB)                # a send out of rank 0
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 1, 0), count=NB, dep_flags=hb.DEP_SEND_SYNC if with_dep else 0)
    return g, lambda X: [X[1], X[0]]


def g_noop_join(with_dep=True):
    g = hb.Graph(3, [NB] * 3, [NB] * 3)
    a, b, c = g.add_subgraph(0), g.add_subgraph(1), g.add_subgraph(2)
    w0 = g.add_wqe(a, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB)
    w1 = g.add_wqe(b, hb.OP_COPY, dst=(Rv, 1, 0), a=(S, 1, 0), count=NB)
    j = g.add_wqe(c, hb.OP_NOOP, dep_flags=hb.DEP_WQE_SYNC | hb.DEP_FENCE, dep_wqe=w0, dep_wqe2=w1 if with_dep else -1)
    g.add_wqe(c, hb.OP_REDUCE, dst=(Rv, 2, 0), a=(Rv, 0, 0), b=(Rv, 1, 0), count=N, dtypes=F3)
    return g, lambda X: [X[0], X[1], _sum(X[0], X[1])]


def g_signal_pair():
    # two subgraphs hand a buffer back and forth with a pair of monotonically increasing signals
    g = hb.Graph(2, [NB, NB], [NB, NB], n_signals=2)
    a, b = g.add_subgraph(0), g.add_subgraph(1)
    g.add_wqe(a, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB)
    g.add_wqe(a, hb.OP_SET, dst=(SIG, 0, 0), value=0, value_per_epoch=1, dep_flags=hb.DEP_SYNC)
    g.add_wqe(b, hb.OP_WAIT, a=(SIG, 0, 0), cmp=hb.CMP_GE, value=0, value_per_epoch=1, dep_flags=hb.DEP_FENCE)
    g.add_wqe(b, hb.OP_REDUCE, dst=(Rv, 1, 0), a=(Rv, 0, 0), b=(S, 1, 0), count=N, dtypes=F3, dep_flags=hb.DEP_FENCE)
    g.add_wqe(b, hb.OP_SET, dst=(SIG, 0, 1), value=0, value_per_epoch=1)
    return g, lambda X: [X[0], _sum(X[0], X[1])]


def g_fanout(with_dep=True):
    # multi-destination forms: a copy into ranks 3, 0, 1 (wrapping), a dependent sum reading one of those
    # copies, and a two-input sum written into ranks 0 and 1
    g = hb.Graph(4, [NB] * 4, [2 * NB, 2 * NB, NB, NB])
    sg = g.add_subgraph(3)
    w0 = g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 3, 0), a=(S, 3, 0), count=NB, ndst=3)
    g.add_wqe(sg, hb.OP_REDUCE, dst=(Rv, 2, 0), a=(Rv, 1, 0), b=(S, 0, 0), count=N, dtypes=F3,
              dep_flags=hb.DEP_WQE_SYNC if with_dep else 0, dep_wqe=w0)
    g.add_wqe(sg, hb.OP_REDUCE_N, dst=(Rv, 0, NB), a=(S, 2, 0), count=N, nsrc=2, ndst=2, dtypes=F3)
    return g, lambda X: [np.concatenate([X[3], _sum(X[2], X[3])]), np.concatenate([X[3], _sum(X[2], X[3])]),
                         _sum(X[3], X[0]), X[3]]


CASES = {"fanout": g_fanout, "fence": g_fence, "sync": g_sync, "wqe_sync": g_wqe_sync, "recv_sync": g_recv_sync,
         "send_sync": g_send_sync, "noop_join": g_noop_join}


@pytest.mark.parametrize("name", sorted(CASES))
def test_dependency_kind_on_host(name):
    g, want = CASES[name](True)
    R = len(want(_x(4)))
    X = _x(R, seed=1)
    p = g.compile(OPTS)
    assert p.check_hazards() == 0
    for seed in range(0, 12):
        Y = interpret(p, X, seed)
        for r, w in enumerate(want(X)):
            assert np.array_equal(Y[r].view(np.float32), w), (name, seed, r)
    # without the dependency the checker must object
    g2, _ = CASES[name](False)
    assert g2.compile(OPTS).check_hazards() > 0


def test_fanout_destinations_are_bounds_checked_one_by_one():
    g = hb.Graph(3, [NB] * 3, [NB, NB // 2, NB])
    sg = g.add_subgraph(0)
    with pytest.raises(hb.HcclError) as e:
        g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB, ndst=3)   # rank 1's buffer is too short
    assert e.value.status == hb.ERR_INVALID_ARG
    assert g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 2, 0), a=(S, 0, 0), count=NB, ndst=2) == 0  # ranks 2 and 0
    i = g.compile(OPTS).info()
    assert i.schedule_bytes == 3 * NB   # one read, two writes


def test_recv_sync_does_not_cover_local_copies():
    g, _ = g_recv_sync(True, read_local=True)
    assert g.compile(OPTS).check_hazards() > 0


def test_check_hazards_flag_rejects_at_compile_time():
    g, _ = g_fence(False)
    with pytest.raises(hb.HcclError) as e:
        g.compile(dict(OPTS, flags=hb.FLAG_CHECK_HAZARDS))
    assert e.value.status == hb.ERR_HAZARD


def test_signal_pair_on_host():
    g, want = g_signal_pair()
    X = _x(2, seed=2)
    p = g.compile(OPTS)
    for seed in range(0, 8):
        Y = interpret(p, X, seed)
        for r, w in enumerate(want(X)):
            assert np.array_equal(Y[r].view(np.float32), w)


def test_wqe_validation():
    g = hb.Graph(2, [NB, NB], [NB, NB], scratch_bytes=NB)
    sg = g.add_subgraph(0)
    def bad(status, **kw):
        with pytest.raises(hb.HcclError) as e:
            g.add_wqe(sg, **kw)
        assert e.value.status == status, kw
    bad(hb.ERR_INVALID_ARG, op=hb.OP_COPY, dst=(S, 0, 0), a=(S, 1, 0), count=16)             # send buffers are read-only
    bad(hb.ERR_INVALID_ARG, op=hb.OP_COPY, dst=(Rv, 0, 8), a=(S, 1, 0), count=NB)            # out of bounds
    bad(hb.ERR_OVERLAP, op=hb.OP_COPY, dst=(Rv, 0, 0), a=(Rv, 0, 8), count=64)
    bad(hb.ERR_DTYPE, op=hb.OP_REDUCE, dst=(Rv, 0, 0), a=(S, 0, 0), b=(S, 1, 0), count=4, dtypes=(9, 0, 0))
    bad(hb.ERR_ALIGNMENT, op=hb.OP_REDUCE, dst=(Rv, 0, 2), a=(S, 0, 0), b=(S, 1, 0), count=4, dtypes=F3)
    bad(hb.ERR_OVERLAP, op=hb.OP_REDUCE, dst=(Rv, 0, 4), a=(Rv, 0, 0), b=(S, 1, 0), count=4, dtypes=F3)   # shifted alias
    bad(hb.ERR_INVALID_ARG, op=hb.OP_REDUCE_N, dst=(Rv, 0, 0), a=(S, 0, 0), count=4, nsrc=3, dtypes=F3)
    bad(hb.ERR_INVALID_ARG, op=hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 1, 0), count=16, ndst=3)     # more destinations than ranks
    bad(hb.ERR_INVALID_ARG, op=hb.OP_COPY, dst=(SC, 0, 0), a=(S, 1, 0), count=16, ndst=2)     # scratch has no ranks to fan out over
    bad(hb.ERR_OVERLAP, op=hb.OP_COPY, dst=(Rv, 1, 0), a=(Rv, 0, 0), count=16, ndst=2)        # second destination is the source
    bad(hb.ERR_INVALID_ARG, op=hb.OP_REDUCE_N, dst=(SC, 0, 0), a=(S, 0, 0), count=4, nsrc=2, ndst=2, dtypes=F3)
    bad(hb.ERR_INVALID_ARG, op=hb.OP_WAIT, a=(SIG, 0, 0), cmp=hb.CMP_GE)                      # no signal slots declared
    bad(hb.ERR_INVALID_ARG, op=hb.OP_NOOP, dep_flags=hb.DEP_WQE_SYNC, dep_wqe=5)             # dependency on the future
    ok = g.add_wqe(sg, hb.OP_REDUCE, dst=(Rv, 0, 0), a=(Rv, 0, 0), b=(S, 1, 0), count=N, dtypes=F3)   # A=A+B
    assert ok == 0


# ------------------------------------------------------------------ the same graphs on the GPU
@pytest.mark.gpu
@pytest.mark.parametrize("name", sorted(CASES) + ["signal_pair"])
@pytest.mark.parametrize("budget", [1, 2, 8])
@pytest.mark.parametrize("engine", [hb.ENGINE_LSU, hb.ENGINE_BULK], ids=["lsu", "bulk"])
def test_dependency_kind_on_gpu(name, budget, engine):
    from gpu_helpers import run_plan
    g, want = (g_signal_pair() if name == "signal_pair" else CASES[name](True))
    R = len(want(_x(4)))
    X = _x(R, seed=3)
    p = g.compile(dict(OPTS, sm_budget=budget, engine=engine))
    Y = run_plan(p, X, iters=5)
    for r, w in enumerate(want(X)):
        assert np.array_equal(Y[r].view(np.float32), w), (name, r)
