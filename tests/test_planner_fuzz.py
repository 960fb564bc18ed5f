"""Seeded random planner configurations run by the host interpreter in random dependency-respecting orders:
every plan must be free of hazards and give the schedule-ordered oracle's bits whatever the order."""
import numpy as np
import pytest

from helpers import interpret
from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth


def _options(rng):
    o = dict(sm_budget=int(rng.choice([1, 3, 8, 148])), engine=int(rng.choice([0, hb.ENGINE_LSU, hb.ENGINE_BULK])),
             tile_bytes=int(rng.choice([0, 128, 512, 4096])), chunk_bytes=int(rng.choice([0, 256, 2048])))
    if rng.random() < 0.4:
        o["chain_group"] = int(rng.choice([1, 2, 5]))
    if rng.random() < 0.4:
        o["flags"] = int(rng.choice([hb.FLAG_DYNAMIC_TICKETS, hb.FLAG_STATIC_CHAINS, hb.FLAG_LEVEL_MAJOR, hb.FLAG_STAGED_RING]))
    return o


@pytest.mark.parametrize("seed", range(60))
def test_random_allreduce_plans(seed):
    rng = np.random.default_rng(seed)
    R = int(rng.integers(1, 10))
    n = int(rng.choice([0, 1, R, R + 1, 63, 1025, int(rng.integers(1, 5000))]))
    dt = int(rng.choice([hb.FP32, hb.BF16, hb.FP16]))
    algos = [hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_RING_FUSED, hb.ALGO_TREE, hb.ALGO_FANOUT]
    o = _options(rng)
    racks = [L for L in (2, 3, 4) if R % L == 0 and R // L >= 2]
    if racks:
        algos.append(hb.ALGO_RING_2LEVEL)
        o["rack_size"] = int(rng.choice(racks))
    algo = int(rng.choice(algos))
    X = synth.normal_ranks(R, n, dt, seed=seed)
    p = hb.hccl_plan_allreduce(R, n, dt, algo, o)
    assert p.check_hazards() == 0, (seed, R, n, dt, algo, o)
    if algo in (hb.ALGO_ONESHOT, hb.ALGO_FANOUT) or R == 1:
        want = orc.allreduce_oneshot_f32(dt, X)
    elif algo == hb.ALGO_TREE:
        want = orc.allreduce_tree_f32(dt, X)
    elif algo == hb.ALGO_RING_2LEVEL:
        want = orc.allreduce_ring2_f32(dt, X, R // o["rack_size"], o["rack_size"])
    else:
        want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for order in (0, seed + 1):
        Y = interpret(p, X, order)
        for r in range(R):
            assert np.array_equal(Y[r].view(np.uint8), want[r].view(np.uint8)), (seed, R, n, dt, algo, o, order, r)


@pytest.mark.parametrize("seed", range(30))
def test_random_alltoallv_and_allgather_plans(seed):
    rng = np.random.default_rng(500 + seed)
    R = int(rng.integers(1, 9))
    o = _options(rng)
    C = rng.integers(0, 30, size=(R, R)).astype(np.int64)
    C[rng.random((R, R)) < 0.25] = 0
    row = int(rng.choice([1, 3, 8]))
    X = [rng.integers(0, 256, size=max(int(C[s].sum()), 1) * row * 2, dtype=np.uint8) for s in range(R)]
    p = hb.hccl_plan_alltoallv(R, C, None, None, None, hb.BF16, row, o)
    assert p.check_hazards() == 0
    SD, RD = orc.packed_displs(C)
    want = [np.full(int(C[:, d].sum()) * row * 2, 0xA5, dtype=np.uint8) for d in range(R)]
    orc.alltoallv(X, want, C, SD, RD, row * 2)
    Y = interpret(p, X, seed + 1)
    for d in range(R):
        assert np.array_equal(Y[d], want[d]), (seed, d)
    counts = [int(c) for c in rng.integers(0, 400, size=R)]
    algos = [hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_FANOUT]
    racks = [L for L in (2, 4) if R % L == 0 and R // L >= 2]
    if racks:
        algos.append(hb.ALGO_RING_2LEVEL)
        o["rack_size"] = int(rng.choice(racks))
    algo = int(rng.choice(algos))
    Xg = [rng.integers(0, 2 ** 16, size=c, dtype=np.uint16) for c in counts]
    q = hb.hccl_plan_allgather(R, counts, 0, hb.BF16, algo, o)
    assert q.check_hazards() == 0, (seed, R, counts, algo, o)
    wantg = np.concatenate(Xg) if sum(counts) else np.zeros(0, np.uint16)
    Yg = interpret(q, [x if x.size else np.zeros(4, np.uint16) for x in Xg], seed + 2)
    for r in range(R):
        assert np.array_equal(Yg[r].view(np.uint16), wantg), (seed, R, counts, algo, o, r)
