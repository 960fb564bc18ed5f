"""Seeded random configurations of the AllReduce / AllGather planners and executor options against the
schedule-ordered oracles: rank counts, sizes, element types, algorithms, engines, block counts, dispatch modes."""
import numpy as np
import pytest

from gpu_helpers import run_plan
from helpers import np_dtype
from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

pytestmark = pytest.mark.gpu


def _options(rng):
    o = dict(sm_budget=int(rng.choice([1, 2, 5, 16, 148])), engine=int(rng.choice([0, hb.ENGINE_LSU, hb.ENGINE_BULK])))
    if rng.random() < 0.5:
        o["tile_bytes"] = int(rng.choice([256, 1024, 4096, 49152]))
    if rng.random() < 0.5:
        o["chunk_bytes"] = int(rng.choice([512, 4096, 65536]))
    if rng.random() < 0.3:
        o["chain_group"] = int(rng.choice([1, 2, 7]))
    if rng.random() < 0.3:
        o["flags"] = int(rng.choice([hb.FLAG_DYNAMIC_TICKETS, hb.FLAG_STATIC_CHAINS, hb.FLAG_LEVEL_MAJOR]))
    if o["engine"] != hb.ENGINE_BULK and rng.random() < 0.2:
        o.update(light=1, threads=int(rng.choice([128, 256, 512])))
    if o["engine"] != hb.ENGINE_LSU and rng.random() < 0.4:      # bulk engine (or the library's choice): stage ring and block shape
        o.update(stage_kib=int(rng.choice([12, 20, 24, 36, 48, 96])), stages=int(rng.choice([0, 2, 3, 5, 8])))
        if rng.random() < 0.5:
            o["threads"] = int(rng.choice([128, 160, 224, 352, 512]))
    if rng.random() < 0.2:
        o["quantum"] = int(rng.choice([1, 2, 5]))               # short-lived blocks (ignored by plans that run as static chains)
    return o


@pytest.mark.parametrize("seed", range(48))
def test_random_allreduce(seed):
    rng = np.random.default_rng(1000 + seed)
    R = int(rng.integers(2, 13))
    n = int(rng.choice([1, R - 1, R, R + 1, 255, 4097, int(rng.integers(1, 60000))]))
    dt = int(rng.choice([hb.FP32, hb.BF16, hb.FP16]))
    algos = [hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_RING_FUSED, hb.ALGO_TREE, hb.ALGO_FANOUT, hb.ALGO_AUTO]
    o = _options(rng)
    racks = [L for L in (2, 3, 4) if R % L == 0 and R // L >= 2]
    if racks:
        algos.append(hb.ALGO_RING_2LEVEL)
        o["rack_size"] = int(rng.choice(racks))
    algo = int(rng.choice(algos))
    X = synth.normal_ranks(R, n, dt, seed=seed)
    p = hb.hccl_plan_allreduce(R, n, dt, algo, o)
    Y = run_plan(p, X, iters=2, misalign=int(rng.choice([0, 0, 4, 8])) if dt == hb.FP32 else int(rng.choice([0, 0, 2, 6])))
    if algo in (hb.ALGO_ONESHOT, hb.ALGO_FANOUT, hb.ALGO_AUTO):
        want = orc.allreduce_oneshot_f32(dt, X)
    elif algo == hb.ALGO_TREE:
        want = orc.allreduce_tree_f32(dt, X)
    elif algo == hb.ALGO_RING_2LEVEL:
        L = o["rack_size"]
        want = orc.allreduce_ring2_f32(dt, X, R // L, L)
    else:
        want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for r in range(R):
        assert np.array_equal(Y[r].view(np.uint8), want[r].view(np.uint8)), (seed, R, n, dt, algo, o, r)


@pytest.mark.parametrize("seed", range(24))
def test_random_allgather(seed):
    rng = np.random.default_rng(2000 + seed)
    R = int(rng.integers(1, 13))
    counts = [int(c) for c in rng.integers(0, 3000, size=R)]
    dt = int(rng.choice([hb.FP32, hb.BF16]))
    algos = [hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_FANOUT]
    o = _options(rng)
    racks = [L for L in (2, 3, 4) if R % L == 0 and R // L >= 2]
    if racks:
        algos.append(hb.ALGO_RING_2LEVEL)
        o["rack_size"] = int(rng.choice(racks))
    algo = int(rng.choice(algos))
    X = [rng.integers(0, 2 ** 16, size=c * (2 if dt == hb.FP32 else 1), dtype=np.uint16) for c in counts]
    p = hb.hccl_plan_allgather(R, counts, 0, dt, algo, o)
    Y = run_plan(p, [x if x.size else np.zeros(8, np.uint16) for x in X], iters=2)
    want = np.concatenate(X) if sum(counts) else np.zeros(0, np.uint16)
    for r in range(R):
        assert np.array_equal(Y[r].view(np.uint16), want), (seed, R, counts, algo, o, r)


@pytest.mark.parametrize("seed", range(24))
def test_random_reducescatter(seed):
    rng = np.random.default_rng(3000 + seed)
    R = int(rng.integers(1, 13))
    counts = [int(c) for c in rng.integers(0, 5000, size=R)]
    if rng.random() < 0.3:
        counts[int(rng.integers(0, R))] = 0
    n = sum(counts)
    dt = int(rng.choice([hb.FP32, hb.BF16, hb.FP16]))
    algo = int(rng.choice([hb.ALGO_RING, hb.ALGO_RING_FUSED, hb.ALGO_ONESHOT]))
    o = _options(rng)
    X = synth.normal_ranks(R, max(n, 1), dt, seed=seed)
    X = [x[:n] if n else x[:0] for x in X]
    p = hb.hccl_plan_reducescatter(R, counts, n, dt, algo, o)
    Y = run_plan(p, [x if x.size else np.zeros(8, np_dtype(dt)) for x in X], iters=2)
    offs = np.concatenate([[0], np.cumsum(counts)])
    if algo == hb.ALGO_ONESHOT:
        whole = orc.allreduce_oneshot_f32(dt, X)[0] if n else np.zeros(0, np_dtype(dt))
        want = [whole[offs[r]:offs[r + 1]] for r in range(R)]
    else:
        want = orc.reducescatter_ring_f32(dt, X, np.array(counts, dtype=np.int64))
    for r in range(R):
        assert np.array_equal(Y[r].view(np.uint8), want[r].view(np.uint8)), (seed, R, counts, dt, algo, o, r)


@pytest.mark.parametrize("seed", range(24))
def test_random_forwarded_rings(seed):
    """Rings on the bulk engine with static chains (the forwarding kernel) at sizes of several pieces per chunk: random
    rank counts, ragged counts, operand misalignment, tile sizes and block counts; ReduceScatter with uneven shards
    (shards off the 16-byte grid run item by item inside the same kernel), AllReduce and AllGather with aligned blocks."""
    rng = np.random.default_rng(4000 + seed)
    R = int(rng.integers(2, 20))
    dt = int(rng.choice([hb.FP32, hb.BF16, hb.FP16]))
    o = dict(engine=hb.ENGINE_BULK, sm_budget=int(rng.choice([1, 3, 16, 148])))
    if rng.random() < 0.6:
        o["tile_bytes"] = int(rng.choice([4096, 28672, 57344, 100000, 262144]))
    if rng.random() < 0.4:
        o["chunk_bytes"] = int(rng.choice([4096, 65536, 1 << 20]))
    mis = int(rng.choice([0, 0, 4, 8, 12])) if dt == hb.FP32 else int(rng.choice([0, 0, 2, 6, 10]))
    kind = int(rng.integers(0, 3))
    if kind == 0:
        n = int(rng.integers(1, 600000))
        X = synth.normal_ranks(R, n, dt, seed=seed)
        p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, o)
        want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    elif kind == 1:
        grid = int(rng.choice([1, 8]))
        counts = [grid * int(c) for c in rng.integers(0, 60000 // grid, size=R)]
        if rng.random() < 0.3:
            counts[int(rng.integers(0, R))] = 0
        n = max(sum(counts), 1)
        X = [x[:sum(counts)] for x in synth.normal_ranks(R, n, dt, seed=seed)]
        p = hb.hccl_plan_reducescatter(R, counts, sum(counts), dt, hb.ALGO_RING, o)
        want = orc.reducescatter_ring_f32(dt, X, np.array(counts, dtype=np.int64))
        X = [x if x.size else np.zeros(8, np_dtype(dt)) for x in X]
    else:
        counts = [8 * int(c) for c in rng.integers(0, 9000, size=R)]
        X = [synth.normal_ranks(1, max(c, 1), dt, seed=seed * 31 + r)[0][:c] for r, c in enumerate(counts)]
        p = hb.hccl_plan_allgather(R, counts, 0, dt, hb.ALGO_RING, o)
        want = orc.allgatherv(X)
        X = [x if x.size else np.zeros(8, np_dtype(dt)) for x in X]
    assert p.info().engine == hb.ENGINE_BULK and p.check_hazards() == 0
    Y = run_plan(p, X, iters=2, misalign=mis)
    for r in range(R):
        w = want[r].view(np.uint8)
        assert np.array_equal(Y[r][:w.size], w), (seed, kind, R, dt, o, mis, r)


@pytest.mark.parametrize("seed", range(32))
def test_random_alltoallv(seed):
    """AllToAllv with random rank counts, row sizes (rows that are and are not multiples of 16 bytes), count matrices
    (uniform, mostly empty, one heavy pair), packed layouts and explicit displacements with gaps, engines, tile and
    stage geometry, block counts, short-lived blocks and buffer misalignment; bit-exact against the oracle, guard
    bands and the gaps between segments untouched."""
    rng = np.random.default_rng(5000 + seed)
    R = int(rng.integers(1, 25))
    dt = int(rng.choice([hb.FP32, hb.BF16, hb.FP16]))
    row_elems = int(rng.choice([1, 3, 7, 8, 64, 128, 250, 256]))
    rb = row_elems * hb.ELEM_BYTES[dt]
    hi = int(rng.choice([3, 40, 400])) if rb * R < 8000 else int(rng.choice([3, 40]))
    C = rng.integers(0, hi + 1, size=(R, R)).astype(np.int64)
    shape = int(rng.integers(0, 3))
    if shape == 1:
        C *= (rng.random((R, R)) < 0.2)
    elif shape == 2:
        C[int(rng.integers(0, R)), int(rng.integers(0, R))] = 20 * hi
    packed = bool(rng.random() < 0.5)
    if packed:
        SD, RD = orc.packed_displs(C)
        send_rows = C.sum(axis=1)
    else:
        # send segments may overlap each other (the same rows sent to several peers); receive segments are disjoint, with gaps
        send_rows = np.full(R, int(C.sum(axis=1).max()) + 2)
        SD = rng.integers(0, int(send_rows[0]) - int(C.max()) + 1, size=(R, R))
        RD = np.zeros((R, R), dtype=np.int64)
        for d in range(R):
            o = int(rng.integers(0, 3))
            for s in rng.permutation(R):
                RD[d, s] = o
                o += int(C[s, d]) + int(rng.integers(0, 3))
    X = [rng.integers(0, 256, size=max(int(send_rows[s]) * rb, 16), dtype=np.uint8) for s in range(R)]
    o = dict(sm_budget=int(rng.choice([1, 2, 5, 16, 148])), engine=int(rng.choice([0, hb.ENGINE_LSU, hb.ENGINE_BULK])))
    if rng.random() < 0.6:
        o["tile_bytes"] = int(rng.choice([256, 1000, 4096, 49152, 245760]))
    if o["engine"] != hb.ENGINE_LSU and rng.random() < 0.4:
        o.update(stage_kib=int(rng.choice([12, 24, 48, 96])), stages=int(rng.choice([0, 2, 3, 8])), copy_by_warps=int(rng.choice([0, 1, 2])))
    if o["engine"] != hb.ENGINE_BULK and rng.random() < 0.2:
        o.update(light=1, threads=int(rng.choice([64, 128, 256])))
    if rng.random() < 0.2:
        o["quantum"] = int(rng.choice([1, 3]))
    mis = int(rng.choice([0, 0, 1, 2, 4, 8]))
    p = hb.hccl_plan_alltoallv(R, C, None if packed else SD, C.T.copy(), None if packed else RD, dt, row_elems, o)
    assert p.check_hazards() == 0
    Y = run_plan(p, X, iters=2, misalign=mis)
    Yw = [np.full(p.extents(r)[1], 0xA5, dtype=np.uint8) for r in range(R)]
    orc.alltoallv([x[:int(send_rows[s]) * rb] for s, x in enumerate(X)], Yw, C, SD, RD, rb)
    for r in range(R):
        assert np.array_equal(Y[r], Yw[r]), (seed, R, dt, row_elems, packed, o, mis, r)
