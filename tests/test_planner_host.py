"""Planner checked on the CPU: the compiled tables, run by the library's host interpreter in random
dependency-respecting orders, must reproduce the oracle; the hazard checker must find every pair of
conflicting work items ordered. No GPU needed."""
import numpy as np
import pytest

from helpers import assert_reduction_close, interpret, np_dtype
from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

DTYPES = [hb.FP32, hb.BF16, hb.FP16]
SMALL = dict(tile_bytes=256, chunk_bytes=1024, chain_group=2, sm_budget=4)


def test_library_exports_every_declared_symbol():
    import ctypes
    import os
    import re
    lib = ctypes.CDLL(hb.LIBRARY_PATH)
    header = open(os.path.join(os.path.dirname(__file__), "..", "include", "hccl.h")).read()
    declared = set(re.findall(r"\b(hccl_[a-z_0-9]+)\s*\(", header))
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(lib, name), name
    assert set(hb.EXPORTS) == declared
    assert lib.hccl_version() >= 100
    assert hb.hccl_opts_for_overlap() == dict(engine=hb.ENGINE_LSU, light=1, threads=128, sm_budget=12)
    i = hb.hccl_plan_alltoallv(4, np.full((4, 4), 100), None, None, None, hb.BF16, 64, hb.hccl_opts_for_overlap()).info()
    assert (i.engine, i.threads, i.sm_budget) == (hb.ENGINE_LSU, 128, 12)


def test_config1_plan_shape():
    p = hb.hccl_plan_allreduce(4, 1 << 20, hb.FP32, hb.ALGO_RING)
    i = p.info()
    assert (i.n_wqe, i.chain_depth) == (24, 6)
    assert i.schedule_bytes == 60 << 20 and i.compulsory_bytes == 32 << 20
    assert i.scratch_bytes == 0
    assert p.check_hazards() == 0


def test_config3_and_5_byte_accounting():
    # ReduceScatter R=16 bf16, 2 MiB granules: 146 bytes of schedule traffic per output position
    n = 1 << 22
    p = hb.hccl_plan_reducescatter(16, None, n, hb.BF16)
    i = p.info()
    assert i.schedule_bytes == 146 * n and i.compulsory_bytes == 34 * n
    assert i.n_wqe == 16 * 15 * ((n // 16 * 2 + (2 << 20) - 1) // (2 << 20))
    # AllReduce R=8 bf16, m bytes per rank: ring 47 m, one-shot 72 m
    for m in (4096, 1 << 20):
        assert hb.hccl_plan_allreduce(8, m // 2, hb.BF16, hb.ALGO_RING).info().schedule_bytes == 47 * m
        assert hb.hccl_plan_allreduce(8, m // 2, hb.BF16, hb.ALGO_ONESHOT).info().schedule_bytes == 72 * m
        # destinations fused: every input read once, every output written once = the compulsory bytes
        i = hb.hccl_plan_allreduce(8, m // 2, hb.BF16, hb.ALGO_FANOUT).info()
        assert i.schedule_bytes == 16 * m == i.compulsory_bytes and i.chain_depth == 1
        # binary tree: 3 levels of sums + 3 levels of copies; per output position 4 x (2+2+4) + 2 x (4+4+4) +
        # (4+4+2) reduce bytes and 7 x (2+2) copy bytes = 94 bytes (the ring's figure), at depth 6 instead of 14
        i = hb.hccl_plan_allreduce(8, m // 2, hb.BF16, hb.ALGO_TREE).info()
        assert i.chain_depth == 6 and i.n_wqe % 14 == 0 and i.schedule_bytes == 47 * m


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("algo", [hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_RING_FUSED, hb.ALGO_FANOUT, hb.ALGO_TREE])
@pytest.mark.parametrize("R,n", [(1, 5), (2, 9), (3, 2), (4, 257), (5, 1000), (8, 4099), (4, 0), (4, 3), (7, 9001), (13, 700)])
def test_allreduce_plans_match_oracle(R, n, dt, algo):
    X = synth.normal_ranks(R, n, dt, seed=R * 100 + n)
    p = hb.hccl_plan_allreduce(R, n, dt, algo, SMALL)
    assert p.check_hazards() == 0
    exact = orc.sum_f64(dt, X)
    want = orc.allreduce(dt, X)
    if algo in (hb.ALGO_ONESHOT, hb.ALGO_FANOUT):  # the fused form sums in the one-shot's order
        bitwise = orc.allreduce_oneshot_f32(dt, X)
    elif algo == hb.ALGO_TREE:
        bitwise = orc.allreduce_tree_f32(dt, X)
    else:
        bitwise = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for seed in (0, 1, 2):
        Y = interpret(p, X, seed)
        for r in range(R):
            got = Y[r].view(np_dtype(dt))
            assert_reduction_close(dt, got, exact, want[r], "rank %d" % r)
            # same FP32 adds in the same order as the schedule-ordered oracle: identical bits
            assert np.array_equal(got.view(np.uint8), bitwise[r].view(np.uint8))


@pytest.mark.parametrize("flags", [0, hb.FLAG_LEVEL_MAJOR, hb.FLAG_STAGED_RING])
@pytest.mark.parametrize("dt", DTYPES)
def test_ring_variants_same_bits(dt, flags):
    R, n = 6, 3001
    X = synth.normal_ranks(R, n, dt, seed=77)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(SMALL, flags=flags))
    assert p.check_hazards() == 0
    want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for seed in (0, 5):
        Y = interpret(p, X, seed)
        for r in range(R):
            assert np.array_equal(Y[r].view(np_dtype(dt)).view(np.uint8), want[r].view(np.uint8))


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("algo", [hb.ALGO_RING, hb.ALGO_RING_FUSED])
@pytest.mark.parametrize("R,counts", [(2, [3, 4]), (4, None), (5, [0, 7, 1000, 1, 300]), (16, None), (3, [0, 0, 11])])
def test_reducescatter_plans_match_oracle(R, counts, dt, algo):
    n = 4099 if counts is None else sum(counts)
    rc = np.diff(orc.floor_chunk_offsets(n, R)) if counts is None else np.array(counts)
    X = synth.normal_ranks(R, n, dt, seed=R + n, std=0.02)
    p = hb.hccl_plan_reducescatter(R, counts, n, dt, algo, SMALL)
    assert p.check_hazards() == 0
    want = orc.reducescatter(dt, X, rc)
    bitwise = orc.reducescatter_ring_f32(dt, X, rc)
    exact = orc.sum_f64(dt, X)
    offs = np.concatenate([[0], np.cumsum(rc)])
    for seed in (0, 3):
        Y = interpret(p, X, seed)
        for r in range(R):
            got = Y[r].view(np_dtype(dt))
            assert got.size == rc[r]
            assert_reduction_close(dt, got, exact[offs[r]:offs[r + 1]], want[r])
            assert np.array_equal(got.view(np.uint8), bitwise[r].view(np.uint8))


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("R,counts", [(2, [3, 4]), (4, None), (5, [0, 7, 1000, 1, 300]), (3, [0, 0, 11])])
def test_reducescatter_oneshot_is_the_oneshot_allreduce_cut_into_shards(R, counts, dt):
    n = 4099 if counts is None else sum(counts)
    offs = orc.floor_chunk_offsets(n, R) if counts is None else np.concatenate([[0], np.cumsum(counts)])
    X = synth.normal_ranks(R, n, dt, seed=R + n, std=0.02)
    p = hb.hccl_plan_reducescatter(R, counts, n, dt, hb.ALGO_ONESHOT, SMALL)
    assert p.check_hazards() == 0 and p.info().chain_depth <= 1
    whole = orc.allreduce_oneshot_f32(dt, X)[0]
    exact, want = orc.sum_f64(dt, X), orc.reducescatter(dt, X, np.diff(offs))
    Y = interpret(p, X, 3)
    for r in range(R):
        got = Y[r].view(np_dtype(dt))
        assert np.array_equal(got, whole[offs[r]:offs[r + 1]])
        assert_reduction_close(dt, got, exact[offs[r]:offs[r + 1]], want[r])


def test_reducescatter_rejects_bad_counts():
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_reducescatter(4, [1, 2, 3, 4], 11, hb.BF16)
    assert e.value.status == hb.ERR_COUNT_MISMATCH
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_allreduce(4, 10, 7)
    assert e.value.status == hb.ERR_DTYPE
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_allreduce(0, 10, hb.FP32)
    assert e.value.status == hb.ERR_INVALID_ARG
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_allreduce(hb.MAX_RANKS + 1, 10, hb.FP32)
    assert e.value.status == hb.ERR_INVALID_ARG


@pytest.mark.parametrize("algo", [hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_FANOUT])
@pytest.mark.parametrize("R,counts", [(1, [5]), (4, [3, 0, 1000, 17]), (8, None)])
def test_allgather_plans_match_oracle(R, counts, algo):
    dt = hb.BF16
    cs = counts if counts is not None else [321] * R
    rng = np.random.default_rng(R)
    X = [rng.integers(0, 65536, size=c, dtype=np.uint16) for c in cs]
    p = hb.hccl_plan_allgather(R, counts, 321, dt, algo, SMALL)
    assert p.check_hazards() == 0
    want = orc.allgatherv(X)
    for seed in (0, 9):
        Y = interpret(p, X, seed)
        for r in range(R):
            assert np.array_equal(Y[r].view(np.uint16), want[r])


def _a2a_case(R, seed, row_elems, dt, hi=9, packed=True):
    rng = np.random.default_rng(seed)
    C = synth.uniform_counts(R, seed, hi=hi)
    C[rng.integers(0, R), rng.integers(0, R)] = 0
    rb = row_elems * hb.ELEM_BYTES[dt]
    if packed:
        SD, RD = orc.packed_displs(C)
        send_rows = C.sum(axis=1)
    else:
        send_rows = np.full(R, int(C.sum(axis=1).max()) + 2)
        SD = rng.integers(0, int(send_rows[0]) - int(C.max()) + 1, size=(R, R))
        RD = np.zeros((R, R), dtype=np.int64)
        for d in range(R):
            o = int(rng.integers(0, 3))
            for s in rng.permutation(R):
                RD[d, s] = o
                o += int(C[s, d]) + int(rng.integers(0, 3))
    X = [rng.integers(0, 256, size=int(send_rows[s]) * rb, dtype=np.uint8) for s in range(R)]
    return C, SD, RD, X, rb


@pytest.mark.parametrize("R", [1, 2, 3, 5, 8])
@pytest.mark.parametrize("packed", [True, False])
def test_alltoallv_plans_match_oracle(R, packed):
    dt, row_elems = hb.BF16, 7            # 14-byte rows: nothing is 16-byte aligned
    C, SD, RD, X, rb = _a2a_case(R, 100 + R, row_elems, dt, packed=packed)
    p = hb.hccl_plan_alltoallv(R, C, None if packed else SD, C.T.copy(), None if packed else RD, dt, row_elems,
                               dict(SMALL, tile_bytes=256))
    assert p.check_hazards() == 0
    Yw = [np.full(p.extents(r)[1], 0xA5, dtype=np.uint8) for r in range(R)]
    orc.alltoallv(X, Yw, C, SD, RD, rb)
    for seed in (0, 4):
        Y = interpret(p, X, seed)
        for r in range(R):
            assert np.array_equal(Y[r], Yw[r])        # gaps keep the sentinel
    i = p.info()
    assert i.schedule_bytes == 2 * int(C.sum()) * rb == i.compulsory_bytes
    assert i.n_wqe == int((C > 0).sum())              # zero-length segments cost nothing


def test_alltoallv_validation():
    C = np.array([[1, 2], [3, 4]])
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_alltoallv(2, C, None, C, None, hb.FP16, 4)        # recvcounts must be the transpose
    assert e.value.status == hb.ERR_COUNT_MISMATCH
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_alltoallv(2, C, None, None, [[0, 2], [0, 1]], hb.FP16, 4)   # rank 0: rows [0,1) and [2,5) fine; rank 1: [0,2) and [1,5) overlap
    assert e.value.status == hb.ERR_OVERLAP
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_alltoallv(2, [[1, -1], [0, 0]], None, None, None, hb.FP16, 4)
    assert e.value.status == hb.ERR_INVALID_ARG
    # overlapping sends are legal
    p = hb.hccl_plan_alltoallv(2, C, [[0, 0], [0, 0]], None, None, hb.FP16, 4)
    assert p.info().n_wqe == 4


def test_all_zero_counts_is_an_empty_plan():
    p = hb.hccl_plan_alltoallv(3, np.zeros((3, 3), dtype=np.int64), None, None, None, hb.BF16, 128)
    assert p.info().n_tiles == 0 and p.info().schedule_bytes == 0
    assert interpret(p, [np.zeros(1, dtype=np.uint8)] * 3) is not None


# ------------------------------------------------------------------ two-level (rack-aware) schedules
@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("G,L,n", [(2, 2, 37), (2, 3, 1000), (4, 4, 4099), (3, 5, 257), (2, 2, 3), (2, 2, 0)])
def test_two_level_allreduce_matches_oracle(G, L, n, dt):
    R = G * L
    X = synth.normal_ranks(R, n, dt, seed=G * 7 + L)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING_2LEVEL, dict(SMALL, rack_size=L, chunk_bytes=512, chain_group=3))
    assert p.check_hazards() == 0
    bitwise = orc.allreduce_ring2_f32(dt, X, G, L)
    exact, want = orc.sum_f64(dt, X), orc.allreduce(dt, X)
    for seed in (0, 1, 2):
        Y = interpret(p, X, seed)
        for r in range(R):
            got = Y[r].view(np_dtype(dt))
            assert np.array_equal(got.view(np.uint8), bitwise[r].view(np.uint8))
            assert_reduction_close(dt, got, exact, want[r])
    # fewer dependent steps than the flat ring, and fewer bytes between racks
    flat = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(SMALL, rack_size=L)).info()
    i = p.info()
    if n >= R:
        assert i.chain_depth == 2 * (L - 1) + 2 * (G - 1) < flat.chain_depth
        assert i.crossrack_bytes < flat.crossrack_bytes


def test_two_level_degenerates_to_the_flat_ring():
    X = synth.normal_ranks(4, 100, hb.BF16, seed=1)
    want = orc.allreduce_ring_f32(hb.BF16, X, orc.floor_chunk_offsets(100, 4))
    for rack in (1, 4):
        p = hb.hccl_plan_allreduce(4, 100, hb.BF16, hb.ALGO_RING_2LEVEL, dict(SMALL, rack_size=rack))
        Y = interpret(p, X)
        assert np.array_equal(Y[0].view(np.uint16), want[0])
    with pytest.raises(hb.HcclError) as e:
        hb.hccl_plan_allreduce(6, 100, hb.BF16, hb.ALGO_RING_2LEVEL, dict(rack_size=4))
    assert e.value.status == hb.ERR_INVALID_ARG
    # fewer ranks than the default rack of 16 is a single rack: the flat ring, not a refusal
    X8 = synth.normal_ranks(8, 333, hb.BF16, seed=2)
    p = hb.hccl_plan_allreduce(8, 333, hb.BF16, hb.ALGO_RING_2LEVEL, SMALL)
    Y = interpret(p, X8)
    assert np.array_equal(Y[3].view(np.uint16), orc.allreduce_ring_f32(hb.BF16, X8, orc.floor_chunk_offsets(333, 8))[3])
    rng = np.random.default_rng(8)
    Xg = [rng.integers(0, 65536, size=50, dtype=np.uint16) for _ in range(6)]
    pg = hb.hccl_plan_allgather(6, None, 50, hb.BF16, hb.ALGO_RING_2LEVEL, SMALL)
    Yg = interpret(pg, Xg)
    assert np.array_equal(Yg[5].view(np.uint16), orc.allgatherv(Xg)[5])


@pytest.mark.parametrize("G,L", [(2, 2), (2, 3), (4, 4), (8, 16)])
def test_two_level_allgather_matches_oracle(G, L):
    R = G * L
    rng = np.random.default_rng(G * 100 + L)
    cs = [int(c) for c in rng.integers(0, 200, size=R)]
    cs[0] = 0
    X = [rng.integers(0, 65536, size=c, dtype=np.uint16) for c in cs]
    p = hb.hccl_plan_allgather(R, cs, 0, hb.BF16, hb.ALGO_RING_2LEVEL, dict(SMALL, rack_size=L, tile_bytes=64, chunk_bytes=128, chain_group=3))
    assert p.check_hazards() == 0
    want = orc.allgatherv(X)
    for seed in (0, 3):
        Y = interpret(p, X, seed)
        for r in range(R):
            assert np.array_equal(Y[r].view(np.uint16), want[r])
    flat = hb.hccl_plan_allgather(R, cs, 0, hb.BF16, hb.ALGO_RING, dict(SMALL, rack_size=L)).info()
    assert p.info().chain_depth == 1 + (G - 1) + (L - 1) <= flat.chain_depth
    assert p.info().crossrack_bytes < flat.crossrack_bytes


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("R,n", [(4, 1000), (5, 4099), (8, 257)])
def test_bidirectional_ring_matches_oracle(R, n, dt):
    es = hb.ELEM_BYTES[dt]
    granule = 64
    X = synth.normal_ranks(R, n, dt, seed=R * 3 + n)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(SMALL, chunk_bytes=granule * es, flags=hb.FLAG_BIDIRECTIONAL))
    assert p.check_hazards() == 0
    so, sc, sd = orc.bidirectional_segments(n, R, granule)
    want = orc.allreduce_ring_dir_f32(dt, X, so, sc, sd)
    for seed in (0, 1):
        Y = interpret(p, X, seed)
        for r in range(R):
            assert np.array_equal(Y[r].view(np_dtype(dt)).view(np.uint8), want[r].view(np.uint8))
    # reduce-scatter: rank c keeps chunk c of the same sums
    rs = hb.hccl_plan_reducescatter(R, None, n, dt, hb.ALGO_RING, dict(SMALL, chunk_bytes=granule * es, flags=hb.FLAG_BIDIRECTIONAL))
    assert rs.check_hazards() == 0
    offs = orc.floor_chunk_offsets(n, R)
    Y = interpret(rs, X, 2)
    for r in range(R):
        assert np.array_equal(Y[r].view(np_dtype(dt)).view(np.uint8), want[0][offs[r]:offs[r + 1]].view(np.uint8))


# ----------------------------------------------------------------- rings for the forwarding kernel (bulk engine, static chains)
@pytest.mark.parametrize("dt", DTYPES)
def test_bulk_engine_rings_are_independent_chains_with_a_slot_each(dt):
    """On the bulk engine a ring's chains get a scratch slot each (nothing is recycled, so nothing links them) and
    the packet carries no device counter; the hazard checker and the random-order interpreter agree with the oracle."""
    R, n = 5, 20011
    X = synth.normal_ranks(R, n, dt, seed=78)
    opts = dict(engine=hb.ENGINE_BULK, tile_bytes=2048, chunk_bytes=8192, sm_budget=6)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, opts)
    i = p.info()
    assert i.engine == hb.ENGINE_BULK and i.static_chains > 0 and i.n_syncs == 0 and p.check_hazards() == 0
    want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for seed in (0, 1):
        Y = interpret(p, X, seed)
        for r in range(R):
            assert np.array_equal(Y[r].view(np.uint8), want[r].view(np.uint8))
    p = hb.hccl_plan_reducescatter(R, None, n, dt, hb.ALGO_RING, opts)
    assert p.info().static_chains > 0 and p.info().n_syncs == 0 and p.check_hazards() == 0
    Y = interpret(p, X, 2)
    for r, w in enumerate(orc.reducescatter_ring_f32(dt, X, np.diff(orc.floor_chunk_offsets(n, R)))):
        assert np.array_equal(Y[r].view(np.uint8), w.view(np.uint8))
    # a hop-by-hop AllGather is a set of chains of copies of one source each: forwarded too
    pg = hb.hccl_plan_allgather(R, None, 776, dt, hb.ALGO_RING, opts)
    assert pg.info().static_chains > 0 and pg.info().n_syncs == 0 and pg.check_hazards() == 0
    Xg = [x[:776] for x in X]
    for r, w in enumerate(orc.allgatherv(Xg)):
        assert np.array_equal(interpret(pg, Xg, 4)[r].view(np.uint8), w.view(np.uint8))
    # what is not a set of simple chains keeps tickets and counters on this engine
    assert hb.hccl_plan_allreduce(8, 4099, dt, hb.ALGO_TREE, dict(opts, flags=hb.FLAG_STATIC_CHAINS)).info().static_chains == 0


def test_engine_left_to_the_library_for_rings():
    big = hb.hccl_plan_allreduce(8, 1 << 22, hb.BF16, hb.ALGO_RING).info()
    assert big.engine == hb.ENGINE_BULK and big.static_chains >= 148 and big.n_syncs == 0
    assert hb.hccl_plan_allreduce(8, 1 << 18, hb.BF16, hb.ALGO_RING).info().engine == hb.ENGINE_LSU
    assert hb.hccl_plan_allreduce(64, 1 << 18, hb.BF16, hb.ALGO_RING).info().engine == hb.ENGINE_BULK
    assert hb.hccl_plan_reducescatter(16, None, 1 << 26, hb.BF16, hb.ALGO_RING).info().static_chains > 0      # config 3
    assert hb.hccl_plan_allreduce(8, 1 << 22, hb.BF16, hb.ALGO_RING, dict(flags=hb.FLAG_LEVEL_MAJOR)).info().engine == hb.ENGINE_LSU   # another issue order: as before


def test_forwarding_tiles_fill_the_blocks():
    """Tile choice for the forwarding kernel: one round of the 148 blocks where the ring is small enough for that,
    many chains of one or two pieces per tile where it is large; every chain has a scratch slot of its own."""
    c1 = hb.hccl_plan_allreduce(4, 1 << 20, hb.FP32, hb.ALGO_RING).info()                    # config 1
    assert c1.engine == hb.ENGINE_BULK and c1.static_chains == 148 and c1.n_tiles == 148 * 6 and c1.scratch_bytes == 0
    c3 = hb.hccl_plan_reducescatter(16, None, 1 << 26, hb.BF16, hb.ALGO_RING).info()           # config 3
    assert c3.engine == hb.ENGINE_BULK and c3.static_chains >= 8 * 148 and c3.n_tiles == c3.static_chains * 15
    assert c3.tile_bytes <= 2 * 14336 * 4 and c3.scratch_bytes == (1 << 26) * 4                # at most two pieces per tile; a slot per chain
    mid = hb.hccl_plan_allreduce(16, 1 << 21, hb.BF16, hb.ALGO_RING).info()
    assert mid.engine == hb.ENGINE_BULK and 74 <= mid.static_chains <= 148                     # one round
    few = hb.hccl_plan_allreduce(16, 1 << 21, hb.BF16, hb.ALGO_RING, dict(sm_budget=8)).info()
    assert few.sm_budget == 8 and few.static_chains >= 8


# ----------------------------------------------------------------- static chains (a chain of tiles stays in one block)
@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("algo", [hb.ALGO_RING, hb.ALGO_RING_FUSED])
def test_static_chains_and_tickets_give_the_same_bits(algo, dt):
    R, n = 5, 20011
    X = synth.normal_ranks(R, n, dt, seed=77)
    want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    base = dict(tile_bytes=2048, chunk_bytes=8192, sm_budget=6)
    for flags, chained in ((0, True), (hb.FLAG_DYNAMIC_TICKETS, False)):
        p = hb.hccl_plan_allreduce(R, n, dt, algo, dict(base, flags=flags))
        i = p.info()
        assert (i.n_syncs == 0) == chained and (i.static_chains > 0) == chained   # no device counter is left when the chains are static
        assert p.check_hazards() == 0
        for seed in (0, 3, 4):
            Y = interpret(p, X, seed)
            for r in range(R):
                assert np.array_equal(Y[r].view(np.uint8), want[r].view(np.uint8))
    # ReduceScatter and the hop-by-hop AllGather take the same route
    rc = np.diff(orc.floor_chunk_offsets(n, R))
    p = hb.hccl_plan_reducescatter(R, None, n, dt, hb.ALGO_RING, base)
    assert p.info().n_syncs == 0 and p.check_hazards() == 0
    Y = interpret(p, X, 5)
    for r, w in enumerate(orc.reducescatter_ring_f32(dt, X, rc)):
        assert np.array_equal(Y[r].view(np.uint8), w.view(np.uint8))
    p = hb.hccl_plan_allgather(R, None, 777, dt, hb.ALGO_RING, base)
    assert p.info().n_syncs == 0 and p.check_hazards() == 0
    Xg = [x[:777] for x in X]
    for r, w in enumerate(orc.allgatherv(Xg)):
        assert np.array_equal(interpret(p, Xg, 6)[r].view(np.uint8), w.view(np.uint8))


def test_static_chains_need_independent_groups_of_equal_length():
    NB = 4096
    S, Rv = hb.BUF_SEND, hb.BUF_RECV
    opts = dict(tile_bytes=1024, sm_budget=4, flags=hb.FLAG_STATIC_CHAINS)
    E = hb.DEP_WQE_SYNC | hb.DEP_ELEMENTWISE
    # two chains of two copies each: eligible
    g = hb.Graph(2, [NB, NB], [2 * NB, 2 * NB])
    sg = g.add_subgraph(0)
    a = g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB)
    b = g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, 0), a=(S, 1, 0), count=NB)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, NB), a=(Rv, 0, 0), count=NB, dep_flags=E, dep_wqe=a)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, NB), a=(Rv, 1, 0), count=NB, dep_flags=E, dep_wqe=b)
    p = g.compile(opts)
    assert p.info().n_syncs == 0 and p.info().n_tiles == 16 and p.check_hazards() == 0
    rng = np.random.default_rng(0)
    X = [rng.integers(0, 256, NB, dtype=np.uint8) for _ in range(2)]
    for seed in range(6):
        Y = interpret(p, X, seed)
        assert np.array_equal(Y[0], np.concatenate([X[0], X[1]])) and np.array_equal(Y[1], np.concatenate([X[1], X[0]]))
    # a WQE with two successors (a fork) still makes one group: the block runs its three WQEs in issue order
    g = hb.Graph(2, [NB, NB], [2 * NB, 2 * NB])
    sg = g.add_subgraph(0)
    a = g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, 0), a=(Rv, 0, 0), count=NB, dep_flags=E, dep_wqe=a)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, NB), a=(Rv, 0, 0), count=NB, dep_flags=E, dep_wqe=a)
    p = g.compile(opts)
    assert p.info().static_chains == 4 and p.info().n_syncs == 0 and p.check_hazards() == 0
    for seed in range(4):
        Y = interpret(p, X, seed)
        assert np.array_equal(Y[0][:NB], X[0]) and np.array_equal(Y[1], np.concatenate([X[0], X[0]]))
    # groups of different lengths (a chain of two and a single WQE): the compiler keeps tickets and counters
    g = hb.Graph(2, [NB, NB], [2 * NB, 2 * NB])
    sg = g.add_subgraph(0)
    a = g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, 0), a=(Rv, 0, 0), count=NB, dep_flags=E, dep_wqe=a)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, NB), a=(S, 1, 0), count=NB)
    p = g.compile(opts)
    assert p.info().static_chains == 0 and p.info().n_syncs > 0 and p.check_hazards() == 0
    # a dependency on a whole WQE (not tile by tile) also keeps them
    g = hb.Graph(2, [NB, NB], [2 * NB, 2 * NB])
    sg = g.add_subgraph(0)
    a = g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, 0), a=(Rv, 0, 0), count=NB, dep_flags=hb.DEP_WQE_SYNC, dep_wqe=a)
    p = g.compile(opts)
    assert p.info().static_chains == 0 and p.info().n_syncs > 0
    # chains that touch the same bytes without a link between them: static or not, the checker objects
    g = hb.Graph(2, [NB, NB], [2 * NB, 2 * NB])
    sg = g.add_subgraph(0)
    a = g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, 0), a=(S, 0, 0), count=NB)
    b = g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, 0), a=(S, 1, 0), count=NB)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 1, NB), a=(Rv, 0, 0), count=NB, dep_flags=E, dep_wqe=a)
    g.add_wqe(sg, hb.OP_COPY, dst=(Rv, 0, NB), a=(Rv, 1, NB), count=NB, dep_flags=E, dep_wqe=b)   # reads the other chain's output
    p = g.compile(opts)
    assert p.info().n_syncs == 0 and p.check_hazards() > 0


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("R", [2, 3, 4, 5, 8])
def test_static_chains_on_degenerate_sizes(R, dt):
    """Default options (the planner asks for static chains by itself): empty chunks, one-element chunks, sizes
    around the rank count, several granules per chunk."""
    for n in (0, 1, 2, R - 1, R, R + 1, 17, 255, 257, 5000):
        X = synth.normal_ranks(R, n, dt, seed=R * 31 + n)
        want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
        p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(chunk_bytes=512, sm_budget=3))
        assert p.check_hazards() == 0
        if n >= R:
            assert p.info().static_chains > 0
        for seed in (0, 2):
            Y = interpret(p, X, seed)
            for r in range(R):
                assert np.array_equal(Y[r].view(np.uint8), want[r].view(np.uint8)), (n, r)


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("R,n", [(2, 600), (5, 3001), (8, 4099), (13, 700)])
def test_tree_as_groups_inside_one_block(R, n, dt):
    """The tree's sums have two predecessors each, so a granule's WQEs form one group (not a chain); with
    HCCL_FLAG_STATIC_CHAINS a block runs tile k of the whole group in issue order. Same bits as with tickets."""
    X = synth.normal_ranks(R, n, dt, seed=R + n)
    want = orc.allreduce_tree_f32(dt, X)
    for flags, grouped in ((hb.FLAG_STATIC_CHAINS, True), (hb.FLAG_DYNAMIC_TICKETS, False)):
        p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_TREE, dict(tile_bytes=512, chunk_bytes=2048, chain_group=64, sm_budget=5, flags=flags))
        i = p.info()
        assert (i.static_chains > 0) == grouped and p.check_hazards() == 0
        for seed in (0, 7):
            Y = interpret(p, X, seed)
            for r in range(R):
                assert np.array_equal(Y[r].view(np.uint8), want[r].view(np.uint8)), (flags, r)


def test_two_level_allgather_runs_as_groups_by_default():
    p = hb.hccl_plan_allgather(8, None, 500, hb.BF16, hb.ALGO_RING_2LEVEL, dict(rack_size=4, tile_bytes=256))
    i = p.info()
    assert i.static_chains > 0 and i.n_syncs == 0 and p.check_hazards() == 0
    q = hb.hccl_plan_allgather(8, None, 500, hb.BF16, hb.ALGO_RING_2LEVEL, dict(rack_size=4, tile_bytes=256, flags=hb.FLAG_DYNAMIC_TICKETS))
    assert q.info().static_chains == 0 and q.info().n_syncs > 0 and q.check_hazards() == 0
    assert q.info().crossrack_bytes == i.crossrack_bytes and q.info().schedule_bytes == i.schedule_bytes
    rng = np.random.default_rng(1)
    X = [rng.integers(0, 65536, size=500, dtype=np.uint16) for _ in range(8)]
    want = orc.allgatherv(X)
    for plan in (p, q):
        Y = interpret(plan, X, 3)
        for r in range(8):
            assert np.array_equal(Y[r].view(np.uint16), want[r])


def test_allreduce_auto_picks_by_size():
    small = hb.hccl_plan_allreduce(8, 1 << 19, hb.BF16, hb.ALGO_AUTO).info()       # 8 x 1 MiB: one-shot
    assert small.chain_depth == 1 and small.schedule_bytes == hb.hccl_plan_allreduce(8, 1 << 19, hb.BF16, hb.ALGO_ONESHOT).info().schedule_bytes
    large = hb.hccl_plan_allreduce(8, 1 << 23, hb.BF16, hb.ALGO_AUTO).info()       # 8 x 16 MiB: ring
    assert large.chain_depth == 14 and large.schedule_bytes == hb.hccl_plan_allreduce(8, 1 << 23, hb.BF16, hb.ALGO_RING).info().schedule_bytes
    assert hb.hccl_plan_allreduce(64, 1 << 19, hb.BF16, hb.ALGO_AUTO).info().chain_depth == 126   # 64 x 1 MiB: ring
    for fn in (hb.hccl_plan_reducescatter, hb.hccl_plan_allgather):
        with pytest.raises(hb.HcclError):
            fn(4, None, 1024, hb.BF16, hb.ALGO_AUTO)


def test_header_is_plain_c_and_links_against_the_library(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 and a C program must link and run against the
    library (host-only calls: no GPU needed)."""
    import os
    import subprocess
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    src = tmp_path / "use_hccl.c"
    src.write_text(
        '#include <stdio.h>\n#include "hccl.h"\n'
        "int main(void) {\n"
        "    hccl_plan_t* p = NULL;\n"
        "    hccl_plan_info_t info;\n"
        "    if (hccl_plan_allreduce(4, 1 << 20, HCCL_FP32, HCCL_ALGO_RING, NULL, &p) != HCCL_OK) return 1;\n"
        "    if (hccl_plan_info(p, &info) != HCCL_OK) return 2;\n"
        '    printf("%lld %lld %s\\n", (long long)info.n_wqe, (long long)info.schedule_bytes, hccl_status_string(HCCL_ERR_TIMEOUT));\n'
        "    hccl_plan_destroy(p);\n"
        "    return hccl_plan_allreduce(0, 1, HCCL_FP32, HCCL_ALGO_RING, NULL, &p) == HCCL_ERR_INVALID_ARG ? 0 : 3;\n"
        "}\n")
    exe = tmp_path / "use_hccl"
    libdir = os.path.dirname(hb.LIBRARY_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-I", os.path.join(root, "include"), str(src),
                           "-o", str(exe), "-L", libdir, "-l:" + os.path.basename(hb.LIBRARY_PATH), "-Wl,-rpath," + libdir])
    out = subprocess.check_output([str(exe)]).decode().split()
    assert out[0] == "24" and out[1] == str(60 << 20) and "timed" in " ".join(out[2:])
