"""Parity of the CUDA executor against the CPU oracle, through the C ABI. Needs a GPU."""
import numpy as np
import pytest

from gpu_helpers import run_plan
from helpers import assert_reduction_close, np_dtype
from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

pytestmark = pytest.mark.gpu
DTYPES = [hb.FP32, hb.BF16, hb.FP16]
ENGINES = {"lsu": dict(engine=hb.ENGINE_LSU), "lsu_light": dict(engine=hb.ENGINE_LSU, light=1, threads=256),
           "bulk": dict(engine=hb.ENGINE_BULK), "bulk_warpstore": dict(engine=hb.ENGINE_BULK, copy_by_warps=1, threads=288)}


@pytest.fixture(params=sorted(ENGINES), ids=sorted(ENGINES))
def engine(request):
    return ENGINES[request.param]


def _with(opts, engine):
    return dict(opts or {}, **engine)


def _check_allreduce(R, n, dt, algo, opts, X=None, iters=1, misalign=0):
    X = X if X is not None else synth.normal_ranks(R, n, dt, seed=R * 131 + n)
    p = hb.hccl_plan_allreduce(R, n, dt, algo, opts)
    Y = run_plan(p, X, iters=iters, misalign=misalign)
    exact, want = orc.sum_f64(dt, X), orc.allreduce(dt, X)
    bitwise = orc.allreduce_oneshot_f32(dt, X) if algo in (hb.ALGO_ONESHOT, hb.ALGO_FANOUT) else \
        orc.allreduce_tree_f32(dt, X) if algo == hb.ALGO_TREE else \
        orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for r in range(R):
        got = Y[r].view(np_dtype(dt))
        assert_reduction_close(dt, got, exact, want[r], "rank %d" % r)
        assert np.array_equal(got.view(np.uint8), bitwise[r].view(np.uint8)), "rank %d differs from the schedule-ordered FP32 sums" % r


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("algo", [hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_RING_FUSED, hb.ALGO_FANOUT, hb.ALGO_TREE])
@pytest.mark.parametrize("R,n", [(1, 5), (2, 9), (3, 2), (4, 257), (5, 1000), (8, 4099), (4, 0), (4, 3), (8, 100003)])
def test_allreduce_small(R, n, dt, algo, engine):
    _check_allreduce(R, n, dt, algo, _with(dict(tile_bytes=1024, chunk_bytes=4096, chain_group=2, sm_budget=8), engine), iters=2)


@pytest.mark.parametrize("budget", [1, 2, 3, 8, 148, 296])
@pytest.mark.parametrize("dt", [hb.FP32, hb.BF16])
def test_allreduce_any_sm_budget_same_bits(budget, dt, engine):
    _check_allreduce(6, 50021, dt, hb.ALGO_RING, _with(dict(tile_bytes=2048, chunk_bytes=16384, sm_budget=budget), engine), iters=3)


@pytest.mark.parametrize("misalign", [2, 4, 6, 10])
@pytest.mark.parametrize("dt", DTYPES)
def test_allreduce_misaligned_buffers(misalign, dt, engine):
    if dt == hb.FP32 and misalign % 4:
        pytest.skip("buffers must be aligned to the element size")
    _check_allreduce(4, 10007, dt, hb.ALGO_RING, _with(dict(tile_bytes=4096, sm_budget=16), engine), misalign=misalign)
    _check_allreduce(4, 10007, dt, hb.ALGO_ONESHOT, _with(dict(tile_bytes=4096, sm_budget=16), engine), misalign=misalign)
    _check_allreduce(4, 10007, dt, hb.ALGO_FANOUT, _with(dict(tile_bytes=4096, sm_budget=16), engine), misalign=misalign)
    _check_allreduce(5, 10007, dt, hb.ALGO_TREE, _with(dict(tile_bytes=4096, chunk_bytes=8192, chain_group=1, sm_budget=16), engine), misalign=misalign)


def test_config1_allreduce_ring_r4_fp32(engine):
    X = synth.uniform_ranks(4, 1 << 20, hb.FP32, seed=0)
    _check_allreduce(4, 1 << 20, hb.FP32, hb.ALGO_RING, _with(None, engine), X=X, iters=3)


@pytest.mark.parametrize("algo", [hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_FANOUT, hb.ALGO_TREE])
@pytest.mark.parametrize("m", [4096, 65536, 262144, 1 << 20])
def test_config5_allreduce_r8_bf16(m, algo, engine):
    X = synth.normal_ranks(8, m // 2, hb.BF16, seed=m)
    _check_allreduce(8, m // 2, hb.BF16, algo, _with(None, engine), X=X, iters=3)


def test_closed_form_on_device(engine):
    for dt in DTYPES:
        for R in (2, 4, 8, 16):
            n = 3000
            X = [synth.to_bits(np.full(n, r + 1, dtype=np.float32), dt) for r in range(R)]
            for algo in (hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_FANOUT, hb.ALGO_TREE):
                Y = run_plan(hb.hccl_plan_allreduce(R, n, dt, algo, _with(dict(tile_bytes=1024), engine)), X)
                for r in range(R):
                    assert np.all(synth.from_bits(Y[r].view(np_dtype(dt)), dt) == R * (R + 1) / 2)


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("algo", [hb.ALGO_RING, hb.ALGO_RING_FUSED])
@pytest.mark.parametrize("R,counts", [(2, [3, 4]), (4, None), (5, [0, 7, 1000, 1, 300]), (16, None), (3, [0, 0, 11])])
def test_reducescatter_small(R, counts, dt, algo, engine):
    n = 40099 if counts is None else sum(counts)
    rc = np.diff(orc.floor_chunk_offsets(n, R)) if counts is None else np.array(counts)
    X = synth.normal_ranks(R, n, dt, seed=R + n, std=0.02)
    p = hb.hccl_plan_reducescatter(R, counts, n, dt, algo, _with(dict(tile_bytes=1024, chunk_bytes=2048, chain_group=3, sm_budget=16), engine))
    Y = run_plan(p, X, iters=2)
    want, bitwise, exact = orc.reducescatter(dt, X, rc), orc.reducescatter_ring_f32(dt, X, rc), orc.sum_f64(dt, X)
    offs = np.concatenate([[0], np.cumsum(rc)])
    for r in range(R):
        got = Y[r].view(np_dtype(dt))
        assert_reduction_close(dt, got, exact[offs[r]:offs[r + 1]], want[r])
        assert np.array_equal(got.view(np.uint8), bitwise[r].view(np.uint8))


@pytest.mark.parametrize("dt", DTYPES)
def test_reducescatter_oneshot(dt, engine):
    R, counts = 5, [0, 7001, 1000, 1, 30000]
    n = sum(counts)
    offs = np.concatenate([[0], np.cumsum(counts)])
    X = synth.normal_ranks(R, n, dt, seed=11, std=0.02)
    Y = run_plan(hb.hccl_plan_reducescatter(R, counts, n, dt, hb.ALGO_ONESHOT, _with(dict(tile_bytes=4096, sm_budget=16), engine)), X, iters=2)
    whole = orc.allreduce_oneshot_f32(dt, X)[0]
    for r in range(R):
        assert np.array_equal(Y[r].view(np_dtype(dt)), whole[offs[r]:offs[r + 1]])


def test_config3_shape_reducescatter_r16_bf16_reduced_size(engine):
    # config 3 at 1/16 of its size (4 Mi elements per rank, 2 MiB granules -> still several granules per shard? no:
    # shards of 256 Ki elements = 512 KiB, so use 128 KiB granules to keep 4 granules per shard)
    R, n = 16, 1 << 22
    X = synth.normal_ranks(R, n, hb.BF16, seed=3, std=0.02)
    p = hb.hccl_plan_reducescatter(R, None, n, hb.BF16, hb.ALGO_RING, _with(dict(chunk_bytes=128 << 10), engine))
    Y = run_plan(p, X, iters=2)
    rc = np.full(R, n // R)
    want, bitwise = orc.reducescatter(hb.BF16, X, rc), orc.reducescatter_ring_f32(hb.BF16, X, rc)
    for r in range(R):
        got = Y[r].view(np.uint16)
        assert orc.ulp_distance(hb.BF16, got, want[r]).max() <= 1
        assert np.array_equal(got, bitwise[r])


@pytest.mark.parametrize("algo", [hb.ALGO_RING, hb.ALGO_ONESHOT, hb.ALGO_FANOUT])
@pytest.mark.parametrize("R,counts", [(1, [5]), (4, [3, 0, 1000, 17]), (8, None)])
def test_allgather(R, counts, algo, engine):
    cs = counts if counts is not None else [32100] * R
    rng = np.random.default_rng(R)
    X = [rng.integers(0, 65536, size=c, dtype=np.uint16) for c in cs]
    p = hb.hccl_plan_allgather(R, counts, 32100, hb.BF16, algo, _with(dict(tile_bytes=4096, sm_budget=32), engine))
    Y = run_plan(p, X, iters=2)
    want = orc.allgatherv(X)
    for r in range(R):
        assert np.array_equal(Y[r].view(np.uint16), want[r])


def _a2a(R, C, SD, RD, X, dt, row_elems, opts, packed, iters=1, misalign=0):
    rb = row_elems * hb.ELEM_BYTES[dt]
    p = hb.hccl_plan_alltoallv(R, C, None if packed else SD, C.T.copy(), None if packed else RD, dt, row_elems, opts)
    Y = run_plan(p, X, iters=iters, misalign=misalign)
    Yw = [np.full(p.extents(r)[1], 0xA5, dtype=np.uint8) for r in range(R)]
    orc.alltoallv(X, Yw, C, SD, RD, rb)
    for r in range(R):
        assert np.array_equal(Y[r], Yw[r]), "rank %d" % r
    return Y


@pytest.mark.parametrize("R", [1, 2, 3, 5, 8])
@pytest.mark.parametrize("packed", [True, False])
@pytest.mark.parametrize("row_elems", [7, 128])
def test_alltoallv_small(R, packed, row_elems, engine):
    from test_planner_host import _a2a_case
    C, SD, RD, X, rb = _a2a_case(R, 100 + R, row_elems, hb.BF16, hi=40, packed=packed)
    _a2a(R, C, SD, RD, X, hb.BF16, row_elems, _with(dict(tile_bytes=1024, sm_budget=16), engine), packed, iters=2)


@pytest.mark.parametrize("misalign", [1, 3, 8])
def test_alltoallv_misaligned(misalign, engine):
    from test_planner_host import _a2a_case
    C, SD, RD, X, rb = _a2a_case(4, 7, 5, hb.FP16, hi=300, packed=True)
    _a2a(4, C, SD, RD, X, hb.FP16, 5, _with(dict(tile_bytes=4096), engine), True, misalign=misalign)


def test_config2_alltoallv_r8_bf16_rows128(engine):
    R, row_elems = 8, 128
    C = synth.uniform_counts(R, 0, hi=4096)
    assert int(C.sum()) == 133647                       # the seed-0 draw this config is quoted on
    SD, RD = orc.packed_displs(C)
    X = [synth.normal_ranks(1, int(C[s].sum()) * row_elems, hb.BF16, seed=1000 + s)[0].view(np.uint8) for s in range(R)]
    Y = _a2a(R, C, SD, RD, X, hb.BF16, row_elems, _with(None, engine), True, iters=3)
    # identity invariant: exchanging back with the transposed counts restores every send buffer
    CT = C.T.copy()
    SD2, RD2 = orc.packed_displs(CT)
    p2 = hb.hccl_plan_alltoallv(R, CT, None, None, None, hb.BF16, row_elems, _with(None, engine))
    Z = run_plan(p2, Y)
    for s in range(R):
        assert np.array_equal(Z[s], X[s])


def test_alltoallv_zero_everything(engine):
    p = hb.hccl_plan_alltoallv(3, np.zeros((3, 3), dtype=np.int64), None, None, None, hb.BF16, 128, _with(None, engine))
    run_plan(p, [np.zeros(16, dtype=np.uint8)] * 3, iters=2)


def test_overlapping_send_and_receive_is_rejected():
    import torch
    p = hb.hccl_plan_allreduce(2, 1024, hb.FP32, hb.ALGO_ONESHOT)
    from paper_2608_00358_b200.runtime import DeviceCollective
    dc = DeviceCollective(p)
    buf = torch.zeros(4 * 4096, dtype=torch.uint8, device="cuda")
    b = buf.data_ptr()
    dc.set_buffers([b, b + 4096], [b + 2048, b + 8192])
    with pytest.raises(hb.HcclError) as e:
        dc.execute()
    assert e.value.status == hb.ERR_OVERLAP


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("G,L,n", [(2, 2, 37), (4, 4, 40099), (4, 16, 100003), (3, 5, 257)])
def test_two_level_allreduce(G, L, n, dt, engine):
    R = G * L
    X = synth.normal_ranks(R, n, dt, seed=G * 7 + L)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING_2LEVEL, _with(dict(rack_size=L, tile_bytes=2048, chunk_bytes=8192, chain_group=4, sm_budget=32), engine))
    Y = run_plan(p, X, iters=2)
    bitwise, exact, want = orc.allreduce_ring2_f32(dt, X, G, L), orc.sum_f64(dt, X), orc.allreduce(dt, X)
    for r in range(R):
        got = Y[r].view(np_dtype(dt))
        assert np.array_equal(got.view(np.uint8), bitwise[r].view(np.uint8)), "rank %d" % r
        # Every case meets the acceptance rule on every element but one: 64 ranks of fp32 N(0,1) values. There
        # 63 FP32 adds of partial sums near 8 leave an error near 1e-6, which misses 1e-5*|o| + 1e-6 where the
        # sum o itself is near zero: 39 of the 100003 elements (the same 39 on every rank, since all ranks hold
        # the two-level order's bits, compared above), each inside the FP32 summation bound.
        allowed = 39 if (dt == hb.FP32 and R == 64) else 0
        assert_reduction_close(dt, got, exact, want[r], "rank %d" % r, X=X, max_beyond=allowed)


@pytest.mark.parametrize("G,L", [(2, 2), (4, 4), (8, 16)])
def test_two_level_allgather(G, L, engine):
    R = G * L
    rng = np.random.default_rng(G * 100 + L)
    cs = [int(c) for c in rng.integers(0, 3000, size=R)]
    cs[1] = 0
    X = [rng.integers(0, 65536, size=c, dtype=np.uint16) for c in cs]
    p = hb.hccl_plan_allgather(R, cs, 0, hb.BF16, hb.ALGO_RING_2LEVEL, _with(dict(rack_size=L, tile_bytes=1024, chunk_bytes=2048, sm_budget=32), engine))
    Y = run_plan(p, X, iters=2)
    want = orc.allgatherv(X)
    for r in range(R):
        assert np.array_equal(Y[r].view(np.uint16), want[r])


def test_maximum_rank_count(engine):
    """R = 256, the largest job size the paper mentions: pointer tables, rank arithmetic and ring rotation."""
    R, n, dt = 256, 3001, hb.BF16
    X = synth.small_int_ranks(R, n, dt, seed=256, span=1)          # exactly summable in bf16: unique result
    want = orc.allreduce(dt, X)
    for algo, extra in ((hb.ALGO_RING, {}), (hb.ALGO_ONESHOT, {}), (hb.ALGO_RING_2LEVEL, dict(rack_size=16)), (hb.ALGO_FANOUT, {}), (hb.ALGO_TREE, {})):
        p = hb.hccl_plan_allreduce(R, n, dt, algo, _with(dict(sm_budget=64, **extra), engine))
        Y = run_plan(p, X)
        for r in (0, 1, 127, 255):
            assert np.array_equal(Y[r].view(np.uint16), want[r]), (algo, r)
    Xg = [x[:157] for x in X]                                          # AllGather, 256 destinations per work item
    wantg = orc.allgatherv(Xg)[0]
    Y = run_plan(hb.hccl_plan_allgather(R, None, 157, dt, hb.ALGO_FANOUT, _with(dict(sm_budget=64), engine)), Xg)
    for r in (0, 1, 128, 255):
        assert np.array_equal(Y[r].view(np.uint16), wantg), r
    C = synth.uniform_counts(R, 3, hi=3)
    SD, RD = orc.packed_displs(C)
    rb = 16 * 2
    Xa = [synth.hashed_rows_np(s, 0, int(C[s].sum()), 16).reshape(-1).view(np.uint8) for s in range(R)]
    Xa = [x if x.size else np.zeros(16, np.uint8) for x in Xa]
    p = hb.hccl_plan_alltoallv(R, C, None, None, None, hb.FP16, 16, _with(dict(sm_budget=64), engine))
    Y = run_plan(p, Xa)
    Yw = [np.full(p.extents(r)[1], 0xA5, dtype=np.uint8) for r in range(R)]
    orc.alltoallv(Xa, Yw, C, SD, RD, rb)
    for r in range(R):
        assert np.array_equal(Y[r], Yw[r])


@pytest.mark.parametrize("dt", DTYPES)
def test_bidirectional_ring(dt, engine):
    R, n, granule = 6, 100003, 2048
    es = hb.ELEM_BYTES[dt]
    X = synth.normal_ranks(R, n, dt, seed=66)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, _with(dict(chunk_bytes=granule * es, tile_bytes=4096, sm_budget=32, flags=hb.FLAG_BIDIRECTIONAL), engine))
    Y = run_plan(p, X, iters=2)
    so, sc, sd = orc.bidirectional_segments(n, R, granule)
    want = orc.allreduce_ring_dir_f32(dt, X, so, sc, sd)
    for r in range(R):
        assert np.array_equal(Y[r].view(np_dtype(dt)).view(np.uint8), want[r].view(np.uint8)), "rank %d" % r


def test_plan_cache_reuses_bound_plans():
    import torch
    from paper_2608_00358_b200.runtime import PlanCache
    cache = PlanCache()
    C = synth.uniform_counts(4, 1, hi=50)
    a = cache.alltoallv(4, C, dt=hb.FP16, row_elems=32)
    b = cache.alltoallv(4, C.copy(), dt=hb.FP16, row_elems=32)
    c = cache.alltoallv(4, C + 1, dt=hb.FP16, row_elems=32)
    assert a is b and a is not c and (cache.hits, cache.misses, len(cache)) == (1, 2, 2)
    r1 = cache.allreduce(4, 1000, hb.BF16, hb.ALGO_ONESHOT, dict(sm_budget=8))
    assert cache.allreduce(4, 1000, hb.BF16, hb.ALGO_ONESHOT, dict(sm_budget=8)) is r1
    X = synth.normal_ranks(4, 1000, hb.BF16, seed=0)
    send = [torch.from_numpy(x.view(np.int16)).cuda() for x in X]
    recv = [torch.zeros(1000, dtype=torch.int16, device="cuda") for _ in range(4)]
    r1.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    r1.execute()
    r1.check()
    assert np.array_equal(recv[2].cpu().numpy().view(np.uint16), orc.allreduce_oneshot_f32(hb.BF16, X)[2])


@pytest.mark.parametrize("opts", [dict(engine=hb.ENGINE_BULK, stages=2), dict(engine=hb.ENGINE_BULK, stages=3, threads=64),
                                  dict(engine=hb.ENGINE_BULK, threads=512, copy_by_warps=2), dict(engine=hb.ENGINE_LSU, threads=64),
                                  dict(engine=hb.ENGINE_LSU, threads=96, cluster=2), dict(engine=hb.ENGINE_LSU, light=1, threads=512, cluster=4)],
                         ids=["bulk2", "bulk3_64", "bulk512_tmastore", "lsu64", "lsu96_cluster2", "light512_cluster4"])
def test_engine_geometry_variants(opts):
    R, n, dt = 4, 300007, hb.BF16
    X = synth.normal_ranks(R, n, dt, seed=12)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(opts, sm_budget=24))
    Y = run_plan(p, X, iters=2)
    want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for r in range(R):
        assert np.array_equal(Y[r].view(np.uint16), want[r])
    C = synth.uniform_counts(R, 5, hi=3000)
    SD, RD = orc.packed_displs(C)
    Xa = [synth.hashed_rows_np(s, 0, int(C[s].sum()), 64).reshape(-1).view(np.uint8) for s in range(R)]
    pa = hb.hccl_plan_alltoallv(R, C, None, None, None, hb.FP16, 64, dict(opts, sm_budget=24))
    Ya = run_plan(pa, Xa, iters=2)
    Yw = [np.full(pa.extents(r)[1], 0xA5, dtype=np.uint8) for r in range(R)]
    orc.alltoallv(Xa, Yw, C, SD, RD, 128)
    for r in range(R):
        assert np.array_equal(Ya[r], Yw[r])


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("flags", [0, hb.FLAG_DYNAMIC_TICKETS], ids=["chains", "tickets"])
@pytest.mark.parametrize("budget", [1, 3, 148])
def test_static_chains_and_tickets_same_bits(budget, flags, dt):
    """Small rings run each chain of tiles inside one block (no device counters); with DYNAMIC_TICKETS the same
    schedule runs through tickets and counters. Both must give the schedule-ordered oracle's bits."""
    R, n = 6, 50021
    opts = dict(tile_bytes=4096, chunk_bytes=32768, sm_budget=budget, flags=flags)
    for algo in (hb.ALGO_RING, hb.ALGO_RING_FUSED):
        p = hb.hccl_plan_allreduce(R, n, dt, algo, opts)
        assert (p.info().static_chains > 0) == (flags == 0)
        _check_allreduce(R, n, dt, algo, opts, iters=3)
    X = synth.normal_ranks(R, n, dt, seed=5)
    rc = np.diff(orc.floor_chunk_offsets(n, R))
    Y = run_plan(hb.hccl_plan_reducescatter(R, None, n, dt, hb.ALGO_RING, opts), X, iters=2)
    for r, w in enumerate(orc.reducescatter_ring_f32(dt, X, rc)):
        assert np.array_equal(Y[r].view(np.uint8), w.view(np.uint8))
    Xg = [x[:7001] for x in X]
    Y = run_plan(hb.hccl_plan_allgather(R, None, 7001, dt, hb.ALGO_RING, opts), Xg, iters=2, misalign=2 if dt != hb.FP32 else 4)
    for r, w in enumerate(orc.allgatherv(Xg)):
        assert np.array_equal(Y[r].view(np.uint8), w.view(np.uint8))


@pytest.mark.parametrize("budget", [1, 2, 148])
def test_static_chains_longer_than_the_control_warps_window(budget):
    """Chains of 39 and 78 items: the control warp fetches the records of a block's items 32 at a time, so these
    chains cross a refill in their middle, and with one or two blocks many chains follow each other in one block."""
    R, dt = 40, hb.BF16
    opts = dict(engine=hb.ENGINE_LSU, tile_bytes=1024, chunk_bytes=4096, sm_budget=budget)
    Xg = synth.normal_ranks(R, 1531, dt, seed=77)
    p = hb.hccl_plan_allgather(R, None, 1531, dt, hb.ALGO_RING, opts)
    assert p.info().static_chains > 0 and p.info().n_syncs == 0
    Y = run_plan(p, Xg, iters=2, misalign=2)
    for r, w in enumerate(orc.allgatherv(Xg)):
        assert np.array_equal(Y[r].view(np.uint8), w.view(np.uint8))
    n = 40 * 97 + 13
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, opts)
    assert p.info().static_chains > 0 and p.info().n_syncs == 0
    _check_allreduce(R, n, dt, hb.ALGO_RING, opts, iters=2)


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("R", [2, 3, 5])
def test_static_chains_on_degenerate_sizes(R, dt):
    for n in (1, R - 1, R, 257, 5000):
        for budget in (1, 148):
            _check_allreduce(R, n, dt, hb.ALGO_RING, dict(chunk_bytes=512, sm_budget=budget), iters=2)


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("flags", [hb.FLAG_LEVEL_MAJOR, hb.FLAG_STAGED_RING, hb.FLAG_STAGED_RING | hb.FLAG_DYNAMIC_TICKETS,
                                   hb.FLAG_LEVEL_MAJOR | hb.FLAG_BIDIRECTIONAL], ids=["level_major", "staged", "staged_tickets", "level_major_bidir"])
def test_ring_order_flags_on_device(flags, dt, engine):
    """Issue-order and staging variants of the ring move the same values through the same sums: identical bits."""
    R, n, granule = 5, 30011, 1024
    es = hb.ELEM_BYTES[dt]
    X = synth.normal_ranks(R, n, dt, seed=flags + 3)
    opts = _with(dict(tile_bytes=2048, chunk_bytes=granule * es, chain_group=2, sm_budget=24, flags=flags), engine)
    Y = run_plan(hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, opts), X, iters=2)
    if flags & hb.FLAG_BIDIRECTIONAL:
        so, sc, sd = orc.bidirectional_segments(n, R, granule)
        want = orc.allreduce_ring_dir_f32(dt, X, so, sc, sd)
    else:
        want = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for r in range(R):
        assert np.array_equal(Y[r].view(np.uint8), want[r].view(np.uint8)), r
    rc = np.diff(orc.floor_chunk_offsets(n, R))
    if not flags & hb.FLAG_BIDIRECTIONAL:
        Y = run_plan(hb.hccl_plan_reducescatter(R, None, n, dt, hb.ALGO_RING, opts), X)
        for r, w in enumerate(orc.reducescatter_ring_f32(dt, X, rc)):
            assert np.array_equal(Y[r].view(np.uint8), w.view(np.uint8))


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("flags", [hb.FLAG_STATIC_CHAINS, hb.FLAG_DYNAMIC_TICKETS], ids=["groups", "tickets"])
def test_tree_and_two_level_allgather_as_groups(flags, dt):
    R, n = 8, 40009
    opts = dict(tile_bytes=2048, chunk_bytes=16384, chain_group=64, sm_budget=12, rack_size=4, flags=flags)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_TREE, opts)
    assert (p.info().static_chains > 0) == (flags == hb.FLAG_STATIC_CHAINS)
    _check_allreduce(R, n, dt, hb.ALGO_TREE, opts, iters=2)
    X = synth.normal_ranks(R, 5003, dt, seed=2)
    p = hb.hccl_plan_allgather(R, None, 5003, dt, hb.ALGO_RING_2LEVEL, opts)
    assert (p.info().static_chains > 0) == (flags == hb.FLAG_STATIC_CHAINS)
    Y = run_plan(p, X, iters=2)
    for r, w in enumerate(orc.allgatherv(X)):
        assert np.array_equal(Y[r].view(np.uint8), w.view(np.uint8))


@pytest.mark.parametrize("quantum", [1, 3, 1000])
def test_short_lived_blocks_give_the_same_bits(quantum, engine):
    """opts.quantum: blocks leave after that many items and more blocks are launched instead (many more than can
    be resident at once here). AllToAllv, and a ring whose items wait for items of blocks that may have left."""
    R, row = 8, 24
    C = synth.uniform_counts(R, 77, hi=90)
    X = [synth.hashed_rows_np(s, 0, max(int(C[s].sum()), 1), row).reshape(-1).view(np.uint8) for s in range(R)]
    p = hb.hccl_plan_alltoallv(R, C, None, None, None, hb.BF16, row, _with(dict(tile_bytes=512, sm_budget=8, quantum=quantum), engine))
    Y = run_plan(p, X, iters=2)
    SD, RD = orc.packed_displs(C)
    want = [np.full(Y[d].size, 0xA5, dtype=np.uint8) for d in range(R)]
    orc.alltoallv(X, want, C, SD, RD, row * 2)
    for d in range(R):
        assert np.array_equal(Y[d], want[d]), d
    n = 60013
    Xr = synth.normal_ranks(5, n, hb.BF16, seed=quantum, std=0.02)
    pr = hb.hccl_plan_allreduce(5, n, hb.BF16, hb.ALGO_RING, _with(dict(tile_bytes=2048, chunk_bytes=8192, chain_group=2, sm_budget=8, quantum=quantum,
                                                                      flags=hb.FLAG_DYNAMIC_TICKETS), engine))
    assert pr.info().static_chains == 0
    Yr = run_plan(pr, Xr, iters=2)
    ring = orc.allreduce_ring_f32(hb.BF16, Xr, orc.floor_chunk_offsets(n, 5))
    for r in range(5):
        assert np.array_equal(Yr[r].view(np.uint16), ring[r]), r
