"""The forwarding kernel (static chains on the bulk engine): a block walks a piece through all steps of a ring chain
with the running FP32 sums in registers; every step's result is still stored, none is read back (ring schedule of
the paper's Sec. II-A.2). Parity against the schedule-ordered FP32 oracle, bit for bit, and against the FP64
definition within the stated tolerance."""
import numpy as np
import pytest

from gpu_helpers import run_plan
from helpers import assert_reduction_close, np_dtype
from oracle import oracle as orc
from paper_2608_00358_b200 import binding as hb
from paper_2608_00358_b200 import synth

pytestmark = pytest.mark.gpu

DTYPES = [hb.FP32, hb.BF16, hb.FP16]
FORWARD = dict(engine=hb.ENGINE_BULK)   # the ring planners then ask for static chains with a scratch slot per chain


def _ring_cases():
    # (R, elements per rank, misalignment in bytes): whole pieces, ragged tails (n mod 8 != 0), fewer elements than ranks,
    # several pieces per tile, operands that are not 16-byte aligned (those chains run item by item)
    return [(3, 17, 0), (4, 40000, 0), (6, 123457, 0), (16, 16 * 9000 + 5, 0), (8, 8 * 14336 * 3, 0), (5, 70001, 4), (7, 5, 0)]


@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("budget", [1, 7, 148])
def test_reducescatter_and_allreduce_rings_in_the_forwarding_kernel(budget, dt):
    for R, n, mis in _ring_cases():
        opts = dict(FORWARD, sm_budget=budget, chunk_bytes=65536)
        X = synth.normal_ranks(R, n, dt, seed=R * 1000 + n)
        offs = orc.floor_chunk_offsets(n, R)
        p = hb.hccl_plan_reducescatter(R, None, n, dt, hb.ALGO_RING, opts)
        i = p.info()
        assert i.engine == hb.ENGINE_BULK and i.static_chains > 0 and i.n_syncs == 0 and p.check_hazards() == 0, (R, n)
        Y = run_plan(p, X, iters=2, misalign=mis if dt == hb.FP32 else mis // 2)
        for r, w in enumerate(orc.reducescatter_ring_f32(dt, X, np.diff(offs))):
            assert np.array_equal(Y[r].view(np.uint8)[:w.view(np.uint8).size], w.view(np.uint8)), ("reducescatter", R, n, r)
        p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, opts)
        i = p.info()
        assert i.engine == hb.ENGINE_BULK and i.static_chains > 0 and i.n_syncs == 0 and p.check_hazards() == 0, (R, n)
        Y = run_plan(p, X, iters=2, misalign=mis if dt == hb.FP32 else mis // 2)
        exact, want = orc.sum_f64(dt, X), orc.allreduce(dt, X)
        ring = orc.allreduce_ring_f32(dt, X, offs)
        for r in range(R):
            got = Y[r].view(np_dtype(dt))
            assert np.array_equal(got.view(np.uint8), ring[r].view(np.uint8)), ("allreduce", R, n, r)
            assert_reduction_close(dt, got, exact, want[r], "rank %d" % r)


def test_chunks_off_the_16_byte_boundary_are_forwarded_too():
    """R = 3 and 6 with a power-of-two count: no chunk starts on a multiple of 8 elements. Every piece then begins with
    the few elements before the first 16-byte boundary (the partials' scratch slots are shifted to the same phase), and
    the library picks the kernel by itself."""
    for R, n in ((3, 1 << 20), (6, (1 << 20) + 3)):
        for dt in (hb.BF16, hb.FP32):
            X = synth.normal_ranks(R, n, dt, seed=R + n)
            p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING)
            assert p.info().engine == hb.ENGINE_BULK and p.info().static_chains > 0 and p.check_hazards() == 0
            Y = run_plan(p, X, iters=2)
            ring = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
            for r in range(R):
                assert np.array_equal(Y[r].view(np.uint8), ring[r].view(np.uint8)), (R, n, dt, r)


def test_default_options_choose_the_forwarding_kernel_for_large_rings():
    """With about a chain of tiles per SM or more the planners pick it themselves; small rings stay on the register engine."""
    big = hb.hccl_plan_allreduce(8, 1 << 22, hb.BF16, hb.ALGO_RING).info()
    assert big.engine == hb.ENGINE_BULK and big.static_chains >= 148 and big.n_syncs == 0
    small = hb.hccl_plan_allreduce(8, 1 << 18, hb.BF16, hb.ALGO_RING).info()
    assert small.engine == hb.ENGINE_LSU and small.static_chains > 0
    rs = hb.hccl_plan_reducescatter(16, None, 1 << 23, hb.BF16, hb.ALGO_RING).info()
    assert rs.engine == hb.ENGINE_BULK and rs.static_chains >= 148 and rs.n_syncs == 0
    # a schedule that is not a set of simple chains keeps the tickets on the bulk engine
    tree = hb.hccl_plan_allreduce(64, 1 << 22, hb.BF16, hb.ALGO_TREE, dict(engine=hb.ENGINE_BULK, rack_size=16)).info()
    assert tree.static_chains == 0 and tree.n_syncs > 0
    tick = hb.hccl_plan_allreduce(8, 1 << 22, hb.BF16, hb.ALGO_RING, dict(flags=hb.FLAG_DYNAMIC_TICKETS)).info()
    assert tick.static_chains == 0


def test_large_ring_with_default_options_matches_the_oracle():
    """R = 8 x 4 Mi bf16 (the planner's own choice of engine, tiles and slots) on sampled ranks, every element."""
    R, n, dt = 8, 1 << 22, hb.BF16
    X = synth.normal_ranks(R, n, dt, seed=11, std=0.02)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING)
    assert p.info().engine == hb.ENGINE_BULK and p.info().static_chains > 0
    Y = run_plan(p, X, iters=2)
    ring = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    for r in range(R):
        assert np.array_equal(Y[r].view(np.uint8), ring[r].view(np.uint8)), r


def test_maximum_rank_count_in_the_forwarding_kernel():
    """R = 256: chains of 510 items (255 sums, 255 copies) fill the kernel's step table."""
    R, n, dt = 256, 256 * 40 + 3, hb.BF16
    X = synth.small_int_ranks(R, n, dt, seed=256, span=1)          # exactly summable in bf16: unique result
    want = orc.allreduce(dt, X)
    p = hb.hccl_plan_allreduce(R, n, dt, hb.ALGO_RING, dict(FORWARD, sm_budget=64))
    assert p.info().static_chains > 0 and p.info().engine == hb.ENGINE_BULK
    Y = run_plan(p, X)
    for r in (0, 1, 127, 255):
        assert np.array_equal(Y[r].view(np.uint16), want[r]), r


def test_trace_of_a_forwarded_ring_is_complete():
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective, enable_trace
    R, n, dt = 6, 6 * 20000, hb.BF16
    p = hb.hccl_plan_reducescatter(R, None, n, dt, hb.ALGO_RING, dict(FORWARD, sm_budget=5))
    X = synth.normal_ranks(R, n, dt, seed=3)
    send = [torch.from_numpy(x.view(np.int16)).cuda() for x in X]
    recv = [torch.zeros(n // R, dtype=torch.int16, device="cuda") for _ in range(R)]
    dc = DeviceCollective(p)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    tr = enable_trace(p)
    dc.execute()
    torch.cuda.synchronize()
    dc.check()
    rows = tr.cpu().numpy()[:p.info().n_tiles]
    assert (rows[:, 1] != 0).all() and (rows[:, 3] >= rows[:, 1]).all()      # every item was claimed and finished
    assert ((rows[:, 0] & 0xffffffff) == np.arange(p.info().n_tiles)).all()
    p.set_trace(0, 0)


def test_hand_built_chains_with_copies_wider_than_the_stages():
    """A work packet built WQE by WQE: two chains of bf16 + bf16 -> FP32 (scratch) -> + bf16 -> FP32 (receive buffer of rank 0),
    followed by 13 copies of that FP32 result round the ranks. The stages are sized for the 16-bit operands, so the FP32
    copies must go out from the registers although there are enough of them for the staged form. Against numpy."""
    import torch
    from paper_2608_00358_b200.runtime import DeviceCollective
    R, n = 14, 2 * 14336 + 1000                      # elements per chain: two whole pieces and a ragged third
    es, T = 2, 20000                               # tiles of 20000 elements: a whole piece and a part of one
    g = hb.Graph(R, [2 * n * es] * R, [2 * n * 4] * R, scratch_bytes=2 * n * 4)
    dep = hb.DEP_WQE_SYNC | hb.DEP_ELEMENTWISE
    for c in range(2):
        sg = g.add_subgraph(c)
        so, fo = c * n * es, c * n * 4
        w = g.add_wqe(sg, hb.OP_REDUCE, dst=(hb.BUF_SCRATCH, 0, fo), a=(hb.BUF_SEND, 0, so), b=(hb.BUF_SEND, 1, so), count=n,
                      dtypes=(hb.FP32, hb.BF16, hb.BF16), tile_count=T)
        w = g.add_wqe(sg, hb.OP_REDUCE, dst=(hb.BUF_RECV, 0, fo), a=(hb.BUF_SCRATCH, 0, fo), b=(hb.BUF_SEND, 2, so), count=n,
                      dtypes=(hb.FP32, hb.FP32, hb.BF16), dep_flags=dep, dep_wqe=w, tile_count=T)
        for r in range(1, R):
            w = g.add_wqe(sg, hb.OP_COPY, dst=(hb.BUF_RECV, r, fo), a=(hb.BUF_RECV, r - 1, fo), count=n * 4, dep_flags=dep, dep_wqe=w, tile_count=T * 4)
    p = g.compile(dict(engine=hb.ENGINE_BULK, flags=hb.FLAG_STATIC_CHAINS, sm_budget=3))
    assert p.info().static_chains > 0 and p.info().n_syncs == 0 and p.check_hazards() == 0
    X = synth.normal_ranks(R, 2 * n, hb.BF16, seed=41)
    send = [torch.from_numpy(x.view(np.int16)).cuda() for x in X]
    recv = [torch.zeros(2 * n, dtype=torch.float32, device="cuda") for _ in range(R)]
    dc = DeviceCollective(p)
    dc.set_buffers([t.data_ptr() for t in send], [t.data_ptr() for t in recv])
    for _ in range(2):
        dc.execute()
    torch.cuda.synchronize()
    dc.check()
    f = [(x.astype(np.uint32) << 16).view(np.float32) for x in X[:3]]
    want = (f[0] + f[1]) + f[2]
    for r in range(R):
        assert np.array_equal(recv[r].cpu().numpy().view(np.uint32), want.view(np.uint32)), r


def test_hop_by_hop_allgather_forwarded_as_bytes():
    """A flat-ring AllGather is a set of chains of copies of one source each: a piece is loaded once and stored to every
    hop's destination. Equal blocks, blocks of different (16-byte aligned) sizes, 256 ranks (256 copies per chain: the
    most one piece can take), and a block size off the 16-byte grid (then the library keeps the register engine)."""
    for dt in DTYPES:
        es = hb.ELEM_BYTES[dt]
        for R, counts in ((5, None), (7, [8 * (3 + 5 * r) for r in range(7)]), (6, [0, 64, 8, 0, 40000, 16])):
            n = 30008 if counts is None else None
            X = [synth.normal_ranks(1, (n if counts is None else max(counts[r], 1)), dt, seed=50 + r)[0][:(n if counts is None else counts[r])] for r in range(R)]
            p = hb.hccl_plan_allgather(R, counts, n or 0, dt, hb.ALGO_RING)
            assert p.info().engine == hb.ENGINE_BULK and p.info().static_chains > 0 and p.info().n_syncs == 0 and p.check_hazards() == 0
            Y = run_plan(p, X, iters=2)
            for r, w in enumerate(orc.allgatherv(X)):
                assert np.array_equal(Y[r].view(np.uint8)[:w.view(np.uint8).size], w.view(np.uint8)), (dt, R, r)
        assert hb.hccl_plan_allgather(4, None, 1001, dt, hb.ALGO_RING).info().engine == (hb.ENGINE_BULK if (1001 * es) % 16 == 0 else hb.ENGINE_LSU)
    R, n = 256, 72
    X = [synth.normal_ranks(1, n, hb.BF16, seed=r)[0] for r in range(R)]
    p = hb.hccl_plan_allgather(R, None, n, hb.BF16, hb.ALGO_RING, dict(sm_budget=32))
    assert p.info().engine == hb.ENGINE_BULK and p.info().static_chains > 0
    Y = run_plan(p, X)
    want = orc.allgatherv(X)
    for r in (0, 1, 128, 255):
        assert np.array_equal(Y[r].view(np.uint8)[:want[r].view(np.uint8).size], want[r].view(np.uint8)), r
