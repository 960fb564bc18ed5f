"""Pins for the CPU oracle: everything here checks oracle/ against something
other than itself: closed forms, invariants, hand-worked fixtures, library
routines on special cases, and brute force on tiny inputs. No GPU needed."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2608_00358_b200 import synth

FP32, BF16, FP16 = 0, 1, 2
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
DTYPES = [FP32, BF16, FP16]


def _parse_val(tok):
    return float.fromhex(tok) if "p" in tok.lower() else float(tok)


# ---------------------------------------------------------------- conversions
def test_rounding_ties_fixture():
    names = {"fp32": FP32, "bf16": BF16, "fp16": FP16}
    n = 0
    with open(os.path.join(GOLDEN, "rounding_ties.txt")) as f:
        for line in f:
            line = line.split("#")[0].split()
            if not line:
                continue
            dt, val, want = names[line[0]], _parse_val(line[1]), int(line[2], 16)
            got = orc.round_to(dt, np.array([val]))
            bits = int(got.view(np.uint32)[0]) if dt == FP32 else int(got[0])
            assert bits == want, (line, hex(bits))
            n += 1
    assert n >= 25


def test_fp16_rounding_matches_numpy_direct_conversion():
    # numpy converts float64 -> float16 in one correctly rounded step
    rng = np.random.default_rng(1)
    x = np.concatenate([
        rng.standard_normal(20000), rng.standard_normal(20000) * 1e-5, rng.standard_normal(2000) * 3e4,
        rng.uniform(-7e-8, 7e-8, 5000), np.array([0.0, -0.0, 65504.0, 65519.999, 65520.0, -65520.0, 1e9, 2.0 ** -24])])
    with np.errstate(over="ignore"):
        want = x.astype(np.float16).view(np.uint16)
    got = orc.round_to(FP16, x)
    assert np.array_equal(got, want)


def test_bf16_rounding_of_fp32_values_matches_torch():
    # torch rounds float32 -> bfloat16 to nearest even in one step; a float32 value is exact in float64
    rng = np.random.default_rng(2)
    with np.errstate(over="ignore"):   # the largest draws overflow to infinity on purpose
        x = np.concatenate([
            rng.standard_normal(50000).astype(np.float32),
            (rng.standard_normal(5000) * 1e-39).astype(np.float32),   # fp32 subnormals
            (rng.standard_normal(5000) * 1e38).astype(np.float32),
            np.array([0.0, -0.0, 3.3895314e38, 3.4028235e38, -3.4028235e38, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8],
                     dtype=np.float32)])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = orc.round_to(BF16, x.astype(np.float64))
    assert np.array_equal(got, want)


def test_fp32_rounding_matches_numpy():
    rng = np.random.default_rng(3)
    x = np.concatenate([rng.standard_normal(50000), rng.standard_normal(5000) * 1e-41,
                        rng.standard_normal(500) * 1e38, np.array([3.5e38, -3.5e38, 0.0, -0.0])])
    with np.errstate(over="ignore"):
        want = x.astype(np.float32).view(np.uint32)
    got = orc.round_to(FP32, x).view(np.uint32)
    assert np.array_equal(got, want)


@pytest.mark.parametrize("dt", [BF16, FP16])
def test_widen_all_16bit_patterns_roundtrip(dt):
    bits = np.arange(65536, dtype=np.uint16)
    v = orc.widen(dt, bits)
    lib = synth.from_bits(bits, dt)     # numpy (fp16) / torch (bf16) library widening
    finite = np.isfinite(lib)
    assert np.array_equal(np.isnan(v), np.isnan(lib))
    assert np.array_equal(v[~np.isnan(lib)], lib[~np.isnan(lib)])
    # widening then rounding is the identity on every finite pattern
    back = orc.round_to(dt, v[finite])
    assert np.array_equal(back, bits[finite])


# ------------------------------------------------------------- NMC primitive
@pytest.mark.parametrize("dta,dtb,dtd", list(itertools.product(DTYPES, DTYPES, DTYPES)))
def test_nmc_sum_against_numpy_float32_add(dta, dtb, dtd):
    rng = np.random.default_rng(10 + dta * 9 + dtb * 3 + dtd)
    n = 4099
    a = synth.to_bits(rng.standard_normal(n).astype(np.float32), dta)
    b = synth.to_bits((rng.standard_normal(n) * 3).astype(np.float32), dtb)
    got = orc.nmc(dtd, dta, a, dtb, b)
    # numpy float32 add is one IEEE fp32 add; the final conversion is the pinned rounding above
    s32 = synth.from_bits(a, dta).astype(np.float32) + synth.from_bits(b, dtb).astype(np.float32)
    assert s32.dtype == np.float32
    want = synth.to_bits(s32, dtd)
    assert np.array_equal(got.view(np.uint8), want.view(np.uint8))


def test_nmc_copy_form_and_fp32_add_is_not_fp64_add():
    a = np.array([1.0, 2.0 ** 24, -3.5], dtype=np.float32)
    assert np.array_equal(orc.nmc(FP32, FP32, a), a)
    # 2^24 + 1 is not representable in fp32: an FP32 add must return 2^24 (tie to even)
    b = np.array([0.0, 1.0, 0.0], dtype=np.float32)
    out = orc.nmc(FP32, FP32, a, FP32, b)
    assert out[1] == np.float32(2.0 ** 24)


# --------------------------------------------------------------- closed forms
@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("R", [1, 2, 3, 4, 8, 16, 25, 64])
def test_allreduce_rank_constant_closed_form(R, dt):
    n = 37
    X = [synth.to_bits(np.full(n, r + 1, dtype=np.float32), dt) for r in range(R)]
    want_val = R * (R + 1) / 2
    if dt == BF16 and R == 25:
        # 325 needs 9 significand bits: nearest bf16 values are 324 and 326, tie -> even significand (324)
        want_val = 324.0
    Y = orc.allreduce(dt, X)
    for r in range(R):
        assert np.all(synth.from_bits(Y[r], dt) == want_val)
    # the schedule-ordered variants reach the same exact value when no add rounds
    if not (dt == BF16 and R == 25):
        for Yv in (orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R)), orc.allreduce_oneshot_f32(dt, X)):
            for r in range(R):
                assert np.all(synth.from_bits(Yv[r], dt) == want_val)


@pytest.mark.parametrize("dt", DTYPES)
def test_allreduce_position_sensitive_closed_form(dt):
    R, n = 6, 101
    i = np.arange(n)
    X = [synth.to_bits(((r + 1) * (i % 7)).astype(np.float32), dt) for r in range(R)]
    want = (R * (R + 1) // 2) * (i % 7)          # <= 126: exact in every type
    for Y in (orc.allreduce(dt, X), orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R)),
              orc.allreduce_oneshot_f32(dt, X)):
        for r in range(R):
            assert np.array_equal(synth.from_bits(Y[r], dt), want.astype(np.float64))


def test_ring_order_is_the_stated_chain():
    # R = 3, one element per chunk; values chosen so the FP32 result depends on the order of the adds.
    big, one = np.float32(2.0 ** 24), np.float32(1.0)
    # chunk c is summed as (X_{c+1} + X_{c+2}) + X_c
    X = [np.array([one, big, -big], dtype=np.float32),      # rank 0
         np.array([big, one, one], dtype=np.float32),       # rank 1
         np.array([-big, -big, big], dtype=np.float32)]     # rank 2
    Y = orc.allreduce_ring_f32(FP32, X, [0, 1, 2, 3])
    # chunk 0: (X1 + X2) + X0 = (2^24 - 2^24) + 1 = 1
    # chunk 1: (X2 + X0) + X1 = (-2^24 + 2^24) + 1 = 1
    # chunk 2: (X0 + X1) + X2 = (-2^24 + 1 -> -2^24+1 exactly representable) + 2^24 = 1
    assert list(Y[0]) == [1.0, 1.0, 1.0]
    # rank order 0,1,2 instead: element 0: (1 + 2^24) -> 2^24 (the 1 is lost), then - 2^24 = 0
    Z = orc.allreduce_oneshot_f32(FP32, X)
    assert Z[0][0] == 0.0 and Z[2][0] == 0.0
    # and the FP64 definition keeps everything
    assert list(orc.allreduce(FP32, X)[1]) == [1.0, 1.0, 1.0]


# ----------------------------------------------------------------- invariants
@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("R,n", [(2, 9), (4, 257), (5, 17), (8, 255), (16, 64)])
def test_sums_match_numpy_and_invariants(R, n, dt):
    X = synth.normal_ranks(R, n, dt, seed=R * 1000 + n)
    Y = orc.allreduce(dt, X)
    # library special case: numpy's float64 reduction over the rank axis (same order 0..R-1)
    s = np.add.reduce(np.stack([synth.from_bits(x, dt) for x in X]), axis=0)
    assert np.array_equal(orc.sum_f64(dt, X), s)
    if dt == FP16:
        assert np.array_equal(Y[0], s.astype(np.float16).view(np.uint16))
    if dt == FP32:
        assert np.array_equal(Y[0], s.astype(np.float32))
    # (b) identical on all ranks
    for r in range(1, R):
        assert np.array_equal(Y[r], Y[0])
    # (a) ReduceScatter shards concatenated = AllReduce, for ragged shard sizes
    rc = np.diff(orc.floor_chunk_offsets(n, R))
    S = orc.reducescatter(dt, X, rc)
    assert np.array_equal(np.concatenate(S), Y[0])
    rc2 = np.zeros(R, dtype=np.int64)
    rc2[0], rc2[-1] = n // 3, n - n // 3
    assert np.array_equal(np.concatenate(orc.reducescatter(dt, X, rc2)), Y[0])
    # ring-ordered scatter concatenated = ring-ordered AllReduce
    A = orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))
    assert np.array_equal(np.concatenate(orc.reducescatter_ring_f32(dt, X, rc)), A[0])
    # fp32-ordered results stay within the acceptance rule of the FP64 definition
    for V in (A[0], orc.allreduce_oneshot_f32(dt, X)[0]):
        if dt == FP32:
            assert np.all(np.abs(V.astype(np.float64) - s) <= 1e-5 * np.abs(s) + 1e-6)
        else:
            assert orc.ulp_distance(dt, V, Y[0]).max() <= 1


@pytest.mark.parametrize("dt", DTYPES)
def test_rank_permutation_and_power_of_two_scaling(dt):
    R, n = 7, 300
    X = synth.small_int_ranks(R, n, dt, seed=5)           # exactly summable
    Y = orc.allreduce(dt, X)[0]
    perm = [3, 0, 6, 1, 5, 2, 4]
    assert np.array_equal(orc.allreduce(dt, [X[p] for p in perm])[0], Y)
    assert np.array_equal(orc.allreduce_ring_f32(dt, [X[p] for p in perm], orc.floor_chunk_offsets(n, R))[0], Y)
    X4 = [synth.to_bits((synth.from_bits(x, dt) * 4).astype(np.float32), dt) for x in X]
    assert np.array_equal(synth.from_bits(orc.allreduce(dt, X4)[0], dt), 4 * synth.from_bits(Y, dt))


def test_r1_is_a_copy():
    for dt in DTYPES:
        X = synth.normal_ranks(1, 33, dt, seed=9)
        assert np.array_equal(orc.allreduce(dt, X)[0], X[0])
        assert np.array_equal(orc.reducescatter(dt, X, [33])[0], X[0])
        assert np.array_equal(orc.allreduce_ring_f32(dt, X, [0, 33])[0], X[0])
    X = [np.arange(40, dtype=np.uint8)]
    Y = [np.zeros(40, dtype=np.uint8)]
    orc.alltoallv(X, Y, [[10]], [[0]], [[0]], 4)
    assert np.array_equal(Y[0], X[0])


def test_ulp_distance_definition():
    a = np.array([0x0000, 0x8000, 0x0001, 0x3f80, 0x3f80, 0xbf80], dtype=np.uint16)
    b = np.array([0x8000, 0x0001, 0x8001, 0x3f81, 0x3f7f, 0xbf82], dtype=np.uint16)
    assert list(orc.ulp_distance(BF16, a, b)) == [0, 1, 2, 1, 1, 2]


# ------------------------------------------------------------------ AllToAllv
def test_alltoallv_hand_worked_fixture():
    d = {}
    with open(os.path.join(GOLDEN, "alltoallv_two_ranks.txt")) as f:
        for line in f:
            t = line.split("#")[0].split()
            if t:
                d[t[0]] = [int(v) for v in t[1:]]
    R = d["R"][0]
    X = [np.array(d["X%d" % r], dtype=np.int32).view(np.uint8) for r in range(R)]
    Y = [np.full(len(d["Y%d" % r]) * 4, 0xEE, dtype=np.uint8) for r in range(R)]
    C = np.array(d["C"]).reshape(R, R)
    SD = np.array(d["SD"]).reshape(R, R)
    RD = np.array(d["RD"]).reshape(R, R)
    # the fixture's packed receive displacements are what the packing rule gives
    assert np.array_equal(orc.packed_displs(C)[1], RD)
    orc.alltoallv(X, Y, C, SD, RD, 4)
    for r in range(R):
        assert list(Y[r].view(np.int32)) == d["Y%d" % r]


def _fancy_alltoallv(X, C, SD, RD, row_bytes, recv_rows, fill):
    """Second, differently written reference: numpy fancy indexing, one gather per destination."""
    R = C.shape[0]
    out = []
    for d in range(R):
        y = np.full((recv_rows[d], row_bytes), fill, dtype=np.uint8)
        for s in range(R):
            k = np.arange(C[s, d])
            y[RD[d, s] + k] = X[s].reshape(-1, row_bytes)[SD[s, d] + k]
        out.append(y.reshape(-1))
    return out


def test_alltoallv_every_count_matrix_r2():
    row_bytes = 3                                     # odd row size: byte granularity
    for cs in itertools.product(range(3), repeat=4):
        C = np.array(cs).reshape(2, 2)
        SD, RD = orc.packed_displs(C)
        X = [np.arange(100 * s, 100 * s + int(C[s].sum()) * row_bytes, dtype=np.uint8) for s in range(2)]
        recv_rows = C.sum(axis=0)
        Y = [np.full(int(recv_rows[d]) * row_bytes, 0xAB, dtype=np.uint8) for d in range(2)]
        orc.alltoallv(X, Y, C, SD, RD, row_bytes)
        want = _fancy_alltoallv(X, C, SD, RD, row_bytes, recv_rows, 0xAB)
        for d in range(2):
            assert np.array_equal(Y[d], want[d])


@pytest.mark.parametrize("R", [1, 2, 3, 4, 5, 8])
def test_alltoallv_random_gaps_overlapping_sends(R):
    rng = np.random.default_rng(40 + R)
    row_bytes = 6
    C = rng.integers(0, 6, size=(R, R))
    C[rng.integers(0, R), rng.integers(0, R)] = 0
    send_rows = int(C.sum(axis=1).max()) + 3
    SD = rng.integers(0, send_rows - C.max() + 1, size=(R, R))        # arbitrary: overlaps and gaps allowed
    # receive side: shuffled segment order with gaps of 0..2 rows, never overlapping
    RD = np.zeros((R, R), dtype=np.int64)
    recv_rows = np.zeros(R, dtype=np.int64)
    for d in range(R):
        o = int(rng.integers(0, 3))
        for s in rng.permutation(R):
            RD[d, s] = o
            o += int(C[s, d]) + int(rng.integers(0, 3))
        recv_rows[d] = o
    X = [rng.integers(0, 256, size=send_rows * row_bytes, dtype=np.uint8) for _ in range(R)]
    Y = [np.full(int(recv_rows[d]) * row_bytes, 0x5A, dtype=np.uint8) for d in range(R)]
    orc.alltoallv(X, Y, C, SD, RD, row_bytes)
    want = _fancy_alltoallv(X, C, SD, RD, row_bytes, recv_rows, 0x5A)   # gaps keep the sentinel
    for d in range(R):
        assert np.array_equal(Y[d], want[d])
    # restricted to one destination: only that rank is written
    Y2 = [np.full(int(recv_rows[d]) * row_bytes, 0x5A, dtype=np.uint8) for d in range(R)]
    orc.alltoallv(X, Y2, C, SD, RD, row_bytes, dst_only=R - 1)
    assert np.array_equal(Y2[R - 1], want[R - 1])
    for d in range(R - 1):
        assert np.all(Y2[d] == 0x5A)


@pytest.mark.parametrize("R,seed", [(3, 0), (8, 0), (8, 1)])
def test_alltoallv_transpose_roundtrip_is_identity_and_conserves_rows(R, seed):
    row_elems = 16
    C = synth.uniform_counts(R, seed, hi=9)
    SD, RD = orc.packed_displs(C)
    X = [synth.hashed_rows_np(s, 0, int(C[s].sum()), row_elems).reshape(-1).view(np.uint8) for s in range(R)]
    recv_rows = C.sum(axis=0)
    Y = [np.zeros(int(recv_rows[d]) * row_elems * 2, dtype=np.uint8) for d in range(R)]
    orc.alltoallv(X, Y, C, SD, RD, row_elems * 2)
    # conservation: bytes and the multiset of rows
    assert sum(y.size for y in Y) == sum(x.size for x in X)
    rows = lambda bufs: sorted(bytes(r) for b in bufs for r in b.reshape(-1, row_elems * 2))
    assert rows(X) == rows(Y)
    # second exchange with the transposed counts brings every send buffer back
    CT = C.T.copy()
    SD2, RD2 = orc.packed_displs(CT)
    Z = [np.zeros_like(x) for x in X]
    orc.alltoallv(Y, Z, CT, SD2, RD2, row_elems * 2)
    for s in range(R):
        assert np.array_equal(Z[s], X[s])


def test_allgatherv_is_concatenation():
    X = [np.arange(5, dtype=np.float32), np.arange(0, dtype=np.float32), np.arange(3, dtype=np.float32) + 10]
    Y = orc.allgatherv(X)
    for y in Y:
        assert np.array_equal(y, np.concatenate(X))


# ----------------------------------------------------------- input generators
def test_hashed_rows_host_and_torch_agree_and_are_finite():
    a = synth.hashed_rows_np(5, 1000, 64, 256)
    b = synth.hashed_rows_torch(5, 1000, 64, 256, "cpu").numpy().view(np.uint16)
    assert np.array_equal(a, b)
    assert np.all((a & 0x7C00) != 0x7C00)
    assert len(np.unique(a)) > 10000
    assert not np.array_equal(a, synth.hashed_rows_np(6, 1000, 64, 256))
    assert np.array_equal(a[3:5], synth.hashed_rows_np(5, 1003, 2, 256))


def test_config_count_draws():
    C = synth.uniform_counts(8, 0)
    assert C.shape == (8, 8) and C.min() >= 0 and C.max() <= 4096
    Z = synth.zipf_counts(64, 0)
    assert Z.min() >= 1 and Z.max() == 32768


# ------------------------------------------------------------- two-level ring order
@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("G,L", [(2, 2), (2, 3), (4, 4), (3, 5), (1, 4), (4, 1)])
def test_two_level_ring_order(G, L, dt):
    R, n = G * L, 211
    # exactly summable data: the order cannot matter, the result must be the plain sum on every rank
    X = synth.small_int_ranks(R, n, dt, seed=G * 10 + L)
    want = orc.allreduce(dt, X)
    Y = orc.allreduce_ring2_f32(dt, X, G, L)
    for r in range(R):
        assert np.array_equal(Y[r], want[r])
    # random data: within the acceptance rule of the FP64 definition
    X = synth.normal_ranks(R, n, dt, seed=G * 100 + L)
    Y, want, s = orc.allreduce_ring2_f32(dt, X, G, L), orc.allreduce(dt, X), orc.sum_f64(dt, X)
    if dt == FP32:
        assert np.all(np.abs(Y[0].astype(np.float64) - s) <= 1e-5 * np.abs(s) + 1e-6)
    else:
        assert orc.ulp_distance(dt, Y[0], want[0]).max() <= 1
    # with a single rack, or racks of one rank, it is the flat ring
    if G == 1:
        assert np.array_equal(Y[0], orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, L))[0])


def test_two_level_order_is_racks_first():
    # G = 2 racks of L = 2, one element per sub-chunk; values make the FP32 result depend on the grouping.
    big, one = np.float32(2.0 ** 24), np.float32(1.0)
    # sub-chunk (j, k): racks' partials P_g = X_{g,j+1} + X_{g,j}, total = P_{k+1} + P_k
    # element 0 is (j=0,k=0): P_0 = X[1] + X[0], P_1 = X[3] + X[2], total = P_1 + P_0
    X = [np.full(4, v, dtype=np.float32) for v in (big, one, -big, one)]     # ranks (0,0) (0,1) (1,0) (1,1)
    Y = orc.allreduce_ring2_f32(FP32, X, 2, 2)
    # racks first: (1 + 2^24) -> 2^24 and (1 - 2^24) -> -2^24 + 1 exactly; total = 1
    assert np.all(Y[0] == 1.0)
    # the flat ring adds rank by rank and loses nothing different here? (X1 + X2) + X3 + X0 = ((1 - 2^24) + 1) + 2^24 = 2
    assert orc.allreduce_ring_f32(FP32, X, [0, 1, 2, 3, 4])[0][0] == 2.0
    assert orc.allreduce(FP32, X)[0][0] == 2.0


# ------------------------------------------------------------- bidirectional ring order
@pytest.mark.parametrize("dt", DTYPES)
def test_bidirectional_ring_order(dt):
    R, n, granule = 5, 403, 32
    so, sc, sd = orc.bidirectional_segments(n, R, granule)
    assert so[0] == 0 and so[-1] == n and np.all(np.diff(so) > 0) and set(sd) == {1, -1}
    X = synth.small_int_ranks(R, n, dt, seed=8)               # exact: order cannot matter
    Y = orc.allreduce_ring_dir_f32(dt, X, so, sc, sd)
    assert np.array_equal(Y[0], orc.allreduce(dt, X)[0]) and np.array_equal(Y[R - 1], Y[0])
    # all segments forwards = the unidirectional ring
    X = synth.normal_ranks(R, n, dt, seed=9)
    fwd = orc.allreduce_ring_dir_f32(dt, X, so, sc, np.ones_like(sd))
    assert np.array_equal(fwd[0], orc.allreduce_ring_f32(dt, X, orc.floor_chunk_offsets(n, R))[0])
    # backwards on ranks listed in reverse = forwards on the original list (a mirror image of the ring)
    Xr = X[::-1]
    scr = (R - 1 - sc)
    # chunk ranges move with the mirror only if chunks are equal-sized; use one segment per equal chunk
    n2 = 50 * R
    X2 = synth.normal_ranks(R, n2, dt, seed=10)
    so2, sc2, _ = orc.bidirectional_segments(n2, R, 10 ** 9)
    back = orc.allreduce_ring_dir_f32(dt, X2, so2, sc2, -np.ones_like(sc2))
    # element i of chunk c backwards: ((X_{c-1}+X_{c-2})+...)+X_c. Mirror ranks r -> R-1-r: chunk c' = R-1-c forwards
    mirrored = [np.concatenate([x[(R - 1 - c) * 50:(R - c) * 50] for c in range(R)]) for x in X2[::-1]]
    fwd2 = orc.allreduce_ring_f32(dt, mirrored, orc.floor_chunk_offsets(n2, R))
    unmirror = np.concatenate([fwd2[0][(R - 1 - c) * 50:(R - c) * 50] for c in range(R)])
    assert np.array_equal(back[0], unmirror)
    del Xr, scr


def test_bidirectional_order_example():
    big, one = np.float32(2.0 ** 24), np.float32(1.0)
    # R = 3, chunk 0, one element. forwards: (X1 + X2) + X0; backwards: (X2 + X1) + X0 -- same pair first, so use
    # chunk 1: forwards (X2 + X0) + X1, backwards (X0 + X2) + X1: also the same pair. With R = 4, chunk 0:
    # forwards ((X1 + X2) + X3) + X0, backwards ((X3 + X2) + X1) + X0.
    X = [np.array([v], dtype=np.float32) for v in (one, big, one, -big)]       # X0..X3
    so, sc = np.array([0, 1]), np.array([0])
    f = orc.allreduce_ring_dir_f32(FP32, X, so, sc, np.array([1]))[0][0]      # ((2^24 + 1) - 2^24) + 1 = 0 + 1 = 1
    b = orc.allreduce_ring_dir_f32(FP32, X, so, sc, np.array([-1]))[0][0]     # ((-2^24 + 1) + 2^24) + 1 = 1 + 1 = 2
    assert f == 1.0 and b == 2.0


# ----------------------------------------------------------------- binary-tree order
@pytest.mark.parametrize("dt", DTYPES)
@pytest.mark.parametrize("R", [1, 2, 3, 4, 5, 6, 7, 8, 13, 16, 64])
def test_tree_order_built_from_the_pinned_two_input_sum(R, dt):
    """The tree is pairs of neighbours, level by level, an odd one out moving up unchanged. Rebuilt here from
    numpy float32 adds (a different implementation of the FP32 add than the oracle's C) and checked against
    the closed form R(R+1)/2 on rank-constant inputs."""
    n = 97
    X = synth.normal_ranks(R, n, dt, seed=R * 7 + 1)
    v = [synth.from_bits(x, dt).astype(np.float32) for x in X]
    while len(v) > 1:
        nxt = [v[2 * j] + v[2 * j + 1] for j in range(len(v) // 2)]   # numpy float32 add
        if len(v) % 2:
            nxt.append(v[-1])
        v = nxt
    want = orc.round_to(dt, v[0].astype(np.float64))
    Y = orc.allreduce_tree_f32(dt, X)
    for r in range(R):
        assert np.array_equal(Y[r], want)
    # within the acceptance rule of the FP64 definition
    ref, s = orc.allreduce(dt, X)[0], orc.sum_f64(dt, X)
    if dt == FP32:
        assert np.all(np.abs(Y[0].astype(np.float64) - s) <= 1e-5 * np.abs(s) + 1e-6)
    else:
        assert orc.ulp_distance(dt, Y[0], ref).max() <= 1
    # closed form, exact in every type for these R
    if R in (1, 2, 4, 8, 16, 64):
        Xc = [synth.to_bits(np.full(n, r + 1, dtype=np.float32), dt) for r in range(R)]
        assert np.all(synth.from_bits(orc.allreduce_tree_f32(dt, Xc)[0], dt) == R * (R + 1) / 2)


def test_tree_order_example():
    # R = 5: ((x0 + x1) + (x2 + x3)) + x4. Values chosen so that other orders give other FP32 results.
    big, one = np.float32(2.0 ** 24), np.float32(1.0)
    X = [np.array([v], dtype=np.float32) for v in (big, one, one, -big, one)]
    # (2^24 + 1) -> 2^24 ; (1 - 2^24) -> -2^24 + 1 exactly ; sum = 1 ; + 1 = 2
    assert orc.allreduce_tree_f32(FP32, X)[3][0] == 2.0
    # rank order 0..4: ((2^24 + 1) + 1) -> 2^24, - 2^24 = 0, + 1 = 1
    assert orc.allreduce_oneshot_f32(FP32, X)[0][0] == 1.0
    assert orc.allreduce(FP32, X)[0][0] == 3.0      # the FP64 definition keeps every 1
    # swapping the two members of a pair changes nothing (FP32 addition commutes exactly)
    Xs = [X[1], X[0], X[3], X[2], X[4]]
    assert orc.allreduce_tree_f32(FP32, Xs)[0][0] == 2.0
