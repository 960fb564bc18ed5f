/*
 * CPU oracle for the collective hot path (test infrastructure, not product code).
 *
 * Plain, slow, single-threaded C. Each function is the textbook definition of
 * the result that the paper's collectives produce, written out directly; no
 * schedule, no blocking, no vectorisation. It shares no code with the CUDA
 * library and is used only by the tests, by the smoke check and by the
 * benchmark's CPU-baseline leg.
 *
 * What the paper fixes, and where:
 *   - Sec. II-A.2, "Near Memory Compute": the offload engine performs copies
 *     and sums (S=A+B, A=A+B, B=A+B, A=B) on BF16/FP16/FP32 buffers, does its
 *     arithmetic in FP32 and re-quantises when the stored type differs.
 *     -> oracle_nmc() below: one FP32 add, one round-to-nearest-even store.
 *   - Sec. III-B.2 and Sec. V-A/V-D: the collectives are the standard ones
 *     (AllReduce, ReduceScatter, AllGather, AllToAllv) with MPI-style meaning.
 *     A ring or an "all-to-all style" kernel is a schedule that reaches the
 *     same result, so the oracle for a collective is its definition:
 *     the sum over ranks, accumulated in FP64 in rank order 0..R-1 and rounded
 *     once, directly, to the output type.
 *   - Sec. III-B.2, ring AllReduce example (Fig. 5): the order in which a
 *     unidirectional ring adds the ranks' contributions.
 *     -> oracle_allreduce_ring_f32(): the same sums taken step by step in
 *     FP32 in ring order, so a ring executor can also be compared bit for bit.
 *
 * Element types: 0 = fp32, 1 = bf16, 2 = fp16 (raw IEEE bit patterns).
 * Rounding: round-to-nearest-even, subnormals kept, overflow to infinity.
 *
 * Pins (tests/test_oracle_pins.py): closed forms, invariants, numpy/torch
 * library routines on special cases, hand-built rounding ties, brute force on
 * tiny inputs. Every exported function has at least one such pin.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { OR_FP32 = 0, OR_BF16 = 1, OR_FP16 = 2 };

static int elem_size(int dt) { return dt == OR_FP32 ? 4 : 2; }

/* ---- exact widening to double ------------------------------------------ */

static double widen_f32(uint32_t bits) {
    float f;
    memcpy(&f, &bits, 4);
    return (double)f;
}

static double widen_bf16(uint16_t h) {
    /* bf16 is the upper half of an fp32 pattern */
    return widen_f32((uint32_t)h << 16);
}

static double widen_fp16(uint16_t h) {
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int m = h & 0x3ff;
    double v;
    if (e == 0)
        v = ldexp((double)m, -24); /* subnormal: m * 2^-24 */
    else if (e == 31)
        v = m ? NAN : INFINITY;
    else
        v = ldexp((double)(m + 1024), e - 25); /* (1 + m/1024) * 2^(e-15) */
    return sign ? -v : v;
}

/* ---- direct rounding double -> small float, nearest-even ------------------
 * p = significand bits including the hidden one, emin = exponent of the
 * smallest normal, emax = exponent of the largest normal. The value is scaled
 * so that one unit in the last place is 1.0, rounded with rint() (ties to even
 * in the default rounding mode) and reassembled. Returns sign, biased exponent
 * and fraction through the out-parameters. */
static void round_small(double x, int p, int emin, int emax, int *sign, int *bexp, uint32_t *frac,
                        int *is_inf, int *is_nan) {
    *is_inf = *is_nan = 0;
    *sign = signbit(x) ? 1 : 0;
    *bexp = 0;
    *frac = 0;
    if (isnan(x)) {
        *is_nan = 1;
        return;
    }
    if (isinf(x)) {
        *is_inf = 1;
        return;
    }
    double a = fabs(x);
    if (a == 0.0) return;
    int e;
    (void)frexp(a, &e); /* a = f * 2^e, f in [0.5,1) -> exponent of leading bit is e-1 */
    int lead = e - 1;
    if (lead < emin) lead = emin;       /* subnormal range: fixed quantum */
    int q = lead - (p - 1);             /* exponent of one ulp */
    double scaled = ldexp(a, -q);       /* exact: power-of-two scaling */
    double r = rint(scaled);            /* ties to even */
    /* r is an integer in [0, 2^p]; 2^p means the rounding carried out */
    double top = ldexp(1.0, p);
    if (r >= top) {
        r = ldexp(1.0, p - 1);
        lead += 1;
        q += 1;
    }
    if (lead > emax) {
        *is_inf = 1;
        return;
    }
    uint32_t mant = (uint32_t)r;
    uint32_t hidden = 1u << (p - 1);
    if (mant >= hidden) {
        *bexp = lead - emin + 1;
        *frac = mant - hidden;
    } else {
        *bexp = 0; /* subnormal (or zero after rounding) */
        *frac = mant;
    }
}

static uint16_t round_to_bf16(double x) {
    int s, be, inf, nan;
    uint32_t fr;
    round_small(x, 8, -126, 127, &s, &be, &fr, &inf, &nan);
    if (nan) return 0x7fc0;
    if (inf) return (uint16_t)((s << 15) | 0x7f80);
    return (uint16_t)((s << 15) | (be << 7) | fr);
}

static uint16_t round_to_fp16(double x) {
    int s, be, inf, nan;
    uint32_t fr;
    round_small(x, 11, -14, 15, &s, &be, &fr, &inf, &nan);
    if (nan) return 0x7e00;
    if (inf) return (uint16_t)((s << 15) | 0x7c00);
    return (uint16_t)((s << 15) | (be << 10) | fr);
}

static uint32_t round_to_f32(double x) {
    int s, be, inf, nan;
    uint32_t fr;
    round_small(x, 24, -126, 127, &s, &be, &fr, &inf, &nan);
    if (nan) return 0x7fc00000u;
    if (inf) return ((uint32_t)s << 31) | 0x7f800000u;
    return ((uint32_t)s << 31) | ((uint32_t)be << 23) | fr;
}

static double load_elem(const void *buf, int64_t i, int dt) {
    if (dt == OR_FP32) {
        uint32_t b;
        memcpy(&b, (const char *)buf + 4 * i, 4);
        return widen_f32(b);
    }
    uint16_t h;
    memcpy(&h, (const char *)buf + 2 * i, 2);
    return dt == OR_BF16 ? widen_bf16(h) : widen_fp16(h);
}

static void store_elem(void *buf, int64_t i, int dt, double v) {
    if (dt == OR_FP32) {
        uint32_t b = round_to_f32(v);
        memcpy((char *)buf + 4 * i, &b, 4);
    } else {
        uint16_t h = dt == OR_BF16 ? round_to_bf16(v) : round_to_fp16(v);
        memcpy((char *)buf + 2 * i, &h, 2);
    }
}

/* Exported so the pins can exercise the conversions on their own. */
void oracle_widen(int dt, int64_t n, const void *in, double *out) {
    for (int64_t i = 0; i < n; ++i) out[i] = load_elem(in, i, dt);
}
void oracle_round(int dt, int64_t n, const double *in, void *out) {
    for (int64_t i = 0; i < n; ++i) store_elem(out, i, dt, in[i]);
}

/* ---- Near-memory-compute primitive (Sec. II-A.2) --------------------------
 * dst[i] = round_T( fl32( f32(a[i]) + f32(b[i]) ) ). dst may alias a or b
 * (the in-place forms A=A+B and B=A+B). With b == NULL it is the copy form
 * A=B on n elements of type dt_dst (dt_a must equal dt_dst). */
int oracle_nmc(int dt_dst, void *dst, int dt_a, const void *a, int dt_b, const void *b, int64_t n) {
    if (b == NULL) {
        if (dt_a != dt_dst) return 1;
        memmove(dst, a, (size_t)n * (size_t)elem_size(dt_dst));
        return 0;
    }
    for (int64_t i = 0; i < n; ++i) {
        /* widening a 16-bit value to fp32 is exact, so (float) of the double is too */
        volatile float fa = (float)load_elem(a, i, dt_a);
        volatile float fb = (float)load_elem(b, i, dt_b);
        volatile float s = fa + fb; /* one FP32 add, rounded to nearest even */
        store_elem(dst, i, dt_dst, (double)s);
    }
    return 0;
}

/* ---- AllReduce(sum): Y_r[i] = round_T( sum_q X_q[i] ), all r ------------- */
int oracle_allreduce(int R, int64_t n, int dt, const void *const *X, void *const *Y) {
    if (R < 1 || n < 0) return 1;
    for (int64_t i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int q = 0; q < R; ++q) acc += load_elem(X[q], i, dt);
        for (int r = 0; r < R; ++r) store_elem(Y[r], i, dt, acc);
    }
    return 0;
}

/* ---- ReduceScatter(sum): rank r keeps elements [o_r, o_r + c_r) ---------- */
int oracle_reducescatter(int R, const int64_t *recvcounts, int dt, const void *const *X,
                         void *const *Y) {
    if (R < 1) return 1;
    int64_t o = 0;
    for (int r = 0; r < R; ++r) {
        if (recvcounts[r] < 0) return 1;
        for (int64_t j = 0; j < recvcounts[r]; ++j) {
            double acc = 0.0;
            for (int q = 0; q < R; ++q) acc += load_elem(X[q], o + j, dt);
            store_elem(Y[r], j, dt, acc);
        }
        o += recvcounts[r];
    }
    return 0;
}

/* ---- AllGather(v): Y_r[o_q + j] = X_q[j] for every r, q ------------------ */
int oracle_allgatherv(int R, const int64_t *counts, int elem_bytes, const void *const *X,
                      void *const *Y) {
    if (R < 1 || elem_bytes < 1) return 1;
    for (int r = 0; r < R; ++r) {
        int64_t o = 0;
        for (int q = 0; q < R; ++q) {
            if (counts[q] < 0) return 1;
            memcpy((char *)Y[r] + o * elem_bytes, X[q], (size_t)(counts[q] * elem_bytes));
            o += counts[q];
        }
    }
    return 0;
}

/* ---- AllToAllv ------------------------------------------------------------
 * sendcounts, sdispls are R x R row-major indexed [s][d]; rdispls is indexed
 * [d][s]; all in rows of row_bytes bytes. For every (s, d) and k below
 * sendcounts[s][d]: row rdispls[d][s]+k of Y_d = row sdispls[s][d]+k of X_s.
 * Nothing else in Y is touched. dst_only >= 0 restricts the work to that one
 * destination rank (the definition restricted to one d), which lets a caller
 * check one rank of a problem too large to hold at once. */
int oracle_alltoallv(int R, const int64_t *sendcounts, const int64_t *sdispls,
                     const int64_t *rdispls, int64_t row_bytes, const void *const *X,
                     void *const *Y, int dst_only) {
    if (R < 1 || row_bytes < 1) return 1;
    for (int d = 0; d < R; ++d) {
        if (dst_only >= 0 && d != dst_only) continue;
        for (int s = 0; s < R; ++s) {
            int64_t c = sendcounts[(int64_t)s * R + d];
            if (c < 0) return 1;
            const char *src = (const char *)X[s] + sdispls[(int64_t)s * R + d] * row_bytes;
            char *dst = (char *)Y[d] + rdispls[(int64_t)d * R + s] * row_bytes;
            for (int64_t k = 0; k < c; ++k)
                memcpy(dst + k * row_bytes, src + k * row_bytes, (size_t)row_bytes);
        }
    }
    return 0;
}

/* Packed displacements: the exclusive prefix sum of each rank's counts.
 * sdispls[s][d] = sum_{d' < d} C[s][d'];  rdispls[d][s] = sum_{s' < s} C[s'][d]. */
void oracle_packed_displs(int R, const int64_t *sendcounts, int64_t *sdispls, int64_t *rdispls) {
    for (int s = 0; s < R; ++s) {
        int64_t o = 0;
        for (int d = 0; d < R; ++d) {
            sdispls[(int64_t)s * R + d] = o;
            o += sendcounts[(int64_t)s * R + d];
        }
    }
    for (int d = 0; d < R; ++d) {
        int64_t o = 0;
        for (int s = 0; s < R; ++s) {
            rdispls[(int64_t)d * R + s] = o;
            o += sendcounts[(int64_t)s * R + d];
        }
    }
}

/* ---- Ring order, FP32 partials (Sec. III-B.2 ring example; NMC FP32) ------
 * A unidirectional ring r -> r+1 with R chunks: the chunk that ends on rank c
 * starts as X_{c+1}, and each later rank on the way round adds its own
 * contribution, so element i of chunk c is
 *     ((X_{c+1}[i] + X_{c+2}[i]) + X_{c+3}[i]) + ... + X_c[i]     (ranks mod R)
 * with every add in FP32 and one final rounding to the stored type; the
 * all-gather phase then copies that chunk to every rank. Chunk c covers
 * elements [offs[c], offs[c+1]). offs has R+1 entries, offs[0]=0, offs[R]=n. */
int oracle_allreduce_ring_f32(int R, const int64_t *offs, int dt, const void *const *X,
                              void *const *Y) {
    if (R < 1) return 1;
    for (int c = 0; c < R; ++c) {
        for (int64_t i = offs[c]; i < offs[c + 1]; ++i) {
            volatile float acc = (float)load_elem(X[(c + 1) % R], i, dt);
            for (int t = 2; t <= R; ++t) {
                volatile float x = (float)load_elem(X[(c + t) % R], i, dt);
                acc = acc + x;
            }
            for (int r = 0; r < R; ++r) store_elem(Y[r], i, dt, (double)acc);
        }
    }
    return 0;
}

/* Same sums, scattered: rank c keeps chunk c only (ring ReduceScatter). */
int oracle_reducescatter_ring_f32(int R, const int64_t *recvcounts, int dt, const void *const *X,
                                  void *const *Y) {
    if (R < 1) return 1;
    int64_t o = 0;
    for (int c = 0; c < R; ++c) {
        for (int64_t j = 0; j < recvcounts[c]; ++j) {
            volatile float acc = (float)load_elem(X[(c + 1) % R], o + j, dt);
            for (int t = 2; t <= R; ++t) {
                volatile float x = (float)load_elem(X[(c + t) % R], o + j, dt);
                acc = acc + x;
            }
            store_elem(Y[c], j, dt, (double)acc);
        }
        o += recvcounts[c];
    }
    return 0;
}

/* One-shot ("all-to-all style", Sec. V-F PE collective kernels): every rank
 * sums all R inputs itself, in rank order 0..R-1, FP32 adds, one rounding. */
int oracle_allreduce_oneshot_f32(int R, int64_t n, int dt, const void *const *X, void *const *Y) {
    if (R < 1) return 1;
    for (int64_t i = 0; i < n; ++i) {
        volatile float acc = (float)load_elem(X[0], i, dt);
        for (int q = 1; q < R; ++q) {
            volatile float x = (float)load_elem(X[q], i, dt);
            acc = acc + x;
        }
        for (int r = 0; r < R; ++r) store_elem(Y[r], i, dt, (double)acc);
    }
    return 0;
}

/* Binary-tree order (Sec. III-B.2 mentions tree-based NMC reductions as a user of multi-dependency joins):
 * the R inputs are the leaves, in rank order; each level adds neighbours in pairs, (v_0 + v_1), (v_2 + v_3),
 * ..., and an odd one out moves up unchanged; the levels repeat until one value is left. FP32 adds, one
 * rounding to the stored type at the root; every rank receives the result. */
int oracle_allreduce_tree_f32(int R, int64_t n, int dt, const void *const *X, void *const *Y) {
    if (R < 1 || R > 4096) return 1;
    volatile float v[4096];
    for (int64_t i = 0; i < n; ++i) {
        for (int q = 0; q < R; ++q) v[q] = (float)load_elem(X[q], i, dt);
        int m = R;
        while (m > 1) {
            const int pairs = m / 2;
            for (int j = 0; j < pairs; ++j) v[j] = v[2 * j] + v[2 * j + 1];
            if (m & 1) v[pairs] = v[m - 1];
            m = pairs + (m & 1);
        }
        for (int r = 0; r < R; ++r) store_elem(Y[r], i, dt, (double)v[0]);
    }
    return 0;
}

/* Ring order with a direction per segment (bidirectional rings, Sec. III-B.2: half of the data travels
 * r -> r+1, the other half r -> r-1). Segment s covers elements [seg_off[s], seg_off[s+1]) of chunk
 * seg_chunk[s] and travels in direction seg_dir[s] (+1 or -1): its elements are summed as
 * ((X_{c+d} + X_{c+2d}) + ...) + X_c (indices mod R), FP32 adds, one rounding; every rank gets the result. */
int oracle_allreduce_ring_dir_f32(int R, int nseg, const int64_t *seg_off, const int64_t *seg_chunk,
                                  const int64_t *seg_dir, int dt, const void *const *X, void *const *Y) {
    if (R < 1 || nseg < 0) return 1;
    for (int s = 0; s < nseg; ++s) {
        const int c = (int)seg_chunk[s], d = seg_dir[s] >= 0 ? 1 : -1;
        for (int64_t i = seg_off[s]; i < seg_off[s + 1]; ++i) {
            volatile float acc = (float)load_elem(X[((c + d) % R + R) % R], i, dt);
            for (int t = 2; t <= R; ++t) {
                volatile float x = (float)load_elem(X[((c + d * t) % R + R) % R], i, dt);
                acc = acc + x;
            }
            for (int r = 0; r < R; ++r) store_elem(Y[r], i, dt, (double)acc);
        }
    }
    return 0;
}

/* Two-level ring order (Sec. V-D: topology-aware schedules that keep most exchanges inside a rack).
 * R = G racks of L ranks; rank (g, l) = g*L + l. The buffer is cut into L chunks (offs1, L+1 entries) and
 * every chunk j into G sub-chunks (offs2[j*(G+1) .. j*(G+1)+G], absolute element offsets). For sub-chunk
 * (j, k): first every rack g sums its own L ranks round its ring, P_g = ((X_{g,j+1} + X_{g,j+2}) + ...) +
 * X_{g,j} (local indices mod L); then the racks' partials are summed round the ring of racks,
 * ((P_{k+1} + P_{k+2}) + ...) + P_k (rack indices mod G). Every add is FP32 (partials are never
 * re-quantised), one rounding to the stored type at the end; all ranks receive the result. */
int oracle_allreduce_ring2_f32(int G, int L, const int64_t *offs1, const int64_t *offs2, int dt,
                               const void *const *X, void *const *Y) {
    if (G < 1 || L < 1) return 1;
    const int R = G * L;
    (void)offs1;
    for (int j = 0; j < L; ++j) {
        for (int k = 0; k < G; ++k) {
            const int64_t lo = offs2[j * (G + 1) + k], hi = offs2[j * (G + 1) + k + 1];
            for (int64_t i = lo; i < hi; ++i) {
                volatile float total = 0.0f;
                for (int tg = 1; tg <= G; ++tg) {
                    const int g = (k + tg) % G;
                    volatile float part = (float)load_elem(X[g * L + (j + 1) % L], i, dt);
                    for (int t = 2; t <= L; ++t) {
                        volatile float x = (float)load_elem(X[g * L + (j + t) % L], i, dt);
                        part = part + x;
                    }
                    if (tg == 1) total = part; else total = total + part;
                }
                for (int r = 0; r < R; ++r) store_elem(Y[r], i, dt, (double)total);
            }
        }
    }
    return 0;
}

/* Distance in units in the last place between two stored values of type dt,
 * measured on the monotone integer image of the bit patterns (sign-magnitude
 * mapped to an ordered integer; +0 and -0 coincide). Used by the tests'
 * "within 1 ulp" acceptance rule for 16-bit outputs. */
static int64_t ordered(uint32_t bits, int width) {
    uint32_t signmask = 1u << (width - 1);
    int64_t mag = (int64_t)(bits & (signmask - 1));
    return (bits & signmask) ? -mag : mag;
}
void oracle_ulp_distance(int dt, int64_t n, const void *a, const void *b, int64_t *out) {
    for (int64_t i = 0; i < n; ++i) {
        if (dt == OR_FP32) {
            uint32_t x, y;
            memcpy(&x, (const char *)a + 4 * i, 4);
            memcpy(&y, (const char *)b + 4 * i, 4);
            out[i] = llabs(ordered(x, 32) - ordered(y, 32));
        } else {
            uint16_t x, y;
            memcpy(&x, (const char *)a + 2 * i, 2);
            memcpy(&y, (const char *)b + 2 * i, 2);
            out[i] = llabs(ordered(x, 16) - ordered(y, 16));
        }
    }
}

/* FP64 sums without the final rounding, for the fp32 acceptance rule
 * |g - o| <= 1e-5 |o| + 1e-6 where o is the FP64 sum itself. */
int oracle_sum_f64(int R, int64_t n, int dt, const void *const *X, double *out) {
    if (R < 1) return 1;
    for (int64_t i = 0; i < n; ++i) {
        double acc = 0.0;
        for (int q = 0; q < R; ++q) acc += load_elem(X[q], i, dt);
        out[i] = acc;
    }
    return 0;
}
