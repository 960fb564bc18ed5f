// The bulk (TMA) engine's device code: mbarrier and cp.async.bulk wrappers, the per-piece FP32 add from shared
// memory, and the DMA thread that claims items, resolves dependencies and drives the stage ring.
#pragma once
#include "bulk_layout.h"
#include "device.cuh"

namespace hccl {
// ====================================================================== bulk (TMA) engine
// The same dispatch and dependency protocol, but the data mover is the bulk asynchronous copy unit:
// warp 0 is the DMA warp (one elected thread claims tickets, resolves dependencies and issues
// cp.async.bulk loads into a ring of shared-memory stages); the other warps are the compute warps.
//   COPY   : global -> stage -> global, both hops by cp.async.bulk; no thread touches the data.
//   REDUCE : A and B pieces are loaded into a stage by cp.async.bulk (mbarrier complete_tx), the compute
//            warps add them in FP32 from shared memory and store the result to global with 16-byte stores.
// Anything the bulk unit cannot take (an address or length not a multiple of 16 bytes, multi-input sums)
// is handed to the compute warps as a whole work item for the register path.
namespace bulk {


__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait on an mbarrier phase; gives up when the execution is aborted or the time budget runs out.
static __device__ bool mbar_wait(const ExecParams& p, uint32_t bar, uint32_t parity, unsigned long long budget_ns, uint32_t detail) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long deadline = globaltimer_ns() + budget_ns;
    uint32_t spins = 0;
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 31u) == 0) {
            if (aborted(p)) return false;
            if (globaltimer_ns() > deadline) {
                fail(p, HCCL_ERR_TIMEOUT, detail);
                return false;
            }
        }
    }
}
__device__ __forceinline__ unsigned long long policy_evict_first() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// Partials that a later ring step reads back should outlive the streamed inputs in the L2.
__device__ __forceinline__ unsigned long long policy_evict_last() {
    unsigned long long pol;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
// The data at [p, p + 128) will not be read again before it is rewritten: the L2 may drop the line instead of
// writing it back (p 128-byte aligned).
__device__ __forceinline__ void discard_line(const void* p) { asm volatile("discard.global.L2 [%0], 128;" ::"l"(p) : "memory"); }
__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* gsrc, uint32_t bytes, uint32_t bar, bool hint, unsigned long long pol) {
    if (hint)
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
                     ::"r"(smem_dst), "l"(gsrc), "r"(bytes), "r"(bar), "l"(pol) : "memory");
    else
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_dst), "l"(gsrc), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_store_part(void* gdst, uint32_t smem_src, uint32_t bytes, bool hint, unsigned long long pol) {
    if (hint)
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group.L2::cache_hint [%0], [%1], %2, %3;"
                     ::"l"(gdst), "r"(smem_src), "r"(bytes), "l"(pol) : "memory");
    else
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_store(void* gdst, uint32_t smem_src, uint32_t bytes, bool hint, unsigned long long pol) {
    bulk_store_part(gdst, smem_src, bytes, hint, pol);
    bulk_commit();
}
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
// Wait until at most `pending` of the most recent store groups are still reading shared memory.
__device__ __forceinline__ void bulk_wait_read(unsigned long long pending) {
    switch (pending) {
        case 0: asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); break;
        case 1: asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); break;
        case 2: asm volatile("cp.async.bulk.wait_group.read 2;" ::: "memory"); break;
        case 3: asm volatile("cp.async.bulk.wait_group.read 3;" ::: "memory"); break;
        case 4: asm volatile("cp.async.bulk.wait_group.read 4;" ::: "memory"); break;
        case 5: asm volatile("cp.async.bulk.wait_group.read 5;" ::: "memory"); break;
        case 6: asm volatile("cp.async.bulk.wait_group.read 6;" ::: "memory"); break;
        default: asm volatile("cp.async.bulk.wait_group.read 7;" ::: "memory"); break;
    }
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

// 4 consecutive elements of a stage <-> 4 floats (16-byte or 8-byte shared-memory access)
template <int DT>
__device__ __forceinline__ void lds4(const char* p, float (&f)[4]) {
    if constexpr (DT == HCCL_FP32) {
        const float4 v = *reinterpret_cast<const float4*>(p);
        f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
    } else {
        const uint2 v = *reinterpret_cast<const uint2*>(p);
        if constexpr (DT == HCCL_BF16) {
            f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
            f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
        } else {
            const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
            const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
            f[0] = a.x; f[1] = a.y; f[2] = b.x; f[3] = b.y;
        }
    }
}
// KEEP: the store carries an L2 cache-hint policy (FP32 partials only: they are what a next step reads back)
template <int DT, bool KEEP = false>
__device__ __forceinline__ void stg4(char* p, const float (&f)[4], unsigned long long pol = 0) {
    if constexpr (DT == HCCL_FP32) {
        if constexpr (KEEP)
            asm volatile("st.global.L2::cache_hint.v4.f32 [%0], {%1, %2, %3, %4}, %5;" ::"l"(p), "f"(f[0]), "f"(f[1]), "f"(f[2]), "f"(f[3]), "l"(pol) : "memory");
        else
            __stcg(reinterpret_cast<float4*>(p), make_float4(f[0], f[1], f[2], f[3]));
    } else {
        uint2 v;
        if constexpr (DT == HCCL_BF16) {
            const __nv_bfloat162 a = __floats2bfloat162_rn(f[0], f[1]), b = __floats2bfloat162_rn(f[2], f[3]);
            v.x = *reinterpret_cast<const uint32_t*>(&a); v.y = *reinterpret_cast<const uint32_t*>(&b);
        } else {
            const __half2 a = __floats2half2_rn(f[0], f[1]), b = __floats2half2_rn(f[2], f[3]);
            v.x = *reinterpret_cast<const uint32_t*>(&a); v.y = *reinterpret_cast<const uint32_t*>(&b);
        }
        __stcg(reinterpret_cast<uint2*>(p), v);
    }
}
template <int DA, int DB, int DD, bool KEEP = false>
__device__ __forceinline__ void reduce_piece(const char* sa, const char* sb, char* gdst, uint32_t n, uint32_t ctid, uint32_t cnth, unsigned long long pol = 0) {
    const uint32_t units = n >> 2;
    constexpr int U = 2;
    uint32_t u = ctid;
    for (; u + (U - 1) * cnth < units; u += U * cnth) {
        float a[U][4], b[U][4];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            lds4<DA>(sa + (size_t)(u + k * cnth) * 4 * Elem<DA>::BYTES, a[k]);
            lds4<DB>(sb + (size_t)(u + k * cnth) * 4 * Elem<DB>::BYTES, b[k]);
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
#pragma unroll
            for (int e = 0; e < 4; ++e) a[k][e] = a[k][e] + b[k][e];
            stg4<DD, KEEP>(gdst + (size_t)(u + k * cnth) * 4 * Elem<DD>::BYTES, a[k], pol);
        }
    }
    for (; u < units; u += cnth) {
        float a[4], b[4];
        lds4<DA>(sa + (size_t)u * 4 * Elem<DA>::BYTES, a);
        lds4<DB>(sb + (size_t)u * 4 * Elem<DB>::BYTES, b);
#pragma unroll
        for (int e = 0; e < 4; ++e) a[e] = a[e] + b[e];
        stg4<DD, KEEP>(gdst + (size_t)u * 4 * Elem<DD>::BYTES, a, pol);
    }
}
static __device__ void reduce_piece_dispatch(int da, int db, int dd, const char* sa, const char* sb, char* g, uint32_t n, uint32_t ctid, uint32_t cnth,
                                             bool keep, unsigned long long pol) {
#define RP(A, B, D) reduce_piece<A, B, D>(sa, sb, g, n, ctid, cnth)
#define RP_D(A, B) do { if (dd == HCCL_FP32) { if (keep) reduce_piece<A, B, HCCL_FP32, true>(sa, sb, g, n, ctid, cnth, pol); else RP(A, B, HCCL_FP32); } \
                        else if (dd == HCCL_BF16) RP(A, B, HCCL_BF16); else RP(A, B, HCCL_FP16); } while (0)
#define RP_B(A) do { if (db == HCCL_FP32) RP_D(A, HCCL_FP32); else if (db == HCCL_BF16) RP_D(A, HCCL_BF16); else RP_D(A, HCCL_FP16); } while (0)
    if (da == HCCL_FP32) RP_B(HCCL_FP32); else if (da == HCCL_BF16) RP_B(HCCL_BF16); else RP_B(HCCL_FP16);
#undef RP_B
#undef RP_D
#undef RP
}

// State of the DMA thread.
struct Dma {
    uint32_t ns, lag, sb;  // stages, store lag, bytes per stage
    uint32_t stages, full, empty;  // shared-memory addresses
    char* stages_ptr;
    PieceInfo* info;
    unsigned long long head, tail, groups;
    // stage and mbarrier phase parity of piece `head` and of piece `tail`, stepped along with the counters (a 64-bit
    // division per piece on the one issuing thread would cost more than the issue itself)
    uint32_t head_slot, head_par, tail_slot, tail_par;
    unsigned long long pol;       // evict-first: streamed send data
    unsigned long long pol_keep;  // evict-last: FP32 partials in scratch
    bool ok;
    bool copy_by_warps;
};

// Retire the oldest outstanding piece. A COPY piece is drained to global memory here; REDUCE and TILE
// pieces are finished by the compute warps on their own.
static __device__ void retire_one(const ExecParams& p, Dma& d) {
    const unsigned long long j = d.tail;
    const uint32_t slot = d.tail_slot, parity = d.tail_par;
    PieceInfo& pi = d.info[slot];
    if (pi.kind == PIECE_COPY) {
        if (!mbar_wait(p, d.full + 8 * slot, parity, p.timeout_ns, pi.tile_index)) d.ok = false;
        if (d.ok) {
            if (pi.ndst > 1) {  // one stage, several stores, one group
                for (uint32_t k = 0; k < pi.ndst; ++k) {
                    uint32_t r = pi.rank_dst + k;
                    if (r >= p.R) r -= p.R;
                    bulk_store_part((char*)p.recv[r] + pi.dst_off, d.stages + slot * d.sb, pi.n, pi.evict_first != 0, d.pol);
                }
                bulk_commit();
            } else {
                bulk_store(pi.dst, d.stages + slot * d.sb, pi.n, pi.evict_first != 0, d.pol);
            }
            pi.group = d.groups++;
            if (pi.last && p.trace) trace_put(p.trace, p.trace_cap, pi.tile_index, 3, globaltimer_ns());
            if (pi.last && (pi.signal[0] >= 0 || pi.signal[1] >= 0)) {
                bulk_wait_all();  // the item's bytes are in global memory
                fence_proxy_async();
                __threadfence();
                if (pi.signal[0] >= 0) red_release_add_u32(p.counters + pi.signal[0], 1);
                if (pi.signal[1] >= 0) red_release_add_u32(p.counters + pi.signal[1], 1);
            }
        }
    }
    d.tail = j + 1;
    if (++d.tail_slot == d.ns) {
        d.tail_slot = 0;
        d.tail_par ^= 1u;
    }
}
// The piece just written into stage head_slot has been issued.
__device__ __forceinline__ void advance_head(Dma& d) {
    d.head += 1;
    if (++d.head_slot == d.ns) {
        d.head_slot = 0;
        d.head_par ^= 1u;
    }
}
static __device__ void drain(const ExecParams& p, Dma& d) {
    while (d.tail < d.head) retire_one(p, d);
}
// Make stage (k mod ns) reusable for piece k: its previous piece (k - ns) must be retired, passed by every
// compute warp, and, if it was a COPY, fully read out of shared memory by its store.
static __device__ bool acquire_slot(const ExecParams& p, Dma& d, unsigned long long k, uint32_t detail) {
    if (k < d.ns) return d.ok;
    const unsigned long long j = k - d.ns;
    while (d.tail <= j) retire_one(p, d);
    if (!d.ok) return false;
    const uint32_t slot = d.head_slot, parity = d.head_par ^ 1u;   // k is d.head; piece k - ns used the same stage one phase earlier
    if (!mbar_wait(p, d.empty + 8 * slot, parity, 2 * p.timeout_ns + 1000000000ull, detail)) {
        d.ok = false;
        return false;
    }
    const PieceInfo& pi = d.info[slot];
    if (pi.kind == PIECE_COPY) bulk_wait_read(d.groups - (pi.group + 1));
    return true;
}
// After issuing, keep at most `lag` pieces outstanding so that stores follow loads at a fixed distance.
__device__ __forceinline__ void keep_lag(const ExecParams& p, Dma& d) {
    while (d.ok && d.head - d.tail > d.lag) retire_one(p, d);
}

static __device__ void issue_simple(const ExecParams& p, Dma& d, uint32_t kind, uint32_t cur, const Tile* t, const Desc* ds) {
    const unsigned long long k = d.head;
    if (!acquire_slot(p, d, k, cur)) return;
    const uint32_t slot = d.head_slot;
    PieceInfo& pi = d.info[slot];
    pi.kind = kind;
    pi.n = 0;
    pi.last = 1;
    pi.tile_index = cur;
    pi.signal[0] = t ? t->signal[0] : -1;
    pi.signal[1] = t ? t->signal[1] : -1;
    if (t) pi.tile = *t;
    if (ds) pi.desc = *ds;
    mbar_arrive(d.full + 8 * slot);  // no bytes expected: the phase completes at once
    advance_head(d);
}

// ---- hand-over from the control thread to the DMA thread
// The control thread (first lane of the block's second warp) claims items, fetches their records, waits for their
// dependencies and performs WAIT / SET / NOOP items itself; items that move data are passed on through a small
// ring in shared memory. The three or four dependent trips to the L2 that start an item thus overlap with the
// DMA thread's piece issue instead of stalling it.
constexpr uint32_t QUEUE = 1;                  // prepared items the control thread may be ahead by
enum : uint32_t { Q_ITEM = 0, Q_STOP = 1 };
struct alignas(16) Prepared {
    Tile t;
    Desc ds;
    uint32_t item, kind, waited, pad;
};

// One item on the control thread. Returns 0: stop (no more work, failure or abort), 1: done here (no data to
// move), 2: a data item, its records in t / ds, its dependencies met.
static __device__ int control_item(const ExecParams& p, uint32_t cur, const Tile* preloaded, Tile& t, Desc& ds) {
    if (p.trace) {
        trace_put(p.trace, p.trace_cap, cur, 0, (unsigned long long)cur | ((unsigned long long)blockIdx.x << 32));
        trace_put(p.trace, p.trace_cap, cur, 1, globaltimer_ns());
    }
    t = preloaded ? *preloaded : p.tiles[cur];
    if (t.flags & TILE_FLAG_END) return 0;  // behind the last item of a device-built table: no more work, no failure
    if (!tile_ok(p, t)) {
        fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
        return 0;
    }
    ds = p.descs[t.desc];
    if (!desc_ok(p, ds)) {
        fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
        return 0;
    }
    for (uint32_t w = 0; w < t.wait_cnt; ++w) {
        const Wait x = p.waits[t.wait_off + w];
        if (x.sync >= p.n_syncs) {
            fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
            return 0;
        }
        // an item of this block's own pipeline may be what is waited for: the DMA thread retires (and so publishes)
        // what it has in flight whenever it has nothing to issue
        if (!wait_counter(p, x.sync, x.per_epoch, cur)) return 0;
    }
    if (p.trace) trace_put(p.trace, p.trace_cap, cur, 2, globaltimer_ns());
    switch (ds.op) {
        case HCCL_OP_WAIT: {
            const unsigned long long* addr = (ds.kind_a == HCCL_BUF_SIGNAL ? p.signals : p.user_signals) + ds.off_a;
            if (!wait_signal(p, addr, ds.cmp, ds.value + (unsigned long long)g_epoch * ds.value_per_epoch, cur)) return 0;
            publish_tile(p, t);
            return 1;
        }
        case HCCL_OP_SET: {
            unsigned long long* addr = (ds.kind_dst == HCCL_BUF_SIGNAL ? p.signals : p.user_signals) + ds.off_dst;
            __threadfence();
            st_release_u64(addr, ds.value + (unsigned long long)g_epoch * ds.value_per_epoch);
            publish_tile(p, t);
            return 1;
        }
        case HCCL_OP_NOOP:
            publish_tile(p, t);
            return 1;
        default:
            return 2;
    }
}

// One data item through the DMA thread (records and dependencies were dealt with by the control thread).
// Returns false when the block must stop.
static __device__ bool dma_issue(const ExecParams& p, Dma& d, uint32_t cur, const Tile& t, const Desc& ds) {
    switch (ds.op) {
        case HCCL_OP_COPY: {
            char* dst = buf_base(p, ds.kind_dst, ds.rank_dst) + ds.off_dst + t.start;
            const char* src = buf_base(p, ds.kind_a, ds.rank_a) + ds.off_a + t.start;
            const uint32_t nd = ds.ndst > 1 ? ds.ndst : 1;
            const unsigned long long doff = (unsigned long long)ds.off_dst + t.start;
            auto dstk = [&](uint32_t k) -> char* {
                uint32_t r = ds.rank_dst + k;
                if (r >= p.R) r -= p.R;
                return (char*)p.recv[r] + doff;
            };
            uintptr_t bits = (uintptr_t)dst | (uintptr_t)src;
            for (uint32_t k = 1; k < nd; ++k) bits |= (uintptr_t)dstk(k);
            if ((bits & 15u) != 0 || t.count < 16) {
                issue_simple(p, d, PIECE_TILE, cur, &t, &ds);
                keep_lag(p, d);
                return d.ok;
            }
            const uint32_t body = t.count & ~15u, tailb = t.count - body;
            // the last few bytes (< 16) go through this thread; they belong to the item, so before its last piece
            for (uint32_t i = 0; i < tailb; ++i) {
                const char b = __ldcg(src + body + i);
                dst[body + i] = b;
                for (uint32_t k = 1; k < nd; ++k) dstk(k)[body + i] = b;
            }
            const bool stream = ds.kind_a == HCCL_BUF_SEND;
            for (uint32_t off = 0; off < body && d.ok; off += d.sb) {
                const uint32_t nb = min(d.sb, body - off);
                const unsigned long long k = d.head;
                if (!acquire_slot(p, d, k, cur)) return false;
                const uint32_t slot = d.head_slot;
                PieceInfo& pi = d.info[slot];
                pi.kind = d.copy_by_warps ? PIECE_COPYW : PIECE_COPY;
                pi.n = nb;
                pi.last = (off + nb == body) ? 1u : 0u;
                pi.tile_index = cur;
                pi.dst = dst + off;
                pi.ndst = (uint16_t)nd;
                pi.rank_dst = ds.rank_dst;
                pi.dst_off = doff + off;
                pi.signal[0] = t.signal[0];
                pi.signal[1] = t.signal[1];
                pi.evict_first = stream ? 1 : 0;
                mbar_arrive_expect_tx(d.full + 8 * slot, nb);
                bulk_load(d.stages + slot * d.sb, src + off, nb, d.full + 8 * slot, stream, d.pol);
                advance_head(d);
                keep_lag(p, d);
            }
            return d.ok;
        }
        case HCCL_OP_REDUCE: {
            const uint32_t ea = ds.dt_a == HCCL_FP32 ? 4 : 2, eb = ds.dt_b == HCCL_FP32 ? 4 : 2, ed = ds.dt_dst == HCCL_FP32 ? 4 : 2;
            char* dst = buf_base(p, ds.kind_dst, ds.rank_dst) + ds.off_dst + t.start * ed;
            const char* a = buf_base(p, ds.kind_a, ds.rank_a) + ds.off_a + t.start * ea;
            const char* b = buf_base(p, ds.kind_b, ds.rank_b) + ds.off_b + t.start * eb;
            if ((((uintptr_t)dst | (uintptr_t)a | (uintptr_t)b) & 15u) != 0 || (t.count & 7u) != 0) {
                issue_simple(p, d, PIECE_TILE, cur, &t, &ds);
                keep_lag(p, d);
                return d.ok;
            }
            const uint32_t pe = piece_elems(d.sb, ea, eb);
            for (uint32_t e0 = 0; e0 < t.count && d.ok; e0 += pe) {
                const uint32_t ne = min(pe, t.count - e0);
                const unsigned long long k = d.head;
                if (!acquire_slot(p, d, k, cur)) return false;
                const uint32_t slot = d.head_slot;
                PieceInfo& pi = d.info[slot];
                pi.kind = PIECE_REDUCE;
                pi.n = ne;
                pi.last = (e0 + ne == t.count) ? 1u : 0u;
                pi.tile_index = cur;
                pi.dst = dst + (size_t)e0 * ed;
                pi.signal[0] = t.signal[0];
                pi.signal[1] = t.signal[1];
                pi.dt_a = ds.dt_a; pi.dt_b = ds.dt_b; pi.dt_d = ds.dt_dst;
                pi.b_off = pe * ea;
                // FP32 partials in scratch: kept in the L2 in preference to the streamed inputs (loads and stores carry
                // an evict-last policy); after the step that reads a partial for the last time its lines are discarded
                pi.keep_dst = (ds.kind_dst == HCCL_BUF_SCRATCH && ds.dt_dst == HCCL_FP32) ? 1 : 0;
                pi.discard_src = (ds.cmp & HCCL_HINT_LAST_READ_A) && ds.kind_a == HCCL_BUF_SCRATCH ? a + (size_t)e0 * ea : nullptr;
                pi.discard_bytes = ne * ea;
                mbar_arrive_expect_tx(d.full + 8 * slot, ne * (ea + eb));
                const bool a_keep = ds.kind_a == HCCL_BUF_SCRATCH;
                bulk_load(d.stages + slot * d.sb, a + (size_t)e0 * ea, ne * ea, d.full + 8 * slot, ds.kind_a == HCCL_BUF_SEND || a_keep, a_keep ? d.pol_keep : d.pol);
                bulk_load(d.stages + slot * d.sb + pe * ea, b + (size_t)e0 * eb, ne * eb, d.full + 8 * slot, ds.kind_b == HCCL_BUF_SEND, d.pol);
                advance_head(d);
                keep_lag(p, d);
            }
            return d.ok;
        }
        default:  // REDUCE_N: register path
            issue_simple(p, d, PIECE_TILE, cur, &t, &ds);
            keep_lag(p, d);
            return d.ok;
    }
}

}  // namespace bulk
}  // namespace hccl
