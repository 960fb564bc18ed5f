// Device side shared by every kernel of the library: kernel parameters, memory-ordering primitives, element
// conversion, the COPY / REDUCE / REDUCE_N tile loops of the register path, table checks, and the body of the
// register engine. Included by each kernel's translation unit; everything here has internal or inline linkage.
//
// One launch = one execution of a compiled work packet (paper Sec. III-B.2). The B thread blocks
// play the message engines of Sec. II-A.2: each claims the next work item from a global ticket
// (the dispatch the control core does, Sec. II-A.1), waits on the item's dependency counters (what
// the engine's communication core evaluates), then moves or sums the item's bytes (the near-memory
// compute unit's S=A+B / A=A+B / A=B in FP32) and publishes its completion.
//
// Forward progress does not need all blocks resident: items are numbered in an order in which
// dependencies only point backwards and are claimed in that order, so the holder of ticket i waits
// only on tickets below i, all of which are held by running blocks. Every wait is bounded: on
// expiry the block records HCCL_ERR_TIMEOUT and raises an abort flag that all blocks poll; the
// kernel then ends normally. Nothing here traps.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <atomic>
#include <chrono>
#include <cstddef>
#include <cstring>
#include <mutex>
#include <type_traits>
#include <vector>

#include "plan.hpp"


namespace hccl {

struct ExecParams {
    const Desc* descs;
    const Tile* tiles;
    const Wait* waits;
    uint32_t* counters;
    unsigned long long* signals;
    Control* ctl;
    char* scratch;
    unsigned long long* user_signals;
    unsigned long long* trace;  // optional: 4 words per work item (item | block << 32, claim, start, end in ns), or null
    unsigned long long trace_cap;
    uint32_t n_tiles, n_descs, n_syncs, n_waits;
    uint32_t R, nblocks, n_signals;
    uint32_t quantum;  // ticket dispatch: items a block claims before it leaves (0 = until the packet is done)
    // resident executor only: where the last block out of an execution reports it to the host (doorbell record), and the
    // execution number that counts as the first one
    unsigned long long* host_completed;
    unsigned long long* host_t_done;
    uint32_t first_epoch, pad2;
    unsigned long long timeout_ns;
    long long n_user_signals;
    long long trig_wait_slot, trig_set_slot;
    int trig_cmp;
    int static_tickets;  // no dependencies and no more items than blocks: block b runs item b, no atomics
    uint32_t chain_len, n_chains;  // static chains (chain_len > 0): items [c*chain_len, (c+1)*chain_len) are chain c; block b
                                   // runs its share of the chains one after the other, each in order, without counters
    unsigned long long trig_wait_value, trig_wait_per_epoch, trig_set_value, trig_set_per_epoch;
    const void* send[HCCL_MAX_RANKS];
    void* recv[HCCL_MAX_RANKS];
};

// The execution number ("epoch") of the running launch. It lives on the device: every block derives it from
// the control block (done_epoch of the previous execution + 1), so a launch captured in a CUDA graph finds
// the right epoch on every replay. Kept in shared memory, written once per block at kernel entry.
static __shared__ uint32_t g_epoch;
template <class P>
__device__ __forceinline__ void init_epoch(const P& p) {
    if (threadIdx.x == 0) g_epoch = *(volatile uint32_t*)&p.ctl->done_epoch + 1u;
    __syncthreads();
}

// Per-item timestamps for the optional trace (counters per work packet and per subgraph, paper Sec. V-C).
__device__ __forceinline__ void trace_put(unsigned long long* trace, unsigned long long cap, uint32_t item, int word, unsigned long long v) {
    if (trace && item < cap) trace[(size_t)item * 4 + word] = v;
}

// ------------------------------------------------------------------ device primitives
__device__ __forceinline__ uint32_t ld_acquire_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_add_u32(uint32_t* p, uint32_t v) {
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void st_release_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ uint32_t ld_relaxed_u32(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ unsigned long long globaltimer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ bool compare(unsigned long long v, int cmp, unsigned long long want) {
    switch (cmp) {
        case HCCL_CMP_EQ: return v == want;
        case HCCL_CMP_NE: return v != want;
        case HCCL_CMP_GE: return v >= want;
        case HCCL_CMP_GT: return v > want;
        case HCCL_CMP_LE: return v <= want;
        default: return v < want;
    }
}

// Record a failure once per execution and tell everyone to stop.
template <class P>
__device__ __noinline__ void fail(const P& p, uint32_t code, unsigned long long detail) {
    if (atomicExch(&p.ctl->fail_epoch, g_epoch) != g_epoch) {  // first failure of this execution wins
        p.ctl->status = code;
        p.ctl->detail = detail;
    }
    __threadfence();
    atomicExch(&p.ctl->abort, g_epoch);
}
template <class P>
__device__ __forceinline__ bool aborted(const P& p) { return ld_relaxed_u32(&p.ctl->abort) == g_epoch; }

// Bounded wait until counters[sync] has received epoch * per_epoch bumps (wrap-safe compare).
static __device__ bool wait_counter(const ExecParams& p, uint32_t sync, uint32_t per_epoch, uint32_t tile) {
    const uint32_t* c = p.counters + sync;
    const uint32_t target = g_epoch * per_epoch;
    if ((int32_t)(ld_acquire_u32(c) - target) >= 0) return true;
    const unsigned long long deadline = globaltimer_ns() + p.timeout_ns;
    uint32_t spins = 0;
    for (;;) {
        if ((int32_t)(ld_acquire_u32(c) - target) >= 0) return true;
        if ((++spins & 7u) == 0) {
            if (aborted(p)) return false;
            if (globaltimer_ns() > deadline) {
                fail(p, HCCL_ERR_TIMEOUT, tile);
                return false;
            }
        }
        __nanosleep(spins < 64 ? 20 : 200);
    }
}

template <class P>
__device__ bool wait_signal(const P& p, const unsigned long long* addr, int cmp, unsigned long long want, uint32_t tile) {
    if (compare(ld_acquire_u64(addr), cmp, want)) return true;
    const unsigned long long deadline = globaltimer_ns() + p.timeout_ns;
    uint32_t spins = 0;
    for (;;) {
        if (compare(ld_acquire_u64(addr), cmp, want)) return true;
        if ((++spins & 7u) == 0) {
            if (aborted(p)) return false;
            if (globaltimer_ns() > deadline) {
                fail(p, HCCL_ERR_TIMEOUT, tile);
                return false;
            }
        }
        __nanosleep(spins < 64 ? 40 : 400);
    }
}

__device__ __forceinline__ char* buf_base(const ExecParams& p, int kind, int rank) {
    if (kind == HCCL_BUF_SEND) return (char*)p.send[rank];
    if (kind == HCCL_BUF_RECV) return (char*)p.recv[rank];
    return p.scratch;
}

// ------------------------------------------------------------------ element conversion
template <int DT>
struct Elem;
template <>
struct Elem<HCCL_FP32> {
    static constexpr int BYTES = 4;
    static __device__ __forceinline__ float load(const char* p, long long i) { return __ldcg((const float*)p + i); }
    static __device__ __forceinline__ void store(char* p, long long i, float v) { __stcg((float*)p + i, v); }
};
template <>
struct Elem<HCCL_BF16> {
    static constexpr int BYTES = 2;
    static __device__ __forceinline__ float load(const char* p, long long i) {
        return __uint_as_float((uint32_t)__ldcg((const unsigned short*)p + i) << 16);
    }
    static __device__ __forceinline__ void store(char* p, long long i, float v) {
        __stcg((unsigned short*)p + i, __bfloat16_as_ushort(__float2bfloat16_rn(v)));
    }
};
template <>
struct Elem<HCCL_FP16> {
    static constexpr int BYTES = 2;
    static __device__ __forceinline__ float load(const char* p, long long i) {
        return __half2float(__ushort_as_half(__ldcg((const unsigned short*)p + i)));
    }
    static __device__ __forceinline__ void store(char* p, long long i, float v) {
        __stcg((unsigned short*)p + i, __half_as_ushort(__float2half_rn(v)));
    }
};

// 8 consecutive elements <-> 8 floats, 16-byte accesses. STREAM: data read once and never written by
// this kernel (send buffers) may use the streaming, L1-allocating path; everything else bypasses L1
// so that values written by other blocks during this launch are seen.
template <int DT, bool STREAM>
__device__ __forceinline__ void load8(const char* p, float (&f)[8]) {
    if constexpr (DT == HCCL_FP32) {
        float4 x, y;
        if constexpr (STREAM) {
            x = __ldcs((const float4*)p);
            y = __ldcs((const float4*)p + 1);
        } else {
            x = __ldcg((const float4*)p);
            y = __ldcg((const float4*)p + 1);
        }
        f[0] = x.x; f[1] = x.y; f[2] = x.z; f[3] = x.w; f[4] = y.x; f[5] = y.y; f[6] = y.z; f[7] = y.w;
    } else {
        uint4 v;
        if constexpr (STREAM) v = __ldcs((const uint4*)p); else v = __ldcg((const uint4*)p);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if constexpr (DT == HCCL_BF16) {
                f[2 * k] = __uint_as_float(w[k] << 16);
                f[2 * k + 1] = __uint_as_float(w[k] & 0xffff0000u);
            } else {
                const __half2 h = *reinterpret_cast<const __half2*>(&w[k]);
                const float2 t = __half22float2(h);
                f[2 * k] = t.x;
                f[2 * k + 1] = t.y;
            }
        }
    }
}
template <int DT, bool STREAM>
__device__ __forceinline__ void store8(char* p, const float (&f)[8]) {
    if constexpr (DT == HCCL_FP32) {
        const float4 x = make_float4(f[0], f[1], f[2], f[3]), y = make_float4(f[4], f[5], f[6], f[7]);
        if constexpr (STREAM) {
            __stcs((float4*)p, x);
            __stcs((float4*)p + 1, y);
        } else {
            __stcg((float4*)p, x);
            __stcg((float4*)p + 1, y);
        }
    } else {
        uint32_t w[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if constexpr (DT == HCCL_BF16) {
                const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * k], f[2 * k + 1]);
                w[k] = *reinterpret_cast<const uint32_t*>(&h);
            } else {
                const __half2 h = __floats2half2_rn(f[2 * k], f[2 * k + 1]);
                w[k] = *reinterpret_cast<const uint32_t*>(&h);
            }
        }
        const uint4 v = make_uint4(w[0], w[1], w[2], w[3]);
        if constexpr (STREAM) __stcs((uint4*)p, v); else __stcg((uint4*)p, v);
    }
}

// ------------------------------------------------------------------ COPY (A=B), register path
template <bool STREAM>
__device__ void copy_tile_lsu(char* dst, const char* src, uint32_t n, const uint32_t tid, const uint32_t nth) {
    const uintptr_t da = (uintptr_t)dst, sa = (uintptr_t)src;
    if (((da ^ sa) & 15u) == 0) {
        uint32_t head = (uint32_t)((16u - (da & 15u)) & 15u);
        if (head > n) head = n;
        for (uint32_t i = tid; i < head; i += nth) dst[i] = __ldcg(src + i);
        const uint32_t nv = (n - head) >> 4;
        const uint4* s = (const uint4*)(src + head);
        uint4* d = (uint4*)(dst + head);
        constexpr int U = 8;
        uint32_t base = 0;
        for (; base + U * nth <= nv; base += U * nth) {
            uint4 v[U];
#pragma unroll
            for (int k = 0; k < U; ++k) v[k] = STREAM ? __ldcs(s + base + k * nth + tid) : __ldcg(s + base + k * nth + tid);
#pragma unroll
            for (int k = 0; k < U; ++k) {
                if (STREAM) __stcs(d + base + k * nth + tid, v[k]); else __stcg(d + base + k * nth + tid, v[k]);
            }
        }
        for (uint32_t i = base + tid; i < nv; i += nth) {
            const uint4 v = STREAM ? __ldcs(s + i) : __ldcg(s + i);
            if (STREAM) __stcs(d + i, v); else __stcg(d + i, v);
        }
        const uint32_t done = head + (nv << 4);
        for (uint32_t i = done + tid; i < n; i += nth) dst[i] = __ldcg(src + i);
    } else if (((da ^ sa) & 3u) == 0) {
        uint32_t head = (uint32_t)((4u - (da & 3u)) & 3u);
        if (head > n) head = n;
        for (uint32_t i = tid; i < head; i += nth) dst[i] = __ldcg(src + i);
        const uint32_t nw = (n - head) >> 2;
        const uint32_t* s = (const uint32_t*)(src + head);
        uint32_t* d = (uint32_t*)(dst + head);
        for (uint32_t i = tid; i < nw; i += nth) __stcg(d + i, __ldcg(s + i));
        for (uint32_t i = head + (nw << 2) + tid; i < n; i += nth) dst[i] = __ldcg(src + i);
    } else {
        for (uint32_t i = tid; i < n; i += nth) dst[i] = __ldcg(src + i);
    }
}

// COPY with several destinations: every byte is read once and stored into the receive buffer of each of the
// nd ranks r0, r0+1, ... (mod R) at byte offset doff. Vector path when the source and all destinations
// share their position inside a 16-byte word; otherwise one plain copy per destination.
template <bool STREAM>
__device__ void copy_tile_fanout(const ExecParams& p, const char* src, int r0, int nd, size_t doff, uint32_t n, const uint32_t tid, const uint32_t nth) {
    const int R = (int)p.R;
    auto dst = [&](int k) -> char* {
        int r = r0 + k;
        if (r >= R) r -= R;
        return (char*)p.recv[r] + doff;
    };
    const uintptr_t sa = (uintptr_t)src;
    bool vec = true;
    for (int k = 0; k < nd; ++k) vec = vec && ((((uintptr_t)dst(k)) ^ sa) & 15u) == 0;
    if (!vec) {
        for (int k = 0; k < nd; ++k) copy_tile_lsu<false>(dst(k), src, n, tid, nth);
        return;
    }
    uint32_t head = (uint32_t)((16u - (sa & 15u)) & 15u);
    if (head > n) head = n;
    const uint32_t nv = (n - head) >> 4, done = head + (nv << 4);
    for (uint32_t i = tid; i < head + (n - done); i += nth) {
        const uint32_t j = i < head ? i : done + (i - head);
        const char b = __ldcg(src + j);
        for (int k = 0; k < nd; ++k) dst(k)[j] = b;
    }
    const uint4* s = (const uint4*)(src + head);
    constexpr int U = 4;
    uint32_t base = 0;
    for (; base + U * nth <= nv; base += U * nth) {
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) v[u] = STREAM ? __ldcs(s + base + u * nth + tid) : __ldcg(s + base + u * nth + tid);
        for (int k = 0; k < nd; ++k) {
            uint4* d = (uint4*)(dst(k) + head) + base + tid;
#pragma unroll
            for (int u = 0; u < U; ++u) __stcs(d + u * nth, v[u]);
        }
    }
    for (uint32_t i = base + tid; i < nv; i += nth) {
        const uint4 v = STREAM ? __ldcs(s + i) : __ldcg(s + i);
        for (int k = 0; k < nd; ++k) __stcs((uint4*)(dst(k) + head) + i, v);
    }
}

// ------------------------------------------------------------------ REDUCE (S=A+B and in-place forms)
template <int DA, int DB, int DD, bool STREAM_B>
__device__ void reduce_tile_lsu(char* dst, const char* a, const char* b, uint32_t n, const uint32_t tid, const uint32_t nth) {
    // Vector path when the three operands sit at the same element phase modulo 8 (then one short scalar
    // head aligns all of them to 16 bytes); otherwise element by element.
    const uint32_t pa = (uint32_t)(((uintptr_t)a / Elem<DA>::BYTES) & 7u), pb = (uint32_t)(((uintptr_t)b / Elem<DB>::BYTES) & 7u),
                   pd = (uint32_t)(((uintptr_t)dst / Elem<DD>::BYTES) & 7u);
    if (pa != pb || pa != pd) {
        for (uint32_t i = tid; i < n; i += nth) Elem<DD>::store(dst, i, Elem<DA>::load(a, i) + Elem<DB>::load(b, i));
        return;
    }
    uint32_t head = (8u - pa) & 7u;
    if (head > n) head = n;
    if (tid < head) Elem<DD>::store(dst, tid, Elem<DA>::load(a, tid) + Elem<DB>::load(b, tid));
    const uint32_t nv = (n - head) >> 3;
    const char* av = a + (size_t)head * Elem<DA>::BYTES;
    const char* bv = b + (size_t)head * Elem<DB>::BYTES;
    char* dv = dst + (size_t)head * Elem<DD>::BYTES;
    constexpr int U = 4;
    uint32_t base = 0;
    for (; base + U * nth <= nv; base += U * nth) {
        float fa[U][8], fb[U][8];
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const size_t i = base + k * nth + tid;
            load8<DA, false>(av + i * 8 * Elem<DA>::BYTES, fa[k]);
            load8<DB, STREAM_B>(bv + i * 8 * Elem<DB>::BYTES, fb[k]);
        }
#pragma unroll
        for (int k = 0; k < U; ++k) {
            const size_t i = base + k * nth + tid;
#pragma unroll
            for (int e = 0; e < 8; ++e) fa[k][e] = fa[k][e] + fb[k][e];
            store8<DD, false>(dv + i * 8 * Elem<DD>::BYTES, fa[k]);
        }
    }
    for (uint32_t i = base + tid; i < nv; i += nth) {
        float fa[8], fb[8];
        load8<DA, false>(av + (size_t)i * 8 * Elem<DA>::BYTES, fa);
        load8<DB, STREAM_B>(bv + (size_t)i * 8 * Elem<DB>::BYTES, fb);
#pragma unroll
        for (int e = 0; e < 8; ++e) fa[e] = fa[e] + fb[e];
        store8<DD, false>(dv + (size_t)i * 8 * Elem<DD>::BYTES, fa);
    }
    for (uint32_t i = head + (nv << 3) + tid; i < n; i += nth) Elem<DD>::store(dst, i, Elem<DA>::load(a, i) + Elem<DB>::load(b, i));
}

template <int DA, int DB, bool SB>
__device__ __forceinline__ void reduce_dispatch_d(int dd, char* dst, const char* a, const char* b, uint32_t n, uint32_t tid, uint32_t nth) {
    if (dd == HCCL_FP32) reduce_tile_lsu<DA, DB, HCCL_FP32, SB>(dst, a, b, n, tid, nth);
    else if (dd == HCCL_BF16) reduce_tile_lsu<DA, DB, HCCL_BF16, SB>(dst, a, b, n, tid, nth);
    else reduce_tile_lsu<DA, DB, HCCL_FP16, SB>(dst, a, b, n, tid, nth);
}
template <int DA, bool SB>
__device__ __forceinline__ void reduce_dispatch_b(int db, int dd, char* dst, const char* a, const char* b, uint32_t n, uint32_t tid, uint32_t nth) {
    if (db == HCCL_FP32) reduce_dispatch_d<DA, HCCL_FP32, SB>(dd, dst, a, b, n, tid, nth);
    else if (db == HCCL_BF16) reduce_dispatch_d<DA, HCCL_BF16, SB>(dd, dst, a, b, n, tid, nth);
    else reduce_dispatch_d<DA, HCCL_FP16, SB>(dd, dst, a, b, n, tid, nth);
}
template <bool SB>
__device__ void reduce_dispatch(int da, int db, int dd, char* dst, const char* a, const char* b, uint32_t n, uint32_t tid, uint32_t nth) {
    if (da == HCCL_FP32) reduce_dispatch_b<HCCL_FP32, SB>(db, dd, dst, a, b, n, tid, nth);
    else if (da == HCCL_BF16) reduce_dispatch_b<HCCL_BF16, SB>(db, dd, dst, a, b, n, tid, nth);
    else reduce_dispatch_b<HCCL_FP16, SB>(db, dd, dst, a, b, n, tid, nth);
}

// ------------------------------------------------------------------ REDUCE_N (multi-input sum, fixed order)
// Barrier over `nthreads` threads that also ANDs a predicate over them.
__device__ __forceinline__ bool named_sync_and(uint32_t id, uint32_t nthreads, bool pred) {
    uint32_t out;
    asm volatile(
        "{\n\t.reg .pred q, r;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.and.pred r, %2, %3, q;\n\tselp.u32 %0, 1, 0, r;\n\t}"
        : "=r"(out) : "r"((uint32_t)pred), "r"(id), "r"(nthreads) : "memory");
    return out != 0;
}
constexpr uint32_t BARRIER_WORKERS = 5;  // named barrier of the register engine's worker threads alone
// Shared memory for the operand addresses of one REDUCE_N item (sources, then destinations): one array for all
// element-type instantiations, and none in kernels that never ask for it.
template <bool USED>
__device__ __forceinline__ const char** operand_table() {
    __shared__ const char* s_operands[USED ? 2 * HCCL_MAX_RANKS : 1];
    return s_operands;
}

// TABLE (register engine, one block per SM): the operand addresses are put into shared memory first, one per
// thread, and the alignment check is one AND over the block's worker threads. Without it every thread walks the
// pointer arrays of the parameter block (constant cache) for every source and destination, one dependent lookup
// after the other, again for every vector it handles. All `nth` threads must call this together (they meet at a
// named barrier).
template <int DS, int DD, bool TABLE>
__device__ void reduce_n_tile(const ExecParams& p, const Desc& d, uint64_t start, uint32_t n, const uint32_t tid, const uint32_t nth) {
    const int R = (int)p.R, nsrc = d.nsrc, r0 = d.rank_a;
    const size_t soff = (size_t)d.off_a + start * Elem<DS>::BYTES;
    // destinations: one, or the receive buffers of nd consecutive ranks at the same offset
    const int nd = d.ndst > 1 ? d.ndst : 1, rd0 = d.rank_dst;
    const size_t doff = (size_t)d.off_dst + start * Elem<DD>::BYTES;
    char* const dst0 = buf_base(p, d.kind_dst, d.rank_dst) + doff;
    auto dstp = [&](int j) -> char* {
        if (j == 0) return dst0;
        int r = rd0 + j;
        if (r >= R) r -= R;
        return (char*)p.recv[r] + doff;
    };
    const bool from_send = d.kind_a == HCCL_BUF_SEND;
    auto src_lookup = [&](int k) -> const char* {
        int r = r0 + k;
        if (r >= R) r -= R;
        return (const char*)(from_send ? p.send[r] : (const void*)p.recv[r]) + soff;
    };
    // same phase for every operand?
    const uint32_t pd = (uint32_t)(((uintptr_t)dst0 / Elem<DD>::BYTES) & 7u);
    bool vec = true;
    const char** const s_src = TABLE ? operand_table<TABLE>() : nullptr;
    char** const s_dst = TABLE ? (char**)(operand_table<TABLE>() + HCCL_MAX_RANKS) : nullptr;
    if constexpr (TABLE) {
        // one operand per warp and round: a constant-cache lookup is fast only when a warp's lanes ask for the same word
        for (int k = (int)(tid >> 5); k < nsrc + nd; k += (int)(nth >> 5)) {
            if (k < nsrc) {
                const char* q = src_lookup(k);
                if ((tid & 31u) == 0) s_src[k] = q;
                vec = vec && ((uint32_t)(((uintptr_t)q / Elem<DS>::BYTES) & 7u) == pd);
            } else {
                char* q = dstp(k - nsrc);
                if ((tid & 31u) == 0) s_dst[k - nsrc] = q;
                vec = vec && ((uint32_t)(((uintptr_t)q / Elem<DD>::BYTES) & 7u) == pd);
            }
        }
        vec = named_sync_and(BARRIER_WORKERS, nth, vec);
    } else {
        for (int k = 0; k < nsrc; ++k) vec = vec && ((uint32_t)(((uintptr_t)src_lookup(k) / Elem<DS>::BYTES) & 7u) == pd);
        for (int j = 1; j < nd; ++j) vec = vec && ((uint32_t)(((uintptr_t)dstp(j) / Elem<DD>::BYTES) & 7u) == pd);
    }
    auto src = [&](int k) -> const char* {
        if constexpr (TABLE) return s_src[k]; else return src_lookup(k);
    };
    auto dst = [&](int j) -> char* {
        if constexpr (TABLE) return s_dst[j]; else return dstp(j);
    };
    if (!vec) {
        for (uint32_t i = tid; i < n; i += nth) {
            float acc = Elem<DS>::load(src(0), i);
            for (int k = 1; k < nsrc; ++k) acc = acc + Elem<DS>::load(src(k), i);
            for (int j = 0; j < nd; ++j) Elem<DD>::store(dst(j), i, acc);
        }
        return;
    }
    uint32_t head = (8u - pd) & 7u;
    if (head > n) head = n;
    const uint32_t nv = (n - head) >> 3;
    auto scalar = [&](uint32_t i) {
        float acc = Elem<DS>::load(src(0), i);
        for (int k = 1; k < nsrc; ++k) acc = acc + Elem<DS>::load(src(k), i);
        for (int j = 0; j < nd; ++j) Elem<DD>::store(dst(j), i, acc);
    };
    if (tid < head) scalar(tid);
    for (uint32_t i = head + (nv << 3) + tid; i < n; i += nth) scalar(i);
    const size_t hs = (size_t)head * Elem<DS>::BYTES;
    // Vector body: the loads of a group of sources are all issued before the first add, so a thread has G
    // 16-byte (or 32-byte) requests in flight; the adds then run in source order.
    constexpr int G = (DS == HCCL_FP32) ? 4 : 8;   // sources fetched together
    constexpr int W = (DS == HCCL_FP32) ? 2 : 1;   // 16-byte words per 8 elements
    const bool stream = (d.cmp & 1u) != 0;         // planner's hint: every source byte is read exactly once
    auto widen = [](const uint4 (&raw)[W], float (&x)[8]) {
        if constexpr (DS == HCCL_FP32) {
            x[0] = __uint_as_float(raw[0].x); x[1] = __uint_as_float(raw[0].y);
            x[2] = __uint_as_float(raw[0].z); x[3] = __uint_as_float(raw[0].w);
            x[4] = __uint_as_float(raw[W - 1].x); x[5] = __uint_as_float(raw[W - 1].y);
            x[6] = __uint_as_float(raw[W - 1].z); x[7] = __uint_as_float(raw[W - 1].w);
        } else {
            const uint32_t wv[4] = {raw[0].x, raw[0].y, raw[0].z, raw[0].w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                if constexpr (DS == HCCL_BF16) {
                    x[2 * h] = __uint_as_float(wv[h] << 16);
                    x[2 * h + 1] = __uint_as_float(wv[h] & 0xffff0000u);
                } else {
                    const float2 t2 = __half22float2(*reinterpret_cast<const __half2*>(&wv[h]));
                    x[2 * h] = t2.x;
                    x[2 * h + 1] = t2.y;
                }
            }
        }
    };
    auto fetch = [&](int k, size_t off, uint4 (&raw)[W]) {
        const uint4* q = reinterpret_cast<const uint4*>(src(k) + off);
#pragma unroll
        for (int w = 0; w < W; ++w) raw[w] = stream ? __ldcs(q + w) : __ldcg(q + w);
    };
    // A group of N consecutive sources starting at k0: N loads in flight, then N adds in source order.
    // INIT: the group's first source starts the sum (x + 0 would turn -0 into +0).
    auto group = [&](auto n_tag, auto init_tag, int k0, size_t off, float (&acc)[8]) {
        constexpr int N = decltype(n_tag)::value;
        constexpr bool INIT = decltype(init_tag)::value;
        uint4 raw[N][W];
#pragma unroll
        for (int j = 0; j < N; ++j) fetch(k0 + j, off, raw[j]);
#pragma unroll
        for (int j = 0; j < N; ++j) {
            float x[8];
            widen(raw[j], x);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = (INIT && j == 0) ? x[e] : acc[e] + x[e];
        }
    };
    using T = std::true_type;
    using F = std::false_type;
    for (uint32_t i = tid; i < nv; i += nth) {
        const size_t off = hs + (size_t)i * 8 * Elem<DS>::BYTES;
        float acc[8];
        int k;
        if (nsrc >= G) { group(std::integral_constant<int, G>{}, T{}, 0, off, acc); k = G; }
        else { group(std::integral_constant<int, 1>{}, T{}, 0, off, acc); k = 1; }
        for (; k + G <= nsrc; k += G) group(std::integral_constant<int, G>{}, F{}, k, off, acc);
        for (; k < nsrc; ++k) group(std::integral_constant<int, 1>{}, F{}, k, off, acc);
        const size_t o = (size_t)head * Elem<DD>::BYTES + (size_t)i * 8 * Elem<DD>::BYTES;
        store8<DD, false>(dst0 + o, acc);
        for (int j = 1; j < nd; ++j) store8<DD, false>(dst(j) + o, acc);
    }
}

template <bool TABLE>
static __device__ void reduce_n_dispatch(const ExecParams& p, const Desc& d, uint64_t start, uint32_t n, uint32_t tid, uint32_t nth) {
#define RN(S, D) reduce_n_tile<S, D, TABLE>(p, d, start, n, tid, nth)
    if (d.dt_a == HCCL_FP32) {
        if (d.dt_dst == HCCL_FP32) RN(HCCL_FP32, HCCL_FP32); else if (d.dt_dst == HCCL_BF16) RN(HCCL_FP32, HCCL_BF16); else RN(HCCL_FP32, HCCL_FP16);
    } else if (d.dt_a == HCCL_BF16) {
        if (d.dt_dst == HCCL_FP32) RN(HCCL_BF16, HCCL_FP32); else if (d.dt_dst == HCCL_BF16) RN(HCCL_BF16, HCCL_BF16); else RN(HCCL_BF16, HCCL_FP16);
    } else {
        if (d.dt_dst == HCCL_FP32) RN(HCCL_FP16, HCCL_FP32); else if (d.dt_dst == HCCL_BF16) RN(HCCL_FP16, HCCL_BF16); else RN(HCCL_FP16, HCCL_FP16);
    }
#undef RN
}

// ------------------------------------------------------------------ one work item, all threads
// The operand addresses of a COPY (one destination) or REDUCE item. With static chains the control warp works them
// out for 32 items at once, one lane per item, so that the worker threads do not each walk from buffer kind and rank
// to a base address and on to the tile's offset before their first load (0.25 us of a chain step of 0.75 us).
struct Resolved {
    char* dst;
    const char* a;
    const char* b;
};
__device__ __forceinline__ bool resolve(const ExecParams& p, const Desc& d, const Tile& t, Resolved& r) {
    if (d.op == HCCL_OP_COPY && d.ndst <= 1) {
        r.a = buf_base(p, d.kind_a, d.rank_a) + d.off_a + t.start;
        r.dst = buf_base(p, d.kind_dst, d.rank_dst) + d.off_dst + t.start;
        r.b = nullptr;
        return true;
    }
    if (d.op == HCCL_OP_REDUCE) {
        r.dst = buf_base(p, d.kind_dst, d.rank_dst) + d.off_dst + t.start * (d.dt_dst == HCCL_FP32 ? 4 : 2);
        r.a = buf_base(p, d.kind_a, d.rank_a) + d.off_a + t.start * (d.dt_a == HCCL_FP32 ? 4 : 2);
        r.b = buf_base(p, d.kind_b, d.rank_b) + d.off_b + t.start * (d.dt_b == HCCL_FP32 ? 4 : 2);
        return true;
    }
    return false;
}

// TABLE: see reduce_n_tile (all `nth` threads call this together and may meet at the workers' named barrier).
// `r`: the item's operand addresses if they have been worked out already, else null.
template <bool TABLE>
static __device__ void run_tile_lsu(const ExecParams& p, const Desc& d, const Tile& t, const uint32_t tid, const uint32_t nth, const Resolved* r = nullptr) {
    if (TABLE && r) {  // only the builds that can afford the code (and ever pass addresses)
        if (d.op == HCCL_OP_COPY) {
            if (d.kind_a == HCCL_BUF_SEND) copy_tile_lsu<true>(r->dst, r->a, t.count, tid, nth); else copy_tile_lsu<false>(r->dst, r->a, t.count, tid, nth);
        } else {
            if (d.kind_b == HCCL_BUF_SEND) reduce_dispatch<true>(d.dt_a, d.dt_b, d.dt_dst, r->dst, r->a, r->b, t.count, tid, nth);
            else reduce_dispatch<false>(d.dt_a, d.dt_b, d.dt_dst, r->dst, r->a, r->b, t.count, tid, nth);
        }
        return;
    }
    switch (d.op) {
        case HCCL_OP_COPY: {
            const char* src = buf_base(p, d.kind_a, d.rank_a) + d.off_a + t.start;
            if (d.ndst > 1) {
                if (d.kind_a == HCCL_BUF_SEND) copy_tile_fanout<true>(p, src, d.rank_dst, d.ndst, (size_t)d.off_dst + t.start, t.count, tid, nth);
                else copy_tile_fanout<false>(p, src, d.rank_dst, d.ndst, (size_t)d.off_dst + t.start, t.count, tid, nth);
                break;
            }
            char* dst = buf_base(p, d.kind_dst, d.rank_dst) + d.off_dst + t.start;
            // send-to-receive copies (AllToAllv, AllGather's first hop) are read once and written once
            if (d.kind_a == HCCL_BUF_SEND) copy_tile_lsu<true>(dst, src, t.count, tid, nth); else copy_tile_lsu<false>(dst, src, t.count, tid, nth);
            break;
        }
        case HCCL_OP_REDUCE: {
            char* dst = buf_base(p, d.kind_dst, d.rank_dst) + d.off_dst + t.start * (d.dt_dst == HCCL_FP32 ? 4 : 2);
            const char* a = buf_base(p, d.kind_a, d.rank_a) + d.off_a + t.start * (d.dt_a == HCCL_FP32 ? 4 : 2);
            const char* b = buf_base(p, d.kind_b, d.rank_b) + d.off_b + t.start * (d.dt_b == HCCL_FP32 ? 4 : 2);
            if (d.kind_b == HCCL_BUF_SEND) reduce_dispatch<true>(d.dt_a, d.dt_b, d.dt_dst, dst, a, b, t.count, tid, nth);
            else reduce_dispatch<false>(d.dt_a, d.dt_b, d.dt_dst, dst, a, b, t.count, tid, nth);
            break;
        }
        case HCCL_OP_REDUCE_N:
            reduce_n_dispatch<TABLE>(p, d, t.start, t.count, tid, nth);
            break;
        default:
            break;
    }
}

// Checks on a table entry before it is used; a failing entry is reported, never dereferenced.
static __device__ bool tile_ok(const ExecParams& p, const Tile& t) {
    if (t.desc >= p.n_descs) return false;
    if ((uint64_t)t.wait_off + t.wait_cnt > p.n_waits) return false;
    for (int k = 0; k < 2; ++k)
        if (t.signal[k] >= (int32_t)p.n_syncs) return false;
    return true;
}
static __device__ bool desc_ok(const ExecParams& p, const Desc& d) {
    if (d.op > HCCL_OP_NOOP) return false;
    if (d.op == HCCL_OP_COPY || d.op == HCCL_OP_REDUCE || d.op == HCCL_OP_REDUCE_N) {
        if (d.kind_dst != HCCL_BUF_RECV && d.kind_dst != HCCL_BUF_SCRATCH) return false;
        if (d.kind_a > HCCL_BUF_SCRATCH) return false;
        if (d.rank_dst >= p.R || d.rank_a >= p.R) return false;
        if (d.op == HCCL_OP_REDUCE && (d.kind_b > HCCL_BUF_SCRATCH || d.rank_b >= p.R)) return false;
        if (d.op != HCCL_OP_COPY && (d.dt_dst > HCCL_FP16 || d.dt_a > HCCL_FP16 || (d.op == HCCL_OP_REDUCE && d.dt_b > HCCL_FP16))) return false;
        if (d.op == HCCL_OP_REDUCE_N && (d.nsrc < 1 || d.nsrc > p.R || d.kind_a > HCCL_BUF_RECV)) return false;
        if (d.op != HCCL_OP_REDUCE && d.ndst > 1 && (d.ndst > p.R || d.kind_dst != HCCL_BUF_RECV)) return false;
    }
    if (d.op == HCCL_OP_WAIT) {
        if (d.kind_a == HCCL_BUF_SIGNAL) return (uint64_t)d.off_a < p.n_signals;
        if (d.kind_a == HCCL_BUF_USER_SIGNAL) return d.off_a >= 0 && d.off_a < p.n_user_signals;
        return false;
    }
    if (d.op == HCCL_OP_SET) {
        if (d.kind_dst == HCCL_BUF_SIGNAL) return (uint64_t)d.off_dst < p.n_signals;
        if (d.kind_dst == HCCL_BUF_USER_SIGNAL) return d.off_dst >= 0 && d.off_dst < p.n_user_signals;
        return false;
    }
    return true;
}

__device__ __forceinline__ void publish_tile(const ExecParams& p, const Tile& t) {
    if (t.signal[0] >= 0 || t.signal[1] >= 0) {
        __threadfence();
        if (t.signal[0] >= 0) red_release_add_u32(p.counters + t.signal[0], 1);
        if (t.signal[1] >= 0) red_release_add_u32(p.counters + t.signal[1], 1);
    }
}

// Last block out: completion value for a device-triggered caller, epoch stamp, clean ticket.
// `lean`: nobody reads the control block or the results before this launch has ended (no completion value to
// publish, not the resident executor), so the end of the kernel orders everything and the fences are left out.
// Returns true in the block that was last.
template <class P>
__device__ bool leave(const P& p, bool lean = false) {
    if (!lean) __threadfence();
    const uint32_t prev = atomicAdd(&p.ctl->exits, 1);
    if (prev == p.nblocks - 1) {
        if (!lean) __threadfence();
        if (p.trig_set_slot >= 0 && !aborted(p)) st_release_u64(p.user_signals + p.trig_set_slot, p.trig_set_value + (unsigned long long)g_epoch * p.trig_set_per_epoch);
        p.ctl->t_last_ns = globaltimer_ns();
        p.ctl->ticket = 0;
        p.ctl->exits = 0;
        if (!lean) __threadfence();
        p.ctl->done_epoch = g_epoch;
        return true;
    }
    return false;
}

// Named barriers of the register engine (id 0 is left to __syncthreads).
__device__ __forceinline__ void named_sync(uint32_t id, uint32_t nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

// Loads and checks the records of work item `cur`. No waiting here.
static __device__ bool fetch_tile(const ExecParams& p, uint32_t cur, Tile& t, Desc& d, const Tile* preloaded = nullptr) {
    if (p.trace) {
        trace_put(p.trace, p.trace_cap, cur, 0, (unsigned long long)cur | ((unsigned long long)blockIdx.x << 32));
        trace_put(p.trace, p.trace_cap, cur, 1, globaltimer_ns());
    }
    t = preloaded ? *preloaded : p.tiles[cur];
    if (t.flags & TILE_FLAG_END) return false;  // behind the last item of a device-built table: no more work, no failure
    if (!tile_ok(p, t)) {
        fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
        return false;
    }
    d = p.descs[t.desc];
    if (!desc_ok(p, d)) {
        fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
        return false;
    }
    return true;
}
// Static chains: a block's items are consecutive table entries known from the start, so the 32 lanes of the control
// warp fetch the records of the next 32 of them at once (one trip to memory for the tiles, one for the
// descriptors) instead of lane 0 paying both trips for every item. `lane`: every lane of the warp calls this.
constexpr uint32_t WINDOW = 32;
// Each lane also runs the checks on its own item, so that lane 0 later only copies the records (its work between two
// items of a chain is on the chain's critical path, one instruction after the other).
// wok: 0 the item fails its checks, 1 it passes, 2 it passes and its operand addresses are in wr.
__device__ __forceinline__ void window_fill(const ExecParams& p, uint32_t first, uint32_t end, uint32_t lane, Tile* wt, Desc* wd, Resolved* wr, uint8_t* wok) {
    const uint32_t idx = first + lane;
    if (idx < end && idx < p.n_tiles) {
        const Tile t = p.tiles[idx];
        wt[lane] = t;
        uint8_t ok = 0;
        if (!(t.flags & TILE_FLAG_END) && tile_ok(p, t)) {
            const Desc d = p.descs[t.desc];
            wd[lane] = d;
            if (desc_ok(p, d)) {
                Resolved r;
                ok = resolve(p, d, t, r) ? 2 : 1;
                if (ok == 2) wr[lane] = r;
            }
        }
        wok[lane] = ok;
    }
    __syncwarp();
}
// An item whose records are in the window.
static __device__ bool fetch_windowed(const ExecParams& p, uint32_t cur, Tile& t, Desc& d, const Tile& wt, const Desc& wd, uint8_t ok) {
    if (p.trace) {
        trace_put(p.trace, p.trace_cap, cur, 0, (unsigned long long)cur | ((unsigned long long)blockIdx.x << 32));
        trace_put(p.trace, p.trace_cap, cur, 1, globaltimer_ns());
    }
    t = wt;
    if (t.flags & TILE_FLAG_END) return false;
    if (!ok) {
        fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
        return false;
    }
    d = wd;
    return true;
}
// One non-blocking look at every dependency counter of the item.
static __device__ bool deps_ready(const ExecParams& p, const Tile& t) {
    for (uint32_t w = 0; w < t.wait_cnt; ++w) {
        const Wait x = p.waits[t.wait_off + w];
        if (x.sync >= p.n_syncs) return false;
        if ((int32_t)(ld_acquire_u32(p.counters + x.sync) - g_epoch * x.per_epoch) < 0) return false;
    }
    return true;
}
// Blocking (bounded) part: dependency counters, then a WAIT's condition; a SET is performed here.
static __device__ bool wait_deps(const ExecParams& p, uint32_t cur, const Tile& t, const Desc& d, bool counters_done) {
    if (!counters_done) {
        for (uint32_t w = 0; w < t.wait_cnt; ++w) {
            const Wait x = p.waits[t.wait_off + w];
            if (x.sync >= p.n_syncs) {
                fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
                return false;
            }
            if (!wait_counter(p, x.sync, x.per_epoch, cur)) return false;
        }
    }
    if (d.op == HCCL_OP_WAIT) {
        const unsigned long long* addr = (d.kind_a == HCCL_BUF_SIGNAL ? p.signals : p.user_signals) + d.off_a;
        if (!wait_signal(p, addr, d.cmp, d.value + (unsigned long long)g_epoch * d.value_per_epoch, cur)) return false;
    } else if (d.op == HCCL_OP_SET) {
        unsigned long long* addr = (d.kind_dst == HCCL_BUF_SIGNAL ? p.signals : p.user_signals) + d.off_dst;
        __threadfence();
        st_release_u64(addr, d.value + (unsigned long long)g_epoch * d.value_per_epoch);
    }
    return true;
}

// Register engine. Warp 0 is the control warp: its first lane claims tickets, fetches the next item's
// records and looks at its dependency counters while the worker warps are still moving the current item,
// and publishes an item's completion while the workers are already on the next one. Two shared-memory
// buffers hold the current and the next item; named barriers FULL[b] (item in buffer b may start) and
// DONE[b] (workers have stored all of it) pair the two sides.
// Static chains: the items of block b (an even share of the chains, contiguous).
__device__ __forceinline__ void chain_range(const ExecParams& p, uint32_t& first_item, uint32_t& end_item) {
    const uint32_t B = p.nblocks, q = p.n_chains / B, rem = p.n_chains % B, b = blockIdx.x;
    const uint32_t c0 = b * q + min(b, rem), c1 = c0 + q + (b < rem ? 1u : 0u);
    first_item = c0 * p.chain_len;
    end_item = c1 * p.chain_len;
}
// The first item of a block, and the one after `cur`.
__device__ __forceinline__ uint32_t first_item(const ExecParams& p, uint32_t& range_end) {
    if (p.chain_len) {
        uint32_t f;
        chain_range(p, f, range_end);
        return f < range_end ? f : p.n_tiles;
    }
    return p.static_tickets ? blockIdx.x : atomicAdd(&p.ctl->ticket, 1);
}
// `left` counts the claims a block may still make (opts.quantum; effectively unbounded when that is 0).
__device__ __forceinline__ uint32_t next_item(const ExecParams& p, uint32_t cur, uint32_t range_end, uint32_t& left) {
    if (p.chain_len) return cur + 1 < range_end ? cur + 1 : p.n_tiles;
    if (p.static_tickets || left == 0) return p.n_tiles;
    --left;
    return atomicAdd(&p.ctl->ticket, 1);
}

template <bool RESIDENT, bool AHEAD>
__device__ __forceinline__ void executor_lsu_body(const ExecParams& p) {
    __shared__ Tile s_tile[2];
    __shared__ Desc s_desc[2];
    __shared__ int s_go[2];
    __shared__ Tile s_wtile[AHEAD ? WINDOW : 1];  // static chains: records of the items [win_base, win_base + WINDOW)
    __shared__ Desc s_wdesc[AHEAD ? WINDOW : 1];
    __shared__ uint8_t s_wok[AHEAD ? WINDOW : 1];   // the checks on them, done by the lane that fetched them
    __shared__ Resolved s_wres[AHEAD ? WINDOW : 1]; // and their operand addresses
    __shared__ Resolved s_res[2];                   // of the items in s_tile / s_desc (valid where s_go says 2)
    const bool window = AHEAD && p.chain_len != 0;
    uint32_t win_base = 0, win_end = 0;  // win_end: end of the block's items
    const uint32_t tid = threadIdx.x, nth = blockDim.x;
    constexpr uint32_t FULL = 1, DONE = 3;  // barrier ids FULL+b, DONE+b
    // Entry. The execution number, the abort word, the first ticket and (with static tickets) the first item's
    // tile record do not depend on one another: thread 0 issues all of these loads before it uses any of
    // them, so a small collective pays one trip to memory here instead of four in a row.
    uint32_t next = 0, abort0 = 0, range_end = 0;
    uint32_t left = p.quantum ? p.quantum - 1u : 0xffffffffu;  // the first claim is made at entry
    Tile pre;
    bool pre_ok = false;
    const bool gated = p.trig_wait_slot >= 0;
    if (tid == 0) {
        if (!gated) {
            next = first_item(p, range_end);
            if (next < p.n_tiles && !window) {
                pre = p.tiles[next];
                pre_ok = true;
            }
        }
        abort0 = *(volatile uint32_t*)&p.ctl->abort;
        g_epoch = *(volatile uint32_t*)&p.ctl->done_epoch + 1u;
    }
    if (window && tid < 32) {  // the tables do not change: they may be read before a trigger has fired
        chain_range(p, win_base, win_end);
        window_fill(p, win_base, win_end, tid, s_wtile, s_wdesc, s_wres, s_wok);
    }
    __syncthreads();
    if (tid >= 32) {
        const uint32_t wtid = tid - 32, nwork = nth - 32;
        for (uint32_t k = 0;; ++k) {
            const uint32_t b = k & 1;
            named_sync(FULL + b, nth);
            if (!s_go[b]) break;
            run_tile_lsu<AHEAD>(p, s_desc[b], s_tile[b], wtid, nwork, s_go[b] == 2 ? &s_res[b] : nullptr);
            if (!window) named_sync(DONE + b, nth);  // static chains: the next item's FULL barrier says it as well
        }
        return;
    }
    // ---- control warp; every lane executes the barriers, lane 0 does the rest
    bool live = true, have = false, ready = false;
    if (tid == 0) {
        if (gated) {
            live = wait_signal(p, p.user_signals + p.trig_wait_slot, p.trig_cmp, p.trig_wait_value + (unsigned long long)g_epoch * p.trig_wait_per_epoch, 0xffffffffu);
            next = first_item(p, range_end);
        }
        if (next == 0) p.ctl->t_first_ns = globaltimer_ns();
    }
    uint32_t cur = 0, prev_item = 0;
    if (window) {
        // Static chains: no item waits for anything but the item before it in this block, and none has anything to
        // publish. One barrier per item then does: FULL[b] lets the workers start item k, and their arrival at
        // it says that item k-1 is stored. The control warp fills the other buffer with item k+1 in the meantime.
        const uint32_t end = min(win_end, p.n_tiles);
        cur = win_base;  // every lane keeps the item numbers (the lanes refill the window together)
        if (tid == 0) {
            const bool h = live && cur < end && !(gated ? aborted(p) : abort0 == g_epoch);
            const bool f = h && fetch_windowed(p, cur, s_tile[0], s_desc[0], s_wtile[0], s_wdesc[0], s_wok[0]);
            if (f && s_wok[0] == 2) s_res[0] = s_wres[0];
            s_go[0] = f ? s_wok[0] : 0;  // 1: run it; 2: run it, its operand addresses are in s_res
        }
        for (uint32_t k = 0;; ++k) {
            const uint32_t b = k & 1;
            named_sync(FULL + b, nth);
            const int go = s_go[b];
            if (tid == 0 && p.trace) {
                const unsigned long long now = globaltimer_ns();
                if (k > 0) trace_put(p.trace, p.trace_cap, prev_item, 3, now);
                if (go) trace_put(p.trace, p.trace_cap, cur, 2, now);
            }
            if (!go) break;
            const uint32_t nx = cur + 1;
            if (nx < end && nx - win_base >= WINDOW) {
                win_base = nx;
                window_fill(p, win_base, win_end, tid, s_wtile, s_wdesc, s_wres, s_wok);
            }
            if (tid == 0) {
                const uint32_t ab = ld_relaxed_u32(&p.ctl->abort);  // asked for first, looked at when the records are in
                const uint32_t slot = nx < end ? nx - win_base : 0;
                const bool h = nx < end && fetch_windowed(p, nx, s_tile[b ^ 1], s_desc[b ^ 1], s_wtile[slot], s_wdesc[slot], s_wok[slot]);
                if (h && s_wok[slot] == 2) s_res[b ^ 1] = s_wres[slot];
                s_go[b ^ 1] = (h && ab != g_epoch) ? s_wok[slot] : 0;
            }
            prev_item = cur;
            cur = nx;
        }
    } else
    for (uint32_t k = 0;; ++k) {
        const uint32_t b = k & 1;
        int32_t sig0 = -1, sig1 = -1;
        bool prev = false;
        if (tid == 0) {
            // item k: its records were fetched during item k-1 (or are fetched now for the first one)
            if (k == 0) {
                cur = next;
                have = live && cur < p.n_tiles && !(gated ? aborted(p) : abort0 == g_epoch);
                if (have) {
                    next = next_item(p, cur, range_end, left);
                    have = fetch_tile(p, cur, s_tile[0], s_desc[0], pre_ok ? &pre : nullptr);
                    ready = have && deps_ready(p, s_tile[0]);
                }
            }
            prev = k > 0;
            if (prev) {
                sig0 = s_tile[b ^ 1].signal[0];
                sig1 = s_tile[b ^ 1].signal[1];
            }
        }
        if (k > 0) named_sync(DONE + (b ^ 1), nth);  // the workers have stored all of item k-1
        if (tid == 0 && p.trace && k > 0) trace_put(p.trace, p.trace_cap, prev_item, 3, globaltimer_ns());
        if (tid == 0) {
            const bool simple = have && ready && s_desc[b].op != HCCL_OP_WAIT && s_desc[b].op != HCCL_OP_SET;
            if (!simple && prev && (sig0 >= 0 || sig1 >= 0)) {
                // item k may have to wait (perhaps for item k-1 itself): publish k-1 first. The release is
                // cumulative: it covers the workers' stores that the DONE barrier ordered before this thread.
                if (sig0 >= 0) red_release_add_u32(p.counters + sig0, 1);
                if (sig1 >= 0) red_release_add_u32(p.counters + sig1, 1);
                sig0 = sig1 = -1;
            }
            bool go = have;  // `have` carries the abort word as the look-ahead saw it; waits look at it again
            if (go && !simple) go = wait_deps(p, cur, s_tile[b], s_desc[b], ready);
            s_go[b] = go ? 1 : 0;
        }
        named_sync(FULL + b, nth);  // workers start item k (or leave)
        const int go = s_go[b];
        if (tid == 0 && p.trace && go) trace_put(p.trace, p.trace_cap, cur, 2, globaltimer_ns());
        prev_item = cur;
        if (tid == 0) {
            if (sig0 >= 0 || sig1 >= 0) {  // publish item k-1 while the workers run item k
                if (sig0 >= 0) red_release_add_u32(p.counters + sig0, 1);
                if (sig1 >= 0) red_release_add_u32(p.counters + sig1, 1);
            }
            if (go) {
                // look ahead: claim, fetch and poll item k+1 behind the workers' back
                cur = next;
                const uint32_t ab = ld_relaxed_u32(&p.ctl->abort);  // asked for first, looked at when the records are in
                have = cur < p.n_tiles;
                if (have) {
                    next = next_item(p, cur, range_end, left);
                    have = fetch_tile(p, cur, s_tile[b ^ 1], s_desc[b ^ 1]);
                    ready = have && deps_ready(p, s_tile[b ^ 1]);
                }
                have = have && ab != g_epoch;
            }
        }
        if (!go) break;
    }
    if (tid == 0) {
        const bool last = leave(p, !RESIDENT && p.trig_set_slot < 0);
        if (RESIDENT && last && p.host_completed && ld_relaxed_u32(&p.ctl->fail_epoch) != g_epoch) {
            // the host learns of a successful execution from the block that ended it, not a poll later from block 0
            // (a failed one is reported by block 0, verdict first)
            asm volatile("st.relaxed.sys.global.u64 [%0], %1;" ::"l"(p.host_t_done), "l"(globaltimer_ns()) : "memory");
            asm volatile("st.release.sys.global.u64 [%0], %1;" ::"l"(p.host_completed), "l"((unsigned long long)(g_epoch - p.first_epoch + 1u)) : "memory");
        }
    }
}

}  // namespace hccl
