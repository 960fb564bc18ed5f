// Persistent executor kernel for sm_100a and the host calls that bind and launch it.
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

// The file can be compiled whole (HCCL_PART undefined or 0) or in four slices that are linked together, so
// that the build compiles its kernels in parallel: 1 = hccl_executor_lsu, 2 = hccl_executor_lsu_light,
// 3 = hccl_executor_bulk, 4 = the resident and device-resident kernels and all host code.
#ifndef HCCL_PART
#define HCCL_PART 0
#endif
#define HCCL_IN_PART(n) (HCCL_PART == 0 || HCCL_PART == (n))

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
    uint32_t R, nblocks, n_signals, pad0;
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
        for (uint32_t i = tid; i < head; i += nth) dst[i] = src[i];
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
template <int DS, int DD>
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
    auto src = [&](int k) -> const char* {
        int r = r0 + k;
        if (r >= R) r -= R;
        return (const char*)(from_send ? p.send[r] : (const void*)p.recv[r]) + soff;
    };
    // same phase for every operand?
    const uint32_t pd = (uint32_t)(((uintptr_t)dst0 / Elem<DD>::BYTES) & 7u);
    bool vec = true;
    for (int k = 0; k < nsrc; ++k) vec = vec && ((uint32_t)(((uintptr_t)src(k) / Elem<DS>::BYTES) & 7u) == pd);
    for (int j = 1; j < nd; ++j) vec = vec && ((uint32_t)(((uintptr_t)dstp(j) / Elem<DD>::BYTES) & 7u) == pd);
    if (!vec) {
        for (uint32_t i = tid; i < n; i += nth) {
            float acc = Elem<DS>::load(src(0), i);
            for (int k = 1; k < nsrc; ++k) acc = acc + Elem<DS>::load(src(k), i);
            for (int j = 0; j < nd; ++j) Elem<DD>::store(dstp(j), i, acc);
        }
        return;
    }
    uint32_t head = (8u - pd) & 7u;
    if (head > n) head = n;
    const uint32_t nv = (n - head) >> 3;
    auto scalar = [&](uint32_t i) {
        float acc = Elem<DS>::load(src(0), i);
        for (int k = 1; k < nsrc; ++k) acc = acc + Elem<DS>::load(src(k), i);
        for (int j = 0; j < nd; ++j) Elem<DD>::store(dstp(j), i, acc);
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
        for (int j = 1; j < nd; ++j) store8<DD, false>(dstp(j) + o, acc);
    }
}

static __device__ void reduce_n_dispatch(const ExecParams& p, const Desc& d, uint64_t start, uint32_t n, uint32_t tid, uint32_t nth) {
#define RN(S, D) reduce_n_tile<S, D>(p, d, start, n, tid, nth)
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
static __device__ void run_tile_lsu(const ExecParams& p, const Desc& d, const Tile& t, const uint32_t tid, const uint32_t nth) {
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
            reduce_n_dispatch(p, d, t.start, t.count, tid, nth);
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
template <class P>
__device__ void leave(const P& p, bool lean = false) {
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
    }
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
__device__ __forceinline__ uint32_t next_item(const ExecParams& p, uint32_t cur, uint32_t range_end) {
    if (p.chain_len) return cur + 1 < range_end ? cur + 1 : p.n_tiles;
    return p.static_tickets ? p.n_tiles : atomicAdd(&p.ctl->ticket, 1);
}

template <bool RESIDENT>
__device__ __forceinline__ void executor_lsu_body(const ExecParams& p) {
    __shared__ Tile s_tile[2];
    __shared__ Desc s_desc[2];
    __shared__ int s_go[2];
    const uint32_t tid = threadIdx.x, nth = blockDim.x;
    constexpr uint32_t FULL = 1, DONE = 3;  // barrier ids FULL+b, DONE+b
    // Entry. The execution number, the abort word, the first ticket and (with static tickets) the first item's
    // tile record do not depend on one another: thread 0 issues all of these loads before it uses any of
    // them, so a small collective pays one trip to memory here instead of four in a row.
    uint32_t next = 0, abort0 = 0, range_end = 0;
    Tile pre;
    bool pre_ok = false;
    const bool gated = p.trig_wait_slot >= 0;
    if (tid == 0) {
        if (!gated) {
            next = first_item(p, range_end);
            if (next < p.n_tiles) {
                pre = p.tiles[next];
                pre_ok = true;
            }
        }
        abort0 = *(volatile uint32_t*)&p.ctl->abort;
        g_epoch = *(volatile uint32_t*)&p.ctl->done_epoch + 1u;
    }
    __syncthreads();
    if (tid >= 32) {
        const uint32_t wtid = tid - 32, nwork = nth - 32;
        for (uint32_t k = 0;; ++k) {
            const uint32_t b = k & 1;
            named_sync(FULL + b, nth);
            if (!s_go[b]) break;
            run_tile_lsu(p, s_desc[b], s_tile[b], wtid, nwork);
            named_sync(DONE + b, nth);
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
                    next = next_item(p, cur, range_end);
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
            bool go = have && !aborted(p);
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
                have = cur < p.n_tiles && !aborted(p);
                if (have) {
                    next = next_item(p, cur, range_end);
                    have = fetch_tile(p, cur, s_tile[b ^ 1], s_desc[b ^ 1]);
                    ready = have && deps_ready(p, s_tile[b ^ 1]);
                }
            }
        }
        if (!go) break;
    }
    if (tid == 0) leave(p, !RESIDENT && p.trig_set_slot < 0);
}

#if HCCL_IN_PART(1)
__global__ void __launch_bounds__(512, 1) hccl_executor_lsu(const __grid_constant__ ExecParams p) { executor_lsu_body<false>(p); }
#else
__global__ void __launch_bounds__(512, 1) hccl_executor_lsu(const __grid_constant__ ExecParams p);
#endif
// Same program compiled to at most 64 registers per thread: two 512-thread blocks (or four of 256) fit one
// SM, and a block of 256 threads leaves three quarters of the register file to whatever else runs there.
#if HCCL_IN_PART(2)
__global__ void __launch_bounds__(512, 2) hccl_executor_lsu_light(const __grid_constant__ ExecParams p) { executor_lsu_body<false>(p); }
#else
__global__ void __launch_bounds__(512, 2) hccl_executor_lsu_light(const __grid_constant__ ExecParams p);
#endif

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

constexpr uint32_t MAX_STAGES = 4;            // 4 x 48 KiB + bookkeeping fits the 227 KB a block may have
constexpr uint32_t STAGE_BYTES = 49152;       // a COPY piece fills a stage; a REDUCE piece splits it into A and B
// Elements per REDUCE piece: as many as fit a stage with both operands, in whole multiples of 512 elements
// (6144 for fp32+fp32, 8192 for fp32+16-bit, 12288 for 16-bit+16-bit).
__host__ __device__ constexpr uint32_t piece_elems(uint32_t ea, uint32_t eb) { return STAGE_BYTES / (ea + eb) / 512 * 512; }

// PIECE_COPY: loaded and stored by the bulk unit. PIECE_COPYW: loaded by the bulk unit, stored by the compute
// warps from shared memory (the stage is free as soon as the warps have read it, without waiting for a
// bulk store to drain, so more of the stage ring is loads in flight).
enum : uint32_t { PIECE_COPY = 0, PIECE_REDUCE = 1, PIECE_TILE = 2, PIECE_EXIT = 3, PIECE_COPYW = 4 };

struct alignas(16) PieceInfo {  // one per stage, in shared memory; written by the DMA thread
    uint32_t kind;
    uint32_t n;           // REDUCE: elements; COPY: bytes
    uint32_t last;        // last piece of its work item: publish the item's completion after it
    uint32_t tile_index;
    char* dst;            // global destination of this piece
    unsigned long long group;  // COPY: sequence number of the bulk store group that drains this stage
    int32_t signal[2];
    uint8_t dt_a, dt_b, dt_d, evict_first;
    uint32_t b_off;       // REDUCE: byte offset of operand B inside the stage
    uint16_t ndst, rank_dst;   // COPY with several destinations: receive buffers of ranks rank_dst .. +ndst-1 (mod R)
    unsigned long long dst_off;  // ... at this byte offset (dst is then the first of them)
    Tile tile;            // PIECE_TILE: the work item and its descriptor for the register path
    Desc desc;
};

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
template <int DT>
__device__ __forceinline__ void stg4(char* p, const float (&f)[4]) {
    if constexpr (DT == HCCL_FP32) {
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
template <int DA, int DB, int DD>
__device__ __forceinline__ void reduce_piece(const char* sa, const char* sb, char* gdst, uint32_t n, uint32_t ctid, uint32_t cnth) {
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
            stg4<DD>(gdst + (size_t)(u + k * cnth) * 4 * Elem<DD>::BYTES, a[k]);
        }
    }
    for (; u < units; u += cnth) {
        float a[4], b[4];
        lds4<DA>(sa + (size_t)u * 4 * Elem<DA>::BYTES, a);
        lds4<DB>(sb + (size_t)u * 4 * Elem<DB>::BYTES, b);
#pragma unroll
        for (int e = 0; e < 4; ++e) a[e] = a[e] + b[e];
        stg4<DD>(gdst + (size_t)u * 4 * Elem<DD>::BYTES, a);
    }
}
static __device__ void reduce_piece_dispatch(int da, int db, int dd, const char* sa, const char* sb, char* g, uint32_t n, uint32_t ctid, uint32_t cnth) {
#define RP(A, B, D) reduce_piece<A, B, D>(sa, sb, g, n, ctid, cnth)
#define RP_D(A, B) do { if (dd == HCCL_FP32) RP(A, B, HCCL_FP32); else if (dd == HCCL_BF16) RP(A, B, HCCL_BF16); else RP(A, B, HCCL_FP16); } while (0)
#define RP_B(A) do { if (db == HCCL_FP32) RP_D(A, HCCL_FP32); else if (db == HCCL_BF16) RP_D(A, HCCL_BF16); else RP_D(A, HCCL_FP16); } while (0)
    if (da == HCCL_FP32) RP_B(HCCL_FP32); else if (da == HCCL_BF16) RP_B(HCCL_BF16); else RP_B(HCCL_FP16);
#undef RP_B
#undef RP_D
#undef RP
}

// State of the DMA thread.
struct Dma {
    uint32_t ns, lag;
    uint32_t stages, full, empty;  // shared-memory addresses
    char* stages_ptr;
    PieceInfo* info;
    unsigned long long head, tail, groups;
    unsigned long long pol;
    bool ok;
    bool copy_by_warps;
};

// Retire the oldest outstanding piece. A COPY piece is drained to global memory here; REDUCE and TILE
// pieces are finished by the compute warps on their own.
static __device__ void retire_one(const ExecParams& p, Dma& d) {
    const unsigned long long j = d.tail;
    const uint32_t slot = (uint32_t)(j % d.ns), parity = (uint32_t)((j / d.ns) & 1);
    PieceInfo& pi = d.info[slot];
    if (pi.kind == PIECE_COPY) {
        if (!mbar_wait(p, d.full + 8 * slot, parity, p.timeout_ns, pi.tile_index)) d.ok = false;
        if (d.ok) {
            if (pi.ndst > 1) {  // one stage, several stores, one group
                for (uint32_t k = 0; k < pi.ndst; ++k) {
                    uint32_t r = pi.rank_dst + k;
                    if (r >= p.R) r -= p.R;
                    bulk_store_part((char*)p.recv[r] + pi.dst_off, d.stages + slot * STAGE_BYTES, pi.n, pi.evict_first != 0, d.pol);
                }
                bulk_commit();
            } else {
                bulk_store(pi.dst, d.stages + slot * STAGE_BYTES, pi.n, pi.evict_first != 0, d.pol);
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
    const uint32_t slot = (uint32_t)(j % d.ns), parity = (uint32_t)((j / d.ns) & 1);
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

static __device__ bool wait_counter_draining(const ExecParams& p, Dma& d, uint32_t sync, uint32_t per_epoch, uint32_t tile) {
    const uint32_t target = g_epoch * per_epoch;
    if ((int32_t)(ld_acquire_u32(p.counters + sync) - target) >= 0) return true;
    drain(p, d);  // the item waited for may sit in this block's own pipeline
    if (!d.ok) return false;
    return wait_counter(p, sync, per_epoch, tile);
}

static __device__ void issue_simple(const ExecParams& p, Dma& d, uint32_t kind, uint32_t cur, const Tile* t, const Desc* ds) {
    const unsigned long long k = d.head;
    if (!acquire_slot(p, d, k, cur)) return;
    const uint32_t slot = (uint32_t)(k % d.ns);
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
    d.head = k + 1;
}

// One work item through the DMA thread. Returns false when the block must stop.
static __device__ bool dma_item(const ExecParams& p, Dma& d, uint32_t cur, const Tile* preloaded = nullptr) {
    if (p.trace) {
        trace_put(p.trace, p.trace_cap, cur, 0, (unsigned long long)cur | ((unsigned long long)blockIdx.x << 32));
        trace_put(p.trace, p.trace_cap, cur, 1, globaltimer_ns());
    }
    const Tile t = preloaded ? *preloaded : p.tiles[cur];
    if (!tile_ok(p, t)) {
        fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
        return false;
    }
    const Desc ds = p.descs[t.desc];
    if (!desc_ok(p, ds)) {
        fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
        return false;
    }
    bool waited = false;
    for (uint32_t w = 0; w < t.wait_cnt; ++w) {
        const Wait x = p.waits[t.wait_off + w];
        if (x.sync >= p.n_syncs) {
            fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
            return false;
        }
        if (!wait_counter_draining(p, d, x.sync, x.per_epoch, cur)) return false;
        waited = true;
    }
    if (waited) fence_proxy_async();  // what the acquired counters cover must be visible to the bulk unit too
    if (p.trace) trace_put(p.trace, p.trace_cap, cur, 2, globaltimer_ns());
    switch (ds.op) {
        case HCCL_OP_WAIT: {
            drain(p, d);
            if (!d.ok) return false;
            const unsigned long long* addr = (ds.kind_a == HCCL_BUF_SIGNAL ? p.signals : p.user_signals) + ds.off_a;
            if (!wait_signal(p, addr, ds.cmp, ds.value + (unsigned long long)g_epoch * ds.value_per_epoch, cur)) return false;
            publish_tile(p, t);
            return true;
        }
        case HCCL_OP_SET: {
            unsigned long long* addr = (ds.kind_dst == HCCL_BUF_SIGNAL ? p.signals : p.user_signals) + ds.off_dst;
            __threadfence();
            st_release_u64(addr, ds.value + (unsigned long long)g_epoch * ds.value_per_epoch);
            publish_tile(p, t);
            return true;
        }
        case HCCL_OP_NOOP:
            publish_tile(p, t);
            return true;
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
            for (uint32_t off = 0; off < body && d.ok; off += STAGE_BYTES) {
                const uint32_t nb = min(STAGE_BYTES, body - off);
                const unsigned long long k = d.head;
                if (!acquire_slot(p, d, k, cur)) return false;
                const uint32_t slot = (uint32_t)(k % d.ns);
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
                bulk_load(d.stages + slot * STAGE_BYTES, src + off, nb, d.full + 8 * slot, stream, d.pol);
                d.head = k + 1;
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
            const uint32_t pe = piece_elems(ea, eb);
            for (uint32_t e0 = 0; e0 < t.count && d.ok; e0 += pe) {
                const uint32_t ne = min(pe, t.count - e0);
                const unsigned long long k = d.head;
                if (!acquire_slot(p, d, k, cur)) return false;
                const uint32_t slot = (uint32_t)(k % d.ns);
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
                mbar_arrive_expect_tx(d.full + 8 * slot, ne * (ea + eb));
                bulk_load(d.stages + slot * STAGE_BYTES, a + (size_t)e0 * ea, ne * ea, d.full + 8 * slot, ds.kind_a == HCCL_BUF_SEND, d.pol);
                bulk_load(d.stages + slot * STAGE_BYTES + pe * ea, b + (size_t)e0 * eb, ne * eb, d.full + 8 * slot, ds.kind_b == HCCL_BUF_SEND, d.pol);
                d.head = k + 1;
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

#if !HCCL_IN_PART(3)
__global__ void __launch_bounds__(512, 1) hccl_executor_bulk(const __grid_constant__ ExecParams p, const uint32_t ns, const uint32_t copy_by_warps);
#else
__global__ void __launch_bounds__(512, 1) hccl_executor_bulk(const __grid_constant__ ExecParams p, const uint32_t ns, const uint32_t copy_by_warps) {
    using namespace bulk;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    char* stages_ptr = reinterpret_cast<char*>(smem_raw);
    PieceInfo* info = reinterpret_cast<PieceInfo*>(stages_ptr + (size_t)ns * STAGE_BYTES);
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(info + ns);  // full[ns], empty[ns]
    const uint32_t tid = threadIdx.x;
    const uint32_t ncw = (blockDim.x >> 5) - 1;  // compute warps
    const uint32_t full = smem_u32(bars), empty = smem_u32(bars + ns);
    // entry: first ticket, its tile record, the abort word and the execution number are loaded together
    uint32_t next0 = 0, abort0 = 0;
    Tile pre;
    bool pre_ok = false;
    const bool gated = p.trig_wait_slot >= 0;
    if (tid == 0) {
        if (!gated) {
            next0 = p.static_tickets ? blockIdx.x : atomicAdd(&p.ctl->ticket, 1);
            if (next0 < p.n_tiles) {
                pre = p.tiles[next0];
                pre_ok = true;
            }
        }
        abort0 = *(volatile uint32_t*)&p.ctl->abort;
        g_epoch = *(volatile uint32_t*)&p.ctl->done_epoch + 1u;
    }
    if (tid == 0) {
        for (uint32_t s = 0; s < ns; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(empty + 8 * s, ncw);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();

    if (tid < 32) {
        if (tid != 0) return;  // one elected thread drives the DMA warp
        Dma d;
        d.ns = ns;
        d.lag = copy_by_warps ? ns : (ns > 2 ? ns - 2 : 1);
        d.copy_by_warps = copy_by_warps != 0;
        d.stages = smem_u32(stages_ptr);
        d.stages_ptr = stages_ptr;
        d.full = full;
        d.empty = empty;
        d.info = info;
        d.head = d.tail = d.groups = 0;
        d.pol = policy_evict_first();
        d.ok = true;
        bool live = true;
        uint32_t next = next0;
        if (gated) {
            live = wait_signal(p, p.user_signals + p.trig_wait_slot, p.trig_cmp, p.trig_wait_value + (unsigned long long)g_epoch * p.trig_wait_per_epoch, 0xffffffffu);
            next = p.static_tickets ? blockIdx.x : atomicAdd(&p.ctl->ticket, 1);
        }
        if (next == 0) p.ctl->t_first_ns = globaltimer_ns();
        bool first = true;
        while (live && d.ok) {
            const uint32_t cur = next;
            if (cur >= p.n_tiles || (first && !gated ? abort0 == g_epoch : aborted(p))) break;
            next = p.static_tickets ? p.n_tiles : atomicAdd(&p.ctl->ticket, 1);
            if (!dma_item(p, d, cur, first && pre_ok ? &pre : nullptr)) break;
            first = false;
        }
        // wind down: finish what is in flight, release the compute warps, leave
        if (d.ok && !aborted(p)) drain(p, d);
        if (d.ok && !aborted(p)) {
            const unsigned long long kx = d.head;
            issue_simple(p, d, PIECE_EXIT, 0xffffffffu, nullptr, nullptr);
            // every compute warp has passed the exit piece = all of this block's results are stored
            if (d.ok && d.head == kx + 1)
                mbar_wait(p, empty + 8 * (uint32_t)(kx % ns), (uint32_t)((kx / ns) & 1), 2 * p.timeout_ns + 1000000000ull, 0xfffffffcu);
        }
        if (!d.ok || aborted(p)) {
            // stop path: no load may still be writing into this block's shared memory when it exits
            for (unsigned long long j = d.tail; j < d.head; ++j) {
                const uint32_t slot = (uint32_t)(j % ns);
                if (info[slot].kind == PIECE_COPY || info[slot].kind == PIECE_REDUCE || info[slot].kind == PIECE_COPYW)
                    mbar_wait(p, full + 8 * slot, (uint32_t)((j / ns) & 1), 1000000000ull, 0xfffffffeu);
            }
        }
        bulk_wait_all();
        // the compute warps must be out of the stages before the block's verdict is given
        leave(p, p.trig_set_slot < 0);
        return;
    }

    // ------------------------------------------------------------ compute warps
    const uint32_t ctid = tid - 32, cnth = ncw * 32;
    for (unsigned long long k = 0;; ++k) {
        const uint32_t slot = (uint32_t)(k % ns), parity = (uint32_t)((k / ns) & 1);
        if (!mbar_wait(p, full + 8 * slot, parity, 2 * p.timeout_ns + 1000000000ull, 0xfffffffdu)) break;
        const PieceInfo& pi = info[slot];
        const uint32_t kind = pi.kind;
        if (kind == PIECE_EXIT) {
            __syncwarp();
            if ((tid & 31u) == 0) mbar_arrive(empty + 8 * slot);  // tells the DMA thread this warp has stored everything
            break;
        }
        if (kind == PIECE_REDUCE) {
            reduce_piece_dispatch(pi.dt_a, pi.dt_b, pi.dt_d, stages_ptr + (size_t)slot * STAGE_BYTES,
                                  stages_ptr + (size_t)slot * STAGE_BYTES + pi.b_off, pi.dst, pi.n, ctid, cnth);
        } else if (kind == PIECE_COPYW) {
            const uint4* src = reinterpret_cast<const uint4*>(stages_ptr + (size_t)slot * STAGE_BYTES);
            uint4* dst = reinterpret_cast<uint4*>(pi.dst);
            const uint32_t nv = pi.n >> 4;
            const bool stream = pi.evict_first != 0;
            if (pi.ndst > 1) {
                const uint32_t nd = pi.ndst, r0 = pi.rank_dst;
                const unsigned long long doff = pi.dst_off;
                constexpr int U = 4;
                uint32_t i = ctid;
                for (; i + (U - 1) * cnth < nv; i += U * cnth) {
                    uint4 v[U];
#pragma unroll
                    for (int u = 0; u < U; ++u) v[u] = src[i + u * cnth];
                    for (uint32_t k = 0; k < nd; ++k) {
                        uint32_t r = r0 + k;
                        if (r >= p.R) r -= p.R;
                        uint4* dk = reinterpret_cast<uint4*>((char*)p.recv[r] + doff) + i;
#pragma unroll
                        for (int u = 0; u < U; ++u) __stcs(dk + u * cnth, v[u]);
                    }
                }
                for (; i < nv; i += cnth) {
                    const uint4 v = src[i];
                    for (uint32_t k = 0; k < nd; ++k) {
                        uint32_t r = r0 + k;
                        if (r >= p.R) r -= p.R;
                        __stcs(reinterpret_cast<uint4*>((char*)p.recv[r] + doff) + i, v);
                    }
                }
            } else
            for (uint32_t i = ctid; i < nv; i += cnth) {
                if (stream) __stcs(dst + i, src[i]); else __stcg(dst + i, src[i]);
            }
        } else if (kind == PIECE_TILE) {
            run_tile_lsu(p, pi.desc, pi.tile, ctid, cnth);
        }
        if (kind != PIECE_COPY && pi.last && p.trace && ctid == 0) trace_put(p.trace, p.trace_cap, pi.tile_index, 3, globaltimer_ns());
        if (kind != PIECE_COPY && pi.last && (pi.signal[0] >= 0 || pi.signal[1] >= 0)) {
            asm volatile("bar.sync 1, %0;" ::"r"(cnth) : "memory");  // every compute warp has stored its share
            if (ctid == 0) {  // release, cumulative over the stores the barrier ordered before this thread
                if (pi.signal[0] >= 0) red_release_add_u32(p.counters + pi.signal[0], 1);
                if (pi.signal[1] >= 0) red_release_add_u32(p.counters + pi.signal[1], 1);
            }
            asm volatile("bar.sync 1, %0;" ::"r"(cnth) : "memory");  // the stage's info is read before it is recycled
        }
        __syncwarp();
        if ((tid & 31u) == 0) mbar_arrive(empty + 8 * slot);
    }
}
#endif  // part 3

#if HCCL_IN_PART(4)
// ====================================================================== resident, doorbell-fed executor
// The register engine as a long-lived kernel (paper Sec. II-A.3 "express doorbells": the work request's
// write is the doorbell; Sec. V-B: re-enqueueing a cached work packet costs microseconds). The blocks stay
// resident and execute the bound plan once per doorbell ring. The doorbell is a 64-byte record in pinned,
// mapped HOST memory: the host rings by storing a larger request number, block 0 polls it, releases all
// blocks through a device-side word, and reports completion (and a failure verdict) back into the record.
// Every wait is bounded: the kernel leaves by itself after idle_ns without a ring, or when told to stop.
struct Doorbell {                       // layout shared with hccl_doorbell_t in hccl.h
    unsigned long long request;         // host -> device: number of executions asked for so far
    unsigned long long completed;       // device -> host: executions finished
    unsigned long long stop;            // host -> device: leave after the current execution
    unsigned long long exited;          // device -> host: the kernel has left (1 = stop, 2 = idle, 3 = failure)
    unsigned long long status, detail;  // device -> host: verdict of the last failed execution
    unsigned long long pad[2];
};

__device__ __forceinline__ unsigned long long ld_sys_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.relaxed.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_sys_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}

__global__ void __launch_bounds__(512, 1) hccl_executor_resident(const __grid_constant__ ExecParams p, Doorbell* db,
                                                                  const unsigned long long idle_ns, const uint32_t first_epoch) {
    __shared__ uint32_t s_cmd;          // epoch to run, or 0 to leave
    uint32_t epoch = first_epoch;       // the next execution's number
    for (;;) {
        if (threadIdx.x == 0) {
            uint32_t cmd = 0;
            if (blockIdx.x == 0) {
                // the previous execution must have been left by every block before anything else happens
                bool ok = true;
                if (epoch != first_epoch) {
                    const unsigned long long deadline = globaltimer_ns() + 2 * p.timeout_ns + 1000000000ull;
                    while (ld_acquire_u32(&p.ctl->done_epoch) != epoch - 1) {
                        if (globaltimer_ns() > deadline) { ok = false; break; }
                        __nanosleep(50);
                    }
                    if (ok) {
                        if (ld_acquire_u32(&p.ctl->fail_epoch) == epoch - 1) {
                            st_sys_u64(&db->status, p.ctl->status);
                            st_sys_u64(&db->detail, p.ctl->detail);
                            ok = false;  // a failed execution leaves the counters inconsistent: stop serving
                        }
                        st_sys_u64(&db->completed, (unsigned long long)(epoch - first_epoch));
                    }
                }
                unsigned long long why = ok ? 0 : 3;
                if (ok) {
                    const unsigned long long deadline = globaltimer_ns() + idle_ns;
                    for (;;) {
                        if (ld_sys_u64(&db->request) > (unsigned long long)(epoch - first_epoch)) { cmd = epoch; break; }
                        if (ld_sys_u64(&db->stop) != 0) { why = 1; break; }
                        if (globaltimer_ns() > deadline) { why = 2; break; }
                        __nanosleep(100);
                    }
                }
                if (cmd == 0) st_sys_u64(&db->exited, why);
                // release the other blocks: server_go carries the epoch to run, or all ones to leave
                asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(&p.ctl->server_go), "r"(cmd ? cmd : 0xffffffffu) : "memory");
            } else {
                const unsigned long long deadline = globaltimer_ns() + idle_ns + 4 * p.timeout_ns + 4000000000ull;
                for (;;) {
                    const uint32_t go = ld_acquire_u32(&p.ctl->server_go);
                    if (go == epoch) { cmd = epoch; break; }
                    if (go == 0xffffffffu || globaltimer_ns() > deadline) break;
                    __nanosleep(50);
                }
            }
            s_cmd = cmd;
        }
        __syncthreads();
        if (s_cmd == 0) break;
        executor_lsu_body<true>(p);     // one execution: tickets, dependencies, data, completion stamp
        __syncthreads();
        ++epoch;
    }
}

// ====================================================================== device-resident AllToAllv
// "AllToAllvDynamic" (paper Sec. IV-B.2): the per-peer row counts are produced on the device (by a routing
// kernel) after the collective has been compiled and possibly already enqueued. The kernel reads the R x R
// count matrix from device memory, derives packed send and receive displacements with warp-level prefix
// sums, cuts every (source, destination) segment into equal-byte tiles, and moves them. Nothing about the
// sizes goes through the host. Every count is validated against the capacities fixed at plan time before a
// single byte is written.
constexpr int DYN_MAX_RANKS = 64;

struct DynParams {
    const long long* counts;       // device, [R*R], counts[s*R+d] rows from s to d
    long long* recvcounts_out;     // device, [R*R] indexed [d*R+s], or null
    long long* rdispls_out;        // device, [R*R] indexed [d*R+s], or null
    Control* ctl;
    unsigned long long* user_signals;
    uint32_t R, nblocks;
    unsigned long long timeout_ns;
    unsigned long long row_bytes, tile_bytes;
    long long trig_wait_slot, trig_set_slot;
    int trig_cmp, pad1;
    unsigned long long trig_wait_value, trig_wait_per_epoch, trig_set_value, trig_set_per_epoch;
    long long max_send_rows[DYN_MAX_RANKS], max_recv_rows[DYN_MAX_RANKS];
    const void* send[DYN_MAX_RANKS];
    void* recv[DYN_MAX_RANKS];
};

__device__ __forceinline__ long long warp_inclusive_scan(long long v, uint32_t lane) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const long long u = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= (uint32_t)o) v += u;
    }
    return v;
}

__global__ void __launch_bounds__(512, 1) hccl_a2a_dynamic(const __grid_constant__ DynParams q) {
    extern __shared__ __align__(16) unsigned char dsm[];
    const uint32_t R = q.R, RR = R * R;
    long long* s_cnt = reinterpret_cast<long long*>(dsm);  // [RR] rows of segment (s,d)
    long long* s_sd = s_cnt + RR;                          // [RR] first row of the segment in X_s
    long long* s_rd = s_sd + RR;                           // [RR] first row of the segment in Y_d
    uint32_t* s_tp = reinterpret_cast<uint32_t*>(s_rd + RR);  // [RR+1] exclusive prefix of tiles per segment
    __shared__ int s_bad;
    __shared__ unsigned long long s_bad_at;
    __shared__ uint32_t s_team_ticket[2];
    __shared__ int s_live;
    const uint32_t tid = threadIdx.x, nth = blockDim.x, lane = tid & 31u, warp = tid >> 5, nwarps = nth >> 5;
    init_epoch(q);
    if (tid == 0) {
        s_bad = 0;
        s_bad_at = 0;
        bool live = true;
        if (q.trig_wait_slot >= 0)
            live = wait_signal(q, q.user_signals + q.trig_wait_slot, q.trig_cmp, q.trig_wait_value + (unsigned long long)g_epoch * q.trig_wait_per_epoch, 0xffffffffu);
        s_live = live ? 1 : 0;
    }
    __syncthreads();
    if (s_live) {
        // ---- metadata from device memory (written by the producer before it released us)
        for (uint32_t i = tid; i < RR; i += nth) {
            const long long c = __ldcg(q.counts + i);
            s_cnt[i] = c;
            if (c < 0 || c > (1ll << 40)) {
                s_bad = 1;
                s_bad_at = i;
            }
        }
        __syncthreads();
        if (!s_bad) {
            // send displacements: exclusive scan of each source's row of counts; one warp per source
            for (uint32_t s = warp; s < R; s += nwarps) {
                long long carry = 0;
                for (uint32_t base = 0; base < R; base += 32) {
                    const uint32_t d = base + lane;
                    const long long v = d < R ? s_cnt[s * R + d] : 0;
                    const long long inc = warp_inclusive_scan(v, lane);
                    if (d < R) s_sd[s * R + d] = carry + inc - v;
                    carry += __shfl_sync(0xffffffffu, inc, 31);
                }
                if (lane == 0 && carry > q.max_send_rows[s]) {
                    s_bad = 1;
                    s_bad_at = (unsigned long long)s * R;
                }
            }
            // receive displacements: exclusive scan down each destination's column; one warp per destination
            for (uint32_t d = warp; d < R; d += nwarps) {
                long long carry = 0;
                for (uint32_t base = 0; base < R; base += 32) {
                    const uint32_t s = base + lane;
                    const long long v = s < R ? s_cnt[s * R + d] : 0;
                    const long long inc = warp_inclusive_scan(v, lane);
                    if (s < R) s_rd[s * R + d] = carry + inc - v;
                    carry += __shfl_sync(0xffffffffu, inc, 31);
                }
                if (lane == 0 && carry > q.max_recv_rows[d]) {
                    s_bad = 1;
                    s_bad_at = d;
                }
            }
            // tiles per segment and their exclusive prefix over (s,d) in row-major order; warp 0
            if (warp == 0) {
                long long carry = 0;
                for (uint32_t base = 0; base < RR; base += 32) {
                    const uint32_t i = base + lane;
                    const long long bytes = i < RR ? s_cnt[i] * (long long)q.row_bytes : 0;
                    const long long v = (bytes + (long long)q.tile_bytes - 1) / (long long)q.tile_bytes;
                    const long long inc = warp_inclusive_scan(v, lane);
                    if (i < RR) s_tp[i] = (uint32_t)(carry + inc - v);
                    carry += __shfl_sync(0xffffffffu, inc, 31);
                }
                if (lane == 0) {
                    s_tp[RR] = (uint32_t)carry;
                    if (carry > 0x7fffffffll) {
                        s_bad = 1;
                        s_bad_at = RR;
                    }
                }
            }
        }
        __syncthreads();
        if (s_bad) {
            if (tid == 0) fail(q, HCCL_ERR_BAD_DESCRIPTOR, s_bad_at);
        } else {
            // what each receiver gets and where, for the kernels that consume the result
            if (blockIdx.x == 0) {
                for (uint32_t i = tid; i < RR; i += nth) {
                    const uint32_t s = i / R, d = i % R;
                    if (q.recvcounts_out) q.recvcounts_out[d * R + s] = s_cnt[i];
                    if (q.rdispls_out) q.rdispls_out[d * R + s] = s_rd[i];
                }
            }
            const uint32_t total = s_tp[RR];
            // The block works as teams of 256 threads, each claiming and copying tiles on its own (named
            // barrier per team), so that one team's gap between two tiles is covered by the other's copy.
            const uint32_t team_size = nth >= 512 ? 256u : nth, n_teams = nth / team_size;
            const uint32_t team = tid / team_size, ltid = tid - team * team_size;
            if (team < n_teams) {
                uint32_t next = 0;
                if (ltid == 0) next = atomicAdd(&q.ctl->ticket, 1);
                for (;;) {
                    if (ltid == 0) {
                        s_team_ticket[team] = next;
                        if (next < total) next = atomicAdd(&q.ctl->ticket, 1);  // one ahead
                    }
                    named_sync(1 + team, team_size);
                    const uint32_t t = s_team_ticket[team];
                    if (t >= total) break;
                    // segment of tile t: the last i with s_tp[i] <= t (zero-length segments share a prefix value
                    // with their successor and are skipped by taking the last one)
                    uint32_t lo = 0, hi = RR;
                    while (hi - lo > 1) {
                        const uint32_t mid = (lo + hi) >> 1;
                        if (s_tp[mid] <= t) lo = mid; else hi = mid;
                    }
                    const uint32_t i = lo, s = i / R, d = i % R;
                    const unsigned long long off = (unsigned long long)(t - s_tp[i]) * q.tile_bytes;
                    const unsigned long long seg = (unsigned long long)s_cnt[i] * q.row_bytes;
                    const uint32_t len = (uint32_t)min((unsigned long long)q.tile_bytes, seg - off);
                    const char* src = (const char*)q.send[s] + (unsigned long long)s_sd[i] * q.row_bytes + off;
                    char* dst = (char*)q.recv[d] + (unsigned long long)s_rd[i] * q.row_bytes + off;
                    copy_tile_lsu<true>(dst, src, len, ltid, team_size);
                    named_sync(1 + team, team_size);  // the ticket word is rewritten only after everyone has read it
                }
            }
        }
    }
    __syncthreads();
    if (tid == 0) leave(q);
}

#endif  // part 4: kernels
}  // namespace hccl

#if HCCL_IN_PART(4)
// ====================================================================== host side
using namespace hccl;

namespace {
thread_local char g_cuda_err[256] = "";
hccl_status_t cuda_fail(cudaError_t e, const char* what) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return HCCL_ERR_CUDA;
}
#define CUDA_TRY(x)                                   \
    do {                                              \
        cudaError_t _e = (x);                         \
        if (_e != cudaSuccess) return cuda_fail(_e, #x); \
    } while (0)
}  // namespace

extern "C" {

const char* hccl_last_cuda_error(void) { return g_cuda_err; }

hccl_status_t hccl_plan_bind(hccl_plan_t* p, void* dev_workspace, size_t bytes, void* stream) {
    if (!p || !dev_workspace) return HCCL_ERR_INVALID_ARG;
    if (((uintptr_t)dev_workspace) % 256) return HCCL_ERR_ALIGNMENT;
    if (bytes < p->layout.total) return HCCL_ERR_WORKSPACE;
    const Layout& L = p->layout;
    std::vector<char> img((size_t)L.scratch, 0);  // control, counters and signals start at zero
    if (!p->descs.empty()) std::memcpy(img.data() + L.descs, p->descs.data(), p->descs.size() * sizeof(Desc));
    if (!p->tiles.empty()) std::memcpy(img.data() + L.tiles, p->tiles.data(), p->tiles.size() * sizeof(Tile));
    if (!p->waits.empty()) std::memcpy(img.data() + L.waits, p->waits.data(), p->waits.size() * sizeof(Wait));
    cudaStream_t s = (cudaStream_t)stream;
    CUDA_TRY(cudaMemcpyAsync(dev_workspace, img.data(), img.size(), cudaMemcpyHostToDevice, s));
    CUDA_TRY(cudaStreamSynchronize(s));
    // opt-in shared memory sizes are set here, once, so that hccl_execute itself is only a launch
    if (p->dynamic) {
        const size_t RR = (size_t)p->R * p->R;
        const size_t smem = RR * 24 + (RR + 1) * 4 + 16;
        if (smem > 48 * 1024) CUDA_TRY(cudaFuncSetAttribute(hccl_a2a_dynamic, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(DYN_MAX_RANKS * DYN_MAX_RANKS * 24 + (DYN_MAX_RANKS * DYN_MAX_RANKS + 1) * 4 + 16)));
    } else if (p->opts.engine == HCCL_ENGINE_BULK) {
        const size_t smem = (size_t)bulk::MAX_STAGES * (bulk::STAGE_BYTES + sizeof(bulk::PieceInfo) + 16) + 128;
        if (smem <= 227 * 1024) CUDA_TRY(cudaFuncSetAttribute(hccl_executor_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)std::min<size_t>(smem, 227 * 1024)));
    }
    p->workspace = dev_workspace;
    p->workspace_bytes = bytes;
    p->epoch = 0;
    p->checked_send.clear();
    p->checked_recv.clear();
    return HCCL_OK;
}

// How the blocks find their work: tickets, one item per block, or static chains.
static int set_dispatch(const hccl_plan_t* p, ExecParams& prm) {
    int blocks = p->opts.sm_budget;
    if ((uint32_t)blocks > prm.n_tiles) blocks = (int)std::max<uint32_t>(prm.n_tiles, 1u);
    prm.chain_len = p->chain_len;
    prm.n_chains = p->n_chains;
    if (p->chain_len) blocks = (int)std::max<uint32_t>(1u, std::min<uint32_t>((uint32_t)blocks, p->n_chains));
    prm.nblocks = (uint32_t)blocks;
    prm.static_tickets = (!p->chain_len && prm.n_waits == 0 && prm.n_tiles <= (uint32_t)blocks) ? 1 : 0;
    return blocks;
}

// Kernel parameters of a bound plan: table addresses inside its workspace, sizes, trigger, rank buffers, and
// how the blocks find their work. Returns the number of blocks to launch.
static int fill_params(const hccl_plan_t* p, ExecParams& prm, const void* const* sendbufs, void* const* recvbufs) {
    char* ws = (char*)p->workspace;
    const Layout& L = p->layout;
    prm.descs = (const Desc*)(ws + L.descs);
    prm.tiles = (const Tile*)(ws + L.tiles);
    prm.waits = (const Wait*)(ws + L.waits);
    prm.counters = (uint32_t*)(ws + L.counters);
    prm.signals = (unsigned long long*)(ws + L.signals);
    prm.ctl = (Control*)(ws + L.control);
    prm.scratch = ws + L.scratch;
    prm.user_signals = (unsigned long long*)p->user_signals;
    prm.trace = (unsigned long long*)p->trace;
    prm.trace_cap = (unsigned long long)p->trace_cap;
    prm.n_tiles = (uint32_t)p->tiles.size();
    prm.n_descs = (uint32_t)p->descs.size();
    prm.n_syncs = (uint32_t)p->sync_per_epoch.size();
    prm.n_waits = (uint32_t)p->waits.size();
    prm.n_signals = (uint32_t)p->n_signals;
    prm.R = (uint32_t)p->R;
    prm.timeout_ns = p->opts.timeout_ns;
    prm.n_user_signals = p->n_user_signals;
    prm.trig_wait_slot = p->trig_wait_slot;
    prm.trig_set_slot = p->trig_set_slot;
    prm.trig_cmp = p->trig_cmp;
    prm.trig_wait_value = p->trig_wait_value;
    prm.trig_wait_per_epoch = p->trig_wait_per_epoch;
    prm.trig_set_value = p->trig_set_value;
    prm.trig_set_per_epoch = p->trig_set_per_epoch;
    for (int r = 0; r < p->R; ++r) {
        prm.send[r] = sendbufs[r];
        prm.recv[r] = recvbufs[r];
    }
    return set_dispatch(p, prm);
}

static hccl_status_t check_buffers(hccl_plan_t* p, const void* const* sendbufs, void* const* recvbufs) {
    const int R = p->R;
    bool same = (int)p->checked_send.size() == R;
    for (int r = 0; same && r < R; ++r) same = p->checked_send[r] == sendbufs[r] && p->checked_recv[r] == recvbufs[r];
    if (same) return HCCL_OK;
    for (int r = 0; r < R; ++r) {
        if ((p->send_bytes[r] > 0 && !sendbufs[r]) || (p->recv_bytes[r] > 0 && !recvbufs[r])) return HCCL_ERR_INVALID_ARG;
        if (((uintptr_t)sendbufs[r] | (uintptr_t)recvbufs[r]) & (uintptr_t)(p->buf_align - 1)) return HCCL_ERR_ALIGNMENT;
    }
    // out-of-place only: no receive extent may intersect a send extent or another receive extent
    for (int d = 0; d < R; ++d) {
        const uintptr_t lo = (uintptr_t)recvbufs[d], hi = lo + (uintptr_t)p->recv_bytes[d];
        if (lo == hi) continue;
        for (int s = 0; s < R; ++s) {
            const uintptr_t slo = (uintptr_t)sendbufs[s], shi = slo + (uintptr_t)p->send_bytes[s];
            if (slo != shi && lo < shi && slo < hi) return HCCL_ERR_OVERLAP;
            if (s > d) {
                const uintptr_t rlo = (uintptr_t)recvbufs[s], rhi = rlo + (uintptr_t)p->recv_bytes[s];
                if (rlo != rhi && lo < rhi && rlo < hi) return HCCL_ERR_OVERLAP;
            }
        }
    }
    p->checked_send.assign(sendbufs, sendbufs + R);
    p->checked_recv.assign(recvbufs, recvbufs + R);
    return HCCL_OK;
}

hccl_status_t hccl_execute(hccl_plan_t* p, const void* const* sendbufs, void* const* recvbufs, void* stream) {
    if (!p || !sendbufs || !recvbufs) return HCCL_ERR_INVALID_ARG;
    if (!p->workspace) return HCCL_ERR_NOT_BOUND;
    hccl_status_t st = check_buffers(p, sendbufs, recvbufs);
    if (st != HCCL_OK) return st;
    if ((p->trig_wait_slot >= 0 || p->trig_set_slot >= 0) && !p->user_signals) return HCCL_ERR_INVALID_ARG;
    if (p->dynamic) {
        if (!p->dyn_counts) return HCCL_ERR_INVALID_ARG;
        static thread_local DynParams q;
        const uint32_t epoch = p->epoch + 1;
        q.counts = (const long long*)p->dyn_counts;
        q.recvcounts_out = (long long*)p->dyn_recvcounts_out;
        q.rdispls_out = (long long*)p->dyn_rdispls_out;
        q.ctl = (Control*)((char*)p->workspace + p->layout.control);
        q.user_signals = (unsigned long long*)p->user_signals;
        q.R = (uint32_t)p->R;
        q.nblocks = (uint32_t)p->opts.sm_budget;
        q.timeout_ns = p->opts.timeout_ns;
        q.row_bytes = (unsigned long long)p->dyn_row_bytes;
        q.tile_bytes = p->opts.tile_bytes;
        q.trig_wait_slot = p->trig_wait_slot;
        q.trig_set_slot = p->trig_set_slot;
        q.trig_cmp = p->trig_cmp;
        q.trig_wait_value = p->trig_wait_value;
        q.trig_wait_per_epoch = p->trig_wait_per_epoch;
        q.trig_set_value = p->trig_set_value;
        q.trig_set_per_epoch = p->trig_set_per_epoch;
        for (int r = 0; r < p->R; ++r) {
            q.max_send_rows[r] = p->dyn_max_send_rows[r];
            q.max_recv_rows[r] = p->dyn_max_recv_rows[r];
            q.send[r] = sendbufs[r];
            q.recv[r] = recvbufs[r];
        }
        const size_t RR = (size_t)p->R * p->R;
        const size_t smem = RR * 24 + (RR + 1) * 4 + 16;
        hccl_a2a_dynamic<<<p->opts.sm_budget, p->opts.threads, smem, (cudaStream_t)stream>>>(q);
        CUDA_TRY(cudaGetLastError());
        p->epoch = epoch;
        return HCCL_OK;
    }
    static thread_local ExecParams prm;  // 4 KB+: keep it off the stack
    const uint32_t epoch = p->epoch + 1;
    const int blocks = fill_params(p, prm, sendbufs, recvbufs);
    if (p->opts.engine == HCCL_ENGINE_BULK) {
        const uint32_t ns = (uint32_t)std::min<int>(std::max<int>(p->opts.stages > 0 ? p->opts.stages : (int)bulk::MAX_STAGES, 2), (int)bulk::MAX_STAGES);
        const size_t smem = (size_t)ns * (bulk::STAGE_BYTES + sizeof(bulk::PieceInfo) + 16) + 128;
        const int threads = std::max(64, p->opts.threads);
        hccl_executor_bulk<<<blocks, threads, smem, (cudaStream_t)stream>>>(prm, ns, (uint32_t)(p->opts.copy_by_warps == 1 || (p->opts.copy_by_warps == 0 && p->opts.sm_budget < 100)));
    } else {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks);
        cfg.blockDim = dim3((unsigned)p->opts.threads);
        cfg.dynamicSmemBytes = 0;
        cfg.stream = (cudaStream_t)stream;
        cudaLaunchAttribute attr[1];
        int nattr = 0;
        if (p->opts.cluster > 1 && blocks % p->opts.cluster == 0) {
            // blocks of one cluster are placed on SMs of one GPC next to each other: a budget of B blocks then
            // takes B / cluster neighbourhoods away from a concurrent kernel instead of B scattered SMs
            attr[nattr].id = cudaLaunchAttributeClusterDimension;
            attr[nattr].val.clusterDim.x = (unsigned)p->opts.cluster;
            attr[nattr].val.clusterDim.y = 1;
            attr[nattr].val.clusterDim.z = 1;
            ++nattr;
        }
        cfg.attrs = attr;
        cfg.numAttrs = (unsigned)nattr;
        if (p->opts.light)
            CUDA_TRY(cudaLaunchKernelEx(&cfg, hccl_executor_lsu_light, prm));
        else
            CUDA_TRY(cudaLaunchKernelEx(&cfg, hccl_executor_lsu, prm));
    }
    CUDA_TRY(cudaGetLastError());
    p->epoch = epoch;
    return HCCL_OK;
}

hccl_status_t hccl_execute_host(hccl_plan_t* p, const void* const* host_send, void* const* host_recv, void* const* dev_send,
                                void* const* dev_recv, void* stream) {
    if (!p || !host_send || !host_recv || !dev_send || !dev_recv) return HCCL_ERR_INVALID_ARG;
    cudaStream_t s = (cudaStream_t)stream;
    for (int r = 0; r < p->R; ++r)
        if (p->send_bytes[r] > 0) CUDA_TRY(cudaMemcpyAsync(dev_send[r], host_send[r], (size_t)p->send_bytes[r], cudaMemcpyHostToDevice, s));
    hccl_status_t st = hccl_execute(p, (const void* const*)dev_send, dev_recv, stream);
    if (st != HCCL_OK) return st;
    for (int r = 0; r < p->R; ++r)
        if (p->recv_bytes[r] > 0) CUDA_TRY(cudaMemcpyAsync(host_recv[r], dev_recv[r], (size_t)p->recv_bytes[r], cudaMemcpyDeviceToHost, s));
    return HCCL_OK;
}

// ---------------------------------------------------------------------- host pipeline (AllToAllv by destination windows)
}  // extern "C"

struct hccl_hostpipe {
    int R = 0;
    int64_t row_bytes = 0;
    std::vector<int64_t> counts;          // [s*R+d] rows
    std::vector<int64_t> sdispl;          // packed, rows
    std::vector<int64_t> recv_rows;       // per destination
    std::vector<int32_t> first_dest;      // n_windows + 1
    std::vector<hccl_plan_t*> plans;      // one per window
    std::vector<size_t> ws_off;           // each sub-plan's slice of the workspace
    size_t ws_total = 0;
    std::vector<cudaEvent_t> in_done, exec_done, out_done;
    cudaEvent_t all_done = nullptr;
    bool bound = false, ran = false;
    ~hccl_hostpipe() {
        for (hccl_plan_t* q : plans) hccl_plan_destroy(q);
        for (cudaEvent_t e : in_done) cudaEventDestroy(e);
        for (cudaEvent_t e : exec_done) cudaEventDestroy(e);
        for (cudaEvent_t e : out_done) cudaEventDestroy(e);
        if (all_done) cudaEventDestroy(all_done);
    }
};

extern "C" {

hccl_status_t hccl_hostpipe_alltoallv_create(int R, const int64_t* sendcounts, hccl_dtype_t dt, int64_t row_elems, int n_windows,
                                             const hccl_opts_t* opts, hccl_hostpipe_t** out) {
    if (!out || !sendcounts || R < 1 || R > HCCL_MAX_RANKS || row_elems < 1 || n_windows < 1) return HCCL_ERR_INVALID_ARG;
    if (dt != HCCL_FP32 && dt != HCCL_BF16 && dt != HCCL_FP16) return HCCL_ERR_DTYPE;
    hccl_hostpipe* hp = new (std::nothrow) hccl_hostpipe();
    if (!hp) return HCCL_ERR_INVALID_ARG;
    hp->R = R;
    hp->row_bytes = row_elems * (dt == HCCL_FP32 ? 4 : 2);
    hp->counts.assign(sendcounts, sendcounts + (size_t)R * R);
    hp->sdispl.assign((size_t)R * R, 0);
    hp->recv_rows.assign(R, 0);
    int64_t total = 0;
    for (int s = 0; s < R; ++s) {
        int64_t acc = 0;
        for (int d = 0; d < R; ++d) {
            const int64_t c = sendcounts[(size_t)s * R + d];
            if (c < 0) {
                delete hp;
                return HCCL_ERR_INVALID_ARG;
            }
            hp->sdispl[(size_t)s * R + d] = acc;
            acc += c;
            hp->recv_rows[d] += c;
            total += c;
        }
    }
    // Contiguous windows of destinations, each closed once the rows received so far reach its cumulative
    // share. The shares taper towards both ends (weights 1, 2, 3, 4, 4, ..., 4, 3, 2, 1): the first copy-in
    // and the last copy-out are the only steps nothing overlaps, so those windows are the small ones.
    const int W = std::min(n_windows, R);
    std::vector<int64_t> cum(W + 1, 0);
    for (int g = 0; g < W; ++g) cum[g + 1] = cum[g] + std::min(std::min(g + 1, W - g), 4);
    hp->first_dest.push_back(0);
    int64_t acc = 0, in_window = 0;
    for (int d = 0; d < R; ++d) {
        acc += hp->recv_rows[d];
        in_window += hp->recv_rows[d];
        const int made = (int)hp->first_dest.size();  // windows closed so far + 1
        if (made < W && (__int128)acc * cum[W] >= (__int128)total * cum[made] && in_window > 0 && d + 1 < R) {
            hp->first_dest.push_back(d + 1);
            in_window = 0;
        }
    }
    hp->first_dest.push_back(R);
    // a trailing window without rows joins the one before it
    while (hp->first_dest.size() > 2) {
        int64_t rows = 0;
        for (int d = hp->first_dest[hp->first_dest.size() - 2]; d < R; ++d) rows += hp->recv_rows[d];
        if (rows > 0) break;
        hp->first_dest.erase(hp->first_dest.end() - 2);
    }
    const int nw = (int)hp->first_dest.size() - 1;
    for (int g = 0; g < nw; ++g) {
        hccl_plan_t* q = nullptr;
        hccl_status_t st = hccl::plan_alltoallv_window(R, sendcounts, nullptr, nullptr, nullptr, dt, row_elems, opts,
                                                       hp->first_dest[g], hp->first_dest[g + 1], &q);
        if (st != HCCL_OK) {
            delete hp;
            return st;
        }
        hp->plans.push_back(q);
        hp->ws_off.push_back(hp->ws_total);
        hp->ws_total += (size_t)((q->layout.total + 255) / 256 * 256);
    }
    *out = hp;
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_windows(const hccl_hostpipe_t* hp, int32_t* n_windows, int32_t* first_dest) {
    if (!hp || !n_windows) return HCCL_ERR_INVALID_ARG;
    *n_windows = (int32_t)hp->plans.size();
    if (first_dest)
        for (size_t i = 0; i < hp->first_dest.size(); ++i) first_dest[i] = hp->first_dest[i];
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_workspace_bytes(const hccl_hostpipe_t* hp, size_t* bytes) {
    if (!hp || !bytes) return HCCL_ERR_INVALID_ARG;
    *bytes = hp->ws_total;
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_bind(hccl_hostpipe_t* hp, void* dev_workspace, size_t bytes, void* stream) {
    if (!hp || !dev_workspace) return HCCL_ERR_INVALID_ARG;
    if (((uintptr_t)dev_workspace) % 256) return HCCL_ERR_ALIGNMENT;
    if (bytes < hp->ws_total) return HCCL_ERR_WORKSPACE;
    for (size_t g = 0; g < hp->plans.size(); ++g) {
        hccl_status_t st = hccl_plan_bind(hp->plans[g], (char*)dev_workspace + hp->ws_off[g], (size_t)hp->plans[g]->layout.total, stream);
        if (st != HCCL_OK) return st;
    }
    if (!hp->all_done) {
        hp->in_done.resize(hp->plans.size());
        hp->exec_done.resize(hp->plans.size());
        hp->out_done.resize(hp->plans.size());
        for (size_t g = 0; g < hp->plans.size(); ++g) {
            CUDA_TRY(cudaEventCreateWithFlags(&hp->in_done[g], cudaEventDisableTiming));
            CUDA_TRY(cudaEventCreateWithFlags(&hp->exec_done[g], cudaEventDisableTiming));
            CUDA_TRY(cudaEventCreateWithFlags(&hp->out_done[g], cudaEventDisableTiming));
        }
        CUDA_TRY(cudaEventCreateWithFlags(&hp->all_done, cudaEventDisableTiming));
    }
    hp->bound = true;
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_execute(hccl_hostpipe_t* hp, const void* const* host_send, void* const* host_recv, void* const* dev_send,
                                    void* const* dev_recv, void* stream_in, void* stream_exec, void* stream_out) {
    if (!hp || !host_send || !host_recv || !dev_send || !dev_recv) return HCCL_ERR_INVALID_ARG;
    if (!hp->bound) return HCCL_ERR_NOT_BOUND;
    cudaStream_t si = (cudaStream_t)stream_in, sx = (cudaStream_t)stream_exec, so = (cudaStream_t)stream_out;
    const int R = hp->R;
    // The staging buffers are reused by the next call. Its copies-in may start once the previous call's last
    // exchange has run (nothing reads the send staging after that), and its exchange of window g once the
    // previous call's copy-out of window g has finished; so one call's drain overlaps the next one's fill.
    if (hp->ran) CUDA_TRY(cudaStreamWaitEvent(si, hp->exec_done.back(), 0));
    for (size_t g = 0; g < hp->plans.size(); ++g) {
        const int d0 = hp->first_dest[g], d1 = hp->first_dest[g + 1];
        for (int s = 0; s < R; ++s) {  // rows of source s bound for destinations d0..d1-1: one contiguous slice
            const int64_t lo = hp->sdispl[(size_t)s * R + d0];
            const int64_t hi = d1 < R ? hp->sdispl[(size_t)s * R + d1] : hp->sdispl[(size_t)s * R + R - 1] + hp->counts[(size_t)s * R + R - 1];
            if (hi > lo)
                CUDA_TRY(cudaMemcpyAsync((char*)dev_send[s] + lo * hp->row_bytes, (const char*)host_send[s] + lo * hp->row_bytes,
                                         (size_t)((hi - lo) * hp->row_bytes), cudaMemcpyHostToDevice, si));
        }
        CUDA_TRY(cudaEventRecord(hp->in_done[g], si));
        CUDA_TRY(cudaStreamWaitEvent(sx, hp->in_done[g], 0));
        if (hp->ran) CUDA_TRY(cudaStreamWaitEvent(sx, hp->out_done[g], 0));
        hccl_status_t st = hccl_execute(hp->plans[g], (const void* const*)dev_send, dev_recv, stream_exec);
        if (st != HCCL_OK) return st;
        CUDA_TRY(cudaEventRecord(hp->exec_done[g], sx));
        CUDA_TRY(cudaStreamWaitEvent(so, hp->exec_done[g], 0));
        for (int d = d0; d < d1; ++d)
            if (hp->recv_rows[d] > 0)
                CUDA_TRY(cudaMemcpyAsync(host_recv[d], dev_recv[d], (size_t)(hp->recv_rows[d] * hp->row_bytes), cudaMemcpyDeviceToHost, so));
        CUDA_TRY(cudaEventRecord(hp->out_done[g], so));
    }
    CUDA_TRY(cudaEventRecord(hp->all_done, so));
    hp->ran = true;
    return HCCL_OK;
}

hccl_status_t hccl_hostpipe_status(hccl_hostpipe_t* hp, hccl_status_t* device_status, int64_t* detail) {
    if (!hp || !device_status) return HCCL_ERR_INVALID_ARG;
    if (!hp->bound) return HCCL_ERR_NOT_BOUND;
    *device_status = HCCL_OK;
    for (hccl_plan_t* q : hp->plans) {
        hccl_status_t ds = HCCL_OK;
        int64_t dd = 0;
        hccl_status_t st = hccl_plan_status(q, &ds, &dd);
        if (st != HCCL_OK) return st;
        if (ds != HCCL_OK) {
            *device_status = ds;
            if (detail) *detail = dd;
            return HCCL_OK;
        }
    }
    if (detail) *detail = 0;
    return HCCL_OK;
}

void hccl_hostpipe_destroy(hccl_hostpipe_t* hp) { delete hp; }

hccl_status_t hccl_plan_status(hccl_plan_t* p, hccl_status_t* device_status, int64_t* detail) {
    if (!p || !device_status) return HCCL_ERR_INVALID_ARG;
    if (!p->workspace) return HCCL_ERR_NOT_BOUND;
    Control c;
    CUDA_TRY(cudaMemcpy(&c, (char*)p->workspace + p->layout.control, sizeof(c), cudaMemcpyDeviceToHost));
    // The device numbers its own executions (so that graph replays count too): the last one failed if the
    // failure stamp carries its number.
    if (c.done_epoch != 0 && c.fail_epoch == c.done_epoch) {
        *device_status = (hccl_status_t)c.status;
        if (detail) *detail = (int64_t)c.detail;
        return HCCL_OK;
    }
    if (c.exits != 0) return HCCL_ERR_BUSY;  // blocks of an execution are still leaving: synchronise first
    *device_status = HCCL_OK;
    if (detail) *detail = (int64_t)c.done_epoch;
    return HCCL_OK;
}

}  // extern "C"

// ====================================================================== resident executor: host side
extern "C" {

hccl_status_t hccl_server_start(hccl_plan_t* p, const void* const* sendbufs, void* const* recvbufs, void* host_doorbell,
                                uint64_t idle_timeout_ns, void* stream) {
    if (!p || !sendbufs || !recvbufs || !host_doorbell) return HCCL_ERR_INVALID_ARG;
    if (!p->workspace) return HCCL_ERR_NOT_BOUND;
    if (p->dynamic || p->server_db) return HCCL_ERR_INVALID_ARG;
    if (((uintptr_t)host_doorbell) % 64) return HCCL_ERR_ALIGNMENT;
    hccl_status_t st = check_buffers(p, sendbufs, recvbufs);
    if (st != HCCL_OK) return st;
    void* dev_db = nullptr;
    CUDA_TRY(cudaHostGetDevicePointer(&dev_db, host_doorbell, 0));  // fails unless the record is pinned, mapped memory
    cudaStream_t s = (cudaStream_t)stream;
    Control c;
    CUDA_TRY(cudaStreamSynchronize(s));
    CUDA_TRY(cudaMemcpy(&c, (char*)p->workspace + p->layout.control, sizeof(c), cudaMemcpyDeviceToHost));
    CUDA_TRY(cudaMemsetAsync((char*)p->workspace + p->layout.control + offsetof(Control, server_go), 0, 4, s));
    std::memset(host_doorbell, 0, sizeof(Doorbell));
    static thread_local ExecParams prm;
    const int blocks = fill_params(p, prm, sendbufs, recvbufs);
    // every block must be resident at once (the blocks wait for each other between executions)
    int dev = 0, sms = 0, per_sm = 0;
    CUDA_TRY(cudaGetDevice(&dev));
    CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, hccl_executor_resident, p->opts.threads, 0));
    if (blocks > sms * per_sm) return HCCL_ERR_INVALID_ARG;
    Doorbell* db = (Doorbell*)dev_db;
    unsigned long long idle = idle_timeout_ns ? idle_timeout_ns : 100000000ull;
    uint32_t first_epoch = c.done_epoch + 1;
    void* args[] = {(void*)&prm, (void*)&db, (void*)&idle, (void*)&first_epoch};
    CUDA_TRY(cudaLaunchCooperativeKernel((const void*)hccl_executor_resident, dim3((unsigned)blocks), dim3((unsigned)p->opts.threads), args, 0, s));
    p->server_db = host_doorbell;
    p->server_rings = 0;
    return HCCL_OK;
}

hccl_status_t hccl_server_ring(hccl_plan_t* p) {
    if (!p || !p->server_db) return HCCL_ERR_INVALID_ARG;
    volatile Doorbell* db = (volatile Doorbell*)p->server_db;
    if (db->exited) return db->exited == 3 ? (hccl_status_t)db->status : HCCL_ERR_TIMEOUT;  // the kernel has left: start it again
    std::atomic_thread_fence(std::memory_order_release);
    db->request = ++p->server_rings;
    return HCCL_OK;
}

hccl_status_t hccl_server_wait(hccl_plan_t* p, uint64_t timeout_ns) {
    if (!p || !p->server_db) return HCCL_ERR_INVALID_ARG;
    volatile Doorbell* db = (volatile Doorbell*)p->server_db;
    const auto t0 = std::chrono::steady_clock::now();
    const uint64_t limit = timeout_ns ? timeout_ns : 5000000000ull;
    for (;;) {
        if (db->completed >= p->server_rings) break;
        if (db->exited) break;
        if ((uint64_t)std::chrono::duration_cast<std::chrono::nanoseconds>(std::chrono::steady_clock::now() - t0).count() > limit) return HCCL_ERR_TIMEOUT;
    }
    std::atomic_thread_fence(std::memory_order_acquire);
    if (db->exited == 3) return (hccl_status_t)db->status;
    if (db->completed < p->server_rings) return HCCL_ERR_TIMEOUT;  // left (idle or stopped) before serving this ring
    return HCCL_OK;
}

hccl_status_t hccl_server_stop(hccl_plan_t* p) {
    if (!p || !p->server_db) return HCCL_ERR_INVALID_ARG;
    volatile Doorbell* db = (volatile Doorbell*)p->server_db;
    db->stop = 1;
    p->epoch += p->server_rings;
    p->server_db = nullptr;
    return HCCL_OK;
}

}  // extern "C"

// ====================================================================== execution without any allocation
// Workspace for callers that cannot obtain device memory of their own: one array that lives in the
// library's device image for the life of the process (every GPU that loads the library holds it).
#define HCCL_NOALLOC_WORKSPACE_BYTES (8u << 20)
static __device__ __align__(256) unsigned char g_noalloc_workspace[HCCL_NOALLOC_WORKSPACE_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_noalloc_addr[kMaxDevices] = {};  // device address of g_noalloc_workspace, per device ordinal
std::mutex g_noalloc_mu;
}  // namespace

extern "C" hccl_status_t hccl_execute_noalloc(hccl_plan_t* p, const void* const* sendbufs, void* const* recvbufs, void* stream) {
    if (!p || !sendbufs || !recvbufs) return HCCL_ERR_INVALID_ARG;
    if (p->layout.total > HCCL_NOALLOC_WORKSPACE_BYTES) {
        snprintf(g_cuda_err, sizeof(g_cuda_err), "plan needs %llu workspace bytes; the built-in workspace holds %u",
                 (unsigned long long)p->layout.total, HCCL_NOALLOC_WORKSPACE_BYTES);
        return HCCL_ERR_WORKSPACE;
    }
    if (p->trig_wait_slot >= 0 || p->trig_set_slot >= 0 || p->dynamic) return HCCL_ERR_INVALID_ARG;  // triggers and device-resident plans belong to bound plans
    int dev = -1;
    CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return HCCL_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_noalloc_mu);  // one user of the array at a time from this process
    if (!g_noalloc_addr[dev]) {
        // In host code the array's name is only a handle; its device address on the current device is
        // looked up once here and that address is what the kernel receives.
        void* ptr = nullptr;
        CUDA_TRY(cudaGetSymbolAddress(&ptr, g_noalloc_workspace));
        if (!ptr || ((uintptr_t)ptr % 256) != 0) return HCCL_ERR_ALIGNMENT;
        g_noalloc_addr[dev] = ptr;
    }
    char* ws = (char*)g_noalloc_addr[dev];
    // same aliasing rules as hccl_execute, checked on every call (nothing is cached for this path)
    const int R = p->R;
    for (int r = 0; r < R; ++r) {
        if ((p->send_bytes[r] > 0 && !sendbufs[r]) || (p->recv_bytes[r] > 0 && !recvbufs[r])) return HCCL_ERR_INVALID_ARG;
        if (((uintptr_t)sendbufs[r] | (uintptr_t)recvbufs[r]) & (uintptr_t)(p->buf_align - 1)) return HCCL_ERR_ALIGNMENT;
    }
    for (int d = 0; d < R; ++d) {
        const uintptr_t lo = (uintptr_t)recvbufs[d], hi = lo + (uintptr_t)p->recv_bytes[d];
        if (lo == hi) continue;
        for (int s = 0; s < R; ++s) {
            const uintptr_t slo = (uintptr_t)sendbufs[s], shi = slo + (uintptr_t)p->send_bytes[s];
            if (slo != shi && lo < shi && slo < hi) return HCCL_ERR_OVERLAP;
            const uintptr_t rlo = (uintptr_t)recvbufs[s], rhi = rlo + (uintptr_t)p->recv_bytes[s];
            if (s > d && rlo != rhi && lo < rhi && rlo < hi) return HCCL_ERR_OVERLAP;
        }
    }
    // The array keeps whatever the previous call left. Everything that must start at zero (control words,
    // dependency counters, signal slots) is rewritten together with this plan's tables; the FP32 scratch
    // behind them is always written before it is read within one execution, so it is left as it is.
    const Layout& L = p->layout;
    static thread_local std::vector<char> img;
    img.assign((size_t)L.scratch, 0);
    if (!p->descs.empty()) std::memcpy(img.data() + L.descs, p->descs.data(), p->descs.size() * sizeof(Desc));
    if (!p->tiles.empty()) std::memcpy(img.data() + L.tiles, p->tiles.data(), p->tiles.size() * sizeof(Tile));
    if (!p->waits.empty()) std::memcpy(img.data() + L.waits, p->waits.data(), p->waits.size() * sizeof(Wait));
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_TRY(cudaMemcpyAsync(ws, img.data(), img.size(), cudaMemcpyHostToDevice, st));
    static thread_local ExecParams prm;
    prm.descs = (const Desc*)(ws + L.descs);
    prm.tiles = (const Tile*)(ws + L.tiles);
    prm.waits = (const Wait*)(ws + L.waits);
    prm.counters = (uint32_t*)(ws + L.counters);
    prm.signals = (unsigned long long*)(ws + L.signals);
    prm.ctl = (Control*)(ws + L.control);
    prm.scratch = ws + L.scratch;
    prm.user_signals = nullptr;
    prm.trace = nullptr;
    prm.trace_cap = 0;
    prm.n_tiles = (uint32_t)p->tiles.size();
    prm.n_descs = (uint32_t)p->descs.size();
    prm.n_syncs = (uint32_t)p->sync_per_epoch.size();
    prm.n_waits = (uint32_t)p->waits.size();
    prm.n_signals = (uint32_t)p->n_signals;
    prm.R = (uint32_t)R;
    prm.timeout_ns = p->opts.timeout_ns;
    prm.n_user_signals = 0;
    prm.trig_wait_slot = -1;
    prm.trig_set_slot = -1;
    prm.trig_cmp = 0;
    prm.trig_wait_value = prm.trig_set_value = prm.trig_wait_per_epoch = prm.trig_set_per_epoch = 0;
    for (int r = 0; r < R; ++r) {
        prm.send[r] = sendbufs[r];
        prm.recv[r] = recvbufs[r];
    }
    const int blocks = set_dispatch(p, prm);
    hccl_executor_lsu<<<blocks, p->opts.threads, 0, st>>>(prm);
    CUDA_TRY(cudaGetLastError());
    // This call owns the shared array until its kernel is done, so it waits here and hands back the
    // device-side verdict itself.
    CUDA_TRY(cudaStreamSynchronize(st));
    Control c;
    CUDA_TRY(cudaMemcpy(&c, ws + L.control, sizeof(c), cudaMemcpyDeviceToHost));
    if (c.fail_epoch == 1) return (hccl_status_t)c.status;
    if (c.done_epoch != 1) return HCCL_ERR_BUSY;
    return HCCL_OK;
}
#endif  // part 4
