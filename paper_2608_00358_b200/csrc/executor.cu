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
#include <cstring>
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
    uint32_t n_tiles, n_descs, n_syncs, n_waits;
    uint32_t epoch, R, nblocks, n_signals;
    unsigned long long timeout_ns;
    long long n_user_signals;
    long long trig_wait_slot, trig_set_slot;
    int trig_cmp, pad0;
    unsigned long long trig_wait_value, trig_set_value;
    const void* send[HCCL_MAX_RANKS];
    void* recv[HCCL_MAX_RANKS];
};

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
__device__ __noinline__ void fail(const ExecParams& p, uint32_t code, unsigned long long detail) {
    if (atomicExch(&p.ctl->fail_epoch, p.epoch) != p.epoch) {  // first failure of this execution wins
        p.ctl->status = code;
        p.ctl->detail = detail;
    }
    __threadfence();
    atomicExch(&p.ctl->abort, p.epoch);
}
__device__ __forceinline__ bool aborted(const ExecParams& p) { return ld_relaxed_u32(&p.ctl->abort) == p.epoch; }

// Bounded wait until counters[sync] has received epoch * per_epoch bumps (wrap-safe compare).
__device__ bool wait_counter(const ExecParams& p, uint32_t sync, uint32_t per_epoch, uint32_t tile) {
    const uint32_t* c = p.counters + sync;
    const uint32_t target = p.epoch * per_epoch;
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

__device__ bool wait_signal(const ExecParams& p, const unsigned long long* addr, int cmp, unsigned long long want, uint32_t tile) {
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
__device__ void copy_tile_lsu(char* dst, const char* src, uint32_t n) {
    const uint32_t tid = threadIdx.x, nth = blockDim.x;
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

// ------------------------------------------------------------------ REDUCE (S=A+B and in-place forms)
template <int DA, int DB, int DD, bool STREAM_B>
__device__ void reduce_tile_lsu(char* dst, const char* a, const char* b, uint32_t n) {
    const uint32_t tid = threadIdx.x, nth = blockDim.x;
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
__device__ __forceinline__ void reduce_dispatch_d(int dd, char* dst, const char* a, const char* b, uint32_t n) {
    if (dd == HCCL_FP32) reduce_tile_lsu<DA, DB, HCCL_FP32, SB>(dst, a, b, n);
    else if (dd == HCCL_BF16) reduce_tile_lsu<DA, DB, HCCL_BF16, SB>(dst, a, b, n);
    else reduce_tile_lsu<DA, DB, HCCL_FP16, SB>(dst, a, b, n);
}
template <int DA, bool SB>
__device__ __forceinline__ void reduce_dispatch_b(int db, int dd, char* dst, const char* a, const char* b, uint32_t n) {
    if (db == HCCL_FP32) reduce_dispatch_d<DA, HCCL_FP32, SB>(dd, dst, a, b, n);
    else if (db == HCCL_BF16) reduce_dispatch_d<DA, HCCL_BF16, SB>(dd, dst, a, b, n);
    else reduce_dispatch_d<DA, HCCL_FP16, SB>(dd, dst, a, b, n);
}
template <bool SB>
__device__ void reduce_dispatch(int da, int db, int dd, char* dst, const char* a, const char* b, uint32_t n) {
    if (da == HCCL_FP32) reduce_dispatch_b<HCCL_FP32, SB>(db, dd, dst, a, b, n);
    else if (da == HCCL_BF16) reduce_dispatch_b<HCCL_BF16, SB>(db, dd, dst, a, b, n);
    else reduce_dispatch_b<HCCL_FP16, SB>(db, dd, dst, a, b, n);
}

// ------------------------------------------------------------------ REDUCE_N (multi-input sum, fixed order)
template <int DS, int DD>
__device__ void reduce_n_tile(const ExecParams& p, const Desc& d, uint64_t start, uint32_t n) {
    const uint32_t tid = threadIdx.x, nth = blockDim.x;
    const int R = (int)p.R, nsrc = d.nsrc, r0 = d.rank_a;
    const size_t soff = (size_t)d.off_a + start * Elem<DS>::BYTES;
    char* dst = buf_base(p, d.kind_dst, d.rank_dst) + d.off_dst + start * Elem<DD>::BYTES;
    const bool from_send = d.kind_a == HCCL_BUF_SEND;
    auto src = [&](int k) -> const char* {
        int r = r0 + k;
        if (r >= R) r -= R;
        return (const char*)(from_send ? p.send[r] : (const void*)p.recv[r]) + soff;
    };
    // same phase for every operand?
    const uint32_t pd = (uint32_t)(((uintptr_t)dst / Elem<DD>::BYTES) & 7u);
    bool vec = true;
    for (int k = 0; k < nsrc; ++k) vec = vec && ((uint32_t)(((uintptr_t)src(k) / Elem<DS>::BYTES) & 7u) == pd);
    if (!vec) {
        for (uint32_t i = tid; i < n; i += nth) {
            float acc = Elem<DS>::load(src(0), i);
            for (int k = 1; k < nsrc; ++k) acc = acc + Elem<DS>::load(src(k), i);
            Elem<DD>::store(dst, i, acc);
        }
        return;
    }
    uint32_t head = (8u - pd) & 7u;
    if (head > n) head = n;
    const uint32_t nv = (n - head) >> 3;
    auto scalar = [&](uint32_t i) {
        float acc = Elem<DS>::load(src(0), i);
        for (int k = 1; k < nsrc; ++k) acc = acc + Elem<DS>::load(src(k), i);
        Elem<DD>::store(dst, i, acc);
    };
    if (tid < head) scalar(tid);
    for (uint32_t i = head + (nv << 3) + tid; i < n; i += nth) scalar(i);
    const size_t hs = (size_t)head * Elem<DS>::BYTES;
    for (uint32_t i = tid; i < nv; i += nth) {
        float acc[8];
        load8<DS, false>(src(0) + hs + (size_t)i * 8 * Elem<DS>::BYTES, acc);
        int k = 1;
        for (; k + 4 <= nsrc; k += 4) {
            float x[4][8];
#pragma unroll
            for (int j = 0; j < 4; ++j) load8<DS, false>(src(k + j) + hs + (size_t)i * 8 * Elem<DS>::BYTES, x[j]);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = acc[e] + x[j][e];
            }
        }
        for (; k < nsrc; ++k) {
            float x[8];
            load8<DS, false>(src(k) + hs + (size_t)i * 8 * Elem<DS>::BYTES, x);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = acc[e] + x[e];
        }
        store8<DD, false>(dst + (size_t)head * Elem<DD>::BYTES + (size_t)i * 8 * Elem<DD>::BYTES, acc);
    }
}

__device__ void reduce_n_dispatch(const ExecParams& p, const Desc& d, uint64_t start, uint32_t n) {
#define RN(S, D) reduce_n_tile<S, D>(p, d, start, n)
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
__device__ void run_tile_lsu(const ExecParams& p, const Desc& d, const Tile& t) {
    switch (d.op) {
        case HCCL_OP_COPY: {
            char* dst = buf_base(p, d.kind_dst, d.rank_dst) + d.off_dst + t.start;
            const char* src = buf_base(p, d.kind_a, d.rank_a) + d.off_a + t.start;
            // send-to-receive copies (AllToAllv, AllGather's first hop) are read once and written once
            if (d.kind_a == HCCL_BUF_SEND) copy_tile_lsu<true>(dst, src, t.count); else copy_tile_lsu<false>(dst, src, t.count);
            break;
        }
        case HCCL_OP_REDUCE: {
            char* dst = buf_base(p, d.kind_dst, d.rank_dst) + d.off_dst + t.start * (d.dt_dst == HCCL_FP32 ? 4 : 2);
            const char* a = buf_base(p, d.kind_a, d.rank_a) + d.off_a + t.start * (d.dt_a == HCCL_FP32 ? 4 : 2);
            const char* b = buf_base(p, d.kind_b, d.rank_b) + d.off_b + t.start * (d.dt_b == HCCL_FP32 ? 4 : 2);
            if (d.kind_b == HCCL_BUF_SEND) reduce_dispatch<true>(d.dt_a, d.dt_b, d.dt_dst, dst, a, b, t.count);
            else reduce_dispatch<false>(d.dt_a, d.dt_b, d.dt_dst, dst, a, b, t.count);
            break;
        }
        case HCCL_OP_REDUCE_N:
            reduce_n_dispatch(p, d, t.start, t.count);
            break;
        default:
            break;
    }
}

// Checks on a table entry before it is used; a failing entry is reported, never dereferenced.
__device__ bool tile_ok(const ExecParams& p, const Tile& t) {
    if (t.desc >= p.n_descs) return false;
    if ((uint64_t)t.wait_off + t.wait_cnt > p.n_waits) return false;
    for (int k = 0; k < 2; ++k)
        if (t.signal[k] >= (int32_t)p.n_syncs) return false;
    return true;
}
__device__ bool desc_ok(const ExecParams& p, const Desc& d) {
    if (d.op > HCCL_OP_NOOP) return false;
    if (d.op == HCCL_OP_COPY || d.op == HCCL_OP_REDUCE || d.op == HCCL_OP_REDUCE_N) {
        if (d.kind_dst != HCCL_BUF_RECV && d.kind_dst != HCCL_BUF_SCRATCH) return false;
        if (d.kind_a > HCCL_BUF_SCRATCH) return false;
        if (d.rank_dst >= p.R || d.rank_a >= p.R) return false;
        if (d.op == HCCL_OP_REDUCE && (d.kind_b > HCCL_BUF_SCRATCH || d.rank_b >= p.R)) return false;
        if (d.op != HCCL_OP_COPY && (d.dt_dst > HCCL_FP16 || d.dt_a > HCCL_FP16 || (d.op == HCCL_OP_REDUCE && d.dt_b > HCCL_FP16))) return false;
        if (d.op == HCCL_OP_REDUCE_N && (d.nsrc < 1 || d.nsrc > p.R || d.kind_a > HCCL_BUF_RECV)) return false;
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

// Thread 0: everything that precedes the data movement of work item `cur`. Returns false to stop.
__device__ bool prepare_tile(const ExecParams& p, uint32_t cur, Tile& t, Desc& d) {
    t = p.tiles[cur];
    if (!tile_ok(p, t)) {
        fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
        return false;
    }
    d = p.descs[t.desc];
    if (!desc_ok(p, d)) {
        fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
        return false;
    }
    for (uint32_t w = 0; w < t.wait_cnt; ++w) {
        const Wait x = p.waits[t.wait_off + w];
        if (x.sync >= p.n_syncs) {
            fail(p, HCCL_ERR_BAD_DESCRIPTOR, cur);
            return false;
        }
        if (!wait_counter(p, x.sync, x.per_epoch, cur)) return false;
    }
    if (d.op == HCCL_OP_WAIT) {
        const unsigned long long* addr = (d.kind_a == HCCL_BUF_SIGNAL ? p.signals : p.user_signals) + d.off_a;
        if (!wait_signal(p, addr, d.cmp, d.value + (unsigned long long)p.epoch * d.value_per_epoch, cur)) return false;
    } else if (d.op == HCCL_OP_SET) {
        unsigned long long* addr = (d.kind_dst == HCCL_BUF_SIGNAL ? p.signals : p.user_signals) + d.off_dst;
        __threadfence();
        st_release_u64(addr, d.value + (unsigned long long)p.epoch * d.value_per_epoch);
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
__device__ void leave(const ExecParams& p) {
    __threadfence();
    const uint32_t prev = atomicAdd(&p.ctl->exits, 1);
    if (prev == p.nblocks - 1) {
        __threadfence();
        if (p.trig_set_slot >= 0 && !aborted(p)) st_release_u64(p.user_signals + p.trig_set_slot, p.trig_set_value);
        p.ctl->t_last_ns = globaltimer_ns();
        p.ctl->ticket = 0;
        p.ctl->exits = 0;
        __threadfence();
        p.ctl->done_epoch = p.epoch;
    }
}

__global__ void __launch_bounds__(512, 1) hccl_executor_lsu(const __grid_constant__ ExecParams p) {
    __shared__ Tile s_tile;
    __shared__ Desc s_desc;
    __shared__ int s_go;
    const uint32_t tid = threadIdx.x;
    uint32_t next = 0;
    bool live = true;
    if (tid == 0) {
        if (p.trig_wait_slot >= 0)
            live = wait_signal(p, p.user_signals + p.trig_wait_slot, p.trig_cmp, p.trig_wait_value, 0xffffffffu);
        next = atomicAdd(&p.ctl->ticket, 1);
        if (next == 0) p.ctl->t_first_ns = globaltimer_ns();
    }
    for (;;) {
        if (tid == 0) {
            const uint32_t cur = next;
            int go = 0;
            if (live && cur < p.n_tiles && !aborted(p)) {
                next = atomicAdd(&p.ctl->ticket, 1);  // claim ahead: its latency hides behind this item
                go = prepare_tile(p, cur, s_tile, s_desc) ? 1 : 0;
            }
            s_go = go;
        }
        __syncthreads();
        if (!s_go) break;
        run_tile_lsu(p, s_desc, s_tile);
        __syncthreads();
        if (tid == 0) publish_tile(p, s_tile);
    }
    if (tid == 0) leave(p);
}

}  // namespace hccl

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
    p->workspace = dev_workspace;
    p->workspace_bytes = bytes;
    p->epoch = 0;
    p->checked_send.clear();
    p->checked_recv.clear();
    return HCCL_OK;
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
    static thread_local ExecParams prm;  // 4 KB+: keep it off the stack
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
    prm.n_tiles = (uint32_t)p->tiles.size();
    prm.n_descs = (uint32_t)p->descs.size();
    prm.n_syncs = (uint32_t)p->sync_per_epoch.size();
    prm.n_waits = (uint32_t)p->waits.size();
    prm.n_signals = (uint32_t)p->n_signals;
    prm.R = (uint32_t)p->R;
    const uint32_t epoch = p->epoch + 1;
    prm.epoch = epoch;
    prm.timeout_ns = p->opts.timeout_ns;
    prm.n_user_signals = p->n_user_signals;
    prm.trig_wait_slot = p->trig_wait_slot;
    prm.trig_set_slot = p->trig_set_slot;
    prm.trig_cmp = p->trig_cmp;
    prm.trig_wait_value = p->trig_wait_value + (uint64_t)epoch * p->trig_wait_per_epoch;
    prm.trig_set_value = p->trig_set_value + (uint64_t)epoch * p->trig_set_per_epoch;
    for (int r = 0; r < p->R; ++r) {
        prm.send[r] = sendbufs[r];
        prm.recv[r] = recvbufs[r];
    }
    int blocks = p->opts.sm_budget;
    if ((uint32_t)blocks > prm.n_tiles) blocks = (int)std::max<uint32_t>(prm.n_tiles, 1u);
    prm.nblocks = (uint32_t)blocks;
    hccl_executor_lsu<<<blocks, p->opts.threads, 0, (cudaStream_t)stream>>>(prm);
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

hccl_status_t hccl_plan_status(hccl_plan_t* p, hccl_status_t* device_status, int64_t* detail) {
    if (!p || !device_status) return HCCL_ERR_INVALID_ARG;
    if (!p->workspace) return HCCL_ERR_NOT_BOUND;
    Control c;
    CUDA_TRY(cudaMemcpy(&c, (char*)p->workspace + p->layout.control, sizeof(c), cudaMemcpyDeviceToHost));
    if (p->epoch == 0) {
        *device_status = HCCL_OK;
        if (detail) *detail = 0;
        return HCCL_OK;
    }
    if (c.fail_epoch == p->epoch) {
        *device_status = (hccl_status_t)c.status;
        if (detail) *detail = (int64_t)c.detail;
        return HCCL_OK;
    }
    if (c.done_epoch != p->epoch) return HCCL_ERR_BUSY;  // the last execution has not finished
    *device_status = HCCL_OK;
    if (detail) *detail = 0;
    return HCCL_OK;
}

}  // extern "C"
