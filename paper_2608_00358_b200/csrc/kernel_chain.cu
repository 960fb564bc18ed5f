// Static chains on the bulk copy unit: a block walks a piece of 14336 elements through every step of its chain with the
// running FP32 sums held in registers.
//
// A ring ReduceScatter (paper Sec. II-A.2: send, receive, compute WQEs, step after step) is, per chunk, a chain of
// S = A + B items in which A of step t+1 is what step t stored. The other engines read that partial back from the
// L2; per element and step that is 4 bytes stored, 4 read back and 2 (bf16) read from the own input through an SM's
// port to the L2, which moves about 63 GB/s of stores and takes loads and stores in turn. Here every step still
// stores its result where its descriptor says, but the thread that stored an element keeps it and adds the next
// step's B to it: 4 bytes stored and 2 loaded per element and step. The B operands (send buffers, which no step
// writes) are fetched ahead by cp.async.bulk into a ring of stages; stores are plain 16-byte stores from registers.
//
// A ring AllReduce's AllGather hops (copies of what the step before stored) are stored from the same registers.
//
// Warp 0: lane 0 is the DMA thread; all 32 lanes fetch and check the records of a chain's steps together. Warps 1-7
// are the compute warps. A piece may start off a 16-byte boundary if all operands of the chain do so by the same
// number of elements: its first few and last few elements are read and stored with plain accesses by one thread each.
// A chain whose steps are not all of the form above (another operation first, an operand at another position inside
// a 16-byte word than the others, B not in a send buffer, an A that is neither a send buffer nor the step before)
// runs item by item through the register path, as the register engine's static chains do.
#include "bulk.cuh"
#include "kernels.cuh"

namespace hccl {
namespace chainfw {
using namespace bulk;

constexpr uint32_t CW = 7, CTH = CW * 32;    // compute warps, compute threads: 8 warps in all, so that a thread may have 255 registers
                                             // (nine warps are given registers like twelve: 168, and the running sums spill)
constexpr int G = 16;                         // groups of 4 elements per compute thread and piece
constexpr uint32_t PIECE = CTH * 4 * G;      // elements per piece: 64 per compute thread (one DMA issue per piece: the fewer the better)
constexpr uint32_t MAX_NS = 6;               // stages: 6 of PIECE * 2 bytes (16-bit operands) or 3 of PIECE * 4 (FP32)
constexpr uint32_t MAX_CDST = 256;           // destinations of one K_C piece: a chain's copies are stored one after the other by one piece
constexpr uint32_t MAX_STEPS = 512;          // items per chain that fit the step table (2 R - 2 for R = 256: 510)

enum : uint32_t { K_A = 0, K_B = 1, K_ITEM = 2, K_EXIT = 3, K_C = 4, K_CM = 5, K_RM = 6 };
constexpr uint32_t CM_MIN16 = 6, CM_MIN32 = 12;  // from this many copies on (16-bit / FP32 values), a chain's copies go out as one K_CM piece
struct alignas(16) Piece {
    char* dst;                  // K_B: where this piece's sums go; K_C: where the held values are copied to (K_CM: the stage's
                                //      destination list says where)
    const char* src0;           // K_A, K_B: where the operand's piece starts; its first `head` and last ((n - head) mod 8)
                                //           elements are read with plain loads, the rest arrives through the stage
    const char* discard;        // K_B: FP32 partial that a non-forwarding engine would read here for the last time (or null)
    uint32_t n;                 // elements in the piece
    uint32_t item;              // work item: K_ITEM runs it whole; trace and failure reports
    uint8_t kind, dt_src, dt_dst, keep;
    uint8_t last, head;         // last piece of its item (trace); elements before the first 16-byte boundary (0..7)
    uint16_t ndst;              // K_CM: destinations (consecutive items from `item` on)
};
struct alignas(8) Step {        // one item of the current chain, tile offset applied
    char* dst;
    const char* a;
    const char* b;
    uint32_t n;
    uint32_t item;
    uint8_t dt_a, dt_b, dt_dst, flags;
};
// Element phase of an address: all operands of a chain must share it, so that one scalar head of (8 - phase) mod 8
// elements brings all of them to a 16-byte boundary together.
// (es is 2 or 4: shifts and masks, no 64-bit division on the one thread that checks every step of every chain)
__device__ __forceinline__ uint32_t phase_of(const void* p, uint32_t es) { return (uint32_t)(((uintptr_t)p >> (es == 4 ? 2 : 1)) & 7u); }
__device__ __forceinline__ bool whole_elements(const void* p, uint32_t es) { return ((uintptr_t)p & (uintptr_t)(es - 1)) == 0; }
enum : uint8_t { S_OK = 1, S_COPY = 2, S_KEEP = 4, S_DISCARD_A = 8 };

template <int DS>
__device__ __forceinline__ void take(const char* stage, uint32_t nv, uint32_t ctid, float (&S)[G][4]) {
#pragma unroll
    for (int k = 0; k < G; ++k) {
        const uint32_t e = (k * CTH + ctid) * 4;
        if (e < nv) lds4<DS>(stage + (size_t)e * Elem<DS>::BYTES, S[k]);
    }
}
// The add and the store are separate steps (three variants by the operand's type, four by the destination's), not
// twelve fused ones: with those inlined side by side the compiler ran out of its 255 registers.
template <int DS>
__device__ __forceinline__ void accumulate(const char* stage, uint32_t nv, uint32_t ctid, float (&S)[G][4]) {
#pragma unroll
    for (int h = 0; h < G; h += 8) {  // eight loads in flight at a time
        float b[8][4];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t e = ((h + k) * CTH + ctid) * 4;
            if (e < nv) lds4<DS>(stage + (size_t)e * Elem<DS>::BYTES, b[k]);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const uint32_t e = ((h + k) * CTH + ctid) * 4;
            if (e < nv) {
#pragma unroll
                for (int j = 0; j < 4; ++j) S[h + k][j] = S[h + k][j] + b[k][j];
            }
        }
    }
}
template <int DD, bool KEEP>
__device__ __forceinline__ void store_all(char* dst, uint32_t nv, uint32_t ctid, const float (&S)[G][4], unsigned long long pol) {
#pragma unroll
    for (int k = 0; k < G; ++k) {
        const uint32_t e = (k * CTH + ctid) * 4;
        if (e < nv) stg4<DD, KEEP>(dst + (size_t)e * Elem<DD>::BYTES, S[k], pol);
    }
}
// The same values, rounded the same way, into shared memory (for the bulk copies of a chain's AllGather hops).
template <int DD>
__device__ __forceinline__ void stage_all(char* out, uint32_t nv, uint32_t ctid, const float (&S)[G][4]) {
#pragma unroll
    for (int k = 0; k < G; ++k) {
        const uint32_t e = (k * CTH + ctid) * 4;
        if (e < nv) {
            if constexpr (DD == HCCL_FP32) {
                *reinterpret_cast<float4*>(out + (size_t)e * 4) = make_float4(S[k][0], S[k][1], S[k][2], S[k][3]);
            } else {
                uint2 v;
                if constexpr (DD == HCCL_BF16) {
                    const __nv_bfloat162 a = __floats2bfloat162_rn(S[k][0], S[k][1]), b = __floats2bfloat162_rn(S[k][2], S[k][3]);
                    v.x = *reinterpret_cast<const uint32_t*>(&a); v.y = *reinterpret_cast<const uint32_t*>(&b);
                } else {
                    const __half2 a = __floats2half2_rn(S[k][0], S[k][1]), b = __floats2half2_rn(S[k][2], S[k][3]);
                    v.x = *reinterpret_cast<const uint32_t*>(&a); v.y = *reinterpret_cast<const uint32_t*>(&b);
                }
                *reinterpret_cast<uint2*>(out + (size_t)e * 2) = v;
            }
        }
    }
}
__device__ __forceinline__ float load_elem(int dt, const char* p, uint32_t i) {
    return dt == HCCL_FP32 ? Elem<HCCL_FP32>::load(p, i) : dt == HCCL_BF16 ? Elem<HCCL_BF16>::load(p, i) : Elem<HCCL_FP16>::load(p, i);
}
__device__ __forceinline__ void store_elem(int dt, char* p, uint32_t i, float v) {
    if (dt == HCCL_FP32) Elem<HCCL_FP32>::store(p, i, v); else if (dt == HCCL_BF16) Elem<HCCL_BF16>::store(p, i, v); else Elem<HCCL_FP16>::store(p, i, v);
}
__device__ __forceinline__ uint32_t esize(int dt) { return dt == HCCL_FP32 ? 4u : 2u; }
// The compute warps' bounded wait, inlined: across a call the 32 running sums of every thread would be written to local
// memory and read back, once per piece (the L1 has little room left beside the stages, so from the L2).
__device__ __forceinline__ bool wait_inline(const ExecParams& p, uint32_t bar, uint32_t parity, unsigned long long budget_ns, uint32_t detail) {
    if (mbar_try_wait(bar, parity)) return true;
    unsigned long long deadline = 0;
    for (uint32_t spins = 1;; ++spins) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spins & 31u) == 0) {
            if (aborted(p)) return false;
            const unsigned long long now = globaltimer_ns();
            if (deadline == 0) deadline = now + budget_ns;
            if (now > deadline) {
                fail(p, HCCL_ERR_TIMEOUT, detail);
                return false;
            }
        }
    }
}
// Bounded wait that does not look at the abort word (for loads that are in flight whatever happens to the execution).
__device__ __forceinline__ void mbar_wait_quiet(uint32_t bar, uint32_t parity, unsigned long long budget_ns) {
    if (mbar_try_wait(bar, parity)) return;
    const unsigned long long deadline = globaltimer_ns() + budget_ns;
    while (!mbar_try_wait(bar, parity) && globaltimer_ns() < deadline) {}
}

}  // namespace chainfw

using namespace chainfw;

// COPIES: the build that also forwards a chain's copies (ring AllReduce). A packet of sums alone (ring ReduceScatter)
// runs in the build without that code: the compiler is at its register limit here, and the extra paths cost the sums'
// loop 6 % (config 3: 0.73 against 0.69 ms).
template <bool COPIES>
__device__ __forceinline__ void executor_chain_body(const ExecParams& p, const uint32_t ns, const uint32_t stage_bytes) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) unsigned long long s_bar[2 * MAX_NS + 1];  // full, empty, and the compute warps' own barrier
    __shared__ Piece s_info[MAX_NS];
    __shared__ Step s_step[MAX_STEPS];
    __shared__ char* s_cdst[MAX_NS][MAX_CDST];  // K_C: where the piece in each stage is copied to
    const uint32_t tid = threadIdx.x;
    const uint32_t stages = smem_u32(smem), full = smem_u32(s_bar), empty = full + 8 * MAX_NS, cbar = empty + 8 * MAX_NS;
    if (tid == 0) {
        for (uint32_t s = 0; s < ns; ++s) {
            mbar_init(full + 8 * s, 1);
            mbar_init(empty + 8 * s, CW);
        }
        mbar_init(cbar, CW);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    init_epoch(p);  // ends with __syncthreads
    const unsigned long long long_wait = 2 * p.timeout_ns + 1000000000ull;
    const bool lean = p.trig_set_slot < 0;

    if (tid >= 32) {
        // ------------------------------------------------------------ compute warps
        const uint32_t ctid = tid - 32, lane = tid & 31u;
        const unsigned long long pol_keep = policy_evict_last();
        float S[G][4];
        float s_tail = 0.f;  // this thread's scalar element of the piece, if it has one
#pragma unroll
        for (int k = 0; k < G; ++k)
#pragma unroll
            for (int j = 0; j < 4; ++j) S[k][j] = 0.f;
        uint32_t cpar = 0;  // phase parity of the compute warps' barrier
        for (uint32_t slot = 0, parity = 0;;) {
            if (!wait_inline(p, full + 8 * slot, parity, long_wait, 0xfffffff7u)) break;
            const Piece pi = s_info[slot];
            if (pi.kind == K_EXIT) {
                if (ctid == 0) {  // the bulk copies of the chains' last pieces must have arrived, not only have left the stages
                    bulk_wait_all();
                    fence_proxy_async();
                }
                if (!lean) __threadfence();
                __syncwarp();
                if (lane == 0) mbar_arrive(empty + 8 * slot);  // tells the DMA thread that everything is stored
                break;
            }
            const char* stage = (const char*)smem + (size_t)slot * stage_bytes;
            // the piece: `head` scalar elements up to the first 16-byte boundary, nv elements in 16-byte groups, the rest scalar again;
            // thread ctid < edge keeps scalar element number ei
            const uint32_t head = pi.head, nv = (pi.n - head) & ~7u, edge = pi.n - nv, ei = ctid < head ? ctid : nv + ctid;
            char* const body = pi.dst + (size_t)head * esize(pi.dt_dst);  // K_B, K_C: where the 16-byte groups go
            if (pi.kind == K_A) {
                if (pi.dt_src == HCCL_FP32) take<HCCL_FP32>(stage, nv, ctid, S);
                else if (pi.dt_src == HCCL_BF16) take<HCCL_BF16>(stage, nv, ctid, S);
                else take<HCCL_FP16>(stage, nv, ctid, S);
                if (ctid < edge) s_tail = load_elem(pi.dt_src, pi.src0, ei);
            } else if (pi.kind == K_B) {
                if (pi.dt_src == HCCL_FP32) accumulate<HCCL_FP32>(stage, nv, ctid, S);
                else if (pi.dt_src == HCCL_BF16) accumulate<HCCL_BF16>(stage, nv, ctid, S);
                else accumulate<HCCL_FP16>(stage, nv, ctid, S);
                if (pi.dt_dst == HCCL_FP32) {
                    if (pi.keep) store_all<HCCL_FP32, true>(body, nv, ctid, S, pol_keep); else store_all<HCCL_FP32, false>(body, nv, ctid, S, pol_keep);
                } else if (pi.dt_dst == HCCL_BF16) {
                    store_all<HCCL_BF16, false>(body, nv, ctid, S, pol_keep);
                } else {
                    store_all<HCCL_FP16, false>(body, nv, ctid, S, pol_keep);
                }
                if (ctid < edge) {
                    s_tail = s_tail + load_elem(pi.dt_src, pi.src0, ei);
                    store_elem(pi.dt_dst, pi.dst, ei, s_tail);
                }
                if (pi.discard) {
                    // whole 128-byte lines inside the partial that a re-reading engine would have read here for the last time
                    const uintptr_t lo = ((uintptr_t)pi.discard + 127u) & ~(uintptr_t)127u, hi = ((uintptr_t)pi.discard + (size_t)pi.n * 4) & ~(uintptr_t)127u;
                    for (uintptr_t a = lo + (uintptr_t)ctid * 128u; a < hi; a += (uintptr_t)CTH * 128u) discard_line((const void*)a);
                }
                if (pi.last && p.trace && ctid == 0) trace_put(p.trace, p.trace_cap, pi.item, 3, globaltimer_ns());
            } else if (COPIES && pi.kind == K_C) {
                // a copy of what this block holds, stored from the registers (chains with few copies)
                if (pi.dt_dst == HCCL_FP32) store_all<HCCL_FP32, false>(body, nv, ctid, S, pol_keep);
                else if (pi.dt_dst == HCCL_BF16) store_all<HCCL_BF16, false>(body, nv, ctid, S, pol_keep);
                else store_all<HCCL_FP16, false>(body, nv, ctid, S, pol_keep);
                if (ctid < edge) store_elem(pi.dt_dst, pi.dst, ei, s_tail);
                if (pi.last && p.trace && ctid == 0) trace_put(p.trace, p.trace_cap, pi.item, 3, globaltimer_ns());
            } else if (COPIES && pi.kind == K_CM) {
                // The chain's copies: the held values, rounded to the copies' type, go into this piece's stage (which no load
                // uses) once; one thread then stores the stage to every destination with cp.async.bulk. One piece for all
                // the copies of a long chain: between two pieces the compute warps wait, which costs as much as storing a copy
                // (with few copies the trip through shared memory and the barrier cost more than that: FP32 R = 4 +13 %, R = 8 +5 %;
                // bf16 R = 8 -6 %, R = 64 -8 %).
                const uint32_t nd = pi.ndst, ed = esize(pi.dt_dst);
                char* const out = (char*)smem + (size_t)slot * stage_bytes;
                if (pi.dt_dst == HCCL_FP32) stage_all<HCCL_FP32>(out, nv, ctid, S);
                else if (pi.dt_dst == HCCL_BF16) stage_all<HCCL_BF16>(out, nv, ctid, S);
                else stage_all<HCCL_FP16>(out, nv, ctid, S);
                if (ctid < edge)
                    for (uint32_t j = 0; j < nd; ++j) store_elem(pi.dt_dst, s_cdst[slot][j], ei, s_tail);
                // the copies end the chain: what follows is another chain's first operand, and the sums need not be kept
                s_tail = 0.f;
#pragma unroll
                for (int k = 0; k < G; ++k)
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) S[k][jj] = 0.f;
                fence_proxy_async();  // this thread's writes to the stage, before the bulk copies read it
                __syncwarp();
                if (lane == 0) mbar_arrive(cbar);
                if (!wait_inline(p, cbar, cpar, long_wait, 0xfffffff2u)) break;
                cpar ^= 1u;
                if (ctid == 0) {
                    if (nv) {
                        for (uint32_t j = 0; j < nd; ++j) bulk_store_part(s_cdst[slot][j] + (size_t)head * ed, smem_u32(out), nv * ed, false, 0);
                        bulk_commit();
                        bulk_wait_read(0);  // the stage is read out: it may be given away (this warp's arrival below)
                    }
                    if (pi.last && p.trace)
                        for (uint32_t j = 0; j < nd; ++j) trace_put(p.trace, p.trace_cap, pi.item + j, 3, globaltimer_ns());
                }
            } else if (COPIES && pi.kind == K_RM) {
                // a piece of a chain of copies: the stage holds the source's bytes; one thread stores it to every destination
                const uint32_t nd = pi.ndst, hb = pi.head, nvb = (pi.n - hb) & ~15u, eb = pi.n - nvb, bi = ctid < hb ? ctid : nvb + ctid;
                if (ctid < eb) {
                    const char v = __ldcg(pi.src0 + bi);
                    for (uint32_t j = 0; j < nd; ++j) s_cdst[slot][j][bi] = v;
                }
                if (ctid == 0) {
                    if (nvb) {
                        for (uint32_t j = 0; j < nd; ++j) bulk_store_part(s_cdst[slot][j] + hb, smem_u32(stage), nvb, false, 0);
                        bulk_commit();
                        bulk_wait_read(0);
                    }
                    if (pi.last && p.trace)
                        for (uint32_t j = 0; j < nd; ++j) trace_put(p.trace, p.trace_cap, pi.item + j, 3, globaltimer_ns());
                }
            } else {  // K_ITEM: the whole item through the register path; items of a chain follow each other in this block
                // the item before must be stored by all compute threads. A bounded wait on an mbarrier, not a named barrier:
                // a warp that has left an aborted execution would leave the others waiting at one for ever
                __syncwarp();
                if (lane == 0) mbar_arrive(cbar);
                if (!wait_inline(p, cbar, cpar, long_wait, 0xfffffff3u)) break;
                cpar ^= 1u;
                const Tile t = p.tiles[pi.item];
                run_tile_lsu<false>(p, p.descs[t.desc], t, ctid, CTH);
                // nothing is forwarded out of an item that ran this way (and the sums need not survive the call)
                s_tail = 0.f;
#pragma unroll
                for (int k = 0; k < G; ++k)
#pragma unroll
                    for (int j = 0; j < 4; ++j) S[k][j] = 0.f;
                if (p.trace && ctid == 0) trace_put(p.trace, p.trace_cap, pi.item, 3, globaltimer_ns());
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(empty + 8 * slot);
            if (++slot == ns) {
                slot = 0;
                parity ^= 1u;
            }
        }
        return;
    }

    // ------------------------------------------------------------ warp 0: DMA thread (lane 0) and the step table (all lanes)
    const uint32_t lane = tid;
    const unsigned long long pol = policy_evict_first();
    uint32_t first = 0, end = 0;
    chain_range(p, first, end);
    end = min(end, p.n_tiles);
    bool ok = true;
    if (lane == 0) {
        if (p.trig_wait_slot >= 0)
            ok = wait_signal(p, p.user_signals + p.trig_wait_slot, p.trig_cmp, p.trig_wait_value + (unsigned long long)g_epoch * p.trig_wait_per_epoch, 0xffffffffu);
        if (ok && aborted(p)) ok = false;
        if (first == 0 && first < end) p.ctl->t_first_ns = globaltimer_ns();
    }
    ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    uint32_t slot = 0, parity = 0;    // next stage to fill and the phase parity of this use of it
    unsigned long long issued = 0;
    // lane 0: make stage `slot` free for a new piece
    auto acquire = [&]() -> bool {
        if (issued >= ns && !mbar_wait(p, empty + 8 * slot, parity ^ 1u, long_wait, 0xfffffff6u)) return false;
        return true;
    };
    auto advance = [&]() {
        ++issued;
        if (++slot == ns) {
            slot = 0;
            parity ^= 1u;
        }
    };
    const uint32_t L = p.chain_len;
    for (uint32_t base = first; ok && L > 0 && base < end; base += L) {
        // ---- the chain's steps: records fetched, checked and resolved by the warp's lanes
        bool good = true, fast = L <= MAX_STEPS;  // a longer chain runs item by item
        for (uint32_t t0 = 0; t0 < L && good; t0 += 32) {
            const uint32_t t = t0 + lane;
            bool g = true, f = true;
            if (t < L) {
                const uint32_t item = base + t;
                Step st;
                st.item = item;
                st.flags = 0;
                st.n = 0;
                st.dst = nullptr; st.a = nullptr; st.b = nullptr;
                st.dt_a = st.dt_b = st.dt_dst = 0;
                const Tile tl = p.tiles[item];
                g = tile_ok(p, tl) && !(tl.flags & TILE_FLAG_END);
                if (g) {
                    const Desc d = p.descs[tl.desc];
                    g = desc_ok(p, d);
                    if (g) {
                        st.flags = S_OK;
                        st.n = tl.count;
                        st.dt_a = d.dt_a; st.dt_b = d.dt_b; st.dt_dst = d.dt_dst;
                        if (COPIES && d.op == HCCL_OP_COPY) {
                            // a copy of what the step before stored (a ring's AllGather hops): the block stores what it holds again
                            // ... or, at the head of a chain of copies alone, of a send buffer (a hop-by-hop AllGather): bytes, not values
                            f = d.ndst <= 1 && (t > 0 || d.kind_a == HCCL_BUF_SEND);
                            st.flags |= S_COPY;
                            st.dst = buf_base(p, d.kind_dst, d.rank_dst) + d.off_dst + tl.start;
                            st.a = buf_base(p, d.kind_a, d.rank_a) + d.off_a + tl.start;
                            st.n = tl.count;  // bytes for now; elements once the type of the held values is known (below)
                            // (its element size is known only from the step before: the phase is checked below)
                        } else {
                            f = d.op == HCCL_OP_REDUCE && d.kind_b == HCCL_BUF_SEND;
                        }
                        if (f && d.op == HCCL_OP_REDUCE) {
                            st.dst = buf_base(p, d.kind_dst, d.rank_dst) + d.off_dst + tl.start * esize(d.dt_dst);
                            st.a = buf_base(p, d.kind_a, d.rank_a) + d.off_a + tl.start * esize(d.dt_a);
                            st.b = buf_base(p, d.kind_b, d.rank_b) + d.off_b + tl.start * esize(d.dt_b);
                            const uint32_t ph = phase_of(st.b, esize(d.dt_b));
                            f = whole_elements(st.b, esize(d.dt_b)) && whole_elements(st.dst, esize(d.dt_dst)) && phase_of(st.dst, esize(d.dt_dst)) == ph &&
                                (t > 0 || (whole_elements(st.a, esize(d.dt_a)) && phase_of(st.a, esize(d.dt_a)) == ph));
                            if (t == 0 && (d.kind_a != HCCL_BUF_SEND || PIECE * esize(d.dt_a) > stage_bytes)) f = false;
                            if (PIECE * esize(d.dt_b) > stage_bytes) f = false;  // the launch sized the stages for 16-bit operands
                            if (d.kind_dst == HCCL_BUF_SCRATCH && d.dt_dst == HCCL_FP32) st.flags |= S_KEEP;
                            if ((d.cmp & HCCL_HINT_LAST_READ_A) && d.kind_a == HCCL_BUF_SCRATCH && d.dt_a == HCCL_FP32) st.flags |= S_DISCARD_A;
                        }
                    }
                }
                if (t < MAX_STEPS) s_step[t] = st;
            }
            good = __all_sync(0xffffffffu, g);
            fast = fast && __all_sync(0xffffffffu, f);
        }
        __syncwarp();
        bool raw_chain = false;
        if (good && fast) {
            // Every step after the first must take exactly what the step before stored: sums first (each takes an FP32 sum),
            // then copies of what the block holds, whose element type is that of the last sum's result. Checked by all lanes,
            // a step each (the one thread that issues the pieces has no time for a walk over every step of every chain).
            uint32_t first_copy = L;
            for (uint32_t t0 = 0; t0 < L; t0 += 32) {
                const uint32_t t = t0 + lane;
                const uint32_t copies = __ballot_sync(0xffffffffu, t < L && (s_step[t].flags & S_COPY));
                if (copies && first_copy == L) first_copy = t0 + (uint32_t)__ffs((int)copies) - 1u;
            }
            if (first_copy < L && L - first_copy > MAX_CDST) fast = false;  // (one piece takes all copies of a chain)
            const bool raw = first_copy == 0;  // copies alone: the bytes of the first source go to every destination
            raw_chain = raw;
            const uint32_t held_dt = first_copy >= 1 && first_copy < L ? s_step[first_copy - 1].dt_dst : 0;  // type of what the copies move
            const uint32_t held_n = first_copy >= 1 && first_copy < L ? s_step[first_copy - 1].n : 0;
            __syncwarp();
            for (uint32_t t0 = 0; t0 < L && fast; t0 += 32) {
                const uint32_t t = t0 + lane;
                bool f = true;
                if (raw && t < L) {
                    const Step& st = s_step[t];
                    f = (st.flags & S_COPY) && (((uintptr_t)st.dst ^ (uintptr_t)s_step[0].a) & 15u) == 0 && st.n == s_step[0].n &&
                        (t == 0 || st.a == s_step[t - 1].dst);
                } else if (t >= 1 && t < L) {
                    Step& st = s_step[t];
                    const Step& pv = s_step[t - 1];  // only fields that no lane rewrites are read from it (dst; for a sum also dt_dst, n)
                    f = st.a == pv.dst;
                    if (t < first_copy) {
                        f = f && !(st.flags & S_COPY) && st.dt_a == HCCL_FP32 && pv.dt_dst == HCCL_FP32 && st.n == pv.n &&
                            phase_of(st.b, esize(st.dt_b)) == phase_of(pv.dst, 4);
                    } else {
                        f = f && (st.flags & S_COPY) && st.n == held_n * esize(held_dt) && whole_elements(st.dst, esize(held_dt)) &&
                            phase_of(st.dst, esize(held_dt)) == phase_of(pv.dst, esize(held_dt));
                        st.dt_dst = (uint8_t)held_dt;
                        st.n = held_n;
                    }
                }
                fast = __all_sync(0xffffffffu, f);
            }
            __syncwarp();
        }
        if (lane == 0) {
            if (!good) {
                fail(p, HCCL_ERR_BAD_DESCRIPTOR, base);
                ok = false;
            } else if (!fast) {
                for (uint32_t t = 0; t < L && ok; ++t) {
                    if (!acquire()) { ok = false; break; }
                    Piece& pi = s_info[slot];
                    pi.kind = K_ITEM;
                    pi.item = base + t;
                    pi.n = 0;
                    if (p.trace) {
                        trace_put(p.trace, p.trace_cap, base + t, 0, (unsigned long long)(base + t) | ((unsigned long long)blockIdx.x << 32));
                        trace_put(p.trace, p.trace_cap, base + t, 1, globaltimer_ns());
                        trace_put(p.trace, p.trace_cap, base + t, 2, globaltimer_ns());
                    }
                    mbar_arrive(full + 8 * slot);
                    advance();
                }
            } else if (raw_chain) {
                // copies alone: a piece of the first source is loaded into a stage once and stored from there to the destination of
                // every copy of the chain (bytes as they are; the few before the first and behind the last 16-byte word by plain accesses)
                const uint32_t nb = s_step[0].n, hb0 = (16u - (uint32_t)((uintptr_t)s_step[0].a & 15u)) & 15u;
                for (uint32_t e0 = 0; e0 < nb && ok; e0 += stage_bytes) {
                    const uint32_t ne = min(stage_bytes, nb - e0), head = min(hb0, ne), nvb = (ne - head) & ~15u;
                    if (!acquire()) { ok = false; break; }
                    Piece& pr = s_info[slot];
                    pr.kind = K_RM;
                    pr.n = ne;
                    pr.item = s_step[0].item;
                    pr.head = (uint8_t)head;
                    pr.last = (e0 + ne == nb) ? 1 : 0;
                    pr.ndst = (uint16_t)L;
                    pr.src0 = s_step[0].a + e0;
                    for (uint32_t j = 0; j < L; ++j) {
                        s_cdst[slot][j] = s_step[j].dst + e0;
                        if (p.trace && e0 == 0) {
                            trace_put(p.trace, p.trace_cap, s_step[j].item, 0, (unsigned long long)s_step[j].item | ((unsigned long long)blockIdx.x << 32));
                            trace_put(p.trace, p.trace_cap, s_step[j].item, 1, globaltimer_ns());
                            trace_put(p.trace, p.trace_cap, s_step[j].item, 2, globaltimer_ns());
                        }
                    }
                    if (nvb) {
                        mbar_arrive_expect_tx(full + 8 * slot, nvb);
                        bulk_load(stages + slot * stage_bytes, s_step[0].a + e0 + head, nvb, full + 8 * slot, true, pol);
                    } else {
                        mbar_arrive(full + 8 * slot);
                    }
                    advance();
                }
            } else {
                const uint32_t n = s_step[0].n;
                const uint32_t h0 = (8u - phase_of(s_step[0].b, esize(s_step[0].dt_b))) & 7u;  // the same for every operand and piece of the chain
                for (uint32_t e0 = 0; e0 < n && ok; e0 += PIECE) {
                    const uint32_t ne = min(PIECE, n - e0), head = min(h0, ne), nv = (ne - head) & ~7u;
                    for (uint32_t t = 0; t < L && ok; ++t) {
                        const Step& st = s_step[t];
                        if (p.trace && e0 == 0) {
                            trace_put(p.trace, p.trace_cap, st.item, 0, (unsigned long long)st.item | ((unsigned long long)blockIdx.x << 32));
                            trace_put(p.trace, p.trace_cap, st.item, 1, globaltimer_ns());
                            trace_put(p.trace, p.trace_cap, st.item, 2, globaltimer_ns());
                        }
                        if (t == 0) {  // the chain's first operand, from a send buffer
                            if (!acquire()) { ok = false; break; }
                            Piece& pa = s_info[slot];
                            const uint32_t ea = esize(st.dt_a);
                            pa.kind = K_A;
                            pa.n = ne;
                            pa.item = st.item;
                            pa.dt_src = st.dt_a;
                            pa.src0 = st.a + (size_t)e0 * ea;
                            pa.head = (uint8_t)head;
                            if (nv) {
                                mbar_arrive_expect_tx(full + 8 * slot, nv * ea);
                                bulk_load(stages + slot * stage_bytes, st.a + (size_t)(e0 + head) * ea, nv * ea, full + 8 * slot, true, pol);
                            } else {
                                mbar_arrive(full + 8 * slot);
                            }
                            advance();
                        }
                        if (st.flags & S_COPY) {
                            // all copies from here on (nothing but copies follows a copy in a chain that got this far)
                            const uint32_t m = min(L - t, MAX_CDST);
                            if (!acquire()) { ok = false; break; }
                            Piece& pc = s_info[slot];
                            pc.n = ne;
                            pc.item = st.item;
                            pc.dt_dst = st.dt_dst;
                            pc.last = (e0 + ne == n) ? 1 : 0;
                            pc.head = (uint8_t)head;
                            // one piece per copy, from the registers: few copies, or values wider than the stages were sized for
                            if (m < (st.dt_dst == HCCL_FP32 ? CM_MIN32 : CM_MIN16) || PIECE * esize(st.dt_dst) > stage_bytes) {
                                pc.kind = K_C;
                                pc.dst = st.dst + (size_t)e0 * esize(st.dt_dst);
                                mbar_arrive(full + 8 * slot);
                                advance();
                                continue;
                            }
                            pc.kind = K_CM;
                            pc.ndst = (uint16_t)m;
                            for (uint32_t j = 0; j < m; ++j) {
                                s_cdst[slot][j] = s_step[t + j].dst + (size_t)e0 * esize(st.dt_dst);
                                if (p.trace && e0 == 0 && j > 0) {
                                    trace_put(p.trace, p.trace_cap, st.item + j, 0, (unsigned long long)(st.item + j) | ((unsigned long long)blockIdx.x << 32));
                                    trace_put(p.trace, p.trace_cap, st.item + j, 1, globaltimer_ns());
                                    trace_put(p.trace, p.trace_cap, st.item + j, 2, globaltimer_ns());
                                }
                            }
                            mbar_arrive(full + 8 * slot);
                            advance();
                            t += m - 1;
                            continue;
                        }
                        if (!acquire()) { ok = false; break; }
                        Piece& pb = s_info[slot];
                        const uint32_t eb = esize(st.dt_b), ed = esize(st.dt_dst);
                        pb.kind = K_B;
                        pb.n = ne;
                        pb.item = st.item;
                        pb.dt_src = st.dt_b;
                        pb.dt_dst = st.dt_dst;
                        pb.keep = (st.flags & S_KEEP) ? 1 : 0;
                        pb.last = (e0 + ne == n) ? 1 : 0;
                        pb.dst = st.dst + (size_t)e0 * ed;
                        pb.src0 = st.b + (size_t)e0 * eb;
                        pb.head = (uint8_t)head;
                        pb.discard = (t > 0 && (st.flags & S_DISCARD_A)) ? st.a + (size_t)e0 * 4 : nullptr;
                        if (nv) {
                            mbar_arrive_expect_tx(full + 8 * slot, nv * eb);
                            bulk_load(stages + slot * stage_bytes, st.b + (size_t)(e0 + head) * eb, nv * eb, full + 8 * slot, true, pol);
                        } else {
                            mbar_arrive(full + 8 * slot);
                        }
                        advance();
                    }
                }
            }
            if (ok && aborted(p)) ok = false;
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
    }
    if (lane != 0) return;
    if (ok && acquire()) {
        // the end marker; the compute warps answer on its `empty` barrier when all their stores are issued
        s_info[slot].kind = K_EXIT;
        mbar_arrive(full + 8 * slot);
        mbar_wait(p, empty + 8 * slot, parity, long_wait, 0xfffffff5u);
    } else {
        // given up (a failure is on record, or the execution was aborted): the compute warps leave at their next bounded
        // wait. Loads already issued still write into this block's stages: wait (bounded) for each of them to land.
        const unsigned long long back = issued < ns ? issued : ns;
        for (unsigned long long k = 0; k < back; ++k) {
            if (slot == 0) {
                slot = ns;
                parity ^= 1u;
            }
            --slot;
            mbar_wait_quiet(full + 8 * slot, parity, 2000000000ull);
        }
    }
    leave(p, lean);
}

__global__ void __launch_bounds__(32 + CTH, 1) hccl_executor_chain(const __grid_constant__ ExecParams p, const uint32_t ns, const uint32_t stage_bytes) {
    executor_chain_body<true>(p, ns, stage_bytes);
}
__global__ void __launch_bounds__(32 + CTH, 1) hccl_executor_chain_sums(const __grid_constant__ ExecParams p, const uint32_t ns, const uint32_t stage_bytes) {
    executor_chain_body<false>(p, ns, stage_bytes);
}

}  // namespace hccl
