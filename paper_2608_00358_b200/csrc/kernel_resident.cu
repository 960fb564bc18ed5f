// The resident, doorbell-fed executor and the device-resident AllToAllv.
#include "kernels.cuh"

namespace hccl {

// ====================================================================== resident, doorbell-fed executor
// The register engine as a long-lived kernel (paper Sec. II-A.3 "express doorbells": the work request's
// write is the doorbell; Sec. V-B: re-enqueueing a cached work packet costs microseconds). The blocks stay
// resident and execute the bound plan once per doorbell ring. The doorbell is a 64-byte record in pinned,
// mapped HOST memory: the host rings by storing a larger request number, block 0 polls it, releases all
// blocks through a device-side word, and reports completion (and a failure verdict) back into the record.
// Every wait is bounded: the kernel leaves by itself after idle_ns without a ring, or when told to stop.

// Acquire at system scope: what the host wrote before it rang (the send buffers' contents among it) is
// ordered before everything this thread does afterwards, the release of the other blocks included.
__device__ __forceinline__ unsigned long long ld_sys_u64(const unsigned long long* p) {
    unsigned long long v;
    asm volatile("ld.acquire.sys.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_sys_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.release.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
// No ordering of its own: made visible to the host by the next release store.
__device__ __forceinline__ void st_sys_relaxed_u64(unsigned long long* p, unsigned long long v) {
    asm volatile("st.relaxed.sys.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
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
                    if (ok && ld_acquire_u32(&p.ctl->fail_epoch) == epoch - 1) {
                        // the verdict first, then (below) the exit code that makes the host look at it; `completed` is
                        // not advanced for a failed execution (a successful one was reported by its last block out)
                        st_sys_relaxed_u64(&db->status, p.ctl->status);
                        st_sys_relaxed_u64(&db->detail, p.ctl->detail);
                        ok = false;  // a failed execution leaves the counters inconsistent: stop serving
                    }
                }
                unsigned long long why = ok ? 0 : 3, t_seen = 0;
                if (ok) {
                    const unsigned long long deadline = globaltimer_ns() + idle_ns;
                    for (uint32_t polls = 0;; ++polls) {
                        // every look at the doorbell is a trip over the host link: the stop word gets one look in eight
                        if (ld_sys_u64(&db->request) > (unsigned long long)(epoch - first_epoch)) {
                            cmd = epoch;
                            t_seen = globaltimer_ns();
                            break;
                        }
                        if ((polls & 7u) == 7u) {
                            if (ld_sys_u64(&db->stop) != 0) { why = 1; break; }
                            if (globaltimer_ns() > deadline) { why = 2; break; }
                        }
                        __nanosleep(50);
                    }
                }
                if (cmd == 0) st_sys_u64(&db->exited, why);
                // release the other blocks: server_go carries the epoch to run, or all ones to leave
                asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(&p.ctl->server_go), "r"(cmd ? cmd : 0xffffffffu) : "memory");
                if (cmd) st_sys_relaxed_u64(&db->t_seen_ns, t_seen);  // off the path of the blocks that were just released
            } else {
                const unsigned long long deadline = globaltimer_ns() + idle_ns + 4 * p.timeout_ns + 4000000000ull;
                for (;;) {
                    const uint32_t go = ld_acquire_u32(&p.ctl->server_go);
                    if (go == epoch) { cmd = epoch; break; }
                    if (go == 0xffffffffu || globaltimer_ns() > deadline) break;
                    __nanosleep(20);
                }
            }
            s_cmd = cmd;
        }
        __syncthreads();
        if (s_cmd == 0) break;
        executor_lsu_body<true, true>(p);    // one execution: tickets, dependencies, data, completion stamp
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


// ====================================================================== device-side table builder (any R up to 256)
// The R x R count matrix does not fit shared memory beyond 64 ranks, and no block needs all of it: block s
// builds the tables of source rank s only. It reads rows 0..s of the counts (coalesced, from the L2): from the
// rows above its own it takes, per destination d, the rows that earlier sources send to d (= its receive
// displacement in Y_d) and the number of tiles those sources produce (= the index of its own first tile); its
// own row gives the send displacements and the tiles per segment, both by block-wide exclusive scans built from
// warp shuffles. No block waits for another one. Every block validates what it reads; the block of the last
// source also holds every destination's total and checks it against the receive capacities. A rejected matrix
// raises the abort word, so the executor launched behind this kernel moves nothing.

// Exclusive scan over the 256 threads of the block (one value per thread); *total = the sum. `s_w` holds 8 words.
__device__ __forceinline__ long long block_exclusive_scan(long long v, long long* s_w, long long* total) {
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const long long inc = warp_inclusive_scan(v, lane);
    if (lane == 31) s_w[warp] = inc;
    __syncthreads();
    long long before = 0, all = 0;
#pragma unroll
    for (uint32_t w = 0; w < 8; ++w) {
        const long long x = s_w[w];
        if (w < warp) before += x;
        all += x;
    }
    __syncthreads();
    *total = all;
    return before + inc - v;
}

__global__ void __launch_bounds__(256, 1) hccl_a2a_patch(const __grid_constant__ PatchParams q) {
    __shared__ long long s_w[8];
    __shared__ uint32_t s_tp[HCCL_MAX_RANKS + 1];   // exclusive prefix of this source's tiles per destination
    __shared__ long long s_bytes[HCCL_MAX_RANKS];   // bytes of segment (s, d)
    __shared__ int s_bad, s_live;
    const uint32_t R = q.R, s = blockIdx.x, d = threadIdx.x;
    init_epoch(q);
    if (d == 0) {
        s_bad = 0;
        bool live = true;
        if (q.trig_wait_slot >= 0)
            live = wait_signal(q, q.user_signals + q.trig_wait_slot, q.trig_cmp, q.trig_wait_value + (unsigned long long)g_epoch * q.trig_wait_per_epoch, 0xffffffffu);
        s_live = live ? 1 : 0;
    }
    __syncthreads();
    if (!s_live) return;   // the wait gave up (recorded by wait_signal) or the execution was aborted
    const long long T = (long long)q.tile_bytes, rb = (long long)q.row_bytes;
    // rows above this source's own: receive displacement of column d and tiles produced so far
    long long col = 0, tiles_before = 0, own = 0;
    bool bad = false;
    if (d < R) {
        for (uint32_t r = 0; r <= s; ++r) {
            const long long c = __ldcg(q.counts + (size_t)r * R + d);
            if (c < 0 || c > (1ll << 40)) { bad = true; break; }
            if (r < s) {
                col += c;
                tiles_before += (c * rb + T - 1) / T;
            } else {
                own = c;
            }
        }
    }
    if (bad) s_bad = 1;
    long long row_total, base_tiles, row_tiles;
    const long long sd = block_exclusive_scan(own, s_w, &row_total);           // send displacement, rows
    (void)block_exclusive_scan(tiles_before, s_w, &base_tiles);                // index of this source's first tile
    const long long my_tiles = (own * rb + T - 1) / T;
    const long long tp = block_exclusive_scan(my_tiles, s_w, &row_tiles);      // first tile of segment (s, d) within the row
    if (d == 0 && row_total > q.max_send_rows[s]) s_bad = 1;
    if (s == R - 1 && d < R && col + own > q.max_recv_rows[d]) s_bad = 1;
    if (d < R) {
        s_tp[d] = (uint32_t)tp;
        s_bytes[d] = own * rb;
    }
    if (d == 0) s_tp[R] = (uint32_t)row_tiles;
    __syncthreads();
    const long long cap = (long long)q.tile_cap - (long long)q.end_tiles;   // real items must leave room for the END markers
    if (s_bad || base_tiles + row_tiles > cap) {
        if (d == 0) fail(q, HCCL_ERR_BAD_DESCRIPTOR, (unsigned long long)s * R);
        return;
    }
    if (d < R) {
        Desc ds;
        memset(&ds, 0, sizeof(ds));
        ds.op = HCCL_OP_COPY;
        ds.kind_dst = HCCL_BUF_RECV;
        ds.kind_a = HCCL_BUF_SEND;
        ds.cmp = HCCL_HINT_READ_ONCE;
        ds.rank_dst = (uint16_t)d;
        ds.rank_a = (uint16_t)s;
        ds.off_dst = col * rb;
        ds.off_a = sd * rb;
        ds.count = own * rb;
        q.descs[(size_t)s * R + d] = ds;
        if (q.recvcounts_out) q.recvcounts_out[(size_t)d * R + s] = own;
        if (q.rdispls_out) q.rdispls_out[(size_t)d * R + s] = col;
    }
    // this source's tiles, spread over the block: tile j of the row belongs to the last destination whose prefix
    // is <= j (destinations with nothing to send share a prefix value with their successor and are skipped)
    for (uint32_t j = d; j < (uint32_t)row_tiles; j += blockDim.x) {
        uint32_t lo = 0, hi = R;
        while (hi - lo > 1) {
            const uint32_t mid = (lo + hi) >> 1;
            if (s_tp[mid] <= j) lo = mid; else hi = mid;
        }
        const unsigned long long start = (unsigned long long)(j - s_tp[lo]) * (unsigned long long)T;
        Tile t;
        t.desc = s * R + lo;
        t.count = (uint32_t)min((unsigned long long)T, (unsigned long long)s_bytes[lo] - start);
        t.start = start;
        t.signal[0] = t.signal[1] = -1;
        t.wait_off = 0;
        t.wait_cnt = 0;
        t.flags = TILE_FLAG_NONE;
        q.tiles[(size_t)base_tiles + j] = t;
    }
    if (s == R - 1) {
        // behind the last item: END markers for every block's current and look-ahead claim
        const size_t n = (size_t)(base_tiles + row_tiles);
        for (uint32_t j = d; j < q.end_tiles; j += blockDim.x) {
            Tile t;
            memset(&t, 0, sizeof(t));
            t.signal[0] = t.signal[1] = -1;
            t.flags = TILE_FLAG_END;
            q.tiles[n + j] = t;
        }
    }
}

}  // namespace hccl
