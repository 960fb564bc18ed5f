// The bulk (TMA) engine's kernel.
#include "bulk.cuh"
#include "kernels.cuh"

namespace hccl {

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
        d.pol_keep = policy_evict_last();
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
    const unsigned long long pol_keep = policy_evict_last();
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
                                  stages_ptr + (size_t)slot * STAGE_BYTES + pi.b_off, pi.dst, pi.n, ctid, cnth, pi.keep_dst != 0, pol_keep);
            if (pi.discard_src) {
                // whole 128-byte lines inside the piece; issued before the item is published, so the slot's next
                // writer is ordered after them
                const uintptr_t lo = ((uintptr_t)pi.discard_src + 127u) & ~(uintptr_t)127u, hi = ((uintptr_t)pi.discard_src + pi.discard_bytes) & ~(uintptr_t)127u;
                for (uintptr_t a = lo + (uintptr_t)ctid * 128u; a < hi; a += (uintptr_t)cnth * 128u) discard_line((const void*)a);
            }
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

}  // namespace hccl
