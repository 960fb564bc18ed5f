// The bulk (TMA) engine's kernel.
#include "bulk.cuh"
#include "kernels.cuh"

namespace hccl {

__global__ void __launch_bounds__(512, 1) hccl_executor_bulk(const __grid_constant__ ExecParams p, const uint32_t ns, const uint32_t copy_by_warps,
                                                              const uint32_t stage_bytes) {
    using namespace bulk;
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ Prepared s_queue[QUEUE];
    __shared__ __align__(8) unsigned long long s_qbar[2 * QUEUE + 1];  // q_full[QUEUE], q_empty[QUEUE], control thread has left
    char* stages_ptr = reinterpret_cast<char*>(smem_raw);
    PieceInfo* info = reinterpret_cast<PieceInfo*>(stages_ptr + (size_t)ns * stage_bytes);
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(info + ns);  // full[ns], empty[ns]
    __shared__ __align__(8) unsigned long long s_stored[MAX_STAGES];  // per stage: every compute warp has stored its share of an item's last piece
    const uint32_t tid = threadIdx.x;
    const uint32_t ncw = (blockDim.x >> 5) - 3;  // compute warps: all but the DMA, control and publishing warps
    const uint32_t full = smem_u32(bars), empty = smem_u32(bars + ns);
    const uint32_t q_full = smem_u32(s_qbar), q_empty = smem_u32(s_qbar + QUEUE), ctl_left = smem_u32(s_qbar + 2 * QUEUE);
    // entry (control thread): first ticket, its tile record, the abort word and the execution number are loaded together
    uint32_t next0 = 0, abort0 = 0;
    Tile pre;
    bool pre_ok = false;
    const bool gated = p.trig_wait_slot >= 0;
    if (tid == 32) {
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
            mbar_init(empty + 8 * s, ncw + 1);   // every compute warp and the publishing warp
        }
        for (uint32_t q = 0; q < 2 * QUEUE + 1; ++q) mbar_init(q_full + 8 * q, 1);
        for (uint32_t s = 0; s < ns; ++s) mbar_init(smem_u32(s_stored) + 8 * s, ncw);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_proxy_async();
    }
    __syncthreads();
    const unsigned long long long_wait = 2 * p.timeout_ns + 1000000000ull;

    if (tid >= 32 && tid < 64) {
        // ------------------------------------------------------------ control thread
        if (tid != 32) return;
        bool live = true;
        uint32_t cur = next0;
        if (gated) {
            live = wait_signal(p, p.user_signals + p.trig_wait_slot, p.trig_cmp, p.trig_wait_value + (unsigned long long)g_epoch * p.trig_wait_per_epoch, 0xffffffffu);
            cur = p.static_tickets ? blockIdx.x : atomicAdd(&p.ctl->ticket, 1);
        }
        if (cur == 0) p.ctl->t_first_ns = globaltimer_ns();
        uint32_t qs = 0, qpar = 0;      // ring position of the next hand-over, phase parity of its barriers
        unsigned long long pushed = 0;
        // hand one record to the DMA thread; false if the DMA thread no longer takes any (failure or abort)
        auto push = [&](uint32_t kind, uint32_t item, const Tile* t, const Desc* ds) -> bool {
            if (pushed >= QUEUE && !mbar_wait(p, q_empty + 8 * qs, qpar ^ 1u, long_wait, 0xfffffffbu)) return false;
            Prepared& e = s_queue[qs];
            e.kind = kind;
            e.item = item;
            if (t) {
                e.t = *t;
                e.ds = *ds;
                e.waited = t->wait_cnt;
            }
            mbar_arrive(q_full + 8 * qs);  // release: the record is written
            ++pushed;
            if (++qs == QUEUE) {
                qs = 0;
                qpar ^= 1u;
            }
            return true;
        };
        bool first = true, consumer_alive = true;
        uint32_t left = p.quantum ? p.quantum - 1u : 0xffffffffu;  // claims this block may still make (opts.quantum)
        while (live) {
            if (cur >= p.n_tiles || (first && !gated ? abort0 == g_epoch : aborted(p))) break;
            // the next ticket is claimed before this item's records are waited for: its latency hides behind them
            uint32_t next = p.n_tiles;
            if (!p.static_tickets && left != 0) {
                --left;
                next = atomicAdd(&p.ctl->ticket, 1);
            }
            Tile t;
            Desc ds;
            const int what = control_item(p, cur, first && pre_ok ? &pre : nullptr, t, ds);
            first = false;
            if (what == 0) break;
            if (what == 2 && !push(Q_ITEM, cur, &t, &ds)) {
                consumer_alive = false;
                break;
            }
            cur = next;
        }
        if (consumer_alive) push(Q_STOP, 0xffffffffu, nullptr, nullptr);
        mbar_arrive(ctl_left);  // no ticket is claimed after this
        return;
    }

    if (tid < 32) {
        // ------------------------------------------------------------ DMA thread
        if (tid != 0) return;
        Dma d;
        d.ns = ns;
        d.sb = stage_bytes;
        d.lag = copy_by_warps ? ns : (ns > 2 ? ns - 2 : 1);
        d.copy_by_warps = copy_by_warps != 0;
        d.stages = smem_u32(stages_ptr);
        d.stages_ptr = stages_ptr;
        d.full = full;
        d.empty = empty;
        d.info = info;
        d.head = d.tail = d.groups = 0;
        d.head_slot = d.head_par = d.tail_slot = d.tail_par = 0;
        d.pol = policy_evict_first();
        d.pol_keep = policy_evict_last();
        d.ok = true;
        uint32_t qs = 0, qpar = 0;
        while (d.ok) {
            // next prepared item; while there is none, what is in flight is retired (a COPY item is published when
            // its last piece retires, and the control thread may be waiting for exactly that)
            bool got = mbar_try_wait(q_full + 8 * qs, qpar);
            if (!got) {
                const unsigned long long deadline = globaltimer_ns() + long_wait;
                uint32_t spins = 0;
                while (!(got = mbar_try_wait(q_full + 8 * qs, qpar))) {
                    if (d.tail < d.head) {
                        retire_one(p, d);
                        if (!d.ok) break;
                        continue;
                    }
                    if ((++spins & 31u) == 0) {
                        if (aborted(p)) break;
                        if (globaltimer_ns() > deadline) {
                            fail(p, HCCL_ERR_TIMEOUT, 0xfffffffau);
                            break;
                        }
                    }
                }
            }
            if (!got) break;
            const Prepared& e = s_queue[qs];
            if (e.kind == Q_STOP) break;
            const uint32_t cur = e.item;
            const Tile t = e.t;
            const Desc ds = e.ds;
            const bool waited = e.waited != 0;
            mbar_arrive(q_empty + 8 * qs);  // the record is in registers: its place may be refilled
            if (++qs == QUEUE) {
                qs = 0;
                qpar ^= 1u;
            }
            if (waited) fence_proxy_async();  // what the control thread's acquired counters cover must be visible to the bulk unit too
            if (!dma_issue(p, d, cur, t, ds)) break;
        }
        // wind down: finish what is in flight, release the compute warps, leave
        if (d.ok && !aborted(p)) drain(p, d);
        if (d.ok && !aborted(p)) {
            const unsigned long long kx = d.head;
            const uint32_t xslot = d.head_slot, xpar = d.head_par;
            issue_simple(p, d, PIECE_EXIT, 0xffffffffu, nullptr, nullptr);
            // every compute warp has passed the exit piece = all of this block's results are stored
            if (d.ok && d.head == kx + 1) mbar_wait(p, empty + 8 * xslot, xpar, long_wait, 0xfffffffcu);
        }
        if (!d.ok || aborted(p)) {
            // stop path: no load may still be writing into this block's shared memory when it exits
            uint32_t slot = d.tail_slot, par = d.tail_par;
            for (unsigned long long j = d.tail; j < d.head; ++j) {
                if (info[slot].kind == PIECE_COPY || info[slot].kind == PIECE_REDUCE || info[slot].kind == PIECE_COPYW)
                    mbar_wait(p, full + 8 * slot, par, 1000000000ull, 0xfffffffeu);
                if (++slot == ns) {
                    slot = 0;
                    par ^= 1u;
                }
            }
        }
        bulk_wait_all();
        // the control thread must have claimed its last ticket before the block's verdict is given (the last block
        // out resets the ticket); on the stop path it notices the abort within a few polls
        {
            const unsigned long long deadline = globaltimer_ns() + 2 * long_wait;
            while (!mbar_try_wait(ctl_left, 0) && globaltimer_ns() < deadline) {
            }
        }
        leave(p, p.trig_set_slot < 0);
        return;
    }

    const uint32_t cnth = ncw * 32;
    if (tid >= 64 && tid < 96) {
        // ------------------------------------------------------------ publishing thread
        // Follows the pieces like a compute warp but moves no data: after the last piece of an item it waits (bounded)
        // on the stage's `stored` barrier until every compute warp has stored its share, and publishes the item's
        // completion. The release has to wait for those stores to be performed, a microsecond or two that no
        // data-moving warp spends this way; it is cumulative over the stores that the barrier ordered before this
        // thread. A stage is recycled only after every warp, this one included, has left it, so a `stored`
        // barrier never sees two items at once.
        if (tid != 64) return;
        const uint32_t stored = smem_u32(s_stored);
        uint32_t stored_parity = 0;  // bit s: phase parity of stage s's `stored` barrier (advances only when it is used)
        for (uint32_t slot = 0, parity = 0;;) {
            if (!mbar_wait(p, full + 8 * slot, parity, long_wait, 0xfffffff9u)) break;
            const PieceInfo& pi = info[slot];
            const uint32_t kind = pi.kind, last = pi.last;
            const int32_t sig0 = pi.signal[0], sig1 = pi.signal[1];
            if (kind != PIECE_EXIT && kind != PIECE_COPY && last && (sig0 >= 0 || sig1 >= 0)) {
                if (!mbar_wait(p, stored + 8 * slot, (stored_parity >> slot) & 1u, long_wait, 0xfffffff8u)) break;
                stored_parity ^= 1u << slot;
                if (sig0 >= 0) red_release_add_u32(p.counters + sig0, 1);
                if (sig1 >= 0) red_release_add_u32(p.counters + sig1, 1);
            }
            mbar_arrive(empty + 8 * slot);
            if (kind == PIECE_EXIT) break;
            if (++slot == ns) {
                slot = 0;
                parity ^= 1u;
            }
        }
        return;
    }

    // ------------------------------------------------------------ compute warps
    const uint32_t ctid = tid - 96;
    const unsigned long long pol_keep = policy_evict_last();
    for (uint32_t slot = 0, parity = 0;;) {
        if (!mbar_wait(p, full + 8 * slot, parity, 2 * p.timeout_ns + 1000000000ull, 0xfffffffdu)) break;
        const PieceInfo& pi = info[slot];
        const uint32_t kind = pi.kind;
        if (kind == PIECE_EXIT) {
            __syncwarp();
            if ((tid & 31u) == 0) mbar_arrive(empty + 8 * slot);  // tells the DMA thread this warp has stored everything
            break;
        }
        if (kind == PIECE_REDUCE) {
            reduce_piece_dispatch(pi.dt_a, pi.dt_b, pi.dt_d, stages_ptr + (size_t)slot * stage_bytes,
                                  stages_ptr + (size_t)slot * stage_bytes + pi.b_off, pi.dst, pi.n, ctid, cnth, pi.keep_dst != 0, pol_keep);
            if (pi.discard_src) {
                // whole 128-byte lines inside the piece; issued before the item is published, so the slot's next
                // writer is ordered after them
                const uintptr_t lo = ((uintptr_t)pi.discard_src + 127u) & ~(uintptr_t)127u, hi = ((uintptr_t)pi.discard_src + pi.discard_bytes) & ~(uintptr_t)127u;
                for (uintptr_t a = lo + (uintptr_t)ctid * 128u; a < hi; a += (uintptr_t)cnth * 128u) discard_line((const void*)a);
            }
        } else if (kind == PIECE_COPYW) {
            const uint4* src = reinterpret_cast<const uint4*>(stages_ptr + (size_t)slot * stage_bytes);
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
            run_tile_lsu<false>(p, pi.desc, pi.tile, ctid, cnth);
        }
        if (kind != PIECE_COPY && pi.last && p.trace && ctid == 0) trace_put(p.trace, p.trace_cap, pi.tile_index, 3, globaltimer_ns());
        // the publishing thread waits on the stage's `stored` barrier for every compute warp's stores of an item's last piece
        const bool tell = kind != PIECE_COPY && pi.last && (pi.signal[0] >= 0 || pi.signal[1] >= 0);
        __syncwarp();
        if ((tid & 31u) == 0) {
            if (tell) mbar_arrive(smem_u32(s_stored) + 8 * slot);
            mbar_arrive(empty + 8 * slot);
        }
        if (++slot == ns) {
            slot = 0;
            parity ^= 1u;
        }
    }
}

}  // namespace hccl
