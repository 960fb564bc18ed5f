// Collective planners: each turns a collective into a work packet of copy/reduce WQEs with
// dependencies (paper Sec. III-B.2; ring AllReduce example of Fig. 5; multiple rings with data
// sharded across them and AllToAllv spread over several subgraphs, Sec. IV-A; all-to-all style
// kernels, Sec. V-F), then compiles it.
#include <algorithm>
#include <cstring>
#include <memory>
#include <numeric>

#include "plan.hpp"

using namespace hccl;

namespace {

struct GraphDeleter {
    void operator()(hccl_graph* g) const { hccl_graph_destroy(g); }
};
using GraphPtr = std::unique_ptr<hccl_graph, GraphDeleter>;

hccl_ref_t ref(int kind, int rank, int64_t off) { return hccl_ref_t{kind, rank, off}; }

hccl_wqe_t blank() {
    hccl_wqe_t w;
    std::memset(&w, 0, sizeof(w));
    w.dep_wqe = -1;
    w.dep_wqe2 = -1;
    return w;
}

// One chain = one granule of one chunk travelling round the ring.
constexpr int64_t kForwardPieceElems = 14336;  // elements the forwarding kernel moves per step and block (kernel_chain.cu)

struct Chain {
    int c;            // chunk index = rank the reduced chunk ends on
    int64_t e0, len;  // element range [e0, e0+len) in the send buffers
    int64_t out_off;  // element offset of e0 inside Y_c for a scatter (AllReduce: == e0)
    int dir;          // +1: the chunk travels r -> r+1; -1: r -> r-1 (bidirectional rings)
};

#define CHECK(x)                         \
    do {                                 \
        hccl_status_t _s = (x);          \
        if (_s != HCCL_OK) return _s;    \
    } while (0)

// Emits the ring schedule for `chains`.
//   gather:  true = AllReduce (reduce-scatter then all-gather), false = ReduceScatter only
//   in_recv: FP32 AllReduce keeps partials in the chunk's slot of the acting rank's receive buffer;
//            otherwise FP32 partials live in a recycled ring of scratch slots.
// Issue order: groups of `group` chains; inside a group step by step, chain by chain, so that a
// tile's predecessor was handed out a whole group-step earlier and the group's partials fit the L2.
hccl_status_t emit_ring(hccl_graph* g, int R, int dt, const std::vector<Chain>& chains, bool gather, bool in_recv,
                        const hccl_opts_t& o, int64_t slot_elems, int n_slots, int64_t tile_elems, bool fused) {
    const int es = elem_bytes(dt);
    const size_t nch = chains.size();
    const bool level_major = (o.flags & HCCL_FLAG_LEVEL_MAJOR) != 0;
    const size_t group = level_major ? std::max<size_t>(nch, 1) : (size_t)o.chain_group;
    const bool staged = (o.flags & HCCL_FLAG_STAGED_RING) != 0 && !in_recv && !fused;
    std::vector<int32_t> sg(nch);
    std::vector<int64_t> last(nch, -1);        // last WQE emitted for each chain
    std::vector<int64_t> last_reduce(nch, -1); // last WQE of the chain that touches its scratch slot
    for (size_t i = 0; i < nch; ++i) CHECK(hccl_graph_add_subgraph(g, chains[i].c, &sg[i]));
    const int rs_steps = R - 1;
    const int ag_steps = gather ? R - 1 : 0;

    for (size_t g0 = 0; g0 < nch; g0 += group) {
        const size_t g1 = std::min(nch, g0 + group);
        const int steps = fused ? 1 + ag_steps : rs_steps + ag_steps;
        for (int step = 0; step < steps; ++step) {
            for (size_t i = g0; i < g1; ++i) {
                const Chain& ch = chains[i];
                const int c = ch.c;
                // (AllReduce: the partial sits at the element phase, modulo 8, of the rank buffers' range it belongs to, so that
                // all operands of a step reach a 16-byte boundary after the same number of elements; slots leave room for it)
                const int64_t slot = (int64_t)(i % (size_t)std::max(n_slots, 1)) * slot_elems * 4 + (gather ? (ch.e0 % 8) * 4 : 0);
                hccl_wqe_t w = blank();
                w.tile_count = tile_elems;
                if (last[i] >= 0) {
                    w.dep_flags = HCCL_DEP_WQE_SYNC | HCCL_DEP_ELEMENTWISE;
                    w.dep_wqe = last[i];
                }
                const bool is_rs = fused ? step == 0 : step < rs_steps;
                if (is_rs && fused) {
                    // the whole chain as one multi-input sum, same order: X_{c+1}, X_{c+2}, ..., X_c
                    w.op = HCCL_OP_REDUCE_N;
                    w.hints = HCCL_HINT_READ_ONCE;
                    w.dtype_dst = w.dtype_a = dt;
                    w.nsrc = R;
                    w.a = ref(HCCL_BUF_SEND, (c + 1) % R, ch.e0 * es);
                    w.dst = ref(HCCL_BUF_RECV, c, ch.out_off * es);
                    w.count = ch.len;
                } else if (is_rs) {
                    const int t = step;
                    const int dir = ch.dir;
                    const int r = (((c + dir * (t + 2)) % R) + R) % R, pr = (((r - dir) % R) + R) % R;
                    const bool first = t == 0, final = t == rs_steps - 1;
                    w.op = HCCL_OP_REDUCE;
                    w.count = ch.len;
                    w.b = ref(HCCL_BUF_SEND, r, ch.e0 * es);
                    w.dtype_b = dt;
                    if (in_recv) {
                        w.dtype_dst = w.dtype_a = dt;
                        w.a = first ? ref(HCCL_BUF_SEND, pr, ch.e0 * es) : ref(HCCL_BUF_RECV, pr, ch.e0 * es);
                        w.dst = ref(HCCL_BUF_RECV, r, ch.e0 * es);
                    } else {
                        w.dtype_a = first ? dt : HCCL_FP32;
                        w.a = first ? ref(HCCL_BUF_SEND, pr, ch.e0 * es) : ref(HCCL_BUF_SCRATCH, 0, slot);
                        w.dtype_dst = final ? dt : HCCL_FP32;
                        w.dst = final ? ref(HCCL_BUF_RECV, c, ch.out_off * es) : ref(HCCL_BUF_SCRATCH, 0, slot);
                        if (final && !first && !staged) w.hints |= HCCL_HINT_LAST_READ_A;  // the chain's partial is dead after this step
                        if (first && !final && i >= (size_t)n_slots && last_reduce[i - n_slots] >= 0) {
                            // the slot is recycled: its previous user must have read it for the last time
                            w.dep_flags |= HCCL_DEP_WQE_SYNC;
                            if (w.dep_wqe < 0) {
                                w.dep_flags &= ~HCCL_DEP_ELEMENTWISE;
                                w.dep_wqe = last_reduce[i - n_slots];
                            } else {
                                w.dep_wqe2 = last_reduce[i - n_slots];
                            }
                        }
                        if (staged && !first) {
                            // Paper-style pair: transfer the predecessor's partial into this rank's staging
                            // slot, then add locally (A=A+B). With one memory the "transfer" is a copy.
                            const int64_t stage = ((int64_t)n_slots + (int64_t)(i % (size_t)n_slots)) * slot_elems * 4;
                            hccl_wqe_t cp = blank();
                            cp.op = HCCL_OP_COPY;
                            cp.tile_count = tile_elems * 4;
                            cp.count = ch.len * 4;
                            cp.a = ref(HCCL_BUF_SCRATCH, 0, slot);
                            cp.dst = ref(HCCL_BUF_SCRATCH, 0, stage);
                            cp.dep_flags = HCCL_DEP_WQE_SYNC | HCCL_DEP_ELEMENTWISE;
                            cp.dep_wqe = last[i];
                            int64_t cid;
                            CHECK(hccl_graph_add_wqe(g, sg[i], &cp, &cid));
                            w.a = ref(HCCL_BUF_SCRATCH, 0, stage);
                            w.dep_wqe = cid;
                        }
                    }
                } else {
                    const int u = fused ? step - 1 : step - rs_steps;
                    const int dst_rank = (((c + ch.dir * (u + 1)) % R) + R) % R, src_rank = (((c + ch.dir * u) % R) + R) % R;
                    w.op = HCCL_OP_COPY;
                    w.tile_count = tile_elems * es;
                    w.count = ch.len * es;
                    w.a = ref(HCCL_BUF_RECV, src_rank, ch.e0 * es);
                    w.dst = ref(HCCL_BUF_RECV, dst_rank, ch.e0 * es);
                }
                int64_t id;
                CHECK(hccl_graph_add_wqe(g, sg[i], &w, &id));
                last[i] = id;
                if (is_rs && !fused && !in_recv) last_reduce[i] = id;
            }
        }
    }
    return HCCL_OK;
}

// Tile size in elements for a ring schedule: `level_elems` elements are worked on by one ring step of all
// chains that run together, and a step should be about one tile per block (a chain advances one step per
// tile, so few, large tiles keep the dependency chain short). With opts.tile_bytes set, that many bytes
// of the widest operand.
int64_t pick_tile_elems(int64_t level_elems, const hccl_opts_t& o, int widest, int op, int64_t chain_len = 0) {
    if (o.tile_bytes) return std::max<int64_t>(64, (int64_t)(o.tile_bytes / (uint64_t)widest));
    const int64_t lo = op == HCCL_OP_REDUCE_N ? 1 << 10 : 4 << 10, hi = op == HCCL_OP_REDUCE_N ? 32 << 10 : 64 << 10;
    if (chain_len > 0 && op == HCCL_OP_REDUCE && o.engine == HCCL_ENGINE_LSU) {
        // Register engine (the bulk engine prefers tiles that are whole stages). Chains of one length: cut each into the same number of tiles so that a step of all chains is a whole
        // number of rounds of the blocks (one round if the tiles stay under the cap). Block b then tends to meet
        // tile b of every step, i.e. its own earlier work, instead of waiting for another block's.
        const int64_t chains = std::max<int64_t>(1, level_elems / chain_len);
        for (int64_t rounds = 1; rounds <= 64; ++rounds) {
            const int64_t per_chain = std::max<int64_t>(1, (int64_t)o.sm_budget * rounds / chains);
            const int64_t tile = ((chain_len + per_chain - 1) / per_chain + 63) / 64 * 64;
            if (tile <= hi) return std::max<int64_t>(tile, std::min<int64_t>(lo, (chain_len + 63) / 64 * 64));
        }
    }
    return default_tile(level_elems, o.sm_budget, 1, lo, hi, sweep_of(o, op));
}

// A ring with at least about one chain of tiles per SM does best in the forwarding kernel (bulk engine, static chains:
// running sums in registers, no partial read back). Measured against the register engine's static chains: AllReduce
// bf16 R=8 0.66 at 8 MiB per rank, a tie at 4 MiB, 1.10 at 1 MiB; FP32 R=4 0.74 at 8 MiB, 1.07 at 4 MiB; bf16 R=64 0.85 at
// 512 KiB, 1.44 at 128 KiB; ReduceScatter bf16 R=16 0.74 at 8 MiB, 0.95 at 2 MiB.
// (A ReduceScatter whose shards do not start on multiples of 8 elements stays where it was: a shard's place in the send
// buffers and its place in the receive buffer then differ in their position inside a 16-byte word, and the kernel would
// run such chains item by item through its few compute warps. An AllReduce has no such problem: the kernel starts
// every piece with the few elements before the first 16-byte boundary, the same number for all operands.)
bool ring_wants_forwarding(int R, int64_t count, bool fused, const hccl_opts_t& o, bool scatter = false, const int64_t* recvcounts = nullptr) {
    int64_t off = 0;
    for (int c = 0; c < R && scatter; ++c) {
        if (off % 8) return false;
        off = recvcounts ? off + recvcounts[c] : (int64_t)(((__int128)(c + 1) * count) / R);
    }
    if (o.chain_group != 0 || (o.flags & (HCCL_FLAG_DYNAMIC_TICKETS | HCCL_FLAG_LEVEL_MAJOR | HCCL_FLAG_STAGED_RING | HCCL_FLAG_BIDIRECTIONAL))) return false;
    return !fused && R > 2 && count * 4 <= (1ll << 30) && (count >= (1ll << 20) || (R >= 32 && count >= (1ll << 18)));
}

// Tile size for the forwarding kernel: the one with the shortest estimated makespan. A block runs its chains of tiles one
// after the other; a chain of `steps` steps over a tile of t elements costs steps x (pieces(t) x 0.45 us + t x 0.05 ns)
// plus about 4 us between two chains (fixed cost per piece and step, store time per element, and the fetch of the next
// chain's records; fitted to measurements: config 3, AllReduce bf16 R=64 x 8 MiB, R=8 x 16 MiB, R=16 x 4 MiB), and the
// blocks need ceil(chains / blocks) rounds. Candidates: every chain of the longest granule cut into k equal tiles.
int64_t forward_tile_elems(const std::vector<Chain>& chains, int blocks, int steps) {
    int64_t maxlen = 0;
    for (const Chain& c : chains) maxlen = std::max(maxlen, c.len);
    if (blocks <= 0 || maxlen <= 0) return kForwardPieceElems;
    double best = 0;
    int64_t best_tile = kForwardPieceElems;
    const int64_t kmax = std::min<int64_t>(4096, std::max<int64_t>(1, maxlen / 256));
    for (int64_t k = 1; k <= kmax; ++k) {
        const int64_t tile = ((maxlen + k - 1) / k + 7) / 8 * 8;
        int64_t n = 0;
        for (const Chain& c : chains) n += (c.len + tile - 1) / tile;
        const double pieces = (double)((tile + kForwardPieceElems - 1) / kForwardPieceElems);
        const double rounds = (double)((n + blocks - 1) / blocks);
        // (tiles of more than two pieces measured about 5 % slower per further piece than this sum: config 3 with 4 / 8 pieces
        // per tile 0.72-0.75 / 0.83 ms against 0.69 with two)
        const double cost = rounds * (steps * (pieces * 0.45 + (double)tile * 0.00005) + 4.0) * (1.0 + 0.05 * std::max(0.0, pieces - 2.0));
        if (best == 0 || cost < best * 0.999) {  // ties go to the larger tile (k grows)
            best = cost;
            best_tile = tile;
        }
    }
    return best_tile;
}

// Ring reductions: with the engine left to the library, large ones feed the adds from shared memory through
// the bulk copy unit (measured 15 % ahead at config 3's size: the loads no longer queue in the LSU), small,
// latency-bound ones stay on the register engine (shorter dependency hand-off).
void fill_ring_opts(hccl_opts_t* o, const hccl_opts_t* in, int64_t input_bytes, bool fused) {
    hccl_opts_t tmp;
    if (in) tmp = *in; else std::memset(&tmp, 0, sizeof(tmp));
    if (tmp.engine == HCCL_ENGINE_AUTO) tmp.engine = (!fused && input_bytes >= (256ll << 20)) ? HCCL_ENGINE_BULK : HCCL_ENGINE_LSU;
    // large multi-input sums are pure streams of loads: two 64-register blocks per SM keep twice the loads in
    // flight (measured 6.06 vs 5.78 TB/s at config 3's size)
    if (fused && tmp.engine == HCCL_ENGINE_LSU && tmp.sm_budget == 0 && tmp.light == 0 && tmp.threads == 0 && input_bytes >= (256ll << 20)) {
        tmp.light = 1;
        tmp.sm_budget = 296;
    }
    fill_default_opts(o, &tmp);
}

// Copy-only schedules: with the engine left to the library, the bulk copy unit moves the bytes
// (measured a few percent ahead of the register path at full budget, and no thread touches the data).
void fill_copy_opts(hccl_opts_t* o, const hccl_opts_t* in) {
    hccl_opts_t tmp;
    if (in) tmp = *in; else std::memset(&tmp, 0, sizeof(tmp));
    if (tmp.engine == HCCL_ENGINE_AUTO) tmp.engine = HCCL_ENGINE_BULK;
    fill_default_opts(o, &tmp);
    // With (nearly) every SM copying, the memory is the limit and three stages per block serve it better than four
    // (config 4: 7.57 vs 7.64 ms); with few blocks each one needs all the bytes in flight it can hold.
    if (o->engine == HCCL_ENGINE_BULK && o->stages == 0 && o->stage_kib == 0 && o->sm_budget >= 100) o->stages = 3;
}

// Chains per group for large rings: the FP32 partials of one group-step (chains x granule x 4 bytes) should fill
// about half the L2 (64 MiB): fewer chains leave a step with too few tiles for the blocks, more push the partials
// out of the L2 between two steps (R = 64 x 32 Mi bf16, granules of 512 Ki elements: 16 / 32 / 48 / 64 chains per
// group 6.5 / 3.5 / 4.3 / 4.3 ms; config 3, granules of 1 Mi: 8 / 16 / 24 chains 1.20 / 0.87 / 1.33 ms).
int32_t l2_chain_group(int64_t granule_elems, size_t n_chains) {
    const int64_t g = (64ll << 20) / std::max<int64_t>(granule_elems * 4, 1);
    return (int32_t)std::max<int64_t>(1, std::min<int64_t>(g, (int64_t)std::max<size_t>(n_chains, 1)));
}

std::vector<Chain> make_chains(int R, const std::vector<int64_t>& offs, bool scatter, int64_t granule_elems, bool bidirectional) {
    // chunk c = [offs[c], offs[c+1]); cut into granules; granule-major order so that consecutive chains
    // belong to different chunks (different final ranks) and a chain group spans the ring evenly
    std::vector<Chain> chains;
    int64_t maxlen = 0;
    for (int c = 0; c < R; ++c) maxlen = std::max(maxlen, offs[c + 1] - offs[c]);
    const int64_t ng = granule_elems > 0 ? (maxlen + granule_elems - 1) / granule_elems : 1;
    for (int64_t k = 0; k < ng; ++k) {
        for (int c = 0; c < R; ++c) {
            const int64_t lo = offs[c] + k * granule_elems, hi = std::min(offs[c + 1], lo + granule_elems);
            if (lo >= hi) continue;  // empty chunks and exhausted chunks are elided
            chains.push_back(Chain{c, lo, hi - lo, scatter ? lo - offs[c] : lo, (bidirectional && (k & 1)) ? -1 : 1});
        }
    }
    return chains;
}


// ---------------------------------------------------------------- two-level (rack-aware) schedules
// R = G racks of L ranks, rank (g, l) = g*L + l. One chain = one granule of one sub-chunk (j, k): chunk j of L,
// cut again into G parts. Stages of a chain, each one WQE per participating rack:
//   reduce inside every rack (L-1 steps, FP32 partial P_g in scratch), reduce across racks (G-1 steps,
//   accumulator Q in scratch, the last step rounds into Y of rank (k, j)), gather across racks (G-1 hops
//   between the ranks with local index j), gather inside every rack (L-1 hops). Only the middle two stages
//   move bytes between racks, and they move 1/L of the data.
struct Chain2 {
    int j, k;
    int64_t e0, len;
};

struct TwoLevel {
    hccl_graph* g;
    int G, L, dt, es;
    int64_t n;            // elements per rank buffer (AllReduce) / total gathered elements (AllGather)
    int64_t tile_elems;
    hccl_opts_t o;
    int rank(int rack, int local) const { return ((rack % G + G) % G) * L + ((local % L + L) % L); }
};

hccl_status_t add_dep_wqe(hccl_graph* g, int32_t sg, hccl_wqe_t& w, int64_t d1, int64_t d2, int64_t* id) {
    w.dep_flags = 0;
    w.dep_wqe = w.dep_wqe2 = -1;
    if (d1 < 0) { d1 = d2; d2 = -1; }
    if (d1 >= 0) {
        w.dep_flags = HCCL_DEP_WQE_SYNC | HCCL_DEP_ELEMENTWISE;
        w.dep_wqe = d1;
        if (d2 >= 0) {
            w.dep_wqe2 = d2;
            w.dep_flags |= HCCL_DEP_ELEMENTWISE2;
        }
    }
    return hccl_graph_add_wqe(g, sg, &w, id);
}

// Gather stages shared by AllReduce and AllGather: the data of a chain sits in Y of rank (k, j) at element
// offset `yoff` (produced by WQE `origin`); it hops to the other racks' rank j, and inside every rack round
// the local ring. `stage` selects which hop to emit (0 .. G-2 across racks, then G-1 .. G+L-3 inside racks).
struct GatherState {
    std::vector<int64_t> arrive;  // per rack: WQE that delivered the data to rank (rack, j)
    std::vector<int64_t> last;    // per rack: last intra-rack hop emitted
};

hccl_status_t emit_gather_stage(const TwoLevel& T, int32_t sg, const Chain2& ch, int64_t yoff_elems, int stage, GatherState& st) {
    const int G = T.G, es = T.es;
    hccl_wqe_t w = blank();
    w.op = HCCL_OP_COPY;
    w.count = ch.len * es;
    w.tile_count = T.tile_elems * es;
    if (stage < G - 1) {
        const int v = stage, src = T.rank(ch.k + v, ch.j), dst = T.rank(ch.k + v + 1, ch.j);
        w.a = ref(HCCL_BUF_RECV, src, yoff_elems * es);
        w.dst = ref(HCCL_BUF_RECV, dst, yoff_elems * es);
        int64_t id;
        CHECK(add_dep_wqe(T.g, sg, w, st.arrive[(ch.k + v) % G], -1, &id));
        st.arrive[(ch.k + v + 1) % G] = id;
        return HCCL_OK;
    }
    const int h = stage - (G - 1);
    for (int rack = 0; rack < G; ++rack) {
        const int src = T.rank(rack, ch.j + h), dst = T.rank(rack, ch.j + h + 1);
        w.a = ref(HCCL_BUF_RECV, src, yoff_elems * es);
        w.dst = ref(HCCL_BUF_RECV, dst, yoff_elems * es);
        int64_t id;
        CHECK(add_dep_wqe(T.g, sg, w, h == 0 ? st.arrive[rack] : st.last[rack], -1, &id));
        st.last[rack] = id;
    }
    return HCCL_OK;
}

hccl_status_t emit_allreduce_2level(const TwoLevel& T, const std::vector<Chain2>& chains) {
    const int G = T.G, L = T.L, dt = T.dt, es = T.es;
    const int64_t Pbytes = T.n * 4;                 // one FP32 image of the buffer per rack, then the accumulator
    auto P = [&](int rack, int64_t e) { return ref(HCCL_BUF_SCRATCH, 0, (int64_t)rack * Pbytes + e * 4); };
    auto Q = [&](int64_t e) { return ref(HCCL_BUF_SCRATCH, 0, (int64_t)G * Pbytes + e * 4); };
    const size_t nch = chains.size(), group = (size_t)T.o.chain_group;
    std::vector<int32_t> sg(nch);
    std::vector<std::vector<int64_t>> p_last(nch, std::vector<int64_t>(G, -1));  // last in-rack reduce per rack
    std::vector<int64_t> q_last(nch, -1);
    std::vector<GatherState> gs(nch);
    for (size_t i = 0; i < nch; ++i) {
        CHECK(hccl_graph_add_subgraph(T.g, T.rank(chains[i].k, chains[i].j), &sg[i]));
        gs[i].arrive.assign(G, -1);
        gs[i].last.assign(G, -1);
    }
    const int stages = (L - 1) + (G - 1) + (G - 1) + (L - 1);
    for (size_t g0 = 0; g0 < nch; g0 += group) {
        const size_t g1 = std::min(nch, g0 + group);
        for (int stage = 0; stage < stages; ++stage) {
            for (size_t i = g0; i < g1; ++i) {
                const Chain2& ch = chains[i];
                if (stage < L - 1) {
                    // sums round each rack's ring: local rank (j+t+2) adds its own data to the rack's partial
                    const int t = stage;
                    for (int rack = 0; rack < G; ++rack) {
                        const int l = (ch.j + t + 2) % L, r = T.rank(rack, l), pr = T.rank(rack, l - 1);
                        hccl_wqe_t w = blank();
                        w.op = HCCL_OP_REDUCE;
                        w.count = ch.len;
                        w.tile_count = T.tile_elems;
                        w.dtype_dst = HCCL_FP32;
                        w.dst = P(rack, ch.e0);
                        w.dtype_b = dt;
                        w.b = ref(HCCL_BUF_SEND, r, ch.e0 * es);
                        if (t == 0) { w.dtype_a = dt; w.a = ref(HCCL_BUF_SEND, pr, ch.e0 * es); }
                        else { w.dtype_a = HCCL_FP32; w.a = P(rack, ch.e0); }
                        CHECK(add_dep_wqe(T.g, sg[i], w, p_last[i][rack], -1, &p_last[i][rack]));
                    }
                } else if (stage < (L - 1) + (G - 1)) {
                    // sums round the ring of racks: rack (k+u+2) adds its partial
                    const int u = stage - (L - 1);
                    const int rk = (ch.k + u + 2) % G, prk = (rk + G - 1) % G;
                    const bool first = u == 0, final = u == G - 2;
                    hccl_wqe_t w = blank();
                    w.op = HCCL_OP_REDUCE;
                    w.count = ch.len;
                    w.tile_count = T.tile_elems;
                    w.dtype_a = w.dtype_b = HCCL_FP32;
                    w.a = first ? P(prk, ch.e0) : Q(ch.e0);
                    w.b = P(rk, ch.e0);
                    if (final) { w.dtype_dst = dt; w.dst = ref(HCCL_BUF_RECV, T.rank(ch.k, ch.j), ch.e0 * es); }
                    else { w.dtype_dst = HCCL_FP32; w.dst = Q(ch.e0); }
                    int64_t id;
                    CHECK(add_dep_wqe(T.g, sg[i], w, first ? p_last[i][prk] : q_last[i], p_last[i][rk], &id));
                    q_last[i] = id;
                    if (final) gs[i].arrive[ch.k] = id;
                } else {
                    CHECK(emit_gather_stage(T, sg[i], ch, ch.e0, stage - (L - 1) - (G - 1), gs[i]));
                }
            }
        }
    }
    return HCCL_OK;
}

std::vector<Chain2> make_chains2(int G, int L, int64_t n, int64_t granule) {
    std::vector<Chain2> out;
    for (int j = 0; j < L; ++j) {
        const int64_t lo = (int64_t)(((__int128)j * n) / L), hi = (int64_t)(((__int128)(j + 1) * n) / L);
        for (int k = 0; k < G; ++k) {
            const int64_t a = lo + (int64_t)(((__int128)k * (hi - lo)) / G), b = lo + (int64_t)(((__int128)(k + 1) * (hi - lo)) / G);
            for (int64_t e = a; e < b; e += granule) out.push_back(Chain2{j, k, e, std::min(granule, b - e)});
        }
    }
    return out;
}

hccl_status_t plan_allreduce_2level(int R, int64_t count, hccl_dtype_t dt, const hccl_opts_t& o_in, hccl_plan_t** out) {
    hccl_opts_t o = o_in;
    const int L = o.rack_size, G = R / L, es = elem_bytes(dt);
    // Up to 256 KiB per rank a block does better walking one tile through all of a chunk's steps by itself than the
    // blocks do handing it on through device counters (measured, bf16: R=64 in racks of 16 0.10-0.11 vs 0.16 ms, R=16
    // in racks of 4 0.027-0.039 vs 0.042-0.049 ms; from 512 KiB on the other way round: 0.23 vs 0.20 ms at 1 MiB).
    if (count * es <= (256ll << 10) && !(o.flags & HCCL_FLAG_DYNAMIC_TICKETS)) o.flags |= HCCL_FLAG_STATIC_CHAINS;
    std::vector<int64_t> ext(R, count * es);
    const int64_t granule = std::max<int64_t>(1, (int64_t)(o.chunk_bytes / (uint64_t)es));
    std::vector<Chain2> chains = make_chains2(G, L, count, granule);
    int64_t maxlen = 0;
    for (const Chain2& c : chains) maxlen = std::max(maxlen, c.len);
    hccl_graph* graw = nullptr;
    CHECK(hccl_graph_create(R, ext.data(), ext.data(), (int64_t)(G + 1) * count * 4, 0, &graw));
    GraphPtr g(graw);
    g->compulsory_bytes = 2ll * R * count * es;
    TwoLevel T{g.get(), G, L, (int)dt, es, count, 0, o};
    const int64_t level = std::min<int64_t>(count * G, (int64_t)o.chain_group * maxlen * G);
    T.tile_elems = pick_tile_elems(level, o, 4, HCCL_OP_REDUCE);
    CHECK(emit_allreduce_2level(T, chains));
    return hccl_graph_compile(g.get(), &o, out);
}


// Two-level AllGather: rank (g, j)'s block first lands in its own receive buffer, then travels to the other
// racks' rank j (the only hops between racks), and every rack passes it round its own ring.
hccl_status_t plan_allgather_2level(int R, const std::vector<int64_t>& offs, hccl_dtype_t dt, const hccl_opts_t& o_in, hccl_plan_t** out) {
    hccl_opts_t o = o_in;
    // all copies of one chunk (its trip round the racks and then round every rack) form one group of linked WQEs:
    // a block can walk a tile through all of them by itself
    if (!(o.flags & HCCL_FLAG_DYNAMIC_TICKETS)) o.flags |= HCCL_FLAG_STATIC_CHAINS;
    const int L = o.rack_size, G = R / L, es = elem_bytes(dt);
    std::vector<int64_t> sext(R), rext(R, offs[R] * es);
    for (int r = 0; r < R; ++r) sext[r] = (offs[r + 1] - offs[r]) * es;
    hccl_graph* graw = nullptr;
    CHECK(hccl_graph_create(R, sext.data(), rext.data(), 0, 0, &graw));
    GraphPtr g(graw);
    g->compulsory_bytes = offs[R] * es + (int64_t)R * offs[R] * es;
    const int64_t granule = std::max<int64_t>(1, (int64_t)(o.chunk_bytes / (uint64_t)es));
    struct Item { Chain2 ch; int64_t src_off; };
    std::vector<Item> items;
    for (int64_t k0 = 0;; ++k0) {  // granule-major, so that consecutive chains start on different ranks
        bool any = false;
        for (int q = 0; q < R; ++q) {
            const int64_t lo = offs[q] + k0 * granule;
            if (lo >= offs[q + 1]) continue;
            any = true;
            items.push_back(Item{Chain2{q % L, q / L, lo, std::min(granule, offs[q + 1] - lo)}, lo - offs[q]});
        }
        if (!any) break;
    }
    TwoLevel T{g.get(), G, L, (int)dt, es, offs[R], 0, o};
    T.tile_elems = o.tile_bytes ? std::max<int64_t>(1, (int64_t)(o.tile_bytes / (uint64_t)es))
                                : default_tile(std::min<int64_t>(offs[R], (int64_t)o.chain_group * granule) * G * es, o.sm_budget, 1, 16 << 10,
                                               o.engine == HCCL_ENGINE_LSU ? 3 * sweep_of(o, HCCL_OP_COPY) : (256 << 10), sweep_of(o, HCCL_OP_COPY)) / es;
    T.tile_elems = std::max<int64_t>(T.tile_elems, 1);
    const size_t nch = items.size(), group = (size_t)o.chain_group;
    std::vector<int32_t> sg(nch);
    std::vector<GatherState> gs(nch);
    for (size_t i = 0; i < nch; ++i) {
        CHECK(hccl_graph_add_subgraph(g.get(), T.rank(items[i].ch.k, items[i].ch.j), &sg[i]));
        gs[i].arrive.assign(G, -1);
        gs[i].last.assign(G, -1);
    }
    const int stages = 1 + (G - 1) + (L - 1);
    if (o.flags & HCCL_FLAG_STATIC_CHAINS) {
        // One block will run an item's copies in this order: own copy, the hops round the racks, then rack by
        // rack the hops round that rack, so that every hop reads what the hop just before it wrote.
        for (size_t i = 0; i < nch; ++i) {
            const Chain2& ch = items[i].ch;
            hccl_wqe_t w = blank();
            w.op = HCCL_OP_COPY;
            w.count = ch.len * es;
            w.tile_count = T.tile_elems * es;
            const int r0 = T.rank(ch.k, ch.j);
            w.a = ref(HCCL_BUF_SEND, r0, items[i].src_off * es);
            w.dst = ref(HCCL_BUF_RECV, r0, ch.e0 * es);
            CHECK(hccl_graph_add_wqe(g.get(), sg[i], &w, &gs[i].arrive[ch.k]));
            for (int stage = 0; stage < G - 1; ++stage) CHECK(emit_gather_stage(T, sg[i], ch, ch.e0, stage, gs[i]));
            for (int rack = 0; rack < G; ++rack) {
                int64_t prev = gs[i].arrive[rack];
                for (int h = 0; h < L - 1; ++h) {
                    hccl_wqe_t c = blank();
                    c.op = HCCL_OP_COPY;
                    c.count = ch.len * es;
                    c.tile_count = T.tile_elems * es;
                    c.a = ref(HCCL_BUF_RECV, T.rank(rack, ch.j + h), ch.e0 * es);
                    c.dst = ref(HCCL_BUF_RECV, T.rank(rack, ch.j + h + 1), ch.e0 * es);
                    CHECK(add_dep_wqe(g.get(), sg[i], c, prev, -1, &prev));
                }
            }
        }
        return hccl_graph_compile(g.get(), &o, out);
    }
    for (size_t g0 = 0; g0 < nch; g0 += group) {
        const size_t g1 = std::min(nch, g0 + group);
        for (int stage = 0; stage < stages; ++stage) {
            for (size_t i = g0; i < g1; ++i) {
                const Chain2& ch = items[i].ch;
                if (stage == 0) {
                    hccl_wqe_t w = blank();
                    w.op = HCCL_OP_COPY;
                    w.count = ch.len * es;
                    w.tile_count = T.tile_elems * es;
                    const int r = T.rank(ch.k, ch.j);
                    w.a = ref(HCCL_BUF_SEND, r, items[i].src_off * es);
                    w.dst = ref(HCCL_BUF_RECV, r, ch.e0 * es);
                    CHECK(hccl_graph_add_wqe(g.get(), sg[i], &w, &gs[i].arrive[ch.k]));
                } else {
                    CHECK(emit_gather_stage(T, sg[i], ch, ch.e0, stage - 1, gs[i]));
                }
            }
        }
    }
    return hccl_graph_compile(g.get(), &o, out);
}

// Binary-tree AllReduce built from the two-input sum alone (Sec. III-B.2 names tree-based NMC reductions):
// per granule, neighbours are added in pairs level by level (an odd one out moves up unchanged) with FP32
// partials in scratch, the root is rounded into rank 0's receive buffer, and a binomial tree of copies
// carries it to every rank. Depth 2*ceil(log2 R) instead of the ring's 2(R-1).
hccl_status_t plan_allreduce_tree(int R, int64_t count, hccl_dtype_t dt, hccl_opts_t o, bool group_given, hccl_plan_t** out) {
    const int es = elem_bytes(dt);
    std::vector<int64_t> ext(R, count * es);
    const int64_t granule = std::max<int64_t>(64, (int64_t)(o.chunk_bytes / (uint64_t)es) / 64 * 64);
    const int64_t ng = count > 0 ? (count + granule - 1) / granule : 0;
    if (!group_given && count * 4 <= (32ll << 20)) o.chain_group = (int32_t)std::max<int64_t>(ng, 1);  // small: all granules together
    const int64_t group = std::max<int64_t>(1, o.chain_group);
    // From about 1 MiB per rank (any size up to 8 ranks) a block does better walking one tile through the whole tree by
    // itself (no hand-over between SMs, 2(R-1) items in a row at about 0.7 us each) than the blocks do sharing the
    // tree's 2 log2 R levels at about 2.5 us per hand-over through a device counter; below that the levels' parallelism
    // wins (measured per execution from a CUDA graph at R = 8: 12.7 vs 15.3 us at 4 KiB, 18.0 vs 19.0 at 64 KiB, 18.1
    // vs 22.7 at 256 KiB, 18.5 vs 38.1 at 1 MiB; at R = 64 and 128 KiB 0.148 vs 0.058 ms).
    if ((R <= 8 || count * es >= (1ll << 20)) && !(o.flags & HCCL_FLAG_DYNAMIC_TICKETS)) o.flags |= HCCL_FLAG_STATIC_CHAINS;
    const int half = (R + 1) / 2;                                 // scratch slots one granule needs
    const int64_t n_sets = std::min<int64_t>(std::max<int64_t>(ng, 1), 2 * group);  // recycled sets of slots
    const int64_t slot_elems = (int64_t)align_up((uint64_t)std::min<int64_t>(granule, std::max<int64_t>(count, 1)), 64);
    const int64_t scratch = R > 2 ? n_sets * half * slot_elems * 4 : 0;
    const int64_t tile_elems = pick_tile_elems(std::min<int64_t>(std::max<int64_t>(count, 1), group * granule), o, 4, HCCL_OP_REDUCE);
    hccl_graph* graw = nullptr;
    CHECK(hccl_graph_create(R, ext.data(), ext.data(), scratch, 0, &graw));
    GraphPtr g(graw);
    g->compulsory_bytes = 2ll * R * count * es;

    struct Node {
        hccl_ref_t ref;
        int dt;
        int leaf;       // leftmost leaf (rank) under this node
        int64_t made;   // WQE that produced it, -1 for a raw input
    };
    std::vector<std::vector<Node>> nodes((size_t)ng);
    std::vector<int32_t> sg((size_t)ng);
    std::vector<int64_t> root((size_t)ng, -1);
    std::vector<std::vector<int64_t>> have((size_t)ng, std::vector<int64_t>(R, -1));  // producer of Y_r's copy of the granule
    int K = 0;
    while ((1 << K) < R) ++K;
    for (int64_t i = 0; i < ng; ++i) {
        CHECK(hccl_graph_add_subgraph(g.get(), 0, &sg[i]));
        const int64_t e0 = i * granule;
        for (int r = 0; r < R; ++r) nodes[i].push_back(Node{ref(HCCL_BUF_SEND, r, e0 * es), dt, r, -1});
    }
    for (int64_t g0 = 0; g0 < ng; g0 += group) {
        const int64_t g1 = std::min(ng, g0 + group);
        // ---- up: K levels of pairwise sums
        for (int level = 0; level < K; ++level) {
            for (int64_t i = g0; i < g1; ++i) {
                const int64_t e0 = i * granule, len = std::min(granule, count - e0);
                std::vector<Node>& v = nodes[i];
                if (v.size() < 2) continue;
                std::vector<Node> next;
                for (size_t j = 0; j + 1 < v.size(); j += 2) {
                    const Node &a = v[j], &b = v[j + 1];
                    const bool final = v.size() == 2;
                    hccl_wqe_t w = blank();
                    w.op = HCCL_OP_REDUCE;
                    w.count = len;
                    w.tile_count = tile_elems;
                    w.a = a.ref; w.dtype_a = a.dt;
                    w.b = b.ref; w.dtype_b = b.dt;
                    Node res;
                    res.leaf = a.leaf;
                    if (final) {
                        res.ref = ref(HCCL_BUF_RECV, 0, e0 * es);
                        res.dt = dt;
                    } else {
                        res.ref = ref(HCCL_BUF_SCRATCH, 0, (((i % n_sets) * half) + a.leaf / 2) * slot_elems * 4);
                        res.dt = HCCL_FP32;
                    }
                    w.dst = res.ref; w.dtype_dst = res.dt;
                    // dependencies: the producers of both operands, tile by tile; a fresh scratch slot of a
                    // recycled set also waits for the set's previous user to have finished with it
                    int64_t d1 = a.made, d2 = b.made;
                    if (!final && a.made < 0 && i >= n_sets && root[i - n_sets] >= 0) d1 = root[i - n_sets];
                    if (d1 < 0) { d1 = d2; d2 = -1; }
                    if (d1 >= 0) {
                        w.dep_flags = HCCL_DEP_WQE_SYNC | HCCL_DEP_ELEMENTWISE;
                        w.dep_wqe = d1;
                        if (d2 >= 0) {
                            w.dep_flags |= HCCL_DEP_ELEMENTWISE2;
                            w.dep_wqe2 = d2;
                        }
                    }
                    CHECK(hccl_graph_add_wqe(g.get(), sg[i], &w, &res.made));
                    if (final) root[i] = res.made;
                    next.push_back(res);
                }
                if (v.size() & 1) next.push_back(v.back());
                v.swap(next);
            }
        }
        // ---- R == 1: the "sum" is a copy
        for (int64_t i = g0; i < g1 && R == 1; ++i) {
            const int64_t e0 = i * granule, len = std::min(granule, count - e0);
            hccl_wqe_t w = blank();
            w.op = HCCL_OP_COPY;
            w.count = len * es;
            w.tile_count = tile_elems * es;
            w.a = ref(HCCL_BUF_SEND, 0, e0 * es);
            w.dst = ref(HCCL_BUF_RECV, 0, e0 * es);
            CHECK(hccl_graph_add_wqe(g.get(), sg[i], &w, &root[i]));
        }
        // ---- down: binomial tree of copies from rank 0
        for (int64_t i = g0; i < g1; ++i) have[i][0] = root[i];
        for (int k = K - 1; k >= 0; --k) {
            for (int64_t i = g0; i < g1; ++i) {
                const int64_t e0 = i * granule, len = std::min(granule, count - e0);
                for (int r = 0; r + (1 << k) < R; r += 1 << (k + 1)) {
                    hccl_wqe_t w = blank();
                    w.op = HCCL_OP_COPY;
                    w.count = len * es;
                    w.tile_count = tile_elems * es;
                    w.a = ref(HCCL_BUF_RECV, r, e0 * es);
                    w.dst = ref(HCCL_BUF_RECV, r + (1 << k), e0 * es);
                    w.dep_flags = HCCL_DEP_WQE_SYNC | HCCL_DEP_ELEMENTWISE;
                    w.dep_wqe = have[i][r];
                    CHECK(hccl_graph_add_wqe(g.get(), sg[i], &w, &have[i][r + (1 << k)]));
                }
            }
        }
    }
    return hccl_graph_compile(g.get(), &o, out);
}

}  // namespace

extern "C" {

constexpr int64_t kOwnSlotBytes = 48ll << 20;

hccl_status_t hccl_plan_allreduce(int R, int64_t count, hccl_dtype_t dt, hccl_algo_t algo, const hccl_opts_t* opts,
                                  hccl_plan_t** out) {
    if (!out || R < 1 || R > HCCL_MAX_RANKS || count < 0) return HCCL_ERR_INVALID_ARG;
    if (!valid_dtype(dt)) return HCCL_ERR_DTYPE;
    // measured crossover of the two forms at R = 8 (about 6 MiB per rank) and R = 64 (about 0.5 MiB per rank)
    if (algo == HCCL_ALGO_AUTO) algo = ((int64_t)R * count * elem_bytes(dt) <= (32ll << 20)) ? HCCL_ALGO_ONESHOT : HCCL_ALGO_RING;
    if (algo != HCCL_ALGO_RING && algo != HCCL_ALGO_ONESHOT && algo != HCCL_ALGO_RING_FUSED && algo != HCCL_ALGO_RING_2LEVEL &&
        algo != HCCL_ALGO_FANOUT && algo != HCCL_ALGO_TREE) return HCCL_ERR_INVALID_ARG;
    hccl_opts_t o;
    // An FP32 ring keeps its partials in the receive buffers (no scratch slot is ever shared between chains), so
    // its chains can stay inside one block at any size; that needs the register engine (measured ahead of the
    // bulk engine with tickets: 0.50 vs 0.57 ms at R = 4 x 64 Mi, 0.63 vs 0.69 ms at R = 16 x 16 Mi).
    const bool fp32_ring = dt == HCCL_FP32 && algo == HCCL_ALGO_RING && R > 1;
    // A 16-bit ring whose FP32 partials take at most 48 MiB gives every chain a scratch slot of its own (no
    // recycling), so its chains are independent too and run as static chains on the register engine (R = 64 x 4 Mi
    // bf16: 0.59 vs 1.50 ms on the bulk engine with tickets; x 8 Mi: 1.05 vs 1.61 ms). From 64 MiB of partials on the
    // bulk engine with chain groups sized for the L2 is ahead (x 16 Mi: 1.81 vs 2.16 ms; x 32 Mi: 3.50 vs 4.01 ms).
    const bool own_slots = algo == HCCL_ALGO_RING && R > 1 && count * 4 <= kOwnSlotBytes && (!opts || opts->chain_group == 0);
    hccl_opts_t pre;
    if (opts) pre = *opts; else std::memset(&pre, 0, sizeof(pre));
    if (algo == HCCL_ALGO_RING && pre.engine == HCCL_ENGINE_AUTO && ring_wants_forwarding(R, count, false, pre)) pre.engine = HCCL_ENGINE_BULK;
    if ((fp32_ring || own_slots) && pre.engine == HCCL_ENGINE_AUTO) pre.engine = HCCL_ENGINE_LSU;
    fill_ring_opts(&o, &pre, (int64_t)R * count * elem_bytes(dt), algo == HCCL_ALGO_RING_FUSED || algo == HCCL_ALGO_ONESHOT || algo == HCCL_ALGO_FANOUT || R == 1);
    if (algo == HCCL_ALGO_RING_2LEVEL) {
        // a single rack (R <= rack_size), or racks of one rank, is the flat ring; only two or more racks must tile R
        if (o.rack_size >= 2 && R > o.rack_size && R % o.rack_size != 0) return HCCL_ERR_INVALID_ARG;
        if ((!opts || opts->chain_group == 0) && count * 4 <= (32ll << 20)) o.chain_group = 1 << 20;  // all chains together
        if (o.rack_size >= 2 && R / o.rack_size >= 2) return plan_allreduce_2level(R, count, dt, o, out);
        algo = HCCL_ALGO_RING;
    }
    if (algo == HCCL_ALGO_TREE) return plan_allreduce_tree(R, count, dt, o, opts && opts->chain_group != 0, out);
    const int es = elem_bytes(dt);
    std::vector<int64_t> ext(R, count * es);
    const int64_t compulsory = 2ll * R * count * es;

    if (R > 1 && algo == HCCL_ALGO_FANOUT) {
        // one sum per element, in the one-shot's order, stored into every receive buffer by the work item that formed it
        hccl_graph* graw = nullptr;
        CHECK(hccl_graph_create(R, ext.data(), ext.data(), 0, 0, &graw));
        GraphPtr g(graw);
        g->compulsory_bytes = compulsory;
        int32_t sg;
        CHECK(hccl_graph_add_subgraph(g.get(), 0, &sg));
        hccl_wqe_t w = blank();
        w.op = HCCL_OP_REDUCE_N;
        w.dtype_dst = w.dtype_a = dt;
        w.count = count;
        w.nsrc = R;
        w.ndst = R;
        w.hints = HCCL_HINT_READ_ONCE;
        w.a = ref(HCCL_BUF_SEND, 0, 0);
        w.dst = ref(HCCL_BUF_RECV, 0, 0);
        CHECK(hccl_graph_add_wqe(g.get(), sg, &w, nullptr));
        return hccl_graph_compile(g.get(), &o, out);
    }
    if (R == 1 || algo == HCCL_ALGO_ONESHOT) {
        hccl_graph* graw = nullptr;
        CHECK(hccl_graph_create(R, ext.data(), ext.data(), 0, 0, &graw));
        GraphPtr g(graw);
        g->compulsory_bytes = compulsory;
        for (int r = 0; r < R; ++r) {
            int32_t sg;
            CHECK(hccl_graph_add_subgraph(g.get(), r, &sg));
            hccl_wqe_t w = blank();
            if (R == 1) {
                w.op = HCCL_OP_COPY;
                w.count = count * es;
                w.a = ref(HCCL_BUF_SEND, 0, 0);
            } else {
                w.op = HCCL_OP_REDUCE_N;
                w.dtype_dst = w.dtype_a = dt;
                w.count = count;
                w.nsrc = R;
                w.a = ref(HCCL_BUF_SEND, 0, 0);  // rank order 0..R-1 for every output: identical bits on all ranks
            }
            w.dst = ref(HCCL_BUF_RECV, r, 0);
            CHECK(hccl_graph_add_wqe(g.get(), sg, &w, nullptr));
        }
        return hccl_graph_compile(g.get(), &o, out);
    }

    const bool fused = algo == HCCL_ALGO_RING_FUSED;
    const bool in_recv = dt == HCCL_FP32 && !fused;
    std::vector<int64_t> offs(R + 1);
    for (int c = 0; c <= R; ++c) offs[c] = (int64_t)(((__int128)c * count) / R);
    const int64_t granule = std::max<int64_t>(1, (int64_t)(o.chunk_bytes / (uint64_t)es));
    std::vector<Chain> chains = make_chains(R, offs, false, granule, (o.flags & HCCL_FLAG_BIDIRECTIONAL) != 0 && !fused);
    int64_t maxlen = 0;
    for (const Chain& ch : chains) maxlen = std::max(maxlen, ch.len);
    // small buffers (all FP32 partials fit the L2 several times over): run every chain together, the
    // dependency chain is then as short as the ring allows; large ones keep chain groups for L2 residency
    // Large rings on the bulk engine run in the forwarding kernel (see hccl_plan_reducescatter): a slot per chain, no recycling
    const bool forward = !fused && R > 2 && o.engine == HCCL_ENGINE_BULK && (!opts || opts->chain_group == 0) && count * 4 <= (1ll << 30) &&
                         !(o.flags & (HCCL_FLAG_DYNAMIC_TICKETS | HCCL_FLAG_LEVEL_MAJOR | HCCL_FLAG_STAGED_RING | HCCL_FLAG_BIDIRECTIONAL));
    if ((!opts || opts->chain_group == 0) && (count * 4 <= (32ll << 20) || own_slots || forward)) o.chain_group = (int32_t)std::max<size_t>(chains.size(), 1);
    else if (!opts || opts->chain_group == 0) o.chain_group = l2_chain_group(maxlen, chains.size());
    // ... and each chain of tiles can then stay inside one block (no slot is recycled, so nothing links the chains)
    // (the fused form has no partials at all: its one sum per granule is followed by copies that hop from the
    // bytes the same block has just written)
    if ((count * 4 <= (32ll << 20) || in_recv || own_slots || fused || forward) && !(o.flags & HCCL_FLAG_DYNAMIC_TICKETS)) o.flags |= HCCL_FLAG_STATIC_CHAINS;
    const bool need_scratch = !in_recv && !fused && R > 2;
    const bool staged = (o.flags & HCCL_FLAG_STAGED_RING) != 0 && need_scratch;
    // level-major order runs every chain's step t before any step t+1, so no slot can be recycled
    const size_t slots_wanted = (o.flags & HCCL_FLAG_LEVEL_MAJOR) ? chains.size() : 2 * (size_t)o.chain_group;
    const int n_slots = need_scratch ? (int)std::min<size_t>(chains.size(), slots_wanted) : 0;
    bool shifted = false;  // some chain starts off a multiple of 8 elements: its partial is shifted to the same phase (emit_ring)
    for (const Chain& ch : chains) shifted = shifted || (ch.e0 % 8) != 0;
    const int64_t slot_elems = (int64_t)align_up((uint64_t)maxlen + (shifted ? 8 : 0), 64);
    const int64_t scratch = need_scratch ? (int64_t)n_slots * slot_elems * 4 * (staged ? 2 : 1) : 0;
    const int64_t weight = count * 4 * (R - 1) + (int64_t)count * es * (R - 1);
    const int64_t level = (o.flags & HCCL_FLAG_LEVEL_MAJOR) ? count : std::min<int64_t>(count, (int64_t)o.chain_group * maxlen);
    (void)weight;
    int64_t tile_elems = fused ? pick_tile_elems(level, o, es * R, HCCL_OP_REDUCE_N) : pick_tile_elems(level, o, in_recv ? es : 4, HCCL_OP_REDUCE, maxlen);
    // large FP32 rings as static chains: two passes of the block's threads per tile keep a block's current
    // partial (written by one step, read by the next) in the L2
    if (forward && !o.tile_bytes) tile_elems = forward_tile_elems(chains, o.sm_budget, 2 * (R - 1));
    if (in_recv && o.engine == HCCL_ENGINE_LSU && !o.tile_bytes && count * 4 > (32ll << 20) && (o.flags & HCCL_FLAG_STATIC_CHAINS))
        tile_elems = 2 * sweep_of(o, HCCL_OP_REDUCE);
    if (!fused && o.engine == HCCL_ENGINE_LSU && (!opts || opts->sm_budget == 0) && maxlen > 0) {
        // a step that is a little short of one round of the blocks: launch exactly that many blocks, so that
        // block b keeps meeting tile b of every step (measured 54 vs 58 us at R = 8, 1 MiB per rank)
        const int64_t per_step = std::max<int64_t>(1, level / maxlen) * ((maxlen + tile_elems - 1) / tile_elems);
        if (per_step < o.sm_budget && per_step * 4 >= (int64_t)o.sm_budget * 3) o.sm_budget = (int32_t)per_step;
    }

    hccl_graph* graw = nullptr;
    CHECK(hccl_graph_create(R, ext.data(), ext.data(), scratch, 0, &graw));
    GraphPtr g(graw);
    g->compulsory_bytes = compulsory;
    CHECK(emit_ring(g.get(), R, dt, chains, true, in_recv, o, slot_elems, n_slots, tile_elems, fused));
    return hccl_graph_compile(g.get(), &o, out);
}

hccl_status_t hccl_plan_reducescatter(int R, const int64_t* recvcounts, int64_t count, hccl_dtype_t dt, hccl_algo_t algo,
                                      const hccl_opts_t* opts, hccl_plan_t** out) {
    if (!out || R < 1 || R > HCCL_MAX_RANKS || count < 0) return HCCL_ERR_INVALID_ARG;
    if (!valid_dtype(dt)) return HCCL_ERR_DTYPE;
    if (algo != HCCL_ALGO_RING && algo != HCCL_ALGO_RING_FUSED && algo != HCCL_ALGO_ONESHOT) return HCCL_ERR_INVALID_ARG;
    hccl_opts_t o, pre;
    if (opts) pre = *opts; else std::memset(&pre, 0, sizeof(pre));
    if (algo == HCCL_ALGO_RING && pre.engine == HCCL_ENGINE_AUTO && ring_wants_forwarding(R, count, false, pre, true, recvcounts)) pre.engine = HCCL_ENGINE_BULK;
    fill_ring_opts(&o, &pre, (int64_t)R * count * elem_bytes(dt), algo != HCCL_ALGO_RING || R == 1);
    const int es = elem_bytes(dt);
    std::vector<int64_t> offs(R + 1, 0);
    if (recvcounts) {
        for (int r = 0; r < R; ++r) {
            if (recvcounts[r] < 0) return HCCL_ERR_INVALID_ARG;
            offs[r + 1] = offs[r] + recvcounts[r];
        }
        if (offs[R] != count) return HCCL_ERR_COUNT_MISMATCH;
    } else {
        for (int c = 0; c <= R; ++c) offs[c] = (int64_t)(((__int128)c * count) / R);
    }
    std::vector<int64_t> sext(R, count * es), rext(R);
    for (int r = 0; r < R; ++r) rext[r] = (offs[r + 1] - offs[r]) * es;
    const int64_t compulsory = (int64_t)R * count * es + count * es;

    hccl_graph* graw = nullptr;
    if (R == 1) {
        CHECK(hccl_graph_create(R, sext.data(), rext.data(), 0, 0, &graw));
        GraphPtr g(graw);
        g->compulsory_bytes = compulsory;
        int32_t sg;
        CHECK(hccl_graph_add_subgraph(g.get(), 0, &sg));
        hccl_wqe_t w = blank();
        w.op = HCCL_OP_COPY;
        w.count = count * es;
        w.a = ref(HCCL_BUF_SEND, 0, 0);
        w.dst = ref(HCCL_BUF_RECV, 0, 0);
        CHECK(hccl_graph_add_wqe(g.get(), sg, &w, nullptr));
        return hccl_graph_compile(g.get(), &o, out);
    }
    if (algo == HCCL_ALGO_ONESHOT) {
        // rank r sums its own shard over all ranks itself, in rank order 0..R-1 (the one-shot AllReduce's order)
        CHECK(hccl_graph_create(R, sext.data(), rext.data(), 0, 0, &graw));
        GraphPtr g(graw);
        g->compulsory_bytes = compulsory;
        for (int r = 0; r < R; ++r) {
            int32_t sg;
            CHECK(hccl_graph_add_subgraph(g.get(), r, &sg));
            if (offs[r + 1] == offs[r]) continue;
            hccl_wqe_t w = blank();
            w.op = HCCL_OP_REDUCE_N;
            w.hints = HCCL_HINT_READ_ONCE;
            w.dtype_dst = w.dtype_a = dt;
            w.count = offs[r + 1] - offs[r];
            w.nsrc = R;
            w.a = ref(HCCL_BUF_SEND, 0, offs[r] * es);
            w.dst = ref(HCCL_BUF_RECV, r, 0);
            CHECK(hccl_graph_add_wqe(g.get(), sg, &w, nullptr));
        }
        return hccl_graph_compile(g.get(), &o, out);
    }
    const bool fused = algo == HCCL_ALGO_RING_FUSED;
    const int64_t granule = std::max<int64_t>(1, (int64_t)(o.chunk_bytes / (uint64_t)es));
    std::vector<Chain> chains = make_chains(R, offs, true, granule, (o.flags & HCCL_FLAG_BIDIRECTIONAL) != 0 && !fused);
    int64_t maxlen = 0;
    for (const Chain& ch : chains) maxlen = std::max(maxlen, ch.len);
    // Large rings on the bulk engine: every chain gets a scratch slot of its own (up to 1 GiB in all), so the chains are
    // independent and run in the forwarding kernel, which keeps a chain's running sums in registers and only stores
    // the partials (config 3: 0.69 vs 0.86 ms through tickets with recycled slots whose partials are read back).
    const bool forward = !fused && R > 2 && o.engine == HCCL_ENGINE_BULK && (!opts || opts->chain_group == 0) && count * 4 <= (1ll << 30) &&
                         !(o.flags & (HCCL_FLAG_DYNAMIC_TICKETS | HCCL_FLAG_LEVEL_MAJOR | HCCL_FLAG_STAGED_RING | HCCL_FLAG_BIDIRECTIONAL));
    if ((!opts || opts->chain_group == 0) && (count * 4 <= (32ll << 20) || forward)) o.chain_group = (int32_t)std::max<size_t>(chains.size(), 1);
    else if (!opts || opts->chain_group == 0) o.chain_group = l2_chain_group(maxlen, chains.size());
    // ... and each chain of tiles can then stay inside one block (no slot is recycled, so nothing links the chains)
    if ((count * 4 <= (32ll << 20) || forward) && !(o.flags & HCCL_FLAG_DYNAMIC_TICKETS)) o.flags |= HCCL_FLAG_STATIC_CHAINS;
    const bool need_scratch = !fused && R > 2;
    const bool staged = (o.flags & HCCL_FLAG_STAGED_RING) != 0 && need_scratch;
    // level-major order runs every chain's step t before any step t+1, so no slot can be recycled
    const size_t slots_wanted = (o.flags & HCCL_FLAG_LEVEL_MAJOR) ? chains.size() : 2 * (size_t)o.chain_group;
    const int n_slots = need_scratch ? (int)std::min<size_t>(chains.size(), slots_wanted) : 0;
    const int64_t slot_elems = (int64_t)align_up((uint64_t)maxlen, 64);
    const int64_t scratch = need_scratch ? (int64_t)n_slots * slot_elems * 4 * (staged ? 2 : 1) : 0;
    const int64_t level = (o.flags & HCCL_FLAG_LEVEL_MAJOR) ? count : std::min<int64_t>(count, (int64_t)o.chain_group * maxlen);
    int64_t tile_elems = fused ? pick_tile_elems(level, o, es * R, HCCL_OP_REDUCE_N) : pick_tile_elems(level, o, 4, HCCL_OP_REDUCE, maxlen);
    if (forward && !o.tile_bytes) tile_elems = forward_tile_elems(chains, o.sm_budget, R - 1);
    CHECK(hccl_graph_create(R, sext.data(), rext.data(), scratch, 0, &graw));
    GraphPtr g(graw);
    g->compulsory_bytes = compulsory;
    CHECK(emit_ring(g.get(), R, dt, chains, false, false, o, slot_elems, n_slots, tile_elems, fused));
    return hccl_graph_compile(g.get(), &o, out);
}

hccl_status_t hccl_plan_allgather(int R, const int64_t* sendcounts, int64_t count, hccl_dtype_t dt, hccl_algo_t algo,
                                  const hccl_opts_t* opts, hccl_plan_t** out) {
    if (!out || R < 1 || R > HCCL_MAX_RANKS || count < 0) return HCCL_ERR_INVALID_ARG;
    if (!valid_dtype(dt)) return HCCL_ERR_DTYPE;
    if (algo != HCCL_ALGO_RING && algo != HCCL_ALGO_ONESHOT && algo != HCCL_ALGO_RING_2LEVEL && algo != HCCL_ALGO_FANOUT) return HCCL_ERR_INVALID_ARG;
    hccl_opts_t o;
    if ((algo == HCCL_ALGO_RING || algo == HCCL_ALGO_RING_2LEVEL) && (!opts || opts->engine == HCCL_ENGINE_AUTO)) {
        // hop-by-hop copies wait on one another item by item: through tickets the register engine hands a finished item
        // on sooner than the bulk engine can (which must drain its stores first). The flat ring's chains of copies run in
        // the forwarding kernel of the bulk engine instead (a piece is loaded once and stored to every hop's destination:
        // R = 128 x 8 KiB per rank 0.040 vs 0.109 ms on the register engine's static chains, x 512 KiB 1.51 vs 1.70 ms, x 4 MiB
        // 11.6 vs 11.5 ms; R = 16 x 2 MiB 0.104 vs 0.153 ms), if every block starts on a 16-byte boundary of the receive buffers
        // (else its chains would run item by item there).
        const int es0 = elem_bytes(dt);
        bool aligned = algo == HCCL_ALGO_RING && !(opts && (opts->flags & HCCL_FLAG_DYNAMIC_TICKETS));
        int64_t off = 0;
        for (int r = 0; r < R && aligned; ++r) {
            if ((off * es0) % 16) aligned = false;
            off += sendcounts ? sendcounts[r] : count;
        }
        hccl_opts_t tmp;
        if (opts) tmp = *opts; else std::memset(&tmp, 0, sizeof(tmp));
        tmp.engine = aligned ? HCCL_ENGINE_BULK : HCCL_ENGINE_LSU;
        fill_default_opts(&o, &tmp);
    } else {
        fill_copy_opts(&o, opts);
    }
    const int es = elem_bytes(dt);
    std::vector<int64_t> offs(R + 1, 0), sext(R), rext(R);
    for (int r = 0; r < R; ++r) {
        const int64_t c = sendcounts ? sendcounts[r] : count;
        if (c < 0) return HCCL_ERR_INVALID_ARG;
        offs[r + 1] = offs[r] + c;
        sext[r] = c * es;
    }
    if (algo == HCCL_ALGO_RING_2LEVEL) {
        if (o.rack_size >= 2 && R > o.rack_size && R % o.rack_size != 0) return HCCL_ERR_INVALID_ARG;
        if (o.rack_size >= 2 && R / o.rack_size >= 2) return plan_allgather_2level(R, offs, dt, o, out);
        algo = HCCL_ALGO_RING;
    }
    for (int r = 0; r < R; ++r) rext[r] = offs[R] * es;
    hccl_graph* graw = nullptr;
    CHECK(hccl_graph_create(R, sext.data(), rext.data(), 0, 0, &graw));
    GraphPtr g(graw);
    g->compulsory_bytes = offs[R] * es + (int64_t)R * offs[R] * es;
    // hop-by-hop copies on the register engine: at most three passes of the block's threads per tile (180 KiB),
    // which keeps what a block has just written (and reads next) inside the L2 (12.5 vs 14.0 ms at R = 128, 4 MiB)
    const int64_t tile_cap = (algo == HCCL_ALGO_RING && o.engine == HCCL_ENGINE_LSU) ? 3 * sweep_of(o, HCCL_OP_COPY) : (256 << 10);
    int64_t tile = o.tile_bytes ? (int64_t)o.tile_bytes : default_tile(offs[R] * es, o.sm_budget, 1, 16 << 10, tile_cap, sweep_of(o, HCCL_OP_COPY));
    // the forwarding kernel moves 28 KiB per piece: at most two pieces per tile (more chains to share out)
    if (!o.tile_bytes && algo == HCCL_ALGO_RING && o.engine == HCCL_ENGINE_BULK && !(o.flags & HCCL_FLAG_DYNAMIC_TICKETS)) tile = std::min<int64_t>(tile, 2 * 28672);
    // one subgraph per chunk q: it first lands in its owner's receive buffer, then goes round (ring)
    // or is read by everyone directly (one-shot)
    std::vector<int32_t> sg(R);
    std::vector<int64_t> last(R, -1);
    for (int q = 0; q < R; ++q) CHECK(hccl_graph_add_subgraph(g.get(), q, &sg[q]));
    if (algo == HCCL_ALGO_FANOUT) {  // chunk q: one read, R writes
        // a work item writes R times what it reads, so its tiles are small: a third of a stage at most
        const int64_t ftile = o.tile_bytes ? (int64_t)o.tile_bytes : default_tile(offs[R] * es, o.sm_budget, 4, 8 << 10, 16 << 10, 64);
        for (int q = 0; q < R; ++q) {
            const int64_t bytes = (offs[q + 1] - offs[q]) * es;
            if (bytes == 0) continue;
            hccl_wqe_t w = blank();
            w.op = HCCL_OP_COPY;
            w.count = bytes;
            w.tile_count = ftile;
            w.ndst = R;
            w.a = ref(HCCL_BUF_SEND, q, 0);
            w.dst = ref(HCCL_BUF_RECV, q, offs[q] * es);
            CHECK(hccl_graph_add_wqe(g.get(), sg[q], &w, nullptr));
        }
        return hccl_graph_compile(g.get(), &o, out);
    }
    // Issue order. One-shot: chunk-major (groups of one chunk), so that the R reads of a chunk follow one another
    // while it is still in the L2. Ring: step-major over all chunks (step 0: own copy; steps 1..R-1: hops).
    // Smaller ring groups would let a hop find the previous hop's bytes in the L2, but then every work item
    // meets an unfinished predecessor; measured at R = 128 that costs more than the DRAM reads it saves.
    const bool oneshot = algo == HCCL_ALGO_ONESHOT;
    const int G = oneshot ? 1 : R;
    // hop-by-hop copies: a block can walk a tile through all its hops by itself (each hop then reads what the
    // same SM has just written)
    if (!oneshot && !(o.flags & HCCL_FLAG_DYNAMIC_TICKETS)) o.flags |= HCCL_FLAG_STATIC_CHAINS;
    for (int q0 = 0; q0 < R; q0 += G) {
        for (int u = 0; u < R; ++u) {
            for (int q = q0; q < std::min(R, q0 + G); ++q) {
                const int64_t bytes = (offs[q + 1] - offs[q]) * es;
                if (bytes == 0) continue;
                hccl_wqe_t w = blank();
                w.op = HCCL_OP_COPY;
                w.count = bytes;
                w.tile_count = tile;
                const int dst_rank = (q + u) % R;
                w.dst = ref(HCCL_BUF_RECV, dst_rank, offs[q] * es);
                if (u == 0 || oneshot) {
                    w.a = ref(HCCL_BUF_SEND, q, 0);
                } else {
                    w.a = ref(HCCL_BUF_RECV, (q + u - 1) % R, offs[q] * es);
                    w.dep_flags = HCCL_DEP_WQE_SYNC | HCCL_DEP_ELEMENTWISE;
                    w.dep_wqe = last[q];
                }
                CHECK(hccl_graph_add_wqe(g.get(), sg[q], &w, &last[q]));
            }
        }
    }
    return hccl_graph_compile(g.get(), &o, out);
}

hccl_status_t hccl_plan_alltoallv(int R, const int64_t* sendcounts, const int64_t* sdispls, const int64_t* recvcounts,
                                  const int64_t* rdispls, hccl_dtype_t dt, int64_t row_elems, const hccl_opts_t* opts,
                                  hccl_plan_t** out) {
    return hccl::plan_alltoallv_window(R, sendcounts, sdispls, recvcounts, rdispls, dt, row_elems, opts, 0, R, out);
}

}  // extern "C"

// The AllToAllv planner restricted to the destinations [d_lo, d_hi): the same validation, displacements and
// buffer extents as the whole exchange, but only the segments bound for those destinations become WQEs.
hccl_status_t hccl::plan_alltoallv_window(int R, const int64_t* sendcounts, const int64_t* sdispls, const int64_t* recvcounts,
                                          const int64_t* rdispls, hccl_dtype_t dt, int64_t row_elems, const hccl_opts_t* opts,
                                          int d_lo, int d_hi, hccl_plan_t** out) {
    if (!out || !sendcounts || R < 1 || R > HCCL_MAX_RANKS || row_elems < 1) return HCCL_ERR_INVALID_ARG;
    if (d_lo < 0 || d_hi > R || d_lo > d_hi) return HCCL_ERR_INVALID_ARG;
    if (!valid_dtype(dt)) return HCCL_ERR_DTYPE;
    hccl_opts_t o;
    fill_copy_opts(&o, opts);
    const int64_t row_bytes = row_elems * elem_bytes(dt);
    const size_t RR = (size_t)R * R;
    for (size_t i = 0; i < RR; ++i) {
        if (sendcounts[i] < 0) return HCCL_ERR_INVALID_ARG;
        if (sendcounts[i] > (INT64_MAX / 4) / row_bytes) return HCCL_ERR_INVALID_ARG;
        if (sdispls && sdispls[i] < 0) return HCCL_ERR_INVALID_ARG;
        if (rdispls && rdispls[i] < 0) return HCCL_ERR_INVALID_ARG;
    }
    // the count matrix seen from the receivers is the transpose of the senders' (with real ranks this is
    // the int64 metadata exchange that precedes the data; with virtual ranks the host transposes it)
    if (recvcounts) {
        for (int s = 0; s < R; ++s)
            for (int d = 0; d < R; ++d)
                if (recvcounts[(size_t)d * R + s] != sendcounts[(size_t)s * R + d]) return HCCL_ERR_COUNT_MISMATCH;
    }
    // packed displacements = exclusive prefix sums
    std::vector<int64_t> sd(RR), rd(RR);
    for (int s = 0; s < R; ++s) {
        int64_t acc = 0;
        for (int d = 0; d < R; ++d) {
            sd[(size_t)s * R + d] = sdispls ? sdispls[(size_t)s * R + d] : acc;
            acc += sendcounts[(size_t)s * R + d];
        }
    }
    for (int d = 0; d < R; ++d) {
        int64_t acc = 0;
        for (int s = 0; s < R; ++s) {
            rd[(size_t)d * R + s] = rdispls ? rdispls[(size_t)d * R + s] : acc;
            acc += sendcounts[(size_t)s * R + d];
        }
    }
    // extents, and receive ranges of one rank must be disjoint
    std::vector<int64_t> sext(R, 0), rext(R, 0);
    int64_t payload = 0;
    for (int s = 0; s < R; ++s)
        for (int d = 0; d < R; ++d) {
            const int64_t c = sendcounts[(size_t)s * R + d];
            if (c == 0) continue;
            payload += c * row_bytes;
            sext[s] = std::max(sext[s], (sd[(size_t)s * R + d] + c) * row_bytes);
            rext[d] = std::max(rext[d], (rd[(size_t)d * R + s] + c) * row_bytes);
        }
    for (int d = 0; d < R; ++d) {
        std::vector<std::pair<int64_t, int64_t>> seg;
        for (int s = 0; s < R; ++s) {
            const int64_t c = sendcounts[(size_t)s * R + d];
            if (c > 0) seg.emplace_back(rd[(size_t)d * R + s], c);
        }
        std::sort(seg.begin(), seg.end());
        for (size_t i = 1; i < seg.size(); ++i)
            if (seg[i - 1].first + seg[i - 1].second > seg[i].first) return HCCL_ERR_OVERLAP;
    }
    hccl_graph* graw = nullptr;
    CHECK(hccl_graph_create(R, sext.data(), rext.data(), 0, 0, &graw));
    GraphPtr g(graw);
    // one subgraph per source rank; zero-length segments produce no WQE at all
    int64_t moved = 0;
    for (int s = 0; s < R; ++s) {
        int32_t sg;
        CHECK(hccl_graph_add_subgraph(g.get(), s, &sg));
        for (int d = d_lo; d < d_hi; ++d) {
            const int64_t c = sendcounts[(size_t)s * R + d];
            if (c == 0) continue;
            moved += c * row_bytes;
            hccl_wqe_t w = blank();
            w.op = HCCL_OP_COPY;
            w.count = c * row_bytes;
            w.a = ref(HCCL_BUF_SEND, s, sd[(size_t)s * R + d] * row_bytes);
            w.dst = ref(HCCL_BUF_RECV, d, rd[(size_t)d * R + s] * row_bytes);
            CHECK(hccl_graph_add_wqe(g.get(), sg, &w, nullptr));
        }
    }
    g->compulsory_bytes = 2 * moved;
    (void)payload;
    return hccl_graph_compile(g.get(), &o, out);
}

extern "C" {

hccl_status_t hccl_plan_alltoallv_dynamic(int R, const int64_t* max_send_rows, const int64_t* max_recv_rows, hccl_dtype_t dt,
                                          int64_t row_elems, const hccl_opts_t* opts, hccl_plan_t** out) {
    if (!out || !max_send_rows || !max_recv_rows || R < 1 || R > HCCL_MAX_RANKS || row_elems < 1) return HCCL_ERR_INVALID_ARG;
    if (!valid_dtype(dt)) return HCCL_ERR_DTYPE;
    const int64_t row_bytes = row_elems * elem_bytes(dt);
    std::vector<int64_t> sext(R), rext(R);
    for (int r = 0; r < R; ++r) {
        if (max_send_rows[r] < 0 || max_recv_rows[r] < 0) return HCCL_ERR_INVALID_ARG;
        if (max_send_rows[r] > (INT64_MAX / 4) / row_bytes || max_recv_rows[r] > (INT64_MAX / 4) / row_bytes) return HCCL_ERR_INVALID_ARG;
        sext[r] = max_send_rows[r] * row_bytes;
        rext[r] = max_recv_rows[r] * row_bytes;
    }
    hccl_opts_t o;
    if (opts) o = *opts; else std::memset(&o, 0, sizeof(o));
    // beyond 64 ranks the one-kernel form has no room for the count matrix; from 1 GiB of capacity on, the ordinary
    // executor on device-built tables is the faster and steadier of the two (R = 64, 25.8 GB: 7.7 ms against 7.7-8.8 ms)
    int64_t capacity = 0;
    for (int r = 0; r < R; ++r) capacity += sext[r];
    const bool device_tables = R > 64 || (o.flags & HCCL_FLAG_DEVICE_TABLES) != 0 || capacity >= (1ll << 30);
    if (device_tables) {
        // Descriptors and tiles are written on the device at execute time and run by the ordinary executor: the
        // plan holds empty tables of the largest size the capacities allow. A source of capacity b bytes yields
        // at most b / tile + R tiles (every destination may end in one partial tile).
        hccl_opts_t oc;
        fill_copy_opts(&oc, &o);
        hccl_graph* graw2 = nullptr;
        CHECK(hccl_graph_create(R, sext.data(), rext.data(), 0, 0, &graw2));
        GraphPtr g2(graw2);
        g2->compulsory_bytes = 0;
        hccl_plan* p = nullptr;
        CHECK(hccl_graph_compile(g2.get(), &oc, &p));
        int64_t total = 0;
        for (int r = 0; r < R; ++r) total += sext[r];
        const uint64_t tile = (opts && opts->tile_bytes) ? std::max<uint64_t>(opts->tile_bytes / 16 * 16, 512)
                                                         : (uint64_t)default_tile(total, p->opts.sm_budget, 2, 16 << 10, 256 << 10, sweep_of(p->opts, HCCL_OP_COPY));
        uint64_t max_tiles = (uint64_t)R * (uint64_t)R;
        for (int r = 0; r < R; ++r) max_tiles += (uint64_t)sext[r] / tile;
        const uint32_t end_tiles = 2u * (uint32_t)std::max(p->opts.sm_budget, 148) + 2u;
        if (max_tiles + end_tiles > 0x7ffffff0ull) {
            delete p;
            return HCCL_ERR_INVALID_ARG;
        }
        p->descs.assign((size_t)R * R, Desc{});
        Tile endt;
        std::memset(&endt, 0, sizeof(endt));
        endt.signal[0] = endt.signal[1] = -1;
        endt.flags = TILE_FLAG_END;
        p->tiles.assign((size_t)(max_tiles + end_tiles), endt);   // until the device has written real ones
        compute_layout(p);
        p->dynamic = true;
        p->dyn_device_tables = true;
        p->dyn_end_tiles = end_tiles;
        p->dyn_row_bytes = row_bytes;
        p->dyn_max_send_rows.assign(max_send_rows, max_send_rows + R);
        p->dyn_max_recv_rows.assign(max_recv_rows, max_recv_rows + R);
        p->opts.tile_bytes = tile;
        p->buf_align = elem_bytes(dt);
        p->info.tile_bytes = (int64_t)tile;
        p->info.n_wqe = (int64_t)R * R;
        p->info.n_tiles = (int64_t)p->tiles.size();
        *out = p;
        return HCCL_OK;
    }
    o.engine = HCCL_ENGINE_LSU;  // the device-resident kernel moves bytes through registers
    hccl_graph* graw = nullptr;
    CHECK(hccl_graph_create(R, sext.data(), rext.data(), 0, 0, &graw));
    GraphPtr g(graw);
    g->compulsory_bytes = 0;  // not known before the counts exist
    hccl_plan* p = nullptr;
    CHECK(hccl_graph_compile(g.get(), &o, &p));
    p->dynamic = true;
    p->dyn_row_bytes = row_bytes;
    p->dyn_max_send_rows.assign(max_send_rows, max_send_rows + R);
    p->dyn_max_recv_rows.assign(max_recv_rows, max_recv_rows + R);
    if (!opts || opts->tile_bytes == 0) p->opts.tile_bytes = (uint64_t)p->opts.threads * 128;  // one pass of all threads
    p->opts.tile_bytes = std::max<uint64_t>(p->opts.tile_bytes, 512);
    p->info.tile_bytes = (int64_t)p->opts.tile_bytes;
    *out = p;
    return HCCL_OK;
}

hccl_status_t hccl_plan_set_dynamic_metadata(hccl_plan_t* p, const int64_t* dev_sendcounts, int64_t* dev_recvcounts_out,
                                             int64_t* dev_rdispls_out) {
    if (!p || !p->dynamic || !dev_sendcounts) return HCCL_ERR_INVALID_ARG;
    if (((uintptr_t)dev_sendcounts | (uintptr_t)dev_recvcounts_out | (uintptr_t)dev_rdispls_out) % 8) return HCCL_ERR_ALIGNMENT;
    p->dyn_counts = dev_sendcounts;
    p->dyn_recvcounts_out = dev_recvcounts_out;
    p->dyn_rdispls_out = dev_rdispls_out;
    return HCCL_OK;
}

}  // extern "C"
