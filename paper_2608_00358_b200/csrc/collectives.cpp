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
struct Chain {
    int c;            // chunk index = rank the reduced chunk ends on
    int64_t e0, len;  // element range [e0, e0+len) in the send buffers
    int64_t out_off;  // element offset of e0 inside Y_c for a scatter (AllReduce: == e0)
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
                const int64_t slot = (int64_t)(i % (size_t)std::max(n_slots, 1)) * slot_elems * 4;
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
                    const int r = (c + t + 2) % R, pr = (r + R - 1) % R;
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
                    const int dst_rank = (c + u + 1) % R, src_rank = (c + u) % R;
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
int64_t pick_tile_elems(int64_t level_elems, const hccl_opts_t& o, int widest, int op) {
    if (o.tile_bytes) return std::max<int64_t>(64, (int64_t)(o.tile_bytes / (uint64_t)widest));
    const int64_t lo = op == HCCL_OP_REDUCE_N ? 1 << 10 : 4 << 10, hi = op == HCCL_OP_REDUCE_N ? 32 << 10 : 64 << 10;
    return default_tile(level_elems, o.sm_budget, 1, lo, hi, sweep_of(o, op));
}

// Copy-only schedules: with the engine left to the library, the bulk copy unit moves the bytes
// (measured a few percent ahead of the register path at full budget, and no thread touches the data).
void fill_copy_opts(hccl_opts_t* o, const hccl_opts_t* in) {
    hccl_opts_t tmp;
    if (in) tmp = *in; else std::memset(&tmp, 0, sizeof(tmp));
    if (tmp.engine == HCCL_ENGINE_AUTO) tmp.engine = HCCL_ENGINE_BULK;
    fill_default_opts(o, &tmp);
}

std::vector<Chain> make_chains(int R, const std::vector<int64_t>& offs, bool scatter, int64_t granule_elems) {
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
            chains.push_back(Chain{c, lo, hi - lo, scatter ? lo - offs[c] : lo});
        }
    }
    return chains;
}

}  // namespace

extern "C" {

hccl_status_t hccl_plan_allreduce(int R, int64_t count, hccl_dtype_t dt, hccl_algo_t algo, const hccl_opts_t* opts,
                                  hccl_plan_t** out) {
    if (!out || R < 1 || R > HCCL_MAX_RANKS || count < 0) return HCCL_ERR_INVALID_ARG;
    if (!valid_dtype(dt)) return HCCL_ERR_DTYPE;
    if (algo != HCCL_ALGO_RING && algo != HCCL_ALGO_ONESHOT && algo != HCCL_ALGO_RING_FUSED) return HCCL_ERR_INVALID_ARG;
    hccl_opts_t o;
    fill_default_opts(&o, opts);
    const int es = elem_bytes(dt);
    std::vector<int64_t> ext(R, count * es);
    const int64_t compulsory = 2ll * R * count * es;

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
    std::vector<Chain> chains = make_chains(R, offs, false, granule);
    int64_t maxlen = 0;
    for (const Chain& ch : chains) maxlen = std::max(maxlen, ch.len);
    const bool need_scratch = !in_recv && !fused && R > 2;
    const bool staged = (o.flags & HCCL_FLAG_STAGED_RING) != 0 && need_scratch;
    // level-major order runs every chain's step t before any step t+1, so no slot can be recycled
    const size_t slots_wanted = (o.flags & HCCL_FLAG_LEVEL_MAJOR) ? chains.size() : 2 * (size_t)o.chain_group;
    const int n_slots = need_scratch ? (int)std::min<size_t>(chains.size(), slots_wanted) : 0;
    const int64_t slot_elems = (int64_t)align_up((uint64_t)maxlen, 64);
    const int64_t scratch = need_scratch ? (int64_t)n_slots * slot_elems * 4 * (staged ? 2 : 1) : 0;
    const int64_t weight = count * 4 * (R - 1) + (int64_t)count * es * (R - 1);
    const int64_t level = (o.flags & HCCL_FLAG_LEVEL_MAJOR) ? count : std::min<int64_t>(count, (int64_t)o.chain_group * maxlen);
    (void)weight;
    const int64_t tile_elems = fused ? pick_tile_elems(level, o, es * R, HCCL_OP_REDUCE_N) : pick_tile_elems(level, o, in_recv ? es : 4, HCCL_OP_REDUCE);

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
    if (algo != HCCL_ALGO_RING && algo != HCCL_ALGO_RING_FUSED) return HCCL_ERR_INVALID_ARG;
    hccl_opts_t o;
    fill_default_opts(&o, opts);
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
    const bool fused = algo == HCCL_ALGO_RING_FUSED;
    const int64_t granule = std::max<int64_t>(1, (int64_t)(o.chunk_bytes / (uint64_t)es));
    std::vector<Chain> chains = make_chains(R, offs, true, granule);
    int64_t maxlen = 0;
    for (const Chain& ch : chains) maxlen = std::max(maxlen, ch.len);
    const bool need_scratch = !fused && R > 2;
    const bool staged = (o.flags & HCCL_FLAG_STAGED_RING) != 0 && need_scratch;
    // level-major order runs every chain's step t before any step t+1, so no slot can be recycled
    const size_t slots_wanted = (o.flags & HCCL_FLAG_LEVEL_MAJOR) ? chains.size() : 2 * (size_t)o.chain_group;
    const int n_slots = need_scratch ? (int)std::min<size_t>(chains.size(), slots_wanted) : 0;
    const int64_t slot_elems = (int64_t)align_up((uint64_t)maxlen, 64);
    const int64_t scratch = need_scratch ? (int64_t)n_slots * slot_elems * 4 * (staged ? 2 : 1) : 0;
    const int64_t level = (o.flags & HCCL_FLAG_LEVEL_MAJOR) ? count : std::min<int64_t>(count, (int64_t)o.chain_group * maxlen);
    const int64_t tile_elems = fused ? pick_tile_elems(level, o, es * R, HCCL_OP_REDUCE_N) : pick_tile_elems(level, o, 4, HCCL_OP_REDUCE);
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
    if (algo != HCCL_ALGO_RING && algo != HCCL_ALGO_ONESHOT) return HCCL_ERR_INVALID_ARG;
    hccl_opts_t o;
    fill_copy_opts(&o, opts);
    const int es = elem_bytes(dt);
    std::vector<int64_t> offs(R + 1, 0), sext(R), rext(R);
    for (int r = 0; r < R; ++r) {
        const int64_t c = sendcounts ? sendcounts[r] : count;
        if (c < 0) return HCCL_ERR_INVALID_ARG;
        offs[r + 1] = offs[r] + c;
        sext[r] = c * es;
    }
    for (int r = 0; r < R; ++r) rext[r] = offs[R] * es;
    hccl_graph* graw = nullptr;
    CHECK(hccl_graph_create(R, sext.data(), rext.data(), 0, 0, &graw));
    GraphPtr g(graw);
    g->compulsory_bytes = offs[R] * es + (int64_t)R * offs[R] * es;
    const int64_t tile = o.tile_bytes ? (int64_t)o.tile_bytes : default_tile(offs[R] * es, o.sm_budget, 1, 16 << 10, 256 << 10, sweep_of(o, HCCL_OP_COPY));
    // one subgraph per chunk q: it first lands in its owner's receive buffer, then goes round (ring)
    // or is read by everyone directly (one-shot)
    std::vector<int32_t> sg(R);
    std::vector<int64_t> last(R, -1);
    for (int q = 0; q < R; ++q) CHECK(hccl_graph_add_subgraph(g.get(), q, &sg[q]));
    const int steps = R;  // step 0: own copy; steps 1..R-1: hops
    for (int u = 0; u < steps; ++u) {
        for (int q = 0; q < R; ++q) {
            const int64_t bytes = (offs[q + 1] - offs[q]) * es;
            if (bytes == 0) continue;
            hccl_wqe_t w = blank();
            w.op = HCCL_OP_COPY;
            w.count = bytes;
            w.tile_count = tile;
            const int dst_rank = (q + u) % R;
            w.dst = ref(HCCL_BUF_RECV, dst_rank, offs[q] * es);
            if (u == 0 || algo == HCCL_ALGO_ONESHOT) {
                w.a = ref(HCCL_BUF_SEND, q, 0);
            } else {
                w.a = ref(HCCL_BUF_RECV, (q + u - 1) % R, offs[q] * es);
                w.dep_flags = HCCL_DEP_WQE_SYNC | HCCL_DEP_ELEMENTWISE;
                w.dep_wqe = last[q];
            }
            CHECK(hccl_graph_add_wqe(g.get(), sg[q], &w, &last[q]));
        }
    }
    return hccl_graph_compile(g.get(), &o, out);
}

hccl_status_t hccl_plan_alltoallv(int R, const int64_t* sendcounts, const int64_t* sdispls, const int64_t* recvcounts,
                                  const int64_t* rdispls, hccl_dtype_t dt, int64_t row_elems, const hccl_opts_t* opts,
                                  hccl_plan_t** out) {
    if (!out || !sendcounts || R < 1 || R > HCCL_MAX_RANKS || row_elems < 1) return HCCL_ERR_INVALID_ARG;
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
    g->compulsory_bytes = 2 * payload;
    // one subgraph per source rank; zero-length segments produce no WQE at all
    for (int s = 0; s < R; ++s) {
        int32_t sg;
        CHECK(hccl_graph_add_subgraph(g.get(), s, &sg));
        for (int d = 0; d < R; ++d) {
            const int64_t c = sendcounts[(size_t)s * R + d];
            if (c == 0) continue;
            hccl_wqe_t w = blank();
            w.op = HCCL_OP_COPY;
            w.count = c * row_bytes;
            w.a = ref(HCCL_BUF_SEND, s, sd[(size_t)s * R + d] * row_bytes);
            w.dst = ref(HCCL_BUF_RECV, d, rd[(size_t)d * R + s] * row_bytes);
            CHECK(hccl_graph_add_wqe(g.get(), sg, &w, nullptr));
        }
    }
    return hccl_graph_compile(g.get(), &o, out);
}

hccl_status_t hccl_plan_alltoallv_dynamic(int R, const int64_t* max_send_rows, const int64_t* max_recv_rows, hccl_dtype_t dt,
                                          int64_t row_elems, const hccl_opts_t* opts, hccl_plan_t** out) {
    if (!out || !max_send_rows || !max_recv_rows || R < 1 || R > 64 || row_elems < 1) return HCCL_ERR_INVALID_ARG;
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
