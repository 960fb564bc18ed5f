// Work-packet builder and its lowering to device tables (paper Sec. III-B.2: work packet ->
// subgraphs -> WQEs with dependency metadata; Sec. I: the host generates the complete description).
#include <algorithm>
#include <cstring>
#include <new>

#include "plan.hpp"

using namespace hccl;

namespace {

bool is_data_op(int op) { return op == HCCL_OP_COPY || op == HCCL_OP_REDUCE || op == HCCL_OP_REDUCE_N; }

// byte extent of a data buffer reference, or -1 if the reference is not a data buffer of this graph
int64_t extent_of(const hccl_graph* g, const hccl_ref_t& r) {
    switch (r.kind) {
        case HCCL_BUF_SEND:
            return (r.rank >= 0 && r.rank < g->R) ? g->send_bytes[r.rank] : -1;
        case HCCL_BUF_RECV:
            return (r.rank >= 0 && r.rank < g->R) ? g->recv_bytes[r.rank] : -1;
        case HCCL_BUF_SCRATCH:
            return g->scratch_bytes;
        default:
            return -1;
    }
}

bool in_bounds(const hccl_graph* g, const hccl_ref_t& r, int64_t bytes) {
    int64_t ext = extent_of(g, r);
    return ext >= 0 && r.offset >= 0 && bytes >= 0 && r.offset <= ext && bytes <= ext - r.offset;
}

bool same_buffer(const hccl_ref_t& x, const hccl_ref_t& y) {
    if (x.kind != y.kind) return false;
    return x.kind == HCCL_BUF_SCRATCH || x.rank == y.rank;
}

bool ranges_intersect(const hccl_ref_t& x, int64_t xb, const hccl_ref_t& y, int64_t yb) {
    if (!same_buffer(x, y) || xb == 0 || yb == 0) return false;
    return x.offset < y.offset + yb && y.offset < x.offset + xb;
}

void push_unique(std::vector<int64_t>& v, int64_t x) {
    if (std::find(v.begin(), v.end(), x) == v.end()) v.push_back(x);
}

int wqe_ndst(const hccl_wqe_t& w) { return (w.op == HCCL_OP_COPY || w.op == HCCL_OP_REDUCE_N) && w.ndst > 1 ? w.ndst : 1; }
// Is `rank` one of the ranks whose receive buffer w writes? Is any other rank?
bool writes_rank(const hccl_wqe_t& w, int rank, int R) {
    if (w.dst.kind != HCCL_BUF_RECV) return false;
    const int k = ((rank - w.dst.rank) % R + R) % R;
    return k < wqe_ndst(w);
}
bool writes_other_rank(const hccl_wqe_t& w, int rank, int R) {
    if (w.dst.kind != HCCL_BUF_RECV) return false;
    return wqe_ndst(w) > 1 ? R > 1 : w.dst.rank != rank;
}

// Does WQE w, issued by a subgraph acting for `rank`, bring data into that rank from another one?
bool is_receive(const hccl_wqe_t& w, int rank, int R) {
    if (!is_data_op(w.op) || !writes_rank(w, rank, R)) return false;
    if (w.op == HCCL_OP_REDUCE_N) return w.nsrc > 1 || w.a.rank != rank;
    bool a_remote = (w.a.kind == HCCL_BUF_SEND || w.a.kind == HCCL_BUF_RECV) && w.a.rank != rank;
    bool b_remote = w.op == HCCL_OP_REDUCE && (w.b.kind == HCCL_BUF_SEND || w.b.kind == HCCL_BUF_RECV) && w.b.rank != rank;
    return a_remote || b_remote;
}
// Does it read this rank's buffers on behalf of another rank (a "send": the buffer is busy until it completes)?
bool is_send(const hccl_wqe_t& w, int rank, int R) {
    if (!is_data_op(w.op)) return false;
    if (!writes_other_rank(w, rank, R)) return false;
    if (w.op == HCCL_OP_REDUCE_N) return true;
    bool a_local = (w.a.kind == HCCL_BUF_SEND || w.a.kind == HCCL_BUF_RECV) && w.a.rank == rank;
    bool b_local = w.op == HCCL_OP_REDUCE && (w.b.kind == HCCL_BUF_SEND || w.b.kind == HCCL_BUF_RECV) && w.b.rank == rank;
    return a_local || b_local;
}

}  // namespace

void hccl::fill_default_opts(hccl_opts_t* o, const hccl_opts_t* in) {
    if (in) *o = *in; else std::memset(o, 0, sizeof(*o));
    if (o->sm_budget <= 0) o->sm_budget = 148;
    if (o->engine == 0) o->engine = HCCL_ENGINE_LSU;
    if (o->chunk_bytes == 0) o->chunk_bytes = 2u << 20;
    if (o->timeout_ns == 0) o->timeout_ns = 2000000000ull;
    if (o->chain_group <= 0) o->chain_group = 16;
    if (o->rack_size <= 0) o->rack_size = 16;
    if (o->threads <= 0) o->threads = o->engine == HCCL_ENGINE_BULK ? 352 : 512;  // bulk: DMA, control and publishing warps + 8 compute warps; register: control warp + 15 workers
    o->threads = std::min(512, std::max(o->engine == HCCL_ENGINE_BULK ? 128 : 64, (o->threads + 31) / 32 * 32));  // the service warps + at least one worker warp
}

extern "C" {

hccl_status_t hccl_graph_create(int R, const int64_t* send_bytes, const int64_t* recv_bytes, int64_t scratch_bytes,
                                int32_t n_signals, hccl_graph_t** out) {
    if (!out || R < 1 || R > HCCL_MAX_RANKS || scratch_bytes < 0 || n_signals < 0) return HCCL_ERR_INVALID_ARG;
    hccl_graph* g = new (std::nothrow) hccl_graph();
    if (!g) return HCCL_ERR_INVALID_ARG;
    g->R = R;
    g->send_bytes.assign(R, 0);
    g->recv_bytes.assign(R, 0);
    for (int r = 0; r < R; ++r) {
        int64_t s = send_bytes ? send_bytes[r] : 0, v = recv_bytes ? recv_bytes[r] : 0;
        if (s < 0 || v < 0) {
            delete g;
            return HCCL_ERR_INVALID_ARG;
        }
        g->send_bytes[r] = s;
        g->recv_bytes[r] = v;
    }
    g->scratch_bytes = scratch_bytes;
    g->n_signals = n_signals;
    *out = g;
    return HCCL_OK;
}

hccl_status_t hccl_graph_add_subgraph(hccl_graph_t* g, int rank, int32_t* subgraph) {
    if (!g || !subgraph || rank < 0 || rank >= g->R) return HCCL_ERR_INVALID_ARG;
    Subgraph s;
    s.rank = rank;
    g->subgraphs.push_back(s);
    *subgraph = (int32_t)g->subgraphs.size() - 1;
    return HCCL_OK;
}

hccl_status_t hccl_graph_add_wqe(hccl_graph_t* g, int32_t subgraph, const hccl_wqe_t* wp, int64_t* wqe_id) {
    if (!g || !wp || subgraph < 0 || subgraph >= (int32_t)g->subgraphs.size()) return HCCL_ERR_INVALID_ARG;
    hccl_wqe_t w = *wp;
    const int64_t id = (int64_t)g->wqes.size();
    if (w.count < 0 || w.tile_count < 0) return HCCL_ERR_INVALID_ARG;
    switch (w.op) {
        case HCCL_OP_COPY: {
            if (w.dst.kind != HCCL_BUF_RECV && w.dst.kind != HCCL_BUF_SCRATCH) return HCCL_ERR_INVALID_ARG;
            if (w.a.kind != HCCL_BUF_SEND && w.a.kind != HCCL_BUF_RECV && w.a.kind != HCCL_BUF_SCRATCH) return HCCL_ERR_INVALID_ARG;
            if (w.ndst < 0 || w.ndst > g->R || (w.ndst > 1 && w.dst.kind != HCCL_BUF_RECV)) return HCCL_ERR_INVALID_ARG;
            if (!in_bounds(g, w.a, w.count)) return HCCL_ERR_INVALID_ARG;
            for (int k = 0; k < wqe_ndst(w); ++k) {
                hccl_ref_t d = w.dst;
                if (k) d.rank = (w.dst.rank + k) % g->R;
                if (!in_bounds(g, d, w.count)) return HCCL_ERR_INVALID_ARG;
                if (ranges_intersect(d, w.count, w.a, w.count)) return HCCL_ERR_OVERLAP;
            }
            break;
        }
        case HCCL_OP_REDUCE: {
            if (!valid_dtype(w.dtype_dst) || !valid_dtype(w.dtype_a) || !valid_dtype(w.dtype_b)) return HCCL_ERR_DTYPE;
            if (w.dst.kind != HCCL_BUF_RECV && w.dst.kind != HCCL_BUF_SCRATCH) return HCCL_ERR_INVALID_ARG;
            const hccl_ref_t* src[2] = {&w.a, &w.b};
            const int sdt[2] = {w.dtype_a, w.dtype_b};
            const int64_t db = w.count * elem_bytes(w.dtype_dst);
            if (!in_bounds(g, w.dst, db)) return HCCL_ERR_INVALID_ARG;
            if (w.dst.offset % elem_bytes(w.dtype_dst)) return HCCL_ERR_ALIGNMENT;
            for (int k = 0; k < 2; ++k) {
                const hccl_ref_t& s = *src[k];
                if (s.kind != HCCL_BUF_SEND && s.kind != HCCL_BUF_RECV && s.kind != HCCL_BUF_SCRATCH) return HCCL_ERR_INVALID_ARG;
                const int64_t sb = w.count * elem_bytes(sdt[k]);
                if (!in_bounds(g, s, sb)) return HCCL_ERR_INVALID_ARG;
                if (s.offset % elem_bytes(sdt[k])) return HCCL_ERR_ALIGNMENT;
                // in-place forms A=A+B / B=A+B: exact alias with equal element size only
                if (ranges_intersect(w.dst, db, s, sb)) {
                    bool exact = s.offset == w.dst.offset && elem_bytes(sdt[k]) == elem_bytes(w.dtype_dst);
                    if (!exact) return HCCL_ERR_OVERLAP;
                }
            }
            break;
        }
        case HCCL_OP_REDUCE_N: {
            if (!valid_dtype(w.dtype_dst) || !valid_dtype(w.dtype_a)) return HCCL_ERR_DTYPE;
            if (w.nsrc < 1 || w.nsrc > g->R) return HCCL_ERR_INVALID_ARG;
            if (w.dst.kind != HCCL_BUF_RECV && w.dst.kind != HCCL_BUF_SCRATCH) return HCCL_ERR_INVALID_ARG;
            if (w.ndst < 0 || w.ndst > g->R || (w.ndst > 1 && w.dst.kind != HCCL_BUF_RECV)) return HCCL_ERR_INVALID_ARG;
            if (w.a.kind != HCCL_BUF_SEND && w.a.kind != HCCL_BUF_RECV) return HCCL_ERR_INVALID_ARG;
            const int64_t db = w.count * elem_bytes(w.dtype_dst), sb = w.count * elem_bytes(w.dtype_a);
            if (w.dst.offset % elem_bytes(w.dtype_dst) || w.a.offset % elem_bytes(w.dtype_a)) return HCCL_ERR_ALIGNMENT;
            if (w.a.rank < 0 || w.a.rank >= g->R) return HCCL_ERR_INVALID_ARG;
            for (int j = 0; j < wqe_ndst(w); ++j) {
                hccl_ref_t d = w.dst;
                if (j) d.rank = (w.dst.rank + j) % g->R;
                if (!in_bounds(g, d, db)) return HCCL_ERR_INVALID_ARG;
                for (int k = 0; k < w.nsrc; ++k) {
                    hccl_ref_t s = w.a;
                    s.rank = (w.a.rank + k) % g->R;
                    if (j == 0 && !in_bounds(g, s, sb)) return HCCL_ERR_INVALID_ARG;
                    if (ranges_intersect(d, db, s, sb)) return HCCL_ERR_OVERLAP;
                }
            }
            break;
        }
        case HCCL_OP_WAIT: {
            if (w.cmp < HCCL_CMP_EQ || w.cmp > HCCL_CMP_LT) return HCCL_ERR_INVALID_ARG;
            if (w.a.kind == HCCL_BUF_SIGNAL) {
                if (w.a.offset < 0 || w.a.offset >= g->n_signals) return HCCL_ERR_INVALID_ARG;
            } else if (w.a.kind == HCCL_BUF_USER_SIGNAL) {
                if (w.a.offset < 0) return HCCL_ERR_INVALID_ARG;
            } else {
                return HCCL_ERR_INVALID_ARG;
            }
            break;
        }
        case HCCL_OP_SET: {
            if (w.dst.kind == HCCL_BUF_SIGNAL) {
                if (w.dst.offset < 0 || w.dst.offset >= g->n_signals) return HCCL_ERR_INVALID_ARG;
            } else if (w.dst.kind == HCCL_BUF_USER_SIGNAL) {
                if (w.dst.offset < 0) return HCCL_ERR_INVALID_ARG;
            } else {
                return HCCL_ERR_INVALID_ARG;
            }
            break;
        }
        case HCCL_OP_NOOP:
            break;
        default:
            return HCCL_ERR_INVALID_ARG;
    }
    if (w.dep_flags & HCCL_DEP_WQE_SYNC) {
        if (w.dep_wqe < 0 || w.dep_wqe >= id) return HCCL_ERR_INVALID_ARG;
        if (w.dep_wqe2 >= id) return HCCL_ERR_INVALID_ARG;
    }

    Subgraph& sg = g->subgraphs[subgraph];
    Wqe q;
    q.w = w;
    q.subgraph = subgraph;
    const size_t first_live = 0;
    (void)first_live;
    // Fence on the previous WQE of this subgraph
    if (sg.fence_pending && !sg.wqes.empty()) push_unique(q.preds_full, sg.wqes.back());
    // position of the first WQE after the last Sync barrier (everything before it is implied by the barrier)
    size_t from = 0;
    if (sg.last_sync >= 0) {
        for (size_t i = 0; i < sg.wqes.size(); ++i)
            if (sg.wqes[i] == sg.last_sync) from = i;
    }
    if (w.dep_flags & HCCL_DEP_SYNC) {
        for (size_t i = from; i < sg.wqes.size(); ++i) push_unique(q.preds_full, sg.wqes[i]);
    }
    if (w.dep_flags & (HCCL_DEP_RECV_SYNC | HCCL_DEP_SEND_SYNC)) {
        for (size_t i = from; i < sg.wqes.size(); ++i) {
            const hccl_wqe_t& p = g->wqes[sg.wqes[i]].w;
            bool hit = sg.wqes[i] == sg.last_sync;  // the barrier stands for everything older
            if ((w.dep_flags & HCCL_DEP_RECV_SYNC) && is_receive(p, sg.rank, g->R)) hit = true;
            if ((w.dep_flags & HCCL_DEP_SEND_SYNC) && is_send(p, sg.rank, g->R)) hit = true;
            if (hit) push_unique(q.preds_full, sg.wqes[i]);
        }
    }
    if (w.dep_flags & HCCL_DEP_WQE_SYNC) {
        if (w.dep_flags & HCCL_DEP_ELEMENTWISE)
            push_unique(q.preds_elem, w.dep_wqe);
        else
            push_unique(q.preds_full, w.dep_wqe);
        if (w.dep_wqe2 >= 0) {
            if (w.dep_flags & HCCL_DEP_ELEMENTWISE2) push_unique(q.preds_elem, w.dep_wqe2); else push_unique(q.preds_full, w.dep_wqe2);
        }
    }
    // a predecessor listed both ways is waited for entirely
    for (int64_t p : q.preds_full) {
        auto it = std::find(q.preds_elem.begin(), q.preds_elem.end(), p);
        if (it != q.preds_elem.end()) q.preds_elem.erase(it);
    }
    sg.fence_pending = (w.dep_flags & HCCL_DEP_FENCE) != 0;
    if (w.dep_flags & HCCL_DEP_SYNC) sg.last_sync = id;
    sg.wqes.push_back(id);
    g->wqes.push_back(std::move(q));
    if (wqe_id) *wqe_id = id;
    return HCCL_OK;
}

void hccl_graph_destroy(hccl_graph_t* g) { delete g; }

hccl_status_t hccl_graph_compile(const hccl_graph_t* g, const hccl_opts_t* opts, hccl_plan_t** out) {
    if (!g || !out) return HCCL_ERR_INVALID_ARG;
    hccl_plan* p = nullptr;
    hccl_status_t st = compile_graph(g, opts, &p);
    if (st != HCCL_OK) return st;
    if (p->opts.flags & HCCL_FLAG_CHECK_HAZARDS) {
        int64_t nv = 0;
        st = hccl_plan_check_hazards(p, &nv);
        if (st == HCCL_OK && nv != 0) st = HCCL_ERR_HAZARD;
        if (st != HCCL_OK) {
            delete p;
            return st;
        }
    }
    *out = p;
    return HCCL_OK;
}

}  // extern "C"

hccl_status_t hccl::compile_graph(const hccl_graph* g, const hccl_opts_t* opts_in, hccl_plan** out) {
    hccl_plan* p = new (std::nothrow) hccl_plan();
    if (!p) return HCCL_ERR_INVALID_ARG;
    fill_default_opts(&p->opts, opts_in);
    p->R = g->R;
    p->send_bytes = g->send_bytes;
    p->recv_bytes = g->recv_bytes;
    p->scratch_bytes = g->scratch_bytes;
    p->n_signals = g->n_signals;
    const size_t n = g->wqes.size();

    // ---- byte accounting and default tile size
    auto widest = [](const hccl_wqe_t& w) -> int64_t {
        if (w.op == HCCL_OP_COPY) return 1;
        if (w.op == HCCL_OP_REDUCE) return std::max(elem_bytes(w.dtype_dst), std::max(elem_bytes(w.dtype_a), elem_bytes(w.dtype_b)));
        if (w.op == HCCL_OP_REDUCE_N) return std::max(elem_bytes(w.dtype_dst), elem_bytes(w.dtype_a));
        return 0;
    };
    int64_t schedule = 0, weight = 0, crossrack = 0;
    const int rack = std::max(1, p->opts.rack_size);
    auto remote = [&](const hccl_ref_t& src, const hccl_ref_t& dst) {
        const bool s_rank = src.kind == HCCL_BUF_SEND || src.kind == HCCL_BUF_RECV, d_rank = dst.kind == HCCL_BUF_RECV;
        return s_rank && d_rank && src.rank / rack != dst.rank / rack;
    };
    for (const Wqe& q : g->wqes) {
        const hccl_wqe_t& w = q.w;
        const int nd = wqe_ndst(w);  // a byte counts as crossing once per destination in another rack
        if (w.op == HCCL_OP_COPY)
            for (int j = 0; j < nd; ++j) {
                hccl_ref_t d = w.dst;
                if (j) d.rank = (w.dst.rank + j) % g->R;
                if (remote(w.a, d)) crossrack += w.count;
            }
        if (w.op == HCCL_OP_REDUCE) {
            if (remote(w.a, w.dst)) crossrack += w.count * elem_bytes(w.dtype_a);
            if (remote(w.b, w.dst)) crossrack += w.count * elem_bytes(w.dtype_b);
        }
        if (w.op == HCCL_OP_REDUCE_N)
            for (int j = 0; j < nd; ++j)
                for (int k = 0; k < w.nsrc; ++k) {
                    hccl_ref_t sr = w.a, d = w.dst;
                    sr.rank = (w.a.rank + k) % g->R;
                    if (j) d.rank = (w.dst.rank + j) % g->R;
                    if (remote(sr, d)) crossrack += w.count * elem_bytes(w.dtype_a);
                }
        if (w.op == HCCL_OP_COPY) schedule += (1 + (int64_t)nd) * w.count;
        if (w.op == HCCL_OP_REDUCE) schedule += w.count * (elem_bytes(w.dtype_a) + elem_bytes(w.dtype_b) + elem_bytes(w.dtype_dst));
        if (w.op == HCCL_OP_REDUCE_N) schedule += w.count * ((int64_t)w.nsrc * elem_bytes(w.dtype_a) + (int64_t)nd * elem_bytes(w.dtype_dst));
        weight += w.count * widest(w);
        if (w.op == HCCL_OP_REDUCE || w.op == HCCL_OP_REDUCE_N) {
            auto need = [&](const hccl_ref_t& r, int dt) {
                if (r.kind == HCCL_BUF_SEND || r.kind == HCCL_BUF_RECV) p->buf_align = std::max(p->buf_align, elem_bytes(dt));
            };
            need(w.dst, w.dtype_dst);
            need(w.a, w.dtype_a);
            if (w.op == HCCL_OP_REDUCE) need(w.b, w.dtype_b);
        }
    }
    // Default tile sizes: about two tiles per block for each kind of operation (latency-bound sizes want few,
    // large tiles; big ones are capped), whole passes of the block's threads. opts.tile_bytes overrides.
    int64_t units[3] = {0, 0, 0};  // COPY bytes, REDUCE elements, REDUCE_N elements of the whole packet
    for (const Wqe& q : g->wqes)
        if (is_data_op(q.w.op)) units[q.w.op] += q.w.count;
    const int B = p->opts.sm_budget;
    const bool fixed = p->opts.tile_bytes != 0;
    const int64_t def_copy = default_tile(units[HCCL_OP_COPY], B, 2, 16 << 10, 256 << 10, sweep_of(p->opts, HCCL_OP_COPY));
    const int64_t def_reduce = default_tile(units[HCCL_OP_REDUCE], B, 2, 4 << 10, 64 << 10, sweep_of(p->opts, HCCL_OP_REDUCE));
    const int64_t def_reduce_n = default_tile(units[HCCL_OP_REDUCE_N], B, 2, 1 << 10, 32 << 10, sweep_of(p->opts, HCCL_OP_REDUCE_N));
    const uint64_t tile_bytes = fixed ? std::max<uint64_t>(p->opts.tile_bytes, 256) : (uint64_t)def_copy;
    p->opts.tile_bytes = tile_bytes;
    (void)weight;

    // ---- tiles per WQE
    std::vector<int64_t> tcount(n), ntiles(n);
    for (size_t i = 0; i < n; ++i) {
        const hccl_wqe_t& w = g->wqes[i].w;
        if (!is_data_op(w.op) || w.count == 0) {
            tcount[i] = 0;
            ntiles[i] = 1;  // a dependency-only work item
            continue;
        }
        int64_t tc = w.tile_count;
        if (tc <= 0) {
            if (fixed)  // caller's tile_bytes, in bytes of the widest operand (all sources together for REDUCE_N)
                tc = std::max<int64_t>(1, (int64_t)(tile_bytes / (uint64_t)(widest(w) * (w.op == HCCL_OP_REDUCE_N ? std::max<int>(w.nsrc, 1) : 1))));
            else
                tc = w.op == HCCL_OP_COPY ? def_copy : (w.op == HCCL_OP_REDUCE ? def_reduce : def_reduce_n);
        }
        tc = std::min<int64_t>(std::max<int64_t>(tc, 1), 0x7fffffff);
        tcount[i] = tc;
        ntiles[i] = (w.count + tc - 1) / tc;
    }

    // ---- which sync objects are needed
    std::vector<char> need_desc(n, 0), need_tile(n, 0);
    std::vector<std::vector<int64_t>> pf(n), pe(n);
    for (size_t j = 0; j < n; ++j) {
        pf[j] = g->wqes[j].preds_full;
        for (int64_t i : g->wqes[j].preds_elem) {
            if (ntiles[i] == ntiles[j]) pe[j].push_back(i); else pf[j].push_back(i);
        }
        for (int64_t i : pf[j]) need_desc[i] = 1;
        for (int64_t i : pe[j]) need_tile[i] = 1;
    }
    // ---- static chains: the packet is a set of independent chains of equal length, linked tile by tile
    std::vector<int64_t> depth(n, 1);
    int64_t max_depth = n ? 1 : 0;
    for (size_t i = 0; i < n; ++i) {
        for (int64_t q : pf[i]) depth[i] = std::max(depth[i], depth[q] + 1);
        for (int64_t q : pe[i]) depth[i] = std::max(depth[i], depth[q] + 1);
        max_depth = std::max(max_depth, depth[i]);
    }
    // On the bulk engine static chains run in the forwarding kernel, which is built for chains of REDUCE items followed by plain copies, and for chains of copies of one source (anything
    // else it runs item by item through its few compute warps): only packets made of such items go there.
    bool chains = (p->opts.flags & HCCL_FLAG_STATIC_CHAINS) != 0 && n > 0 && max_depth > 1;
    if (chains && p->opts.engine != HCCL_ENGINE_LSU) {
        // ... and only simple chains (a ring's): one predecessor, one successor
        std::vector<int> successors(n, 0);
        for (size_t j = 0; j < n && chains; ++j) {
            const hccl_wqe_t& w = g->wqes[j].w;
            if (w.op != HCCL_OP_REDUCE && !(w.op == HCCL_OP_COPY && wqe_ndst(w) <= 1)) chains = false;
            if (pe[j].size() > 1) chains = false;
            for (int64_t i : pe[j])
                if (++successors[(size_t)i] > 1) chains = false;
        }
    }
    // Every dependency must be a tile-by-tile link; WQEs linked (directly or not) form a group that one block runs
    // in issue order, which already has every predecessor before its successors. A ring's chain is such a
    // group; so is a chunk that forks into several racks. Groups must be equally long, so that a block finds
    // its tiles by arithmetic.
    std::vector<int64_t> group_of(n);
    for (size_t j = 0; j < n; ++j) group_of[j] = (int64_t)j;
    auto root = [&](int64_t x) {
        while (group_of[x] != x) x = group_of[x] = group_of[group_of[x]];
        return x;
    };
    for (size_t j = 0; j < n && chains; ++j) {
        const int op = g->wqes[j].w.op;
        if (!pf[j].empty() || op == HCCL_OP_WAIT || op == HCCL_OP_SET) chains = false;
        for (int64_t i : pe[j]) group_of[root((int64_t)j)] = root(i);   // roots keep the smallest id: i < j
    }
    std::vector<std::vector<int64_t>> groups;   // in order of their first WQE
    if (chains) {
        std::vector<int64_t> index_of(n, -1);
        for (size_t j = 0; j < n; ++j) {
            const int64_t r = root((int64_t)j);
            if (index_of[r] < 0) {
                index_of[r] = (int64_t)groups.size();
                groups.emplace_back();
            }
            groups[index_of[r]].push_back((int64_t)j);
        }
        for (const auto& grp : groups) {
            if (grp.size() != groups[0].size()) chains = false;
            for (int64_t w : grp)
                if (ntiles[w] != ntiles[grp[0]]) chains = false;
        }
        if (groups.empty() || groups[0].size() < 2) chains = false;
    }
    if (chains) {
        for (size_t j = 0; j < n; ++j) pe[j].clear();  // the order inside a block replaces every counter
        std::fill(need_tile.begin(), need_tile.end(), 0);
    }
    std::vector<int64_t> desc_sync(n, -1), tile_sync0(n, -1);
    for (size_t i = 0; i < n; ++i) {
        if (need_desc[i]) {
            desc_sync[i] = (int64_t)p->sync_per_epoch.size();
            p->sync_per_epoch.push_back((uint32_t)ntiles[i]);
        }
        if (need_tile[i]) {
            tile_sync0[i] = (int64_t)p->sync_per_epoch.size();
            p->sync_per_epoch.insert(p->sync_per_epoch.end(), (size_t)ntiles[i], 1u);
        }
    }
    if (p->sync_per_epoch.size() > 0x7fffffffull) {
        delete p;
        return HCCL_ERR_INVALID_ARG;
    }

    // ---- descriptors, tiles, waits
    p->descs.resize(n);
    for (size_t i = 0; i < n; ++i) {
        const hccl_wqe_t& w = g->wqes[i].w;
        Desc d;
        std::memset(&d, 0, sizeof(d));
        d.op = (uint8_t)((is_data_op(w.op) && w.count == 0) ? HCCL_OP_NOOP : w.op);
        d.dt_dst = (uint8_t)w.dtype_dst; d.dt_a = (uint8_t)w.dtype_a; d.dt_b = (uint8_t)w.dtype_b;
        d.kind_dst = (uint8_t)w.dst.kind; d.kind_a = (uint8_t)w.a.kind; d.kind_b = (uint8_t)w.b.kind;
        d.cmp = (uint8_t)((w.op == HCCL_OP_WAIT) ? w.cmp : w.hints);  // data ops carry their cache hints here
        d.rank_dst = (uint16_t)w.dst.rank; d.rank_a = (uint16_t)w.a.rank;
        if (w.op == HCCL_OP_COPY || w.op == HCCL_OP_REDUCE_N) d.ndst = (uint16_t)wqe_ndst(w); else d.rank_b = (uint16_t)w.b.rank;
        d.nsrc = (uint16_t)w.nsrc;
        d.off_dst = w.dst.offset; d.off_a = w.a.offset; d.off_b = w.b.offset;
        d.count = w.count;
        d.value = w.value; d.value_per_epoch = w.value_per_epoch;
        p->descs[i] = d;
        if (chains) continue;  // tiles are laid out chain by chain below

        if (pf[i].size() + pe[i].size() > 0xffff) {
            delete p;
            return HCCL_ERR_INVALID_ARG;
        }
        for (int64_t k = 0; k < ntiles[i]; ++k) {
            Tile t;
            std::memset(&t, 0, sizeof(t));
            t.desc = (uint32_t)i;
            if (tcount[i] > 0) {
                t.start = (uint64_t)(k * tcount[i]);
                t.count = (uint32_t)std::min<int64_t>(tcount[i], w.count - k * tcount[i]);
            }
            t.signal[0] = tile_sync0[i] >= 0 ? (int32_t)(tile_sync0[i] + k) : -1;
            t.signal[1] = desc_sync[i] >= 0 ? (int32_t)desc_sync[i] : -1;
            t.wait_off = (uint32_t)p->waits.size();
            for (int64_t q : pf[i]) p->waits.push_back(Wait{(uint32_t)desc_sync[q], (uint32_t)ntiles[q]});
            for (int64_t q : pe[i]) p->waits.push_back(Wait{(uint32_t)(tile_sync0[q] + k), 1u});
            t.wait_cnt = (uint16_t)(p->waits.size() - t.wait_off);
            p->tiles.push_back(t);
        }
        if (p->tiles.size() > 0x7ffffff0ull || p->waits.size() > 0xfffffff0ull) {
            delete p;
            return HCCL_ERR_INVALID_ARG;
        }
    }

    if (chains) {
        // chain c = tile k of every WQE of one group, in issue order; chains are numbered group by group
        const uint64_t group_len = groups[0].size();
        uint64_t n_chains = 0;
        for (const auto& grp : groups) n_chains += (uint64_t)ntiles[grp[0]];
        if (n_chains * group_len > 0x7ffffff0ull) {
            delete p;
            return HCCL_ERR_INVALID_ARG;
        }
        p->tiles.reserve((size_t)(n_chains * group_len));
        for (const auto& grp : groups) {
            for (int64_t k = 0; k < ntiles[grp[0]]; ++k) {
                for (int64_t w : grp) {
                    const hccl_wqe_t& q = g->wqes[w].w;
                    Tile t;
                    std::memset(&t, 0, sizeof(t));
                    t.desc = (uint32_t)w;
                    if (tcount[w] > 0) {
                        t.start = (uint64_t)(k * tcount[w]);
                        t.count = (uint32_t)std::min<int64_t>(tcount[w], q.count - k * tcount[w]);
                    }
                    t.signal[0] = t.signal[1] = -1;
                    p->tiles.push_back(t);
                }
            }
        }
        p->chain_len = (uint32_t)group_len;
        p->n_chains = (uint32_t)n_chains;
        p->opts.sm_budget = (int32_t)std::max<uint64_t>(1, std::min<uint64_t>((uint64_t)p->opts.sm_budget, n_chains));
    }

    compute_layout(p);

    hccl_plan_info_t& I = p->info;
    std::memset(&I, 0, sizeof(I));
    I.n_wqe = (int64_t)n;
    I.n_tiles = (int64_t)p->tiles.size();
    I.n_syncs = (int64_t)p->sync_per_epoch.size();
    I.chain_depth = max_depth;
    I.schedule_bytes = schedule;
    int64_t sb = 0, rb = 0;
    for (int r = 0; r < g->R; ++r) { sb += g->send_bytes[r]; rb += g->recv_bytes[r]; }
    I.compulsory_bytes = g->compulsory_bytes >= 0 ? g->compulsory_bytes : sb + rb;
    I.scratch_bytes = p->scratch_bytes;
    I.send_bytes_total = sb;
    I.recv_bytes_total = rb;
    I.R = g->R;
    I.sm_budget = p->opts.sm_budget;
    I.threads = p->opts.threads;
    I.engine = p->opts.engine;
    // the largest work item actually cut, in bytes of its widest operand (planners set tile sizes per WQE)
    int64_t widest_tile = 0;
    for (size_t i = 0; i < n; ++i) {
        const hccl_wqe_t& w = g->wqes[i].w;
        if (tcount[i] > 0) widest_tile = std::max<int64_t>(widest_tile, std::min<int64_t>(tcount[i], w.count) * widest(w) * (w.op == HCCL_OP_REDUCE_N ? std::max<int>(w.nsrc, 1) : 1));
    }
    I.tile_bytes = widest_tile > 0 ? widest_tile : (int64_t)tile_bytes;
    I.crossrack_bytes = crossrack;
    I.static_chains = (int64_t)p->n_chains;
    *out = p;
    return HCCL_OK;
}

void hccl::compute_layout(hccl_plan* p) {
    Layout& L = p->layout;
    uint64_t o = 0;
    L.control = o; o = align_up(o + sizeof(Control), 256);
    L.counters = o; o = align_up(o + 4ull * std::max<size_t>(p->sync_per_epoch.size(), 1), 256);
    L.signals = o; o = align_up(o + 8ull * std::max<int32_t>(p->n_signals, 1), 256);
    L.descs = o; o = align_up(o + sizeof(Desc) * std::max<size_t>(p->descs.size(), 1), 256);
    L.tiles = o; o = align_up(o + sizeof(Tile) * std::max<size_t>(p->tiles.size(), 1), 256);
    L.waits = o; o = align_up(o + sizeof(Wait) * std::max<size_t>(p->waits.size(), 1), 256);
    L.scratch = o; o = align_up(o + (uint64_t)p->scratch_bytes, 256);
    L.total = o;
    p->chain_wide = p->chain_copies = false;
    for (const Desc& d : p->descs) p->chain_copies = p->chain_copies || d.op == HCCL_OP_COPY;
    for (const Desc& d : p->descs)
        if (d.op == HCCL_OP_REDUCE && (d.dt_b == HCCL_FP32 || (d.kind_a == HCCL_BUF_SEND && d.dt_a == HCCL_FP32))) p->chain_wide = true;
}

extern "C" {

hccl_status_t hccl_plan_workspace_bytes(const hccl_plan_t* p, size_t* bytes) {
    if (!p || !bytes) return HCCL_ERR_INVALID_ARG;
    *bytes = (size_t)p->layout.total;
    return HCCL_OK;
}

hccl_status_t hccl_plan_info(const hccl_plan_t* p, hccl_plan_info_t* out) {
    if (!p || !out) return HCCL_ERR_INVALID_ARG;
    *out = p->info;
    out->epoch = p->epoch;
    return HCCL_OK;
}

hccl_status_t hccl_plan_layout(const hccl_plan_t* p, int64_t offsets[8]) {
    if (!p || !offsets) return HCCL_ERR_INVALID_ARG;
    const Layout& L = p->layout;
    const uint64_t v[8] = {L.control, L.counters, L.signals, L.descs, L.tiles, L.waits, L.scratch, L.total};
    for (int i = 0; i < 8; ++i) offsets[i] = (int64_t)v[i];
    return HCCL_OK;
}

hccl_status_t hccl_plan_extents(const hccl_plan_t* p, int rank, int64_t* send_bytes, int64_t* recv_bytes) {
    if (!p || rank < 0 || rank >= p->R) return HCCL_ERR_INVALID_ARG;
    if (send_bytes) *send_bytes = p->send_bytes[rank];
    if (recv_bytes) *recv_bytes = p->recv_bytes[rank];
    return HCCL_OK;
}

hccl_status_t hccl_plan_set_user_signals(hccl_plan_t* p, void* dev_signals, int64_t n_slots) {
    if (!p || n_slots < 0 || (n_slots > 0 && !dev_signals)) return HCCL_ERR_INVALID_ARG;
    if (((uintptr_t)dev_signals) % 8) return HCCL_ERR_ALIGNMENT;
    p->user_signals = dev_signals;
    p->n_user_signals = n_slots;
    return HCCL_OK;
}

hccl_status_t hccl_plan_set_trace(hccl_plan_t* p, void* dev_trace, int64_t capacity_items) {
    if (!p || capacity_items < 0 || (capacity_items > 0 && !dev_trace)) return HCCL_ERR_INVALID_ARG;
    if (((uintptr_t)dev_trace) % 8) return HCCL_ERR_ALIGNMENT;
    p->trace = capacity_items ? dev_trace : nullptr;
    p->trace_cap = capacity_items;
    return HCCL_OK;
}

hccl_status_t hccl_plan_set_trigger(hccl_plan_t* p, int64_t wait_slot, int32_t cmp, uint64_t wait_value,
                                    uint64_t wait_per_epoch, int64_t set_slot, uint64_t set_value, uint64_t set_per_epoch) {
    if (!p) return HCCL_ERR_INVALID_ARG;
    if (wait_slot >= p->n_user_signals || set_slot >= p->n_user_signals) return HCCL_ERR_INVALID_ARG;
    if (wait_slot >= 0 && (cmp < HCCL_CMP_EQ || cmp > HCCL_CMP_LT)) return HCCL_ERR_INVALID_ARG;
    p->trig_wait_slot = wait_slot;
    p->trig_cmp = cmp;
    p->trig_wait_value = wait_value;
    p->trig_wait_per_epoch = wait_per_epoch;
    p->trig_set_slot = set_slot;
    p->trig_set_value = set_value;
    p->trig_set_per_epoch = set_per_epoch;
    return HCCL_OK;
}

void hccl_plan_destroy(hccl_plan_t* p) { delete p; }

const char* hccl_status_string(hccl_status_t s) {
    switch (s) {
        case HCCL_OK: return "ok";
        case HCCL_ERR_INVALID_ARG: return "invalid argument";
        case HCCL_ERR_DTYPE: return "unsupported element type";
        case HCCL_ERR_COUNT_MISMATCH: return "send/receive counts do not match";
        case HCCL_ERR_OVERLAP: return "overlapping ranges";
        case HCCL_ERR_ALIGNMENT: return "misaligned buffer or offset";
        case HCCL_ERR_WORKSPACE: return "workspace too small";
        case HCCL_ERR_BUSY: return "plan busy";
        case HCCL_ERR_CUDA: return "CUDA runtime error";
        case HCCL_ERR_TIMEOUT: return "device-side wait timed out";
        case HCCL_ERR_BAD_DESCRIPTOR: return "malformed descriptor table";
        case HCCL_ERR_NOT_BOUND: return "plan not bound to a workspace";
        case HCCL_ERR_HAZARD: return "conflicting work items not ordered by a dependency";
    }
    return "unknown status";
}

int hccl_version(void) { return 200; }

void hccl_opts_for_overlap(hccl_opts_t* o) {
    if (!o) return;
    std::memset(o, 0, sizeof(*o));
    o->engine = HCCL_ENGINE_LSU;
    o->light = 1;
    o->threads = 128;
    o->sm_budget = 12;
}

}  // extern "C"
