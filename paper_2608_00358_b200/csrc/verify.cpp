// Host-side verification of compiled plans: a tile-level hazard checker and an interpreter that runs
// the tables on host buffers in a random dependency-respecting order. Debugging aids for schedule
// authors; hccl_execute never comes here.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <map>
#include <random>

#include "plan.hpp"

using namespace hccl;

namespace {

struct Access {
    int buf;         // dense id of the buffer: kind * (MAX_RANKS + 1) + rank
    int64_t lo, hi;  // byte range [lo, hi)
    bool write;
    uint32_t tile;
};

int buf_id(int kind, int rank) { return kind * (HCCL_MAX_RANKS + 1) + (kind == HCCL_BUF_SCRATCH ? 0 : rank); }

void tile_accesses(const hccl_plan* p, uint32_t ti, std::vector<Access>& out) {
    const Tile& t = p->tiles[ti];
    const Desc& d = p->descs[t.desc];
    auto add = [&](int kind, int rank, int64_t off, int64_t bytes, bool w) {
        if (bytes > 0) out.push_back(Access{buf_id(kind, rank), off, off + bytes, w, ti});
    };
    switch (d.op) {
        case HCCL_OP_COPY:
            add(d.kind_a, d.rank_a, d.off_a + (int64_t)t.start, t.count, false);
            for (int j = 0; j < ndst_of(d); ++j)
                add(d.kind_dst, (d.rank_dst + j) % p->R, d.off_dst + (int64_t)t.start, t.count, true);
            break;
        case HCCL_OP_REDUCE: {
            const int ea = elem_bytes(d.dt_a), eb = elem_bytes(d.dt_b), ed = elem_bytes(d.dt_dst);
            add(d.kind_a, d.rank_a, d.off_a + (int64_t)t.start * ea, (int64_t)t.count * ea, false);
            add(d.kind_b, d.rank_b, d.off_b + (int64_t)t.start * eb, (int64_t)t.count * eb, false);
            add(d.kind_dst, d.rank_dst, d.off_dst + (int64_t)t.start * ed, (int64_t)t.count * ed, true);
            break;
        }
        case HCCL_OP_REDUCE_N: {
            const int ea = elem_bytes(d.dt_a), ed = elem_bytes(d.dt_dst);
            for (int k = 0; k < d.nsrc; ++k)
                add(d.kind_a, (d.rank_a + k) % p->R, d.off_a + (int64_t)t.start * ea, (int64_t)t.count * ea, false);
            for (int j = 0; j < ndst_of(d); ++j)
                add(d.kind_dst, (d.rank_dst + j) % p->R, d.off_dst + (int64_t)t.start * ed, (int64_t)t.count * ed, true);
            break;
        }
        case HCCL_OP_WAIT:
            add(d.kind_a, 0, d.off_a * 8, 8, false);
            break;
        case HCCL_OP_SET:
            add(d.kind_dst, 0, d.off_dst * 8, 8, true);
            break;
        default:
            break;
    }
}

inline float bf16_to_f32(uint16_t h) {
    uint32_t u = (uint32_t)h << 16;
    float f;
    std::memcpy(&f, &u, 4);
    return f;
}
inline uint16_t f32_to_bf16(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    if ((u & 0x7fffffffu) > 0x7f800000u) return 0x7fc0;  // NaN
    u += 0x7fffu + ((u >> 16) & 1u);                     // nearest even on the dropped 16 bits
    return (uint16_t)(u >> 16);
}
inline float fp16_to_f32(uint16_t h) {
    const int s = h >> 15, e = (h >> 10) & 31, m = h & 1023;
    float v;
    if (e == 0) v = std::ldexp((float)m, -24);
    else if (e == 31) v = m ? NAN : INFINITY;
    else v = std::ldexp((float)(m | 1024), e - 25);
    return s ? -v : v;
}
inline uint16_t f32_to_fp16(float f) {
    uint32_t u;
    std::memcpy(&u, &f, 4);
    const uint32_t sign = (u >> 16) & 0x8000u;
    u &= 0x7fffffffu;
    if (u > 0x7f800000u) return (uint16_t)(sign | 0x7e00);
    if (u >= 0x477ff000u) return (uint16_t)(sign | 0x7c00);  // >= 65520 rounds to infinity
    if (u < 0x38800000u) {                                   // below the smallest normal: fixed quantum 2^-24
        float a;
        std::memcpy(&a, &u, 4);
        const float q = std::nearbyint(std::ldexp(a, 24));   // ties to even
        return (uint16_t)(sign | (uint32_t)q);
    }
    uint32_t r = u - 0x38000000u;                            // rebias 127 -> 15
    r += 0xfffu + ((r >> 13) & 1u);
    return (uint16_t)(sign | (r >> 13));
}

inline float load_f(const char* p, int dt, int64_t i) {
    if (dt == HCCL_FP32) {
        float f;
        std::memcpy(&f, p + 4 * i, 4);
        return f;
    }
    uint16_t h;
    std::memcpy(&h, p + 2 * i, 2);
    return dt == HCCL_BF16 ? bf16_to_f32(h) : fp16_to_f32(h);
}
inline void store_f(char* p, int dt, int64_t i, float v) {
    if (dt == HCCL_FP32) {
        std::memcpy(p + 4 * i, &v, 4);
    } else {
        uint16_t h = dt == HCCL_BF16 ? f32_to_bf16(v) : f32_to_fp16(v);
        std::memcpy(p + 2 * i, &h, 2);
    }
}

}  // namespace

extern "C" {

hccl_status_t hccl_plan_check_hazards(const hccl_plan_t* p, int64_t* n_violations) {
    if (!p || !n_violations) return HCCL_ERR_INVALID_ARG;
    const size_t nt = p->tiles.size();
    std::vector<Access> acc;
    for (uint32_t i = 0; i < nt; ++i) tile_accesses(p, i, acc);
    std::sort(acc.begin(), acc.end(), [](const Access& x, const Access& y) {
        return x.buf != y.buf ? x.buf < y.buf : (x.lo != y.lo ? x.lo < y.lo : x.tile < y.tile);
    });
    // conflicting pairs (older tile, newer tile), by sweeping each buffer's sorted ranges
    std::vector<std::vector<uint32_t>> partners(nt);
    for (size_t i = 0; i < acc.size(); ++i) {
        for (size_t j = i + 1; j < acc.size() && acc[j].buf == acc[i].buf && acc[j].lo < acc[i].hi; ++j) {
            if (!(acc[i].write || acc[j].write) || acc[i].tile == acc[j].tile) continue;
            uint32_t a = std::min(acc[i].tile, acc[j].tile), b = std::max(acc[i].tile, acc[j].tile);
            partners[b].push_back(a);
        }
    }
    // who bumps each sync object
    std::vector<std::vector<uint32_t>> bumpers(p->sync_per_epoch.size());
    for (uint32_t i = 0; i < nt; ++i)
        for (int k = 0; k < 2; ++k)
            if (p->tiles[i].signal[k] >= 0) bumpers[p->tiles[i].signal[k]].push_back(i);
    int64_t bad = 0;
    std::vector<uint32_t> mark(nt, 0xffffffffu), stack;
    for (uint32_t v = 0; v < nt; ++v) {
        if (partners[v].empty()) continue;
        std::sort(partners[v].begin(), partners[v].end());
        partners[v].erase(std::unique(partners[v].begin(), partners[v].end()), partners[v].end());
        const uint32_t floor = partners[v].front();
        // ancestors of v (through waits -> sync objects -> their bumpers), not below the oldest partner
        stack.assign(1, v);
        mark[v] = v;
        while (!stack.empty()) {
            const uint32_t x = stack.back();
            stack.pop_back();
            const Tile& t = p->tiles[x];
            for (uint32_t w = 0; w < t.wait_cnt; ++w) {
                for (uint32_t y : bumpers[p->waits[t.wait_off + w].sync]) {
                    if (y >= floor && mark[y] != v) {
                        mark[y] = v;
                        stack.push_back(y);
                    }
                }
            }
            // static chains: a tile runs after its predecessor in the chain, in the same block
            if (p->chain_len > 0 && x % p->chain_len != 0 && x - 1 >= floor && mark[x - 1] != v) {
                mark[x - 1] = v;
                stack.push_back(x - 1);
            }
        }
        for (uint32_t u : partners[v])
            if (mark[u] != v) ++bad;
    }
    *n_violations = bad;
    return HCCL_OK;
}

hccl_status_t hccl_plan_interpret_host(const hccl_plan_t* p, const void* const* host_send, void* const* host_recv,
                                       void* host_scratch, uint64_t* host_signals, uint64_t seed) {
    if (!p || !host_send || !host_recv) return HCCL_ERR_INVALID_ARG;
    if (p->scratch_bytes > 0 && !host_scratch) return HCCL_ERR_INVALID_ARG;
    const size_t nt = p->tiles.size();
    std::vector<uint32_t> counters(p->sync_per_epoch.size(), 0);
    std::vector<uint64_t> own_signals(std::max<int32_t>(p->n_signals, 1), 0);
    uint64_t* signals = host_signals ? host_signals : own_signals.data();
    auto base = [&](int kind, int rank) -> char* {
        if (kind == HCCL_BUF_SEND) return (char*)host_send[rank];
        if (kind == HCCL_BUF_RECV) return (char*)host_recv[rank];
        return (char*)host_scratch;
    };
    std::vector<char> done(nt, 0);
    auto ready = [&](const Tile& t) {
        if (p->chain_len > 0) {  // static chains: strictly in order inside a chain
            const size_t i = (size_t)(&t - p->tiles.data());
            if (i % p->chain_len != 0 && !done[i - 1]) return false;
        }
        for (uint32_t w = 0; w < t.wait_cnt; ++w) {
            const Wait& x = p->waits[t.wait_off + w];
            if (counters[x.sync] < x.per_epoch) return false;
        }
        const Desc& d = p->descs[t.desc];
        if (d.op == HCCL_OP_WAIT) {
            if (d.kind_a != HCCL_BUF_SIGNAL) return true;  // user signals are not modelled on the host
            const uint64_t v = signals[d.off_a], want = d.value + d.value_per_epoch;  // epoch 1
            switch (d.cmp) {
                case HCCL_CMP_EQ: return v == want;
                case HCCL_CMP_NE: return v != want;
                case HCCL_CMP_GE: return v >= want;
                case HCCL_CMP_GT: return v > want;
                case HCCL_CMP_LE: return v <= want;
                default: return v < want;
            }
        }
        return true;
    };
    auto run = [&](const Tile& t) {
        const Desc& d = p->descs[t.desc];
        switch (d.op) {
            case HCCL_OP_COPY:
                for (int j = 0; j < ndst_of(d); ++j)
                    std::memmove(base(d.kind_dst, (d.rank_dst + j) % p->R) + d.off_dst + t.start, base(d.kind_a, d.rank_a) + d.off_a + t.start, t.count);
                break;
            case HCCL_OP_REDUCE: {
                const char* a = base(d.kind_a, d.rank_a) + d.off_a;
                const char* b = base(d.kind_b, d.rank_b) + d.off_b;
                char* o = base(d.kind_dst, d.rank_dst) + d.off_dst;
                for (int64_t i = (int64_t)t.start; i < (int64_t)(t.start + t.count); ++i) {
                    volatile float s = load_f(a, d.dt_a, i) + load_f(b, d.dt_b, i);
                    store_f(o, d.dt_dst, i, s);
                }
                break;
            }
            case HCCL_OP_REDUCE_N: {
                for (int64_t i = (int64_t)t.start; i < (int64_t)(t.start + t.count); ++i) {
                    volatile float s = load_f(base(d.kind_a, d.rank_a) + d.off_a, d.dt_a, i);
                    for (int k = 1; k < d.nsrc; ++k) s = s + load_f(base(d.kind_a, (d.rank_a + k) % p->R) + d.off_a, d.dt_a, i);
                    for (int j = 0; j < ndst_of(d); ++j) store_f(base(d.kind_dst, (d.rank_dst + j) % p->R) + d.off_dst, d.dt_dst, i, s);
                }
                break;
            }
            case HCCL_OP_SET:
                if (d.kind_dst == HCCL_BUF_SIGNAL) signals[d.off_dst] = d.value + d.value_per_epoch;
                break;
            default:
                break;
        }
        for (int k = 0; k < 2; ++k)
            if (t.signal[k] >= 0) ++counters[t.signal[k]];
        done[(size_t)(&t - p->tiles.data())] = 1;
    };
    if (seed == 0) {
        for (size_t i = 0; i < nt; ++i) {
            if (!ready(p->tiles[i])) return HCCL_ERR_TIMEOUT;  // ticket order must always be runnable
            run(p->tiles[i]);
        }
        return HCCL_OK;
    }
    std::mt19937_64 rng(seed);
    std::vector<uint32_t> pending(nt);
    for (uint32_t i = 0; i < nt; ++i) pending[i] = i;
    while (!pending.empty()) {
        // collect the tiles that may run now, then run one of them at random
        std::vector<size_t> can;
        for (size_t k = 0; k < pending.size(); ++k)
            if (ready(p->tiles[pending[k]])) can.push_back(k);
        if (can.empty()) return HCCL_ERR_TIMEOUT;  // the graph cannot make progress
        // run a random half of the ready set, in random order, before looking again
        std::shuffle(can.begin(), can.end(), rng);
        const size_t take = std::max<size_t>(1, can.size() / 2);
        std::vector<size_t> chosen(can.begin(), can.begin() + take);
        for (size_t k : chosen) run(p->tiles[pending[k]]);
        std::sort(chosen.begin(), chosen.end(), std::greater<size_t>());
        for (size_t k : chosen) {
            pending[k] = pending.back();
            pending.pop_back();
        }
    }
    return HCCL_OK;
}

}  // extern "C"
