// Host-side objects behind the opaque handles of hccl.h.
#pragma once
#include <algorithm>
#include <cstdint>
#include <string>
#include <vector>

#include "../../include/hccl.h"
#include "tables.h"

namespace hccl {

inline int elem_bytes(int dt) { return dt == HCCL_FP32 ? 4 : 2; }
inline bool valid_dtype(int dt) { return dt == HCCL_FP32 || dt == HCCL_BF16 || dt == HCCL_FP16; }
inline uint64_t align_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

struct Wqe {
    hccl_wqe_t w;
    int32_t subgraph;
    std::vector<int64_t> preds_full;  // WQE ids this one waits for entirely
    std::vector<int64_t> preds_elem;  // WQE ids waited for tile by tile
};

struct Subgraph {
    int rank;
    std::vector<int64_t> wqes;        // ids in issue order
    int64_t last_sync = -1;           // last WQE that carried HCCL_DEP_SYNC
    bool fence_pending = false;       // previous WQE carried HCCL_DEP_FENCE
};

}  // namespace hccl

struct hccl_graph {
    int R = 0;
    std::vector<int64_t> send_bytes, recv_bytes;
    int64_t scratch_bytes = 0;
    int32_t n_signals = 0;
    std::vector<hccl::Subgraph> subgraphs;
    std::vector<hccl::Wqe> wqes;
    int64_t compulsory_bytes = -1;    // planners may state it; -1: derive from extents
};

struct hccl_plan {
    int R = 0;
    hccl_opts_t opts{};
    std::vector<int64_t> send_bytes, recv_bytes;
    int64_t scratch_bytes = 0;
    int32_t n_signals = 0;
    std::vector<hccl::Desc> descs;
    std::vector<hccl::Tile> tiles;
    std::vector<hccl::Wait> waits;
    std::vector<uint32_t> sync_per_epoch;  // bumps each sync object receives per execution
    hccl::Layout layout{};
    // static chains (HCCL_FLAG_STATIC_CHAINS): tiles [c*chain_len, (c+1)*chain_len) form chain c, run in order by one block
    uint32_t chain_len = 0, n_chains = 0;
    bool chain_copies = false;  // forwarding kernel: the packet has COPY items (the build that forwards them too)
    bool chain_wide = false;  // forwarding kernel: an FP32 operand arrives through the stages (3 stages of FP32 pieces instead of 6 of 16-bit ones)
    int buf_align = 1;                     // alignment every send/receive pointer must have (largest element read or written)
    hccl_plan_info_t info{};
    // device-triggered execution (Sec. IV-B.3)
    void* user_signals = nullptr;
    int64_t n_user_signals = 0;
    int64_t trig_wait_slot = -1, trig_set_slot = -1;
    int32_t trig_cmp = 0;
    uint64_t trig_wait_value = 0, trig_wait_per_epoch = 0, trig_set_value = 0, trig_set_per_epoch = 0;
    // device-resident AllToAllv (Sec. IV-B.2): sizes are read from device memory when the kernel runs
    bool dynamic = false;
    bool dyn_device_tables = false;        // descriptors and tiles are written by a kernel at execute time
    uint32_t dyn_end_tiles = 0;            // END markers kept behind the last real tile
    int64_t dyn_row_bytes = 0;
    std::vector<int64_t> dyn_max_send_rows, dyn_max_recv_rows;
    const void* dyn_counts = nullptr;
    void* dyn_recvcounts_out = nullptr;
    void* dyn_rdispls_out = nullptr;
    // optional per-item timestamps
    void* trace = nullptr;
    int64_t trace_cap = 0;
    // resident executor: the caller's doorbell record while a server kernel is running
    void* server_db = nullptr;
    uint64_t server_rings = 0;
    // binding
    void* workspace = nullptr;
    size_t workspace_bytes = 0;
    uint32_t epoch = 0;
    // last pointer set that passed the aliasing check
    std::vector<const void*> checked_send;
    std::vector<void*> checked_recv;
};

namespace hccl {
// Elements (bytes for COPY) that one pass of all data-moving threads of a block covers, per operation.
// Tiles that are whole multiples of it leave no partly idle pass at the end of a tile.
inline int64_t sweep_of(const hccl_opts_t& o, int op) {
    if (o.engine == HCCL_ENGINE_BULK) {
        if (op == HCCL_OP_COPY) return 49152;                 // one stage
        if (op == HCCL_OP_REDUCE) return 24576;               // whole pieces for every operand mix (6144, 8192, 12288)
        return (int64_t)(o.threads - 96) * 8;                 // multi-input sums run on the compute warps
    }
    const int64_t workers = o.threads - 32;
    if (op == HCCL_OP_COPY) return workers * 128;             // 8 x 16 bytes per thread
    if (op == HCCL_OP_REDUCE) return workers * 32;            // 4 x 8 elements per thread
    return workers * 8;                                       // REDUCE_N: 8 elements per thread
}
// Default tile size, in the operation's count units, for work of `total_units` spread over `blocks` blocks:
// about `per_block` tiles per block, a power of two between lo and hi, then whole passes of the threads.
inline int64_t nearest_pow2(int64_t x) {
    int64_t p = 1;
    while (p * 2 <= x) p *= 2;
    return (x - p > 2 * p - x) ? 2 * p : p;
}
inline int64_t round_tile(int64_t target, int64_t sweep);
inline int64_t default_tile(int64_t total_units, int blocks, int per_block, int64_t lo, int64_t hi, int64_t sweep) {
    const int64_t want = nearest_pow2(std::max<int64_t>(1, total_units / std::max(1, blocks * per_block)));
    return round_tile(std::min(hi, std::max(lo, want)), sweep);
}
inline int64_t round_tile(int64_t target, int64_t sweep) {
    if (target >= sweep) return target / sweep * sweep;
    return std::max<int64_t>(64, (target + 63) / 64 * 64);
}
hccl_status_t compile_graph(const hccl_graph* g, const hccl_opts_t* opts, hccl_plan** out);
void compute_layout(hccl_plan* p);  // workspace offsets from the sizes of the plan's tables
void fill_default_opts(hccl_opts_t* o, const hccl_opts_t* in);
hccl_status_t plan_alltoallv_window(int R, const int64_t* sendcounts, const int64_t* sdispls, const int64_t* recvcounts,
                                    const int64_t* rdispls, hccl_dtype_t dt, int64_t row_elems, const hccl_opts_t* opts,
                                    int d_lo, int d_hi, hccl_plan_t** out);
}  // namespace hccl
