// Device-visible tables of a compiled work packet. Plain data, fixed layout: written by the host
// planner, uploaded once at bind time, read by the executor kernel and by the host-side plan checker.
//
// Vocabulary (paper Sec. III-B.2): a WQE becomes one descriptor; a descriptor with data is cut into
// tiles, the unit a thread block ("message engine") claims; a sync object is a device-side counter
// that tiles bump on completion and later tiles wait on (the compiled form of the dependency kinds).
#pragma once
#include <stdint.h>

namespace hccl {

struct alignas(16) Desc {  // 64 bytes
    uint8_t op, dt_dst, dt_a, dt_b;          // hccl_op_t, hccl_dtype_t x3
    uint8_t kind_dst, kind_a, kind_b, cmp;   // hccl_buf_t x3, hccl_cmp_t
    uint16_t rank_dst, rank_a;
    union {
        uint16_t rank_b;                     // REDUCE: rank of operand B
        uint16_t ndst;                       // COPY, REDUCE_N: destinations written (0 and 1 both mean one);
    };                                       // destination k is the receive buffer of rank (rank_dst + k) mod R
    uint16_t nsrc;                           // REDUCE_N only
    int64_t off_dst, off_a, off_b;           // byte offsets (data) or slot index (signals)
    int64_t count;                           // bytes (COPY) or elements (REDUCE, REDUCE_N)
    uint64_t value, value_per_epoch;         // WAIT / SET operand
};
static_assert(sizeof(Desc) == 64, "Desc layout");

// Number of destinations a data descriptor writes.
#if defined(__CUDACC__)
__host__ __device__
#endif
inline int ndst_of(const Desc& d) { return (d.op == 0 /*COPY*/ || d.op == 2 /*REDUCE_N*/) && d.ndst > 1 ? (int)d.ndst : 1; }

struct alignas(16) Tile {  // 32 bytes
    uint32_t desc;      // index into descs
    uint32_t count;     // elements / bytes covered by this tile
    uint64_t start;     // first element / byte of the tile inside its descriptor
    int32_t signal[2];  // sync objects bumped on completion (-1: none): [0] per tile, [1] per descriptor
    uint32_t wait_off;  // first entry in waits[]
    uint16_t wait_cnt;
    uint16_t flags;
};
static_assert(sizeof(Tile) == 32, "Tile layout");

// A waiter in epoch e (1, 2, ...) proceeds when counters[sync] has received e * per_epoch bumps.
struct Wait {
    uint32_t sync;
    uint32_t per_epoch;
};

// First 256 bytes of the workspace. Zeroed at bind time; the last block to leave an execution
// resets `ticket` and `exits` so the next launch starts clean (completion/status, cf. Sec. V-C).
struct Control {
    uint32_t ticket;      // next tile to hand out (dispatch, the control core's job, Sec. II-A.1)
    uint32_t exits;       // blocks that have left this execution
    uint32_t abort;       // == epoch: some block gave up in this execution; everyone drains and leaves
    uint32_t fail_epoch;  // epoch of the last execution that recorded a failure
    uint32_t status;      // hccl_status_t recorded by that failure
    uint32_t done_epoch;  // epoch of the last completed execution
    uint64_t detail;      // tile index behind the failure
    uint64_t t_first_ns, t_last_ns;  // globaltimer at first claim / last exit of the last execution
    uint32_t server_go;   // resident executor: epoch every block may now run, all ones = leave
    uint32_t pad;
};

struct Layout {  // byte offsets inside the workspace
    uint64_t control, counters, signals, descs, tiles, waits, scratch, total;
};

// TILE_FLAG_END: written by the device-side table builder of the device-resident AllToAllv behind the last real work
// item of an execution; a block that claims such an item has no more work (the number of items is then known
// only on the device).
enum : uint16_t { TILE_FLAG_NONE = 0, TILE_FLAG_END = 1 };

}  // namespace hccl
