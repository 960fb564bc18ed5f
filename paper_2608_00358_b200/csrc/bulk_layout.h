// Shared-memory layout of the bulk engine, needed by the kernel and by the host code that sizes its launch.
#pragma once
#include <stdint.h>

#include "tables.h"

namespace hccl {
namespace bulk {

constexpr uint32_t MAX_STAGES = 8;
constexpr uint32_t STAGE_BYTES = 49152;       // default stage: a COPY piece fills a stage; a REDUCE piece splits it into A and B;
                                              // 4 x 48 KiB + bookkeeping fits the 227 KB a block may have
constexpr uint32_t MIN_STAGE_BYTES = 12288, MAX_STAGE_BYTES = 98304;  // opts.stage_kib lies in this range
// Elements per REDUCE piece: as many as fit a stage with both operands, in whole multiples of 512 elements
// (48 KiB stages: 6144 for fp32+fp32, 8192 for fp32+16-bit, 12288 for 16-bit+16-bit).
__host__ __device__ constexpr uint32_t piece_elems(uint32_t stage_bytes, uint32_t ea, uint32_t eb) { return stage_bytes / (ea + eb) / 512 * 512; }
// Stages and stage size of a launch from the options (0 = default), and the dynamic shared memory they need.
struct StageConfig { uint32_t ns, stage_bytes; size_t smem; };
constexpr size_t MAX_DYNAMIC_SMEM = 227 * 1024 - 1024;   // a block may have 227 KB; the kernel's static shared memory comes out of it too

// PIECE_COPY: loaded and stored by the bulk unit. PIECE_COPYW: loaded by the bulk unit, stored by the compute
// warps from shared memory (the stage is free as soon as the warps have read it, without waiting for a
// bulk store to drain, so more of the stage ring is loads in flight).
enum : uint32_t { PIECE_COPY = 0, PIECE_REDUCE = 1, PIECE_TILE = 2, PIECE_EXIT = 3, PIECE_COPYW = 4 };

struct alignas(16) PieceInfo;
StageConfig stage_config(int stages_opt, int stage_kib_opt);

struct alignas(16) PieceInfo {  // one per stage, in shared memory; written by the DMA thread
    uint32_t kind;
    uint32_t n;           // REDUCE: elements; COPY: bytes
    uint32_t last;        // last piece of its work item: publish the item's completion after it
    uint32_t tile_index;
    char* dst;            // global destination of this piece
    unsigned long long group;  // COPY: sequence number of the bulk store group that drains this stage
    int32_t signal[2];
    uint8_t dt_a, dt_b, dt_d, evict_first;
    uint32_t b_off;       // REDUCE: byte offset of operand B inside the stage
    uint32_t keep_dst;    // REDUCE: the result is an FP32 partial in scratch, stored with an evict-last L2 policy
    uint32_t discard_bytes;   // REDUCE: ... and this many bytes from discard_src (operand A's global address, or null)
    const char* discard_src;  //         were read for the last time: their L2 lines may be dropped
    uint16_t ndst, rank_dst;   // COPY with several destinations: receive buffers of ranks rank_dst .. +ndst-1 (mod R)
    unsigned long long dst_off;  // ... at this byte offset (dst is then the first of them)
    Tile tile;            // PIECE_TILE: the work item and its descriptor for the register path
    Desc desc;
};

inline StageConfig stage_config(int stages_opt, int stage_kib_opt) {
    uint32_t sb = stage_kib_opt > 0 ? (uint32_t)stage_kib_opt * 1024u : STAGE_BYTES;
    sb = sb / 1024u * 1024u;
    if (sb < MIN_STAGE_BYTES) sb = MIN_STAGE_BYTES;
    if (sb > MAX_STAGE_BYTES) sb = MAX_STAGE_BYTES;
    const size_t per = (size_t)sb + sizeof(PieceInfo) + 16, room = MAX_DYNAMIC_SMEM - 128;
    uint32_t ns = stages_opt > 0 ? (uint32_t)stages_opt : (uint32_t)(4u * STAGE_BYTES / sb);   // default: the same bytes in flight
    if (ns < 2) ns = 2;
    if (ns > MAX_STAGES) ns = MAX_STAGES;
    while (ns > 2 && ns * per > room) --ns;
    return StageConfig{ns, sb, ns * per + 128};
}

}  // namespace bulk
}  // namespace hccl
