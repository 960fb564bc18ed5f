// Declarations of the library's kernels and of the parameter records only some of them take. Each kernel is
// defined in a translation unit of its own (kernel_*.cu) so that they compile in parallel; the host code
// (executor.cu) launches them through these declarations.
#pragma once
#include "device.cuh"

namespace hccl {

struct Doorbell {                       // layout shared with hccl_doorbell_t in hccl.h
    unsigned long long request;         // host -> device: number of executions asked for so far
    unsigned long long completed;       // device -> host: executions finished
    unsigned long long stop;            // host -> device: leave after the current execution
    unsigned long long exited;          // device -> host: the kernel has left (1 = stop, 2 = idle, 3 = failure)
    unsigned long long status, detail;  // device -> host: verdict of the last failed execution
    unsigned long long t_seen_ns, t_done_ns;  // device -> host: device clock when the last ring was seen / when its execution was over
};

constexpr int DYN_MAX_RANKS = 64;

struct DynParams {
    const long long* counts;       // device, [R*R], counts[s*R+d] rows from s to d
    long long* recvcounts_out;     // device, [R*R] indexed [d*R+s], or null
    long long* rdispls_out;        // device, [R*R] indexed [d*R+s], or null
    Control* ctl;
    unsigned long long* user_signals;
    uint32_t R, nblocks;
    unsigned long long timeout_ns;
    unsigned long long row_bytes, tile_bytes;
    long long trig_wait_slot, trig_set_slot;
    int trig_cmp, pad1;
    unsigned long long trig_wait_value, trig_wait_per_epoch, trig_set_value, trig_set_per_epoch;
    long long max_send_rows[DYN_MAX_RANKS], max_recv_rows[DYN_MAX_RANKS];
    const void* send[DYN_MAX_RANKS];
    void* recv[DYN_MAX_RANKS];
};

// Device-side table builder of the device-resident AllToAllv for any rank count (Sec. IV-B.2: the work requests
// are patched on the device): one block per source rank writes that source's R descriptors and their tiles
// into the bound workspace, where the ordinary executor, launched right behind it, finds them.
struct PatchParams {
    const long long* counts;       // device, [R*R], counts[s*R+d] rows from s to d
    long long* recvcounts_out;     // device, [R*R] indexed [d*R+s], or null
    long long* rdispls_out;        // device, [R*R] indexed [d*R+s], or null
    Control* ctl;
    unsigned long long* user_signals;
    Desc* descs;                   // [R*R] in the workspace, descriptor s*R+d = segment (s, d)
    Tile* tiles;                   // [tile_cap] in the workspace
    uint32_t R, tile_cap;          // tile_cap includes room for end_tiles END markers
    uint32_t end_tiles, pad0;
    unsigned long long timeout_ns;
    unsigned long long row_bytes, tile_bytes;
    long long trig_wait_slot;
    int trig_cmp, pad1;
    unsigned long long trig_wait_value, trig_wait_per_epoch;
    long long max_send_rows[HCCL_MAX_RANKS], max_recv_rows[HCCL_MAX_RANKS];
};

__global__ void __launch_bounds__(256, 1) hccl_a2a_patch(const __grid_constant__ PatchParams q);
__global__ void __launch_bounds__(512, 1) hccl_executor_lsu(const __grid_constant__ ExecParams p);
__global__ void __launch_bounds__(512, 2) hccl_executor_lsu_light(const __grid_constant__ ExecParams p);
__global__ void __launch_bounds__(512, 1) hccl_executor_bulk(const __grid_constant__ ExecParams p, const uint32_t ns, const uint32_t copy_by_warps,
                                                              const uint32_t stage_bytes);
// static chains on the bulk copy unit: running sums forwarded from step to step in registers
constexpr uint32_t CHAIN_SMEM_BYTES = 6 * 28672, CHAIN_PIECE_ELEMS = 14336, CHAIN_THREADS = 256;  // 6 stages of 16-bit pieces or 3 of FP32 pieces
__global__ void __launch_bounds__(256, 1) hccl_executor_chain(const __grid_constant__ ExecParams p, const uint32_t ns, const uint32_t stage_bytes);
__global__ void __launch_bounds__(256, 1) hccl_executor_chain_sums(const __grid_constant__ ExecParams p, const uint32_t ns, const uint32_t stage_bytes);  // packets without copies
__global__ void __launch_bounds__(512, 1) hccl_executor_resident(const __grid_constant__ ExecParams p, Doorbell* db,
                                                                  const unsigned long long idle_ns, const uint32_t first_epoch);
__global__ void __launch_bounds__(512, 1) hccl_a2a_dynamic(const __grid_constant__ DynParams q);

}  // namespace hccl
