// The register engine compiled to at most 64 registers per thread: two 512-thread blocks (or four of 256) fit
// one SM, and a block of 256 threads leaves three quarters of the register file to whatever else runs there.
#include "kernels.cuh"

namespace hccl {

__global__ void __launch_bounds__(512, 2) hccl_executor_lsu_light(const __grid_constant__ ExecParams p) { executor_lsu_body<false, false>(p); }

}  // namespace hccl
