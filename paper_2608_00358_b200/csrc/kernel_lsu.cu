// The register engine, one block per SM (up to 128 registers per thread).
#include "kernels.cuh"

namespace hccl {

__global__ void __launch_bounds__(512, 1) hccl_executor_lsu(const __grid_constant__ ExecParams p) { executor_lsu_body<false, true>(p); }

}  // namespace hccl
