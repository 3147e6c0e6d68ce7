// Launch interface of the attention kernel (implemented in steel_kernel.cu).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "steel_plan.h"

namespace steel {

// Opt the kernels in to their dynamic shared-memory size on the current device.
cudaError_t configure_kernels();

// Enqueue the persistent kernel: `grid` CTAs of 320 threads, one per SM.
cudaError_t launch_attention(int head_dim, const CUtensorMap &map_q, const CUtensorMap &map_k,
                             const CUtensorMap &map_v, const KernelParams &params, int grid, cudaStream_t stream);

}  // namespace steel
