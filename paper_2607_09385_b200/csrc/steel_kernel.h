// Launch interface of the attention kernel (implemented in steel_kernel.cu).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/steel_attn.h"
#include "steel_plan.h"

namespace steel {

// Opt the kernels in to their dynamic shared-memory size on the current device.
cudaError_t configure_kernels();

// Enqueue the persistent kernel: `grid` CTAs of 320 threads, one per SM.
cudaError_t launch_attention(int head_dim, const CUtensorMap &map_q, const CUtensorMap &map_k,
                             const CUtensorMap &map_v, const KernelParams &params, int grid, cudaStream_t stream);

// Tensor maps for the caller's tensors + kernel launch, given list / status pointers already set in
// `params` (implemented in steel_attn.cu).
steel_status_t launch_with_params(const steel_attn_params_t &problem, KernelParams params, int grid,
                                  const void *q, const void *k, const void *v, void *o, float *lse,
                                  cudaStream_t stream);

}  // namespace steel
