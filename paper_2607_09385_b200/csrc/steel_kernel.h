// Launch interface of the attention kernel (implemented in steel_kernel.cu).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>

#include "../../include/steel_attn.h"
#include "steel_plan.h"

namespace steel {

// Opt the kernels in to their dynamic shared-memory size on the current device.
cudaError_t configure_kernels();

// Enqueue the persistent kernel: `grid` CTAs of 384 threads, one per SM.  `exp_emulation` selects the
// build with 0, 12.5, 25 or 50 % of the exponentials on the FMA pipe (values 0..3).
cudaError_t launch_attention(int head_dim, int exp_emulation, const CUtensorMap &map_q, const CUtensorMap &map_k,
                             const CUtensorMap &map_v, const KernelParams &params, int grid, cudaStream_t stream);

// The three tensor maps of one (q, k, v) pointer triple; a caller that runs the same tensors again
// skips the driver's encode calls.
struct TensorMaps {
  CUtensorMap q, k, v;
  const void *q_ptr = nullptr, *k_ptr = nullptr, *v_ptr = nullptr;
};

// Tensor maps for the caller's tensors (taken from `cache` when it holds the same pointers) + kernel
// launch, given list / status pointers already set in `params` (implemented in steel_attn.cu).
steel_status_t launch_with_params(const steel_attn_params_t &problem, KernelParams params, int grid,
                                  const void *q, const void *k, const void *v, void *o, float *lse,
                                  cudaStream_t stream, TensorMaps *cache);

}  // namespace steel
