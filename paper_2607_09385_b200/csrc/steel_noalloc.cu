// steel_attn_run_noalloc: the attention call for callers that must not allocate device memory.
//
// The regular path keeps its work lists (items, per-CTA ranges, key-tile step lists) and its status
// word in buffers that steel_attn_create obtains from cudaMalloc.  Some callers cannot do that: code
// running inside another framework's memory pool with the allocator locked, code on a latency path
// where cudaMalloc's implicit device synchronisation is not acceptable, or a process whose memory
// budget is fixed up front.  For them the same kernel runs with those lists in a fixed-size array
// that is part of the library image: every GPU that loads the library holds kScratchBytes for it
// until the process exits.  Inputs and outputs are still the caller's.
#include <cuda_runtime.h>

#include <mutex>
#include <new>

#include "../../include/steel_attn.h"
#include "steel_kernel.h"
#include "steel_planner.h"

using namespace steel;

namespace {

constexpr size_t kMaxItems = 16384;   // work items (64 bytes each)
constexpr size_t kMaxCtas = 1024;     // persistent CTAs (+1 range entry)
constexpr size_t kMaxSteps = 131072;  // explicit step-list entries of bitmap masks (8 bytes each)
constexpr size_t kOffStatus = 0;
constexpr size_t kOffItems = 256;
constexpr size_t kOffCtaBegin = kOffItems + kMaxItems * sizeof(WorkItem);
constexpr size_t kOffSteps = (kOffCtaBegin + (kMaxCtas + 1) * sizeof(int32_t) + 255) / 256 * 256;
constexpr size_t kScratchBytes = kOffSteps + kMaxSteps * sizeof(StepPair);  // about 2.0 MiB

// In host code this name is only a handle for the symbol, never a device address: the address the
// kernel needs comes from cudaGetSymbolAddress below.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mutex;
unsigned char *g_scratch_addr[kMaxDevices] = {};
int g_sm_count[kMaxDevices] = {};

// Once per device, with that device current: resolve the array's device address, read the SM
// count, opt the kernels in to their shared-memory size.
steel_status_t setup_device(int device, unsigned char **base, int *sm_count) {
  std::lock_guard<std::mutex> lock(g_mutex);
  if (!g_scratch_addr[device]) {
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return STEEL_ERR_CUDA;
    if (prop.major != 10) return STEEL_ERR_CUDA;
    void *ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_scratch) != cudaSuccess || !ptr) return STEEL_ERR_CUDA;
    if (configure_kernels() != cudaSuccess) return STEEL_ERR_CUDA;
    g_sm_count[device] = prop.multiProcessorCount;
    g_scratch_addr[device] = static_cast<unsigned char *>(ptr);
  }
  *base = g_scratch_addr[device];
  *sm_count = g_sm_count[device];
  return STEEL_OK;
}

}  // namespace

extern "C" steel_status_t steel_attn_run_noalloc(const steel_attn_params_t *params, const void *q, const void *k,
                                                 const void *v, void *o, float *lse, void *cuda_stream) {
  if (!q || !k || !v || !o) return STEEL_ERR_INVALID_ARG;
  const uintptr_t align = reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(k) |
                          reinterpret_cast<uintptr_t>(v) | reinterpret_cast<uintptr_t>(o);
  if ((align & 15u) || (reinterpret_cast<uintptr_t>(lse) & 3u)) return STEEL_ERR_INVALID_ARG;
  steel_status_t st = validate_params(params);
  if (st != STEEL_OK) return st;

  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) {
    cudaGetLastError();
    return STEEL_ERR_CUDA;
  }
  if (device < 0 || device >= kMaxDevices) return STEEL_ERR_UNSUPPORTED;
  unsigned char *base = nullptr;
  int sm_count = 0;
  st = setup_device(device, &base, &sm_count);
  if (st != STEEL_OK) {
    cudaGetLastError();
    return st;
  }

  Plan plan;  // host memory only
  try {
    st = build_plan(params, sm_count, &plan, /*exec_stats=*/false);
  } catch (const std::bad_alloc &) {
    return STEEL_ERR_ALLOC;
  }
  if (st != STEEL_OK) return st;
  // the fixed array bounds the problem: refuse, rather than truncate, anything larger
  if (plan.items.size() > kMaxItems || plan.steps.size() > kMaxSteps || plan.cta_begin.size() > kMaxCtas + 1)
    return STEEL_ERR_UNSUPPORTED;

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  // The array still holds the previous call's lists and status word: overwrite the lists, clear the word.
  bool ok = cudaMemsetAsync(base + kOffStatus, 0, sizeof(int32_t), stream) == cudaSuccess &&
            (plan.items.empty() || cudaMemcpyAsync(base + kOffItems, plan.items.data(),
                                                   plan.items.size() * sizeof(WorkItem), cudaMemcpyHostToDevice,
                                                   stream) == cudaSuccess) &&
            cudaMemcpyAsync(base + kOffCtaBegin, plan.cta_begin.data(), plan.cta_begin.size() * sizeof(int32_t),
                            cudaMemcpyHostToDevice, stream) == cudaSuccess &&
            (plan.steps.empty() || cudaMemcpyAsync(base + kOffSteps, plan.steps.data(),
                                                   plan.steps.size() * sizeof(StepPair), cudaMemcpyHostToDevice,
                                                   stream) == cudaSuccess);
  if (!ok) {
    cudaGetLastError();
    return STEEL_ERR_CUDA;
  }
  KernelParams kp;
  kp.items = reinterpret_cast<const WorkItem *>(base + kOffItems);
  kp.cta_begin = reinterpret_cast<const int32_t *>(base + kOffCtaBegin);
  kp.steps = reinterpret_cast<const StepPair *>(base + kOffSteps);
  kp.status = reinterpret_cast<int32_t *>(base + kOffStatus);
  kp.trace = nullptr;
  kp.clock_probe = nullptr;
  kp.timeout_cycles = kDefaultTimeoutCycles;
  kp.stall_cta = -1;
  st = launch_with_params(*params, kp, plan.grid, q, k, v, o, lse, stream, nullptr);
  if (st != STEEL_OK) return st;
  // Blocking by design: the host lists above must outlive the copies, and the status word has to
  // be read before the next call clears it.
  int32_t word = 0;
  if (cudaStreamSynchronize(stream) != cudaSuccess ||
      cudaMemcpy(&word, base + kOffStatus, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) {
    cudaGetLastError();
    return STEEL_ERR_CUDA;
  }
  return word == 0 ? STEEL_OK : STEEL_ERR_TIMEOUT;
}
