// C ABI of the library (see include/steel_attn.h): argument checks, plan upload, tensor maps, launch.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <limits>
#include <new>

#include "../../include/steel_attn.h"
#include "steel_kernel.h"
#include "steel_planner.h"

using namespace steel;

static_assert(sizeof(steel_mask_desc_t) == 32 && sizeof(steel_attn_params_t) == 72, "public struct layout");

struct steel_attn {
  steel_attn_params_t params;
  steel_attn_stats_t stats;
  int device = -1;
  int grid = 0;
  WorkItem *d_items = nullptr;
  int32_t *d_cta_begin = nullptr;
  StepPair *d_steps = nullptr;
  int32_t *d_status = nullptr;
  long long *d_trace = nullptr;  // debug builds only
  long long *d_clock_probe = nullptr;
  long long timeout_cycles = kDefaultTimeoutCycles;
  int32_t stall_cta = -1;
  TensorMaps maps;  // of the last (q, k, v) triple run on this handle
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver entry point is resolved at run time so that the library loads (and its host-only
// functions work) on machines without the CUDA driver.
EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void *f = nullptr;
    cudaDriverEntryPointQueryResult res;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &res) != cudaSuccess ||
        res != cudaDriverEntryPointSuccess)
      f = nullptr;
    return reinterpret_cast<EncodeTiledFn>(f);
  }();
  return fn;
}

// bf16 [matrices, rows, head_dim] viewed as a 3-D tensor; boxes of 128 rows x 64 columns (128 bytes),
// 128-byte swizzle; rows beyond `rows` read as zero.
bool make_map(CUtensorMap *map, const void *base, int head_dim, int64_t rows, int64_t matrices) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[3] = {cuuint64_t(head_dim), cuuint64_t(rows), cuuint64_t(matrices)};
  cuuint64_t strides[2] = {cuuint64_t(head_dim) * 2, cuuint64_t(head_dim) * 2 * cuuint64_t(rows)};
  cuuint32_t box[3] = {64, cuuint32_t(kTile), 1};
  cuuint32_t elem_strides[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, elem_strides,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

void free_device(steel_attn *h) {
  if (h->d_items) cudaFree(h->d_items);
  if (h->d_cta_begin) cudaFree(h->d_cta_begin);
  if (h->d_steps) cudaFree(h->d_steps);
  if (h->d_status) cudaFree(h->d_status);
}

}  // namespace

namespace steel {

// Encode the tensor maps for (q, k, v) unless `cache` holds them already, fill the problem fields
// of `kp` (whose list and status pointers the caller has set) and enqueue the kernel.
steel_status_t launch_with_params(const steel_attn_params_t &p, KernelParams kp, int grid, const void *q,
                                  const void *k, const void *v, void *o, float *lse, cudaStream_t stream,
                                  TensorMaps *cache) {
  TensorMaps local;
  TensorMaps &m = cache ? *cache : local;
  if (m.q_ptr != q || m.k_ptr != k || m.v_ptr != v) {
    m.q_ptr = m.k_ptr = m.v_ptr = nullptr;
    if (!make_map(&m.q, q, p.head_dim, p.seq_q, int64_t(p.batch) * p.heads_q) ||
        !make_map(&m.k, k, p.head_dim, p.seq_kv, int64_t(p.batch) * p.heads_kv) ||
        !make_map(&m.v, v, p.head_dim, p.seq_kv, int64_t(p.batch) * p.heads_kv))
      return STEEL_ERR_CUDA;
    m.q_ptr = q;
    m.k_ptr = k;
    m.v_ptr = v;
  }
  kp.o = o;
  kp.lse = lse;
  kp.heads_q = p.heads_q;
  kp.heads_kv = p.heads_kv;
  kp.seq_q = p.seq_q;
  kp.seq_kv = p.seq_kv;
  kp.mask_flags = p.mask.flags;
  // a window wider than the key sequence hides nothing: clamp it so that the kernel's 32-bit
  // column arithmetic cannot overflow
  kp.window = int32_t(std::min<int64_t>(p.mask.window, int64_t(std::max(p.seq_q, p.seq_kv)) + kTile));
  kp.scale_log2 = p.scale * 1.4426950408889634f;
  if (launch_attention(p.head_dim, p.exp_emulation, m.q, m.k, m.v, kp, grid, stream) != cudaSuccess)
    return STEEL_ERR_CUDA;
  return STEEL_OK;
}

}  // namespace steel

extern "C" {

steel_status_t steel_attn_create(const steel_attn_params_t *params, steel_attn_t **out) {
  if (!out) return STEEL_ERR_INVALID_ARG;
  *out = nullptr;
  steel_status_t st = validate_params(params);
  if (st != STEEL_OK) return st;

  int device = 0;
  cudaDeviceProp prop;
  if (cudaGetDevice(&device) != cudaSuccess || cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
    cudaGetLastError();
    return STEEL_ERR_CUDA;
  }
  if (prop.major != 10) return STEEL_ERR_CUDA;  // the kernel is built for sm_100a only

  Plan plan;
  try {
    st = build_plan(params, prop.multiProcessorCount, &plan);
  } catch (const std::bad_alloc &) {
    return STEEL_ERR_ALLOC;
  }
  if (st != STEEL_OK) return st;

  steel_attn *h = new (std::nothrow) steel_attn();
  if (!h) return STEEL_ERR_ALLOC;
  h->params = *params;
  h->params.mask.bitmap = nullptr;  // the caller's bitmap is not referenced after create
  h->stats = plan.stats;
  h->device = device;
  h->grid = plan.grid;

  const size_t n_items = plan.items.size() ? plan.items.size() : 1, n_steps = plan.steps.size() ? plan.steps.size() : 1;
  bool ok = cudaMalloc(&h->d_items, n_items * sizeof(WorkItem)) == cudaSuccess &&
            cudaMalloc(&h->d_cta_begin, plan.cta_begin.size() * sizeof(int32_t)) == cudaSuccess &&
            cudaMalloc(&h->d_steps, n_steps * sizeof(StepPair)) == cudaSuccess &&
            cudaMalloc(&h->d_status, sizeof(int32_t)) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    free_device(h);
    delete h;
    return STEEL_ERR_ALLOC;
  }
  ok = (plan.items.empty() || cudaMemcpy(h->d_items, plan.items.data(), plan.items.size() * sizeof(WorkItem),
                                         cudaMemcpyHostToDevice) == cudaSuccess) &&
       cudaMemcpy(h->d_cta_begin, plan.cta_begin.data(), plan.cta_begin.size() * sizeof(int32_t),
                  cudaMemcpyHostToDevice) == cudaSuccess &&
       (plan.steps.empty() || cudaMemcpy(h->d_steps, plan.steps.data(), plan.steps.size() * sizeof(StepPair),
                                         cudaMemcpyHostToDevice) == cudaSuccess) &&
       cudaMemset(h->d_status, 0, sizeof(int32_t)) == cudaSuccess && configure_kernels() == cudaSuccess &&
       cudaDeviceSynchronize() == cudaSuccess;
  if (!ok || !encode_fn()) {
    cudaGetLastError();
    free_device(h);
    delete h;
    return STEEL_ERR_CUDA;
  }
  *out = h;
  return STEEL_OK;
}

steel_status_t steel_attn_run(steel_attn_t *h, const void *q, const void *k, const void *v, void *o, float *lse,
                              void *cuda_stream) {
  if (!h || !q || !k || !v || !o) return STEEL_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o) || (reinterpret_cast<uintptr_t>(lse) & 3u))
    return STEEL_ERR_INVALID_ARG;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) return STEEL_ERR_CUDA;
  if (device != h->device) return STEEL_ERR_INVALID_ARG;  // the work lists live on the create-time device
  KernelParams kp{};
  kp.items = h->d_items;
  kp.cta_begin = h->d_cta_begin;
  kp.steps = h->d_steps;
  kp.status = h->d_status;
  kp.trace = h->d_trace;
  kp.clock_probe = h->d_clock_probe;
  kp.timeout_cycles = h->timeout_cycles;
  kp.stall_cta = h->stall_cta;
  return launch_with_params(h->params, kp, h->grid, q, k, v, o, lse, static_cast<cudaStream_t>(cuda_stream), &h->maps);
}

steel_status_t steel_attn_last_status(steel_attn_t *h, void *cuda_stream) {
  if (!h) return STEEL_ERR_INVALID_ARG;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  int32_t word = 0;
  if (cudaStreamSynchronize(stream) != cudaSuccess ||
      cudaMemcpy(&word, h->d_status, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess)
    return STEEL_ERR_CUDA;
  if (word != 0 && cudaMemset(h->d_status, 0, sizeof(int32_t)) != cudaSuccess) return STEEL_ERR_CUDA;
  return word == 0 ? STEEL_OK : STEEL_ERR_TIMEOUT;
}

steel_status_t steel_attn_destroy(steel_attn_t *h) {
  if (!h) return STEEL_OK;
  free_device(h);
  delete h;
  return STEEL_OK;
}

steel_status_t steel_attn_get_stats(const steel_attn_t *h, steel_attn_stats_t *stats) {
  if (!h || !stats) return STEEL_ERR_INVALID_ARG;
  *stats = h->stats;
  return STEEL_OK;
}

steel_status_t steel_attn_plan_host(const steel_attn_params_t *params, steel_attn_stats_t *stats, int32_t *tiles,
                                    int64_t capacity, int64_t *n_tiles) {
  if (!stats) return STEEL_ERR_INVALID_ARG;
  Plan plan;
  steel_status_t st;
  try {
    st = build_plan(params, kPlanHostCtas, &plan);
  } catch (const std::bad_alloc &) {
    return STEEL_ERR_ALLOC;
  }
  if (st != STEEL_OK) return st;
  *stats = plan.stats;
  int64_t n = 0;
  if (tiles) {
    walk_plan(plan, [&](int item, const WorkItem &w, int slot, int, uint32_t entry, bool shared) {
      if (n < capacity) {
        int32_t *rec = tiles + 6 * n;
        rec[0] = item;
        rec[1] = w.batch;
        rec[2] = w.head[slot];
        rec[3] = w.qtile[slot];
        rec[4] = int32_t(entry & kEntryTileMask);
        rec[5] = int32_t(((entry & kEntryPartial) ? 1 : 0) | (shared ? 2 : 0) |
                         (((entry >> kEntrySubShift) & 0xF) << 4));
        ++n;
      }
    }, params);
  }
  if (n_tiles) *n_tiles = n;
  return STEEL_OK;
}

#ifdef STEEL_TRACE
// Debug builds: device buffer of gridDim.x * 32 counters filled by the kernel's roles.
steel_status_t steel_attn_set_trace(steel_attn_t *h, long long *device_buffer) {
  if (!h) return STEEL_ERR_INVALID_ARG;
  h->d_trace = device_buffer;
  return STEEL_OK;
}
#endif

steel_status_t steel_attn_debug_clock_probe(steel_attn_t *h, int64_t *device_pair) {
  if (!h || (reinterpret_cast<uintptr_t>(device_pair) & 7u)) return STEEL_ERR_INVALID_ARG;
  h->d_clock_probe = reinterpret_cast<long long *>(device_pair);
  return STEEL_OK;
}

steel_status_t steel_attn_debug_stall(steel_attn_t *h, int32_t cta, int64_t timeout_cycles) {
  if (!h || cta >= h->grid) return STEEL_ERR_INVALID_ARG;
  h->stall_cta = cta < 0 ? -1 : cta;
  h->timeout_cycles = timeout_cycles > 0 ? timeout_cycles : kDefaultTimeoutCycles;
  return STEEL_OK;
}

const char *steel_status_string(steel_status_t status) {
  switch (status) {
    case STEEL_OK: return "ok";
    case STEEL_ERR_INVALID_ARG: return "invalid argument";
    case STEEL_ERR_UNSUPPORTED: return "unsupported configuration";
    case STEEL_ERR_ALLOC: return "allocation failed";
    case STEEL_ERR_CUDA: return "CUDA error";
    case STEEL_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

}  // extern "C"
