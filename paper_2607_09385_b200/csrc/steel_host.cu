// steel_attn_host_*: the attention call for tensors that live in HOST memory.
//
// The problem is cut into chunks that are independent attention problems with contiguous tensors
// (groups of batch elements when batch > 1, groups of KV heads with their query heads when
// batch == 1).  Each chunk goes host -> device on one stream, through the attention kernel on a
// second and device -> host on a third, so that the copies of one chunk overlap the kernel of
// another and both directions of the host link are busy at once.  Every step of the computation
// runs in the same kernel as steel_attn_run: this file only plans chunks, owns the staging buffers
// and orders copies and launches with events.  It is written against the public C ABI alone.
#include <cuda_runtime.h>

#include <new>
#include <vector>

#include "../../include/steel_attn.h"

struct steel_attn_host {
  steel_attn_params_t params{};
  int device = 0;
  int n_chunks = 1;
  size_t q_chunk_bytes = 0, kv_chunk_bytes = 0, lse_chunk_bytes = 0;
  std::vector<steel_attn_t *> child;  // one per chunk (bitmap masks) or a single shared one
  unsigned char *dq = nullptr, *dk = nullptr, *dv = nullptr, *dout = nullptr;
  float *dlse = nullptr;
  cudaStream_t s_in = nullptr, s_run = nullptr, s_out = nullptr;
  cudaEvent_t ev_begin = nullptr, ev_end = nullptr;
  std::vector<cudaEvent_t> ev_in, ev_run;
};

namespace {

int largest_divisor_up_to(int n, int limit) {
  int best = 1;
  for (int c = 1; c <= n && c <= limit; ++c)
    if (n % c == 0) best = c;
  return best;
}

void release(steel_attn_host *h) {
  if (!h) return;
  int prev = 0;
  const bool switched = cudaGetDevice(&prev) == cudaSuccess && prev != h->device &&
                        cudaSetDevice(h->device) == cudaSuccess;
  for (steel_attn_t *c : h->child) steel_attn_destroy(c);
  for (cudaEvent_t e : h->ev_in) cudaEventDestroy(e);
  for (cudaEvent_t e : h->ev_run) cudaEventDestroy(e);
  if (h->ev_begin) cudaEventDestroy(h->ev_begin);
  if (h->ev_end) cudaEventDestroy(h->ev_end);
  if (h->s_in) cudaStreamDestroy(h->s_in);
  if (h->s_run) cudaStreamDestroy(h->s_run);
  if (h->s_out) cudaStreamDestroy(h->s_out);
  cudaFree(h->dq);
  cudaFree(h->dk);
  cudaFree(h->dv);
  cudaFree(h->dout);
  cudaFree(h->dlse);
  if (switched) cudaSetDevice(prev);
  delete h;
}

}  // namespace

extern "C" steel_status_t steel_attn_host_create(const steel_attn_params_t *params, int32_t max_chunks,
                                                 steel_attn_host_t **out) {
  if (!out) return STEEL_ERR_INVALID_ARG;
  *out = nullptr;
  if (!params) return STEEL_ERR_INVALID_ARG;
  // the planner validates everything else; only what the chunking divides by is needed first
  if (params->batch <= 0 || params->heads_q <= 0 || params->heads_kv <= 0 ||
      params->heads_q % params->heads_kv != 0 || params->seq_q <= 0 || params->seq_kv <= 0 ||
      params->head_dim <= 0)
    return STEEL_ERR_INVALID_ARG;
  steel_attn_host *h = new (std::nothrow) steel_attn_host;
  if (!h) return STEEL_ERR_ALLOC;
  h->params = *params;
  if (cudaGetDevice(&h->device) != cudaSuccess) {
    delete h;
    return STEEL_ERR_CUDA;
  }

  const int limit = max_chunks < 1 ? 1 : max_chunks;
  const bool by_batch = params->batch > 1;
  h->n_chunks = largest_divisor_up_to(by_batch ? params->batch : params->heads_kv, limit);
  steel_attn_params_t cp = *params;
  if (by_batch) {
    cp.batch = params->batch / h->n_chunks;
  } else {
    cp.heads_q = params->heads_q / h->n_chunks;
    cp.heads_kv = params->heads_kv / h->n_chunks;
  }
  const size_t row_bytes = static_cast<size_t>(params->head_dim) * 2;
  h->q_chunk_bytes = static_cast<size_t>(cp.batch) * cp.heads_q * params->seq_q * row_bytes;
  h->kv_chunk_bytes = static_cast<size_t>(cp.batch) * cp.heads_kv * params->seq_kv * row_bytes;
  h->lse_chunk_bytes = static_cast<size_t>(cp.batch) * cp.heads_q * params->seq_q * sizeof(float);

  // The bitmap is indexed by query head and shared across the batch: a head chunk needs its own
  // slice and plan, every other chunking runs all chunks through one plan.
  const bool per_chunk_plan = !by_batch && (params->mask.flags & STEEL_MASK_BITMAP) && h->n_chunks > 1;
  steel_status_t st = STEEL_OK;
  const int n_plans = per_chunk_plan ? h->n_chunks : 1;
  for (int c = 0; c < n_plans && st == STEEL_OK; ++c) {
    steel_attn_params_t p = cp;
    if (per_chunk_plan && params->mask.bitmap) {
      const int64_t bq = params->mask.block_q ? params->mask.block_q : 128;
      const int64_t bk = params->mask.block_kv ? params->mask.block_kv : 128;
      if (bq <= 0 || bk <= 0) {
        st = STEEL_ERR_INVALID_ARG;
        break;
      }
      const int64_t tq = (params->seq_q + bq - 1) / bq, tk = (params->seq_kv + bk - 1) / bk;
      const int64_t words_per_head = tq * ((tk + 31) / 32);
      p.mask.bitmap = params->mask.bitmap + static_cast<int64_t>(c) * cp.heads_q * words_per_head;
    }
    steel_attn_t *child = nullptr;
    st = steel_attn_create(&p, &child);
    if (st == STEEL_OK) h->child.push_back(child);
  }
  if (st != STEEL_OK) {
    release(h);
    return st;
  }

  const size_t n = static_cast<size_t>(h->n_chunks);
  bool ok = cudaMalloc(&h->dq, n * h->q_chunk_bytes) == cudaSuccess &&
            cudaMalloc(&h->dk, n * h->kv_chunk_bytes) == cudaSuccess &&
            cudaMalloc(&h->dv, n * h->kv_chunk_bytes) == cudaSuccess &&
            cudaMalloc(&h->dout, n * h->q_chunk_bytes) == cudaSuccess &&
            cudaMalloc(&h->dlse, n * h->lse_chunk_bytes) == cudaSuccess;
  if (!ok) {
    cudaGetLastError();
    release(h);
    return STEEL_ERR_ALLOC;
  }
  ok = cudaStreamCreateWithFlags(&h->s_in, cudaStreamNonBlocking) == cudaSuccess &&
       cudaStreamCreateWithFlags(&h->s_run, cudaStreamNonBlocking) == cudaSuccess &&
       cudaStreamCreateWithFlags(&h->s_out, cudaStreamNonBlocking) == cudaSuccess &&
       cudaEventCreateWithFlags(&h->ev_begin, cudaEventDisableTiming) == cudaSuccess &&
       cudaEventCreateWithFlags(&h->ev_end, cudaEventDisableTiming) == cudaSuccess;
  for (int c = 0; c < h->n_chunks && ok; ++c) {
    cudaEvent_t a = nullptr, b = nullptr;
    ok = cudaEventCreateWithFlags(&a, cudaEventDisableTiming) == cudaSuccess;
    if (ok) h->ev_in.push_back(a);
    ok = ok && cudaEventCreateWithFlags(&b, cudaEventDisableTiming) == cudaSuccess;
    if (ok) h->ev_run.push_back(b);
  }
  if (!ok) {
    cudaGetLastError();
    release(h);
    return STEEL_ERR_CUDA;
  }
  *out = h;
  return STEEL_OK;
}

extern "C" steel_status_t steel_attn_host_run(steel_attn_host_t *h, const void *q, const void *k,
                                              const void *v, void *o, float *lse, void *cuda_stream) {
  if (!h || !q || !k || !v || !o) return STEEL_ERR_INVALID_ARG;
  int device = -1;
  if (cudaGetDevice(&device) != cudaSuccess) return STEEL_ERR_CUDA;
  if (device != h->device) return STEEL_ERR_INVALID_ARG;
  cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
  const unsigned char *hq = static_cast<const unsigned char *>(q);
  const unsigned char *hk = static_cast<const unsigned char *>(k);
  const unsigned char *hv = static_cast<const unsigned char *>(v);
  unsigned char *ho = static_cast<unsigned char *>(o);

#define STEEL_HOST_CHECK(call) \
  if ((call) != cudaSuccess) { \
    cudaGetLastError(); \
    return STEEL_ERR_CUDA; \
  }
  // everything below starts after the work already queued on the caller's stream
  STEEL_HOST_CHECK(cudaEventRecord(h->ev_begin, user));
  STEEL_HOST_CHECK(cudaStreamWaitEvent(h->s_in, h->ev_begin, 0));
  for (int c = 0; c < h->n_chunks; ++c) {
    const size_t qo = c * h->q_chunk_bytes, ko = c * h->kv_chunk_bytes, lo = c * h->lse_chunk_bytes;
    STEEL_HOST_CHECK(cudaMemcpyAsync(h->dq + qo, hq + qo, h->q_chunk_bytes, cudaMemcpyHostToDevice, h->s_in));
    STEEL_HOST_CHECK(cudaMemcpyAsync(h->dk + ko, hk + ko, h->kv_chunk_bytes, cudaMemcpyHostToDevice, h->s_in));
    STEEL_HOST_CHECK(cudaMemcpyAsync(h->dv + ko, hv + ko, h->kv_chunk_bytes, cudaMemcpyHostToDevice, h->s_in));
    STEEL_HOST_CHECK(cudaEventRecord(h->ev_in[c], h->s_in));

    STEEL_HOST_CHECK(cudaStreamWaitEvent(h->s_run, h->ev_in[c], 0));
    steel_attn_t *child = h->child[h->child.size() == 1 ? 0 : c];
    const steel_status_t st =
        steel_attn_run(child, h->dq + qo, h->dk + ko, h->dv + ko, h->dout + qo,
                       reinterpret_cast<float *>(reinterpret_cast<unsigned char *>(h->dlse) + lo), h->s_run);
    if (st != STEEL_OK) return st;
    STEEL_HOST_CHECK(cudaEventRecord(h->ev_run[c], h->s_run));

    STEEL_HOST_CHECK(cudaStreamWaitEvent(h->s_out, h->ev_run[c], 0));
    STEEL_HOST_CHECK(cudaMemcpyAsync(ho + qo, h->dout + qo, h->q_chunk_bytes, cudaMemcpyDeviceToHost, h->s_out));
    if (lse)
      STEEL_HOST_CHECK(cudaMemcpyAsync(reinterpret_cast<unsigned char *>(lse) + lo,
                                       reinterpret_cast<unsigned char *>(h->dlse) + lo, h->lse_chunk_bytes,
                                       cudaMemcpyDeviceToHost, h->s_out));
  }
  // the caller's stream continues once the last chunk is back in host memory
  STEEL_HOST_CHECK(cudaEventRecord(h->ev_end, h->s_out));
  STEEL_HOST_CHECK(cudaStreamWaitEvent(user, h->ev_end, 0));
#undef STEEL_HOST_CHECK
  return STEEL_OK;
}

extern "C" steel_status_t steel_attn_host_last_status(steel_attn_host_t *h, void *cuda_stream) {
  if (!h) return STEEL_ERR_INVALID_ARG;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) return STEEL_ERR_CUDA;
  steel_status_t worst = STEEL_OK;
  for (steel_attn_t *c : h->child) {
    const steel_status_t st = steel_attn_last_status(c, h->s_run);
    if (st != STEEL_OK) worst = st;
  }
  return worst;
}

extern "C" int32_t steel_attn_host_chunks(const steel_attn_host_t *h) { return h ? h->n_chunks : 0; }

extern "C" steel_status_t steel_attn_host_destroy(steel_attn_host_t *h) {
  if (!h) return STEEL_OK;
  int prev = 0;
  if (cudaGetDevice(&prev) == cudaSuccess && prev == h->device) {
    cudaStreamSynchronize(h->s_in);
    cudaStreamSynchronize(h->s_run);
    cudaStreamSynchronize(h->s_out);
  }
  release(h);
  return STEEL_OK;
}
