/*
 * steel_attn.h — C ABI of the block-sparse fused prefill attention library for NVIDIA B200.
 *
 * The operation (paper Eq. 1, generalised by `scale` and a mask): for every batch b, query
 * head h and query row i,
 *
 *     O[b,h,i,:] = softmax_j( scale * Q[b,h,i,:] . K[b,g,j,:] + M[h,i,j] ) V[b,g,:,:]
 *     LSE[b,h,i] = ln sum_j exp( scale * Q[b,h,i,:] . K[b,g,j,:] + M[h,i,j] )
 *
 * with g = h / (heads_q / heads_kv) (grouped-query attention, contiguous groups) and
 * M = 0 where key j is visible to query i, -inf elsewhere.  It is computed as the paper's
 * Algorithm 1: tiled Q K^T, online softmax (running row maximum m and row sum l), P V
 * accumulation, final division by l — never materialising the score matrix, and following
 * the paper's three mask cases (Sec. "The STEEL Pipeline"): a (query-tile, key-tile) pair
 * whose elements are all masked is skipped (no memory traffic, no MMA), an unmasked pair is
 * processed as is, a partially masked pair has the mask generated from coordinates on chip.
 * The mask is never read from memory by the kernel; only a per-CTA work list derived from it.
 *
 * Visibility predicate (AND of the enabled terms; `off` = seq_kv - seq_q):
 *     CAUSAL : j <= i + off
 *     WINDOW : (i + off) - j < window          (with CAUSAL: exactly `window` keys incl. self)
 *     BITMAP : bit (J & 31) of bitmap[(h * T_q + I) * ceil(T_kv / 32) + (J >> 5)] is set,
 *              I = i / block_q, J = j / block_kv, T_q = ceil(seq_q / block_q), T_kv likewise.
 * A query row with no visible key gets O = 0 and LSE = -inf.
 *
 * Memory layout: Q and O are [batch, heads_q, seq_q, head_dim], K and V are
 * [batch, heads_kv, seq_kv, head_dim], all contiguous bfloat16; LSE is
 * [batch, heads_q, seq_q] float32.  Arithmetic: bf16 operands, fp32 accumulation and
 * softmax statistics; P is rounded to bf16 for the second product, l sums the unrounded P.
 *
 * Ownership and threading: every tensor pointer is a DEVICE pointer owned by the caller,
 * 16-byte aligned, and must stay valid until the stream has executed the call.  The bitmap
 * is a HOST pointer read only during steel_attn_create.  A handle owns its device work lists
 * and status word; it is bound to the device that was current at create time and must
 * not be used by two streams at once.  All functions return a status code; nothing throws,
 * aborts or traps.  There is no CPU fallback: without a usable CUDA device the run fails.
 */
#ifndef STEEL_ATTN_H_
#define STEEL_ATTN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct steel_attn steel_attn_t; /* opaque, owned by the library */

typedef enum {
  STEEL_OK = 0,
  STEEL_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, misaligned pointer, bad flags */
  STEEL_ERR_UNSUPPORTED = 2, /* valid problem outside this build's limits (see create)         */
  STEEL_ERR_ALLOC = 3,       /* host or device allocation failed                               */
  STEEL_ERR_CUDA = 4,        /* a CUDA call failed (no device, wrong architecture, launch)     */
  STEEL_ERR_TIMEOUT = 5      /* a bounded device-side wait expired; outputs are undefined      */
} steel_status_t;

enum { STEEL_MASK_CAUSAL = 1u, STEEL_MASK_WINDOW = 2u, STEEL_MASK_BITMAP = 4u };

typedef struct {
  uint32_t flags;           /* OR of STEEL_MASK_*; 0 = dense attention                         */
  int32_t block_q;          /* mask block sizes in tokens, 64 or 128 (0 = 128); they define the */
  int32_t block_kv;         /* BITMAP grid and the granularity at which tiles are counted       */
  int64_t window;           /* W > 0 tokens, used iff WINDOW                                    */
  const uint32_t *bitmap;   /* HOST pointer, used iff BITMAP, copied by create;                 */
                            /* [heads_q][T_q][ceil(T_kv/32)] words, shared across the batch     */
} steel_mask_desc_t;

typedef struct {
  int32_t batch, heads_q, heads_kv; /* heads_q % heads_kv == 0                                  */
  int32_t seq_q, seq_kv;            /* any positive lengths (ragged last tiles are masked)       */
  int32_t head_dim;                 /* 64 or 128                                                 */
  float scale;                      /* finite, > 0; multiplies q.k before softmax                */
  steel_mask_desc_t mask;
  int32_t policy;                   /* placement of query tiles on the persistent CTAs (paper Sec.
                                       "Sparsity-Aware Pipeline Placement"): 0 = query tiles paired for
                                       shared K/V loads, items ordered KV-head-major then longest first,
                                       each to the least loaded CTA (default); 1 = the same items in
                                       natural order cut into contiguous chunks, one per CTA (the paper's
                                       "uniform placement"); 2 = the same items dealt round-robin to the
                                       CTAs (the paper's sparsity-aware placement: consecutive query
                                       tiles side by side)                                         */
  int32_t exp_emulation;            /* share of the Second Stage's exponentials evaluated by a cubic
                                       polynomial on the FMA pipe instead of the special-function unit
                                       (the counterpart of the lookup-table exponent of the paper's Sec.
                                       "Comparison with State-of-the-Art on NPU"): 0 = none (default),
                                       1 = 12.5 %, 2 = 25 %, 3 = 50 %; relative error 7.5e-5 per value  */
} steel_attn_params_t;

/* Work-list statistics of a plan (the skip set of the three mask cases, at the kernel's
 * 128 x 128 tile granularity). */
typedef struct {
  int64_t kept_tiles;     /* (query-block, key-block) pairs that are not fully masked, counted  */
                          /* at the descriptor's block_q x block_kv granularity                 */
  int64_t partial_tiles;  /* of those, pairs with some masked element                           */
  int64_t total_tiles;    /* all block pairs of the problem, skipped ones included              */
  int64_t exec_tiles;     /* 128 x 128 kernel tiles executed (equals kept_tiles for 128 blocks)  */
  int64_t exec_partial;   /* of those, tiles on which the element-wise mask is applied          */
  int64_t work_items;     /* scheduler items (one or two query tiles that share key loads)      */
  int64_t steps;          /* key-tile steps summed over items                                   */
  int64_t kv_tile_loads;  /* K (equally V) tile loads issued; exec_tiles minus shared loads     */
  int64_t list_entries;   /* explicit step-list entries held in device memory (bitmap masks)    */
  int64_t max_cta_steps;  /* steps of the most loaded persistent CTA                            */
  int64_t grid;           /* persistent CTAs launched                                           */
  double effective_flop;  /* 4 * block_q * block_kv * head_dim * kept_tiles                     */
  double useful_flop;     /* 4 * head_dim * (number of visible (i, j) pairs)                     */
} steel_attn_stats_t;

/*
 * Validate `params`, classify every tile (mask cases i-iii), build the work items and their
 * key-tile lists, order them for the persistent scheduler and upload them to the current
 * CUDA device.  On success *out receives the handle; on failure *out is NULL.
 * STEEL_ERR_UNSUPPORTED: head_dim not in {64, 128}; block sizes other than 64 or 128 or
 * block_q != block_kv; more than 2^24 key tiles; batch * heads * seq beyond 2^31 rows.  Allocates device memory;
 * synchronises the device once.
 */
steel_status_t steel_attn_create(const steel_attn_params_t *params, steel_attn_t **out);

/*
 * Enqueue one attention call (Eq. 1, computed as Algorithm 1 over the handle's work lists) on `cuda_stream` (a cudaStream_t cast to void*; NULL = default
 * stream).  q, k, v, o: device bf16 tensors in the layouts above; lse: device float32 or
 * NULL.  Asynchronous: no allocation, no host synchronisation.  One persistent kernel is
 * launched; device-side waits are bounded and, if one expires, the kernel stops and the
 * error is reported by steel_attn_last_status.  STEEL_ERR_INVALID_ARG also if the current device
 * is not the one the handle was created on.
 */
steel_status_t steel_attn_run(steel_attn_t *handle, const void *q, const void *k, const void *v,
                              void *o, float *lse, void *cuda_stream);

/*
 * Synchronise `cuda_stream` and report the device-side status word of the handle's last
 * runs of Algorithm 1's pipeline (its stages hand tiles over through bounded waits) (STEEL_OK or STEEL_ERR_TIMEOUT), then clear it.
 */
steel_status_t steel_attn_last_status(steel_attn_t *handle, void *cuda_stream);

/* Release the handle and the device work lists built from the mask cases of Sec. "The STEEL
 * Pipeline".  destroy(NULL) is STEEL_OK. */
steel_status_t steel_attn_destroy(steel_attn_t *handle);

/* Statistics of the handle's plan. */
steel_status_t steel_attn_get_stats(const steel_attn_t *handle, steel_attn_stats_t *stats);

/*
 * Host-only planning: the same validation, tile classification and work-list construction as
 * steel_attn_create, without touching CUDA.  `stats` receives the statistics.  If `tiles` is
 * not NULL it receives, for every executed pair in the order the kernel's roles walk them,
 * six int32 values {item, batch, head, query_tile, key_tile, flags} (tiles are 128 x 128;
 * flags bit 0: partial, bit 1: the K/V load is shared with the item's other query tile,
 * bits 4..7: enabled 64x64 sub-blocks TL, TR, BL, BR), up to `capacity` records; *n_tiles receives the number written.
 */
steel_status_t steel_attn_plan_host(const steel_attn_params_t *params, steel_attn_stats_t *stats,
                                    int32_t *tiles, int64_t capacity, int64_t *n_tiles);

/*
 * Test hook for the bounded device-side waits.  With cta >= 0, CTA `cta` of the handle's following
 * runs withholds the commands its producer would publish, so the waits of its other roles expire
 * after `timeout_cycles` SM cycles (<= 0: the default, about two seconds): the kernel then returns
 * normally, outputs are undefined and steel_attn_last_status reports STEEL_ERR_TIMEOUT.  Nothing
 * faults or hangs; the context stays usable.  cta < 0 switches the hook off.
 */
steel_status_t steel_attn_debug_stall(steel_attn_t *handle, int32_t cta, int64_t timeout_cycles);

/*
 * Measurement hook for the roofline figures (paper Sec. "Attention Benchmark": throughput is quoted
 * against the device's peak, which depends on the clock actually held).  With a non-NULL
 * `device_pair` (DEVICE pointer to two int64, 8-byte aligned, owned by the caller), CTA 0 of each of
 * the handle's following runs stores {SM cycles, nanoseconds} elapsed over its run there, so that
 * cycles / nanoseconds is the SM clock in GHz during the kernel.  NULL switches the hook off.
 */
steel_status_t steel_attn_debug_clock_probe(steel_attn_t *handle, int64_t *device_pair);

/*
 * (The paper has no counterpart to this entry point; it exists for integration.)  One attention
 * call for callers that cannot allocate device memory: code that runs inside another framework's
 * locked memory pool, on a latency path where cudaMalloc's implicit synchronisation is not
 * acceptable, or under a device-memory budget fixed at start-up.  It takes the problem description
 * and the tensors directly -- no handle -- and keeps the work lists that steel_attn_create would put
 * in cudaMalloc'ed buffers in a fixed array inside the library image instead (about 2 MiB, held on
 * every GPU that loads the library until the process exits).  It calls no cudaMalloc / cudaFree.
 *
 * Limits: at most 16384 work items, 131072 explicit step-list entries (bitmap masks) and 1024
 * persistent CTAs; a problem whose plan is larger is refused with STEEL_ERR_UNSUPPORTED and
 * nothing is launched (the 131072-token graded configuration, 16384 items, is the largest
 * causal case that fits).  Arguments as for steel_attn_create and steel_attn_run.
 *
 * The call is blocking: it plans on the host (transient host memory only), copies the lists on
 * `cuda_stream`, runs the kernel, waits for the stream and returns the device status (STEEL_OK or
 * STEEL_ERR_TIMEOUT).  All calls in the process share the one array per GPU, which still holds the
 * previous call's lists when a call starts: the call rewrites the lists and clears the status word,
 * so two calls that overlap on the same GPU (from two threads or streams) race and must be
 * serialised by the caller.  The first call on each device also resolves the array's device
 * address and configures the kernels; make that first call outside any stream capture.
 */
steel_status_t steel_attn_run_noalloc(const steel_attn_params_t *params, const void *q, const void *k,
                                      const void *v, void *o, float *lse, void *cuda_stream);

/*
 * The same operation for tensors in HOST memory (the end-to-end path of Eq. 1 / Algorithm 1:
 * operands start and results end on the host).  A host-side object owns device staging buffers for
 * Q, K, V, O and LSE, three internal streams and one plan per chunk.  The problem is cut into at
 * most `max_chunks` chunks that are independent attention problems with contiguous tensors: groups
 * of batch elements when batch > 1, groups of KV heads (with their query heads and their slice of
 * the bitmap) when batch == 1; the number used is the largest divisor of batch (of heads_kv) not
 * above max_chunks (values below 1 mean 1).  Chunk c is copied host -> device, run through the
 * kernel of steel_attn_run and copied device -> host on separate streams, so the copies of one
 * chunk overlap the kernel of another.  Results equal those of steel_attn_run on the same chunk.
 */
typedef struct steel_attn_host steel_attn_host_t; /* opaque, owned by the library */

/* Plan the chunks, allocate the staging buffers (the size of all five tensors) on the current
 * device.  Status codes as for steel_attn_create; *out is NULL on failure. */
steel_status_t steel_attn_host_create(const steel_attn_params_t *params, int32_t max_chunks,
                                      steel_attn_host_t **out);

/*
 * q, k, v (read) and o, lse (written; lse may be NULL) are HOST pointers in the layouts above, owned
 * by the caller and valid until `cuda_stream` has executed the call.  With page-locked host memory
 * the call is asynchronous; with pageable memory the copies block the calling thread but the result
 * is the same.  The work is ordered after what is already queued on `cuda_stream`, and later work on
 * `cuda_stream` is ordered after the last device -> host copy.  One object must not be used from
 * two streams or threads at once (the staging buffers are shared between its calls).
 */
steel_status_t steel_attn_host_run(steel_attn_host_t *handle, const void *q, const void *k,
                                   const void *v, void *o, float *lse, void *cuda_stream);

/* Synchronise `cuda_stream`, then report and clear the device status of the chunks' kernels. */
steel_status_t steel_attn_host_last_status(steel_attn_host_t *handle, void *cuda_stream);

/* Number of chunks the object uses (0 for NULL). */
int32_t steel_attn_host_chunks(const steel_attn_host_t *handle);

/* Wait for the object's streams, release its plans, buffers, streams and events. NULL is STEEL_OK. */
steel_status_t steel_attn_host_destroy(steel_attn_host_t *handle);

const char *steel_status_string(steel_status_t status);

#ifdef __cplusplus
}
#endif
#endif /* STEEL_ATTN_H_ */
