/*
 * restkv.h -- C ABI of librestkv.so: the ReST-KV eviction-scoring hot path on one B200 (sm_100a).
 *
 * For one transformer layer, after prefill attention, the library scores every prefix
 * KV pair of every KV head with the layer-wise output-reconstruction indicator, smooths
 * the scores over the observation-window queries (EMA) and along the token axis (box
 * pooling), selects the B best pairs per head and gathers their K/V rows into a
 * compacted cache.  A split-K decode-attention kernel over such a cache is included so
 * that decode latency over the compacted and the full cache can be timed.
 *
 * Conventions that hold for every entry point unless it says otherwise
 *  - Tensor pointers are DEVICE pointers owned by the caller.  Nothing is allocated,
 *    freed or synchronised by the library after restkv_create(); every call only enqueues
 *    work on the given stream and returns.
 *  - Layouts: Q_obs [batch, n_q_heads, w, head_dim] contiguous, oldest window query first.
 *    K, V [batch, n_kv_heads, n_kv, head_dim] addressed through the element strides in
 *    restkv_shape (head_dim is contiguous).  Query head hq reads KV head hq / (n_q_heads / n_kv_heads).
 *    All base pointers must be 16-byte aligned and all strides multiples of 8 elements.
 *  - n_kv = n + causal_tail.  causal_tail = 0: K,V hold only the n scored prefix rows and every
 *    window query sees every row.  causal_tail = w: the last w rows of K,V are the window tokens'
 *    own pairs; window query i sees trailing row j' only if j' <= i, and those rows receive
 *    the score +inf (the paper's Omega, Eq. 8) so they are always kept.
 *  - Errors are return codes.  A call refused for its arguments, shape, pool parameters or
 *    workspace (INVALID_ARG, UNSUPPORTED, WORKSPACE) has enqueued nothing; RESTKV_ERR_CUDA may
 *    come from the middle of a call's launch sequence.  Conditions detected on the device (a
 *    bounded wait that ran out) set a sticky status word that restkv_poll_status() reads;
 *    kernels never trap.  Check restkv_poll_status() before using the outputs of a call.
 *  - Calls must not overlap on the GPU if they share a workspace.
 *  - The tensor-core kernels behind restkv_score, restkv_evict and restkv_decode (bf16, head_dim 128)
 *    are persistent: their thread blocks wait for one another inside one launch, so each launch
 *    needs every SM of the device for itself.  Do not let two such calls, or one of them and any
 *    other kernel that occupies SMs, run at the same time (two streams without ordering): order
 *    them on one stream or with events.  If SMs are held by something else the waits are bounded:
 *    the kernel gives up after about a second, the outputs of that call are undefined, and
 *    restkv_poll_status() returns RESTKV_ERR_TIMEOUT.
 */
#ifndef RESTKV_H_
#define RESTKV_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RESTKV_OK = 0,
  RESTKV_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, misaligned pointer or stride, bad mode */
  RESTKV_ERR_UNSUPPORTED = 2, /* a shape or mode no kernel covers (stated per entry point) */
  RESTKV_ERR_WORKSPACE = 3,   /* workspace null, misaligned (256 B) or smaller than restkv_workspace_bytes() */
  RESTKV_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed; restkv_last_cuda_error() has the code */
  RESTKV_ERR_TIMEOUT = 5      /* a bounded device-side wait expired (reported by restkv_poll_status) */
} restkv_status;

typedef enum { RESTKV_BF16 = 0, RESTKV_F32 = 1 } restkv_dtype;

typedef struct restkv_handle restkv_handle;

/* The stream argument is a cudaStream_t passed as an opaque pointer (NULL = legacy default stream). */
typedef void* restkv_stream;

typedef struct {
  int batch, n_q_heads, n_kv_heads, head_dim;
  int n_kv;            /* rows in K and V (= scored prefix rows n + causal_tail) */
  int w;               /* observation-window queries per head (the paper's S_w) */
  int causal_tail;     /* 0 or w, see above */
  restkv_dtype dtype;  /* element type of Q_obs, K, V and of the compacted outputs */
  float softmax_scale; /* 0 => 1/sqrt(head_dim) (Eq. 3) */
  long long k_stride_b, k_stride_h, k_stride_n; /* element strides of K; 0,0,0 => contiguous */
  long long v_stride_b, v_stride_h, v_stride_n; /* element strides of V; 0,0,0 => contiguous */
} restkv_shape;

typedef enum { RESTKV_POOL_FIXED = 0, RESTKV_POOL_ADAPTIVE = 1 } restkv_pool_mode;

typedef struct {
  int mode;       /* restkv_pool_mode */
  int width;      /* FIXED: odd box width W >= 1 (the kernel size k of Appendix B) */
  int shift;      /* FIXED: gamma_shift */
  float beta;     /* ADAPTIVE: scaling factor of Eq. 11-12 (paper: 2000) */
  int base_width; /* ADAPTIVE: odd fixed kernel k; the box has width W_s + k - 1, centre shift gamma_shift */
  int budget;     /* ADAPTIVE: B of Eq. 10 (per-query top-B whose mean index gives D_front / D_rear) */
} restkv_pool_params;

/* Creates a handle for the CURRENT device: queries its properties and allocates a 256-byte
 * device status block (the only allocation the library ever makes).  Host pointer out. */
restkv_status restkv_create(restkv_handle** out);
restkv_status restkv_destroy(restkv_handle* h);

/* Bytes of device workspace that score / select / evict / decode need for this shape and budget
 * (256-byte aligned pointer required).  Returns 0 on invalid arguments.  `budget` may be 0 when
 * only restkv_score / restkv_decode are used.  ADAPTIVE pooling needs the larger size reported by
 * restkv_workspace_bytes_adaptive (it stores the per-query indicator, 4*batch*n_q_heads*w*n bytes). */
size_t restkv_workspace_bytes(const restkv_shape* shape, int budget);
size_t restkv_workspace_bytes_adaptive(const restkv_shape* shape, int budget);

/*
 * restkv_score -- Eq. 3 (attention weights and outputs of the window queries), Eq. 7 (indicator
 * A/(1-A) * ||z - v_n||_2 with W_O = identity), Eq. 8-9 (EMA over the w window queries, oldest
 * first, alpha = 1 - ema_decay, seeded with the oldest query), mean over the query heads of each
 * KV head, Eq. 10-12 (ADAPTIVE window) and Eq. 13 (box mean, zero outside the scored rows, divisor
 * always the box width).
 *   Q_obs, K, V  device, dtype per shape->dtype
 *   scores       device float [batch, n_kv_heads, n_kv]; rows >= n receive +inf
 *                When K,V hold a single row (n_kv == 1) every attention weight is 1 and Eq. 7 is 0/0;
 *                the score of that row is defined as 0.
 *   pool_used    optional device int32 [batch, n_kv_heads, 2] receiving (W, gamma) per head, or NULL
 * RESTKV_BF16 with head_dim 128 and w * (n_q_heads/n_kv_heads) == 128 runs on the tcgen05 tensor-core
 * kernels; every other supported shape (head_dim <= 256 and a multiple of 8, w*group <= 256) runs on
 * fp32 SIMT kernels.  RESTKV_ERR_UNSUPPORTED otherwise.
 */
restkv_status restkv_score(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                           const void* V, float ema_decay, const restkv_pool_params* pool, float* scores,
                           int32_t* pool_used, void* workspace, size_t workspace_bytes, restkv_stream stream);

/*
 * restkv_score_from_lse -- restkv_score for a caller that already holds the attention statistics of the window
 * rows.  During prompt prefilling the attention of the last w tokens has been computed anyway (paper, Appendix B,
 * "prompt prefilling"): its outputs and softmax normalisers are exactly what pass 1 of restkv_score would
 * recompute (Eq. 3), so with them the indicator (Eq. 7) and its smoothing (Eq. 8-9, Eq. 13) need one read of K and V.
 *   O_obs    device float [batch, n_q_heads, w, head_dim]: o of every window row over the rows it sees
 *            (softmax(scale * q K^T) V, before the output projection)
 *   LSE_obs  device float [batch, n_q_heads, w]: natural-log sum of exp of that row's scaled logits over the same rows
 *   everything else as for restkv_score; the same kernels, tolerances and error codes apply.
 * The values must belong to the same Q_obs, K, V and softmax scale; nothing checks that.
 */
restkv_status restkv_score_from_lse(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                                    const void* V, const float* O_obs, const float* LSE_obs, float ema_decay,
                                    const restkv_pool_params* pool, float* scores, int32_t* pool_used, void* workspace,
                                    size_t workspace_bytes, restkv_stream stream);

/*
 * restkv_evict_from_lse -- restkv_evict with the window rows' O_obs and LSE_obs given as for
 * restkv_score_from_lse (Appendix B; Eq. 3, 7-9, 13, 14): score, select and compact with one read of K and V.
 * All other arguments, outputs and error codes as for restkv_evict.
 */
restkv_status restkv_evict_from_lse(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                                    const void* V, const float* O_obs, const float* LSE_obs, float ema_decay,
                                    const restkv_pool_params* pool, int budget, float* scores_out, int32_t* indices,
                                    void* K_out, void* V_out, void* workspace, size_t workspace_bytes,
                                    restkv_stream stream);

/*
 * restkv_select -- Eq. 14's argmax_B: per (batch, KV head) the min(budget, n_kv) largest scores,
 * ties to the lower index, indices written in ascending order.
 *   scores   device float [batch, n_kv_heads, n_kv] (+inf allowed, NaN not)
 *   indices  device int32 [batch, n_kv_heads, min(budget, n_kv)]
 */
restkv_status restkv_select(restkv_handle* h, const restkv_shape* shape, const float* scores, int budget,
                            int32_t* indices, void* workspace, size_t workspace_bytes, restkv_stream stream);

/*
 * restkv_compact -- Eq. 14's gather: K_out[b,h,s,:] = K[b,h,indices[b,h,s],:], same for V; bit-exact.
 *   indices       device int32 [batch, n_kv_heads, n_sel], each in [0, n_kv) (out-of-range entries are
 *                 skipped and set the sticky status word)
 *   K_out, V_out  device [batch, n_kv_heads, n_sel, head_dim] contiguous, dtype per shape->dtype
 */
restkv_status restkv_compact(restkv_handle* h, const restkv_shape* shape, const void* K, const void* V,
                             const int32_t* indices, int n_sel, void* K_out, void* V_out, restkv_stream stream);

/*
 * restkv_evict -- the fused path: score, select and compact in one call on one stream (Eq. 3-14).
 *   scores_out   optional device float [batch, n_kv_heads, n_kv] (NULL: kept in the workspace only)
 *   indices      device int32 [batch, n_kv_heads, min(budget, n_kv)]
 *   K_out, V_out device [batch, n_kv_heads, min(budget, n_kv), head_dim]
 */
restkv_status restkv_evict(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                           const void* V, float ema_decay, const restkv_pool_params* pool, int budget,
                           float* scores_out, int32_t* indices, void* K_out, void* V_out, void* workspace,
                           size_t workspace_bytes, restkv_stream stream);

/*
 * restkv_evict_host -- the fused path for callers whose tensors live in HOST memory: copies Q_obs, K, V
 * (contiguous, host, ideally pinned) into caller-provided device staging buffers, runs restkv_evict and
 * copies indices, K_out and V_out back to host memory, all asynchronously on `stream`.  shape strides
 * must be 0 (contiguous).  The device buffers d_* have the sizes of their host counterparts.
 */
restkv_status restkv_evict_host(restkv_handle* h, const restkv_shape* shape, const void* Q_host, const void* K_host,
                                const void* V_host, float ema_decay, const restkv_pool_params* pool, int budget,
                                int32_t* indices_host, void* K_out_host, void* V_out_host, void* d_Q, void* d_K,
                                void* d_V, int32_t* d_indices, void* d_K_out, void* d_V_out, void* workspace,
                                size_t workspace_bytes, restkv_stream stream);

/*
 * restkv_decode -- one decode step (Eq. 3) of every query head over a cache of n_rows rows, split along
 * the rows and merged by log-sum-exp.  Built to time decode over the compacted against the full cache.
 *   q        device [batch, n_q_heads, head_dim]
 *   Kc, Vc   device [batch, n_kv_heads, n_rows, head_dim] contiguous
 *   out      device float [batch, n_q_heads, head_dim]
 *   lse      optional device float [batch, n_q_heads] (natural-log sum of exp of the scaled logits)
 * shape->n_kv, w, causal_tail and the strides are ignored.
 * RESTKV_BF16 with head_dim 128 and up to 128 query heads per KV head runs as plain attention on the tensor-core
 * kernel (the softmax weights are rounded to bf16 before they meet V) when the workspace has the ~10 MB it needs,
 * which every restkv_workspace_bytes() result has; everything else runs on fp32 SIMT kernels, which need
 * batch * n_kv_heads * 64 * group * (head_dim + 2) floats and take 1, 2, 4 or 8 query heads per KV head and rows of
 * 32, 64, ..., 1024 bytes (head_dim * element size a power of two); other shapes return RESTKV_ERR_UNSUPPORTED.
 */
restkv_status restkv_decode(restkv_handle* h, const restkv_shape* shape, const void* q, const void* Kc,
                            const void* Vc, int n_rows, float* out, float* lse, void* workspace,
                            size_t workspace_bytes, restkv_stream stream);

/*
 * restkv_decode_static -- restkv_decode for callers that cannot give it a workspace.  (The paper has no
 * counterpart: this is a packaging variant of the decode step above, not another operation.)
 *
 * Some hosts of this library cannot allocate device memory when they reach the decode step: an inference
 * server that handed the whole GPU to its own memory pool at start-up (a later cudaMalloc fails or eats into
 * the pool's headroom), or a latency-bound token loop that cannot afford the device-wide synchronisation a
 * cudaMalloc / cudaFree pair brings.  For them the split partials live in a 2 MiB array that is part of the
 * library image itself, so this call needs neither a handle (restkv_create allocates a status block) nor a
 * workspace, and it calls no allocating routine of CUDA or of any other library.
 *
 *   shape, q, Kc, Vc, n_rows, out, lse   exactly as for restkv_decode (device pointers, caller-owned)
 *
 * Limits and rules
 *  - Capacity: batch * n_q_heads * (head_dim + 2) floats per split must fit in 524288 floats (2 MiB); larger
 *    shapes return RESTKV_ERR_WORKSPACE and enqueue nothing.  Within the capacity the call uses as many row
 *    splits as fit (at most 64), so very wide batches run with fewer splits than restkv_decode would use.
 *  - Every GPU that loads the library carries the 2 MiB until the process exits.
 *  - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 *    device current) and remembers it; make that first call outside any stream capture.  With CUDA's lazy
 *    module loading that first call is also the moment the driver places the module, array included, in
 *    device memory: a host that hands all device memory to its own pool must make one call (any small
 *    shape) BEFORE it does so, or the first call can fail with RESTKV_ERR_CUDA (out of memory);
 *    restkv_decode_static_last_cuda_error() then returns the cudaError_t.
 *  - All calls on a device share the one array.  A call overwrites every slot it later reads, so nothing from
 *    an earlier call leaks into a result; but two calls whose kernels overlap on the GPU (different streams,
 *    no ordering between them) race on it.  Order them on one stream or with events.
 *  - There is no device status word on this path and no launch counter; errors are the return code only.
 */
int restkv_decode_static_last_cuda_error(void);   /* cudaError_t of the last failed CUDA call of the entry below, 0 if none */
restkv_status restkv_decode_static(const restkv_shape* shape, const void* q, const void* Kc, const void* Vc,
                                   int n_rows, float* out, float* lse, restkv_stream stream);

/* Synchronises `stream`, then returns and clears the sticky device status (RESTKV_OK if none). */
restkv_status restkv_poll_status(restkv_handle* h, restkv_stream stream);

/* Number of kernel launches the library has enqueued through this handle since creation. */
long long restkv_launch_count(const restkv_handle* h);

/* Last CUDA error code seen by this handle (0 = none). */
int restkv_last_cuda_error(const restkv_handle* h);

const char* restkv_error_string(restkv_status s);

/* Profiling aid: while a pair of events is set for kernel `which` (RESTKV_KERNEL_*, not NONE), every call records
 * `start` right before and `stop` right after that kernel's launch on the call's stream, so a caller can time
 * single kernels of the fused path with CUDA events.  start/stop are cudaEvent_t handles created by the caller
 * with timing enabled; passing NULL for both clears the pair.  On the tensor-core path pass 1, the merge and pass 2
 * are one launch, recorded as RESTKV_KERNEL_PASS2 (PASS1 and COMBINE fire on the SIMT path only); in restkv_evict
 * the pooling and the gather run inside the select kernel, recorded as RESTKV_KERNEL_SELECT. */
typedef enum {
  RESTKV_KERNEL_NONE = 0, RESTKV_KERNEL_PASS1 = 1, RESTKV_KERNEL_COMBINE = 2, RESTKV_KERNEL_PASS2 = 3,
  RESTKV_KERNEL_POOL = 4, RESTKV_KERNEL_SELECT = 5, RESTKV_KERNEL_COMPACT = 6
} restkv_kernel_id;
restkv_status restkv_set_profile_events(restkv_handle* h, int which, void* start, void* stop);

/* Kernel choice: 0 = automatic, 1 = force the fp32 SIMT kernels, 2 = require the tensor-core kernel (one persistent
 * launch that runs pass 1, the merge of the partial softmax results and pass 2 with every head in flight; what 0
 * picks when the shape qualifies), 3 = require the tensor-core kernel in its head-sequential form: only as many
 * heads in flight as fit in L2, so that pass 2 re-reads K and V from there (half the DRAM reads, but two grid
 * barriers per head; the slower of the two on today's shapes). */
restkv_status restkv_set_kernel_path(restkv_handle* h, int path);

/* restkv_evict on the tensor-core path with a fixed window lets the score kernel itself pool (Eq. 13), select and
 * gather (Eq. 14) each head, with the head's own thread blocks, as soon as the head's scores are complete (default:
 * on).  With 0 the pooling, selection and gather always run as the separate kernel that other paths use; the results
 * are the same.  Meant for timing the two against each other. */
restkv_status restkv_set_fused_select(restkv_handle* h, int on);
int restkv_last_evict_fused_select(const restkv_handle* h);   /* 1 if the last restkv_evict ran them inside the score kernel */

/* Bound of every device-side wait of the persistent kernels, in SM clocks (default 2e9, about a second).  A wait
 * that runs out sets the sticky status (RESTKV_ERR_TIMEOUT from restkv_poll_status), the kernel stops issuing
 * work, waits for what it already issued and returns; the call's outputs are then undefined.  Meant for tests of
 * that path and for callers that want to fail faster.  The paper has no counterpart. */
restkv_status restkv_set_wait_limit(restkv_handle* h, long long sm_clocks);

/*
 * restkv_evict_budgets -- restkv_evict with a budget of its own for every (batch, KV head): what the layer-wise and
 * head-wise budget allocation strategies of Appendix C hand to the eviction step (the strategies themselves are
 * not part of this library).
 *   budgets      device int32 [batch, n_kv_heads]; head r keeps min(max(budgets[r], 1), max_budget, n_kv) rows
 *   max_budget   >= 1: with S = min(max_budget, n_kv), the row stride of the outputs
 *   indices      device int32 [batch, n_kv_heads, S]: the kept rows of a head ascending, then -1 up to S
 *   K_out, V_out device [batch, n_kv_heads, S, head_dim]: rows past a head's count are left untouched
 *   scores_out, workspace (restkv_workspace_bytes[_adaptive](shape, max_budget)), pool, errors: as restkv_evict.
 * The selection and the gather run in the cluster select kernel (never inside the score kernel).
 */
restkv_status restkv_evict_budgets(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                                   const void* V, float ema_decay, const restkv_pool_params* pool,
                                   const int32_t* budgets, int max_budget, float* scores_out, int32_t* indices,
                                   void* K_out, void* V_out, void* workspace, size_t workspace_bytes,
                                   restkv_stream stream);

/* Ablation variants (Appendix G) as modes of the same kernels.  A handle starts with every field 0: the method as
 * Sections 3.2-3.3 define it.  The setting applies to every later restkv_score, restkv_evict, restkv_evict_host,
 * restkv_score_from_lse, restkv_evict_from_lse and restkv_evict_budgets call through the handle; restkv_select, restkv_compact and the
 * decode calls do not depend on it.
 *   indicator (Appendix G.1, indicator table), per query t and token j:
 *     RECONSTRUCTION  A_t[j] / (1 - A_t[j]) * ||o_t - v_j||_2, Eq. 7
 *     ATTENTION       A_t[j], the attention weight alone
 *     ATTENTION_VNORM A_t[j] * ||v_j||_2
 *   temporal (Appendix G.2, smoothing table), over the w window queries, oldest first, alpha = 1 - ema_decay:
 *     EMA      Eq. 8-9: the recursion from the oldest query on (the newest weighs alpha, the oldest (1-alpha)^(w-1))
 *     MEAN     1/w each
 *     INV_EMA  the same recursion run from the newest query to the oldest (the oldest weighs alpha)
 *     NONE     the newest query's indicator alone
 *   spatial (same table): MEAN = the box mean of Eq. 13; MAX = the maximum over the same box, taps outside the scored
 *     rows counting as 0 like in the mean.  Applies to the fixed and to the adaptive window.
 *   group: MEAN or MAX over the query heads that share a KV head (the paper leaves grouped-query attention open).
 * Every combination is accepted.  The tensor-core kernel carries all of them except where its fp32 temporal chain
 * cannot (EMA with ema_decay = 1; INV_EMA with ema_decay = 0, = 1 or (1/ema_decay)^(w-1) > 2^40): those run on the
 * fp32 SIMT kernels, or return RESTKV_ERR_UNSUPPORTED under restkv_set_kernel_path(h, 2 or 3).  With
 * indicator != RECONSTRUCTION a cache of one visible row scores A = 1 (times ||v||), not the 0 that Eq. 7's 0/0 is
 * defined as.  v == NULL restores the defaults.  RESTKV_ERR_INVALID_ARG on a field out of range. */
typedef enum {
  RESTKV_INDICATOR_RECONSTRUCTION = 0, RESTKV_INDICATOR_ATTENTION = 1, RESTKV_INDICATOR_ATTENTION_VNORM = 2
} restkv_indicator;
typedef enum {
  RESTKV_TEMPORAL_EMA = 0, RESTKV_TEMPORAL_MEAN = 1, RESTKV_TEMPORAL_INV_EMA = 2, RESTKV_TEMPORAL_NONE = 3
} restkv_temporal;
typedef enum { RESTKV_SPATIAL_MEAN = 0, RESTKV_SPATIAL_MAX = 1 } restkv_spatial;
typedef enum { RESTKV_GROUP_MEAN = 0, RESTKV_GROUP_MAX = 1 } restkv_group;
typedef struct {
  int indicator;   /* restkv_indicator */
  int temporal;    /* restkv_temporal */
  int spatial;     /* restkv_spatial */
  int group;       /* restkv_group */
} restkv_variant;
restkv_status restkv_set_variant(restkv_handle* h, const restkv_variant* v);   /* v: host pointer, read during the call */

/*
 * The output projection inside the indicator (Eq. 4 and Eq. 7 as printed: || (o_t - v_j) W_O ||_2, where W_O is the
 * query head's d x d_model slice of the layer's output projection).  A handle starts without one: W_O = identity.
 *
 * restkv_prepare_output_projection -- once per layer: from W_O, device [n_q_heads * head_dim, d_model] row-major
 *   (rows hq*head_dim .. of query head hq; dtype bf16 or f32), fill the caller-owned device buffer `factor`
 *   (256-byte aligned, restkv_output_projection_bytes(n_q_heads, head_dim) bytes) with what the kernels read: per
 *   query head M = W W^T (fp32), a Cholesky factor of M rounded to bf16 and the product of the rounded factor with
 *   its transpose.  Two kernels on `stream`.  head_dim a multiple of 16, at most 128 (else RESTKV_ERR_UNSUPPORTED);
 *   RESTKV_ERR_WORKSPACE if `factor` is misaligned or too small.  A singular M (d_model < head_dim) is accepted;
 *   its null directions get no weight.
 * restkv_set_output_projection -- every later restkv_score / restkv_evict / ..._from_lse / ..._budgets /
 *   restkv_evict_host call through the handle measures Eq. 7's norm through this factor (the buffer must stay
 *   alive and unchanged; NULL returns to the identity).  A call whose shape has other n_q_heads or head_dim than
 *   the factor returns RESTKV_ERR_INVALID_ARG.  The attention-weight indicators of restkv_set_variant have no norm
 *   of an output difference and ignore it.
 */
size_t restkv_output_projection_bytes(int n_q_heads, int head_dim);
restkv_status restkv_prepare_output_projection(restkv_handle* h, int n_q_heads, int head_dim, int d_model,
                                               restkv_dtype dtype, const void* W_O, void* factor,
                                               size_t factor_bytes, restkv_stream stream);
restkv_status restkv_set_output_projection(restkv_handle* h, const void* factor, int n_q_heads, int head_dim);

#ifdef __cplusplus
}
#endif
#endif /* RESTKV_H_ */
