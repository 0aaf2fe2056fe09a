// C ABI of librestkv.so: argument checks, workspace carve-up and kernel sequencing.
#include <cstdio>
#include <cstring>
#include <cmath>
#include <new>

#include "restkv_common.cuh"

struct restkv_handle {
  int device;
  int sm_count;
  unsigned int* dev_status;   // 256-byte device block, word 0 = sticky status bits
  void* tc_state;
  long long launches;
  int last_cuda_error;
  int kernel_path;            // 0 auto, 1 SIMT, 2 tensor core required, 3 tensor core in its head-sequential form
  bool fused_select;          // restkv_evict lets the tensor-core score kernel pool, select and gather when it can
  bool last_evict_fused;      // whether the last restkv_evict did
  long long wait_limit;       // SM clocks a device-side wait may last
  restkv_variant variant;     // ablation variant of the score calls (all 0: the method as printed)
  const void* proj_factor;    // output-projection factor of the score calls (null: identity), caller-owned
  int proj_heads, proj_dim;   // the shape it was prepared for
  cudaEvent_t prof_start[7], prof_stop[7];   // per restkv_kernel_id, null = not timed
};

namespace restkv {

static size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

int pass1_splits(const Problem& p, int sm_count) {
  // one wave of (batch, head, split) blocks over the SMs, at least one 128-token tile per split
  int splits = sm_count / p.BH;
  const int tiles = (p.n_kv + 127) / 128;
  if (splits > tiles) splits = tiles;
  if (splits < 1) splits = 1;
  return splits;
}

static int decode_splits(const Problem& p, int n_rows, int sm_count) {
  int splits = (2 * sm_count + p.BH - 1) / p.BH;
  const int by_rows = (n_rows + 255) / 256;
  if (splits > by_rows) splits = by_rows;
  if (splits > kDecodeMaxSplits) splits = kDecodeMaxSplits;
  if (splits < 1) splits = 1;
  return splits;
}

size_t plan_workspace(const Problem& p, int budget, int sm_count, bool adaptive, void* base, Workspace* ws) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    void* ptr = base ? (void*)((char*)base + off) : nullptr;
    off += align256(bytes);
    return ptr;
  };
  Workspace w{};
  w.splits = pass1_splits(p, sm_count);
  // at least the tensor-core kernel's 128 query rows, so that restkv_decode can use it whatever w * group is
  const size_t BH = (size_t)p.BH, R = (size_t)(p.R > 128 ? p.R : 128), d = (size_t)p.d;
  // partial slots: one per (head, split) on the SIMT path, one per CTA in the persistent tensor-core kernel
  size_t slots = BH * w.splits;
  if (slots < (size_t)sm_count) slots = (size_t)sm_count;
  w.part_m = (float*)take(slots * R * sizeof(float));
  w.part_l = (float*)take(slots * R * sizeof(float));
  w.part_O = (float*)take(slots * R * d * sizeof(float));
  w.counters = (unsigned int*)take(1024);
  w.tile_max = (float*)take(BH * (size_t)((p.n_kv + 127) / 128) * 128 * sizeof(float));
  w.row_M2 = (float*)take(BH * 128 * sizeof(float));
  w.sel_hist = (unsigned int*)take(tc_fused_select_hist_words(p.BH) * sizeof(unsigned int));
  w.sel_sfx = (unsigned int*)take(tc_fused_select_sfx_words(sm_count) * sizeof(unsigned int));
  w.q_pad = (__nv_bfloat16*)take(BH * 128 * 128 * sizeof(__nv_bfloat16));
  w.vnorm = (float*)take(BH * (size_t)p.n_kv * sizeof(float));
  w.fin_m = (float*)take(BH * R * sizeof(float));
  w.fin_l = (float*)take(BH * R * sizeof(float));
  w.O_f32 = (float*)take(BH * R * d * sizeof(float));
  w.O_m2 = (__nv_bfloat16*)take(BH * R * d * sizeof(__nv_bfloat16));
  w.aug = (__nv_bfloat16*)take(BH * R * 64 * sizeof(__nv_bfloat16));
  w.I_hat = (float*)take(BH * (size_t)p.n * sizeof(float));
  w.O_proj = (float*)take(BH * R * d * sizeof(float));
  w.vmv = (float*)take(BH * (size_t)p.G * (size_t)p.n_kv * sizeof(float));
  w.scores = (float*)take(BH * (size_t)p.n_kv * sizeof(float));
  w.pool = (int*)take(BH * 2 * sizeof(int));
  w.dec_part = (float*)take(BH * (size_t)kDecodeMaxSplits * p.G * (d + 2) * sizeof(float));
  if (adaptive) {
    int Bp = budget - p.tail;
    if (Bp > p.n) Bp = p.n;
    if (Bp < 1) Bp = 1;
    w.I_raw = (float*)take((size_t)p.batch * p.Hq * p.w * p.n * sizeof(float));
    w.adaptive_idx = (int32_t*)take((size_t)p.batch * p.Hq * p.w * Bp * sizeof(int32_t));
    w.adaptive_sums = (unsigned long long*)take(BH * 2 * sizeof(unsigned long long));
  }
  w.bytes = off;
  if (ws) *ws = w;
  return off;
}

// The part of the workspace that restkv_decode's tensor-core path uses (phases A and B of the score kernel only).
static size_t plan_decode_tc(int BH, int sm_count, void* base, Workspace* ws) {
  size_t off = 0;
  auto take = [&](size_t bytes) {
    void* ptr = base ? (void*)((char*)base + off) : nullptr;
    off += align256(bytes);
    return ptr;
  };
  Workspace w{};
  const size_t bh = (size_t)BH, slots = (size_t)sm_count;
  w.part_m = (float*)take(slots * 128 * sizeof(float));
  w.part_l = (float*)take(slots * 128 * sizeof(float));
  w.part_O = (float*)take(slots * 128 * 128 * sizeof(float));
  w.counters = (unsigned int*)take(1024);
  w.row_M2 = (float*)take(bh * 128 * sizeof(float));
  w.q_pad = (__nv_bfloat16*)take(bh * 128 * 128 * sizeof(__nv_bfloat16));
  w.O_f32 = (float*)take(bh * 128 * 128 * sizeof(float));
  w.O_m2 = (__nv_bfloat16*)take(bh * 128 * 128 * sizeof(__nv_bfloat16));
  w.aug = (__nv_bfloat16*)take(bh * 128 * 64 * sizeof(__nv_bfloat16));
  w.bytes = off;
  if (ws) *ws = w;
  return off;
}

static bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// Validates the shape and fills Problem.  `need_kv`: check the score-path fields too.
static restkv_status make_problem(const restkv_shape* s, bool need_kv, Problem* out) {
  if (!s) return RESTKV_ERR_INVALID_ARG;
  if (s->batch < 1 || s->n_q_heads < 1 || s->n_kv_heads < 1 || s->head_dim < 1) return RESTKV_ERR_INVALID_ARG;
  if (s->n_q_heads % s->n_kv_heads != 0) return RESTKV_ERR_INVALID_ARG;
  if (s->dtype != RESTKV_BF16 && s->dtype != RESTKV_F32) return RESTKV_ERR_INVALID_ARG;
  Problem p{};
  p.batch = s->batch; p.Hq = s->n_q_heads; p.Hkv = s->n_kv_heads; p.G = p.Hq / p.Hkv; p.d = s->head_dim;
  p.dtype = s->dtype;
  p.BH = p.batch * p.Hkv;
  p.scale = s->softmax_scale != 0.f ? s->softmax_scale : 1.0f / sqrtf((float)p.d);
  if (!(p.scale > 0.f) || !std::isfinite(p.scale)) return RESTKV_ERR_INVALID_ARG;
  if (p.d % 8 != 0) return RESTKV_ERR_UNSUPPORTED;
  if (p.d > 256) return RESTKV_ERR_UNSUPPORTED;
  if (need_kv) {
    if (s->n_kv < 1 || s->w < 1) return RESTKV_ERR_INVALID_ARG;
    if (s->causal_tail != 0 && s->causal_tail != s->w) return RESTKV_ERR_INVALID_ARG;
    p.n_kv = s->n_kv; p.w = s->w; p.tail = s->causal_tail; p.n = p.n_kv - p.tail;
    if (p.n < 1) return RESTKV_ERR_INVALID_ARG;
    p.R = p.w * p.G;
    const bool k0 = s->k_stride_b == 0 && s->k_stride_h == 0 && s->k_stride_n == 0;
    const bool v0 = s->v_stride_b == 0 && s->v_stride_h == 0 && s->v_stride_n == 0;
    p.ksn = k0 ? p.d : s->k_stride_n; p.ksh = k0 ? (long long)p.n_kv * p.d : s->k_stride_h;
    p.ksb = k0 ? (long long)p.Hkv * p.n_kv * p.d : s->k_stride_b;
    p.vsn = v0 ? p.d : s->v_stride_n; p.vsh = v0 ? (long long)p.n_kv * p.d : s->v_stride_h;
    p.vsb = v0 ? (long long)p.Hkv * p.n_kv * p.d : s->v_stride_b;
    const long long strides[6] = {p.ksb, p.ksh, p.ksn, p.vsb, p.vsh, p.vsn};
    for (long long st : strides)
      if (st < 0 || st % 8 != 0) return RESTKV_ERR_INVALID_ARG;
    if (p.ksn < p.d || p.vsn < p.d) return RESTKV_ERR_INVALID_ARG;
  }
  *out = p;
  return RESTKV_OK;
}

// The handle's variant and output projection become part of the problem; false if the projection was prepared
// for another shape.
static bool apply_variant(const restkv_handle* h, Problem* p) {
  p->indicator = h->variant.indicator; p->temporal = h->variant.temporal;
  p->spatial = h->variant.spatial; p->group = h->variant.group;
  p->proj = Projection{};
  if (h->proj_factor) {
    if (h->proj_heads != p->Hq || h->proj_dim != p->d) return false;
    // only Eq. 7 has the projected norm
    if (p->indicator == RESTKV_INDICATOR_RECONSTRUCTION) p->proj = projection_view(h->proj_factor, p->Hq, p->d);
  }
  return true;
}

static restkv_status check_pool(const restkv_pool_params* pp, const Problem& p) {
  if (!pp) return RESTKV_ERR_INVALID_ARG;
  if (pp->mode == RESTKV_POOL_FIXED) {
    if (pp->width < 1 || pp->width % 2 == 0) return RESTKV_ERR_INVALID_ARG;
  } else if (pp->mode == RESTKV_POOL_ADAPTIVE) {
    if (pp->base_width < 1 || pp->base_width % 2 == 0 || !(pp->beta > 0.f)) return RESTKV_ERR_INVALID_ARG;
    if (pp->budget - p.tail < 1) return RESTKV_ERR_INVALID_ARG;
  } else {
    return RESTKV_ERR_INVALID_ARG;
  }
  return RESTKV_OK;
}

static bool simt_supported(const Problem& p) {
  if (p.R > 256) return false;
  const size_t smem1 = ((size_t)2 * p.R * (p.d + 1) + (size_t)2 * 32 * p.d) * sizeof(float);
  return smem1 <= 220 * 1024;
}

struct Call {
  restkv_handle* h;
  cudaStream_t st;
  restkv_status fail(cudaError_t e) {
    h->last_cuda_error = (int)e;
    return RESTKV_ERR_CUDA;
  }
};

#define RESTKV_LAUNCH(call, id, expr, count)                                                    \
  do {                                                                                          \
    const bool prof__ = (call).h->prof_start[(id)] != nullptr;                                  \
    if (prof__) cudaEventRecord((call).h->prof_start[(id)], (call).st);                         \
    cudaError_t e__ = (expr);                                                                   \
    if (e__ != cudaSuccess) return (call).fail(e__);                                            \
    if (prof__) cudaEventRecord((call).h->prof_stop[(id)], (call).st);                          \
    (call).h->launches += (count);                                                              \
  } while (0)

// score: pass 1, combine, pass 2, window parameters and, when `scores` is non-null, pooling.  With `scores`
// null the caller pools (the fused path does it inside the select kernel).
static restkv_status run_score(Call& c, const Problem& p, const Workspace& ws, const void* Q, const void* K,
                               const void* V, float ema_decay, const restkv_pool_params* pool, float* scores,
                               int32_t* pool_used, const FusedSelect* sel = nullptr, bool* sel_done = nullptr,
                               const float* O_given = nullptr, const float* LSE_given = nullptr) {
  const bool adaptive = pool->mode == RESTKV_POOL_ADAPTIVE;
  // the tensor-core pass 2 carries the temporal weights as an fp32 Horner chain, which Eq. 9 with alpha = 0 and
  // some inverted EMAs do not fit: those run on the SIMT kernels
  // (the adaptive window needs the per-query indicators, which the tensor-core kernel writes out only when it runs
  // pass 1 itself)
  bool use_tc = tc_supported(p) && c.h->tc_state != nullptr && !(adaptive && O_given) &&
                tc_variant_supported(p, ema_decay);
  if (p.n_kv == 1 && p.indicator != RESTKV_INDICATOR_RECONSTRUCTION) use_tc = false;
  if (p.proj.M && !tc_vmv_supported(p)) use_tc = false;
  if (c.h->kernel_path == 1) use_tc = false;
  if (c.h->kernel_path >= 2 && !use_tc) return RESTKV_ERR_UNSUPPORTED;
  if (!use_tc && !simt_supported(p)) return RESTKV_ERR_UNSUPPORTED;
  if (p.n_kv == 1 && p.indicator == RESTKV_INDICATOR_RECONSTRUCTION) {
    // A single visible row has A = 1 and nothing to redistribute its weight to: the indicator is
    // 0/0 there and is defined as 0 (Eq. 7 has no value), so no kernel is needed.
    cudaError_t e = cudaMemsetAsync(ws.I_hat, 0, (size_t)p.BH * p.n * sizeof(float), c.st);
    if (e == cudaSuccess && adaptive)
      e = cudaMemsetAsync(ws.I_raw, 0, (size_t)p.batch * p.Hq * p.w * p.n * sizeof(float), c.st);
    if (e != cudaSuccess) return c.fail(e);
  } else if (O_given) {
    // the window rows' outputs and log-sum-exps come from the caller: pass 1 and the merge are not needed
    RESTKV_LAUNCH(c, RESTKV_KERNEL_COMBINE, launch_from_lse_prep(p, ws, O_given, LSE_given, use_tc, c.st), 1);
    if (use_tc && p.proj.M)
      RESTKV_LAUNCH(c, RESTKV_KERNEL_PASS1,
                    launch_tc_vmv(c.h->tc_state, p, V, ws.vmv, c.h->sm_count, c.h->wait_limit, c.h->dev_status, c.st), 1);
    if (use_tc) {
      const bool with_sel = sel && c.h->fused_select &&
                            tc_fused_select_supported(p, c.h->sm_count, false, sel->keep, sel->W, sel->gamma);
      RESTKV_LAUNCH(c, RESTKV_KERNEL_PASS2,
                    launch_tc_fused(c.h->tc_state, p, ws, Q, K, V, ema_decay, c.h->sm_count, false, false,
                                    c.h->wait_limit, with_sel ? sel : nullptr, O_given, nullptr, c.h->dev_status, c.st), 1);
      if (sel_done) *sel_done = with_sel;
    } else {
      Workspace wsl = ws;
      wsl.O_f32 = const_cast<float*>(O_given);
      if (p.proj.M) RESTKV_LAUNCH(c, RESTKV_KERNEL_COMBINE, launch_projection_rows(p, O_given, ws.O_proj, c.st), 1);
      RESTKV_LAUNCH(c, RESTKV_KERNEL_PASS2,
                    launch_simt_pass2(p, wsl, Q, K, V, ema_decay, adaptive ? ws.I_raw : nullptr, c.st), 1);
    }
  } else if (use_tc) {
    // pass 1, merge and pass 2 in one persistent launch (timed as "pass 2"); path 3 keeps only as many heads in
    // flight as fit in L2 so that pass 2 re-reads K and V from there
    const bool reuse_l2 = c.h->kernel_path == 3;
    if (p.proj.M)   // the tokens' own terms under the output projection, by a kernel of its own (timed as "pass 1")
      RESTKV_LAUNCH(c, RESTKV_KERNEL_PASS1,
                    launch_tc_vmv(c.h->tc_state, p, V, ws.vmv, c.h->sm_count, c.h->wait_limit, c.h->dev_status, c.st), 1);
    const bool with_sel = sel && c.h->fused_select &&
                          tc_fused_select_supported(p, c.h->sm_count, reuse_l2, sel->keep, sel->W, sel->gamma);
    RESTKV_LAUNCH(c, RESTKV_KERNEL_PASS2,
                  launch_tc_fused(c.h->tc_state, p, ws, Q, K, V, ema_decay, c.h->sm_count, reuse_l2, false,
                                  c.h->wait_limit, with_sel ? sel : nullptr, nullptr, adaptive ? ws.I_raw : nullptr,
                                  c.h->dev_status, c.st), 1);
    if (sel_done) *sel_done = with_sel;
  } else {
    RESTKV_LAUNCH(c, RESTKV_KERNEL_PASS1, launch_simt_pass1(p, ws, Q, K, V, c.st), 1);
    RESTKV_LAUNCH(c, RESTKV_KERNEL_COMBINE, launch_combine(p, ws, c.st), 1);
    if (p.proj.M) RESTKV_LAUNCH(c, RESTKV_KERNEL_COMBINE, launch_projection_rows(p, ws.O_f32, ws.O_proj, c.st), 1);
    RESTKV_LAUNCH(c, RESTKV_KERNEL_PASS2, launch_simt_pass2(p, ws, Q, K, V, ema_decay, adaptive ? ws.I_raw : nullptr, c.st), 1);
  }
  if (adaptive) {
    int nl = 0;
    cudaError_t e = launch_adaptive_params(p, ws, pool->budget, pool->beta, pool->base_width, c.st, &nl);
    if (e != cudaSuccess) return c.fail(e);
    c.h->launches += nl;
  }
  if (scores)
    RESTKV_LAUNCH(c, RESTKV_KERNEL_POOL,
                  launch_pool(p, ws, adaptive ? ws.pool : nullptr, pool->width, pool->shift, scores, pool_used, c.st), 1);
  return RESTKV_OK;
}

static restkv_status check_ws(const Problem& p, int budget, int sm_count, bool adaptive, void* workspace,
                              size_t bytes, Workspace* ws) {
  if (!workspace || ((uintptr_t)workspace & 255u) != 0) return RESTKV_ERR_WORKSPACE;
  const size_t need = plan_workspace(p, budget, sm_count, adaptive, workspace, ws);
  if (bytes < need) return RESTKV_ERR_WORKSPACE;
  return RESTKV_OK;
}

}  // namespace restkv

using namespace restkv;

extern "C" {

restkv_status restkv_create(restkv_handle** out) {
  if (!out) return RESTKV_ERR_INVALID_ARG;
  *out = nullptr;
  restkv_handle* h = new (std::nothrow) restkv_handle();
  if (!h) return RESTKV_ERR_CUDA;
  cudaError_t e = cudaGetDevice(&h->device);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&h->sm_count, cudaDevAttrMultiProcessorCount, h->device);
  int major = 0;
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, h->device);
  if (e == cudaSuccess && major != 10) { delete h; return RESTKV_ERR_UNSUPPORTED; }   // sm_100a only
  if (e == cudaSuccess) e = cudaMalloc((void**)&h->dev_status, 256);
  if (e == cudaSuccess) e = cudaMemset(h->dev_status, 0, 256);
  if (e != cudaSuccess) { delete h; return RESTKV_ERR_CUDA; }
  h->tc_state = nullptr;
  if (tc_init(&h->tc_state) != cudaSuccess || tc_fused_init() != cudaSuccess) h->tc_state = nullptr;
  h->wait_limit = 2000000000ll;
  h->fused_select = true;
  h->last_evict_fused = false;
  h->variant = restkv_variant{0, 0, 0, 0};
  h->proj_factor = nullptr;
  h->proj_heads = h->proj_dim = 0;
  h->launches = 0;
  h->last_cuda_error = 0;
  h->kernel_path = 0;
  for (int i = 0; i < 7; ++i) h->prof_start[i] = h->prof_stop[i] = nullptr;
  *out = h;
  return RESTKV_OK;
}

restkv_status restkv_destroy(restkv_handle* h) {
  if (!h) return RESTKV_ERR_INVALID_ARG;
  cudaFree(h->dev_status);
  delete h;
  return RESTKV_OK;
}

static int sm_count_or_default() {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) {
    int v = 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) sms = v;
  }
  return sms;
}

size_t restkv_workspace_bytes(const restkv_shape* shape, int budget) {
  Problem p;
  if (make_problem(shape, true, &p) != RESTKV_OK || budget < 0) return 0;
  return plan_workspace(p, budget, sm_count_or_default(), false, nullptr, nullptr);
}

size_t restkv_workspace_bytes_adaptive(const restkv_shape* shape, int budget) {
  Problem p;
  if (make_problem(shape, true, &p) != RESTKV_OK || budget < 1) return 0;
  return plan_workspace(p, budget, sm_count_or_default(), true, nullptr, nullptr);
}

restkv_status restkv_score(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                           const void* V, float ema_decay, const restkv_pool_params* pool, float* scores,
                           int32_t* pool_used, void* workspace, size_t workspace_bytes, restkv_stream stream) {
  if (!h || !Q_obs || !K || !V || !scores) return RESTKV_ERR_INVALID_ARG;
  if (!aligned16(Q_obs) || !aligned16(K) || !aligned16(V) || !aligned16(scores)) return RESTKV_ERR_INVALID_ARG;
  if (!(ema_decay >= 0.f && ema_decay <= 1.f)) return RESTKV_ERR_INVALID_ARG;
  Problem p;
  restkv_status s = make_problem(shape, true, &p);
  if (s != RESTKV_OK) return s;
  if (!apply_variant(h, &p)) return RESTKV_ERR_INVALID_ARG;
  if ((s = check_pool(pool, p)) != RESTKV_OK) return s;
  Workspace ws;
  const bool adaptive = pool->mode == RESTKV_POOL_ADAPTIVE;
  if ((s = check_ws(p, adaptive ? pool->budget : 0, h->sm_count, adaptive, workspace, workspace_bytes, &ws)) !=
      RESTKV_OK)
    return s;
  Call c{h, (cudaStream_t)stream};
  return run_score(c, p, ws, Q_obs, K, V, ema_decay, pool, scores, pool_used);
}

restkv_status restkv_score_from_lse(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                                    const void* V, const float* O_obs, const float* LSE_obs, float ema_decay,
                                    const restkv_pool_params* pool, float* scores, int32_t* pool_used, void* workspace,
                                    size_t workspace_bytes, restkv_stream stream) {
  if (!h || !Q_obs || !K || !V || !O_obs || !LSE_obs || !scores) return RESTKV_ERR_INVALID_ARG;
  if (!aligned16(Q_obs) || !aligned16(K) || !aligned16(V) || !aligned16(O_obs) || !aligned16(scores))
    return RESTKV_ERR_INVALID_ARG;
  if (!(ema_decay >= 0.f && ema_decay <= 1.f)) return RESTKV_ERR_INVALID_ARG;
  Problem p;
  restkv_status s = make_problem(shape, true, &p);
  if (s != RESTKV_OK) return s;
  if (!apply_variant(h, &p)) return RESTKV_ERR_INVALID_ARG;
  if ((s = check_pool(pool, p)) != RESTKV_OK) return s;
  Workspace ws;
  const bool adaptive = pool->mode == RESTKV_POOL_ADAPTIVE;
  if ((s = check_ws(p, adaptive ? pool->budget : 0, h->sm_count, adaptive, workspace, workspace_bytes, &ws)) !=
      RESTKV_OK)
    return s;
  Call c{h, (cudaStream_t)stream};
  return run_score(c, p, ws, Q_obs, K, V, ema_decay, pool, scores, pool_used, nullptr, nullptr, O_obs, LSE_obs);
}

restkv_status restkv_select(restkv_handle* h, const restkv_shape* shape, const float* scores, int budget,
                            int32_t* indices, void* workspace, size_t workspace_bytes, restkv_stream stream) {
  if (!h || !scores || !indices || budget < 1) return RESTKV_ERR_INVALID_ARG;
  Problem p;
  restkv_status s = make_problem(shape, true, &p);
  if (s != RESTKV_OK) return s;
  Workspace ws;
  if ((s = check_ws(p, budget, h->sm_count, false, workspace, workspace_bytes, &ws)) != RESTKV_OK) return s;
  Call c{h, (cudaStream_t)stream};
  RESTKV_LAUNCH(c, RESTKV_KERNEL_SELECT,
                launch_select(p.BH, p.n, p.n_kv, budget, nullptr, nullptr, nullptr, 1, 0, false, const_cast<float*>(scores), indices, nullptr,
                              nullptr, nullptr, nullptr, nullptr, nullptr, c.st), 1);
  return RESTKV_OK;
}

restkv_status restkv_compact(restkv_handle* h, const restkv_shape* shape, const void* K, const void* V,
                             const int32_t* indices, int n_sel, void* K_out, void* V_out, restkv_stream stream) {
  if (!h || !K || !V || !indices || !K_out || !V_out || n_sel < 1) return RESTKV_ERR_INVALID_ARG;
  if (!aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out)) return RESTKV_ERR_INVALID_ARG;
  Problem p;
  restkv_status s = make_problem(shape, true, &p);
  if (s != RESTKV_OK) return s;
  Call c{h, (cudaStream_t)stream};
  RESTKV_LAUNCH(c, RESTKV_KERNEL_COMPACT, launch_compact(p, K, V, indices, n_sel, K_out, V_out, h->dev_status, c.st), 1);
  return RESTKV_OK;
}

// budgets non-null: per (batch, KV head) budgets on the device; `budget` is then the row stride of the outputs.
static restkv_status evict_impl(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                                const void* V, const float* O_obs, const float* LSE_obs, float ema_decay,
                                const restkv_pool_params* pool, int budget, const int32_t* budgets, float* scores_out,
                                int32_t* indices,
                                void* K_out, void* V_out, void* workspace, size_t workspace_bytes,
                                restkv_stream stream) {
  if (!h || !Q_obs || !K || !V || !indices || !K_out || !V_out || budget < 1) return RESTKV_ERR_INVALID_ARG;
  if (!aligned16(Q_obs) || !aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out))
    return RESTKV_ERR_INVALID_ARG;
  if (scores_out && !aligned16(scores_out)) return RESTKV_ERR_INVALID_ARG;
  if (!(ema_decay >= 0.f && ema_decay <= 1.f)) return RESTKV_ERR_INVALID_ARG;
  Problem p;
  restkv_status s = make_problem(shape, true, &p);
  if (s != RESTKV_OK) return s;
  if (!apply_variant(h, &p)) return RESTKV_ERR_INVALID_ARG;
  if ((s = check_pool(pool, p)) != RESTKV_OK) return s;
  Workspace ws;
  const bool adaptive = pool->mode == RESTKV_POOL_ADAPTIVE;
  const int ws_budget = adaptive ? (pool->budget > budget ? pool->budget : budget) : budget;
  if ((s = check_ws(p, ws_budget, h->sm_count, adaptive, workspace, workspace_bytes, &ws)) != RESTKV_OK) return s;
  Call c{h, (cudaStream_t)stream};
  float* scores = scores_out ? scores_out : ws.scores;
  // With a fixed window the tensor-core score kernel pools, selects and gathers each head itself, right after the
  // head's scores are complete and with the head's own CTAs; otherwise the kernels below do.
  const int keep_rows = budget < p.n_kv ? budget : p.n_kv;
  FusedSelect sel{keep_rows, pool->width, pool->shift, scores, indices, K_out, V_out};
  bool sel_done = false;
  if ((s = run_score(c, p, ws, Q_obs, K, V, ema_decay, pool, nullptr, nullptr, (adaptive || budgets) ? nullptr : &sel,
                     &sel_done, O_obs, LSE_obs)) != RESTKV_OK)
    return s;
  h->last_evict_fused = sel_done;
  if (sel_done) return RESTKV_OK;
  // Pooling (Eq. 13) runs inside the select kernel, which also writes the pooled scores.  So does the gather
  // (Eq. 14) while the select kernel's clusters fit the GPU in one wave; with more (batch, head) rows than that the
  // stand-alone gather, which spreads over every SM, is the faster one.
  // (with per-head budgets the index rows have unused tails, which only the select kernel's own gather skips)
  const bool fuse_gather = p.BH * 8 <= h->sm_count || budgets != nullptr;
  RESTKV_LAUNCH(c, RESTKV_KERNEL_SELECT,
                launch_select(p.BH, p.n, p.n_kv, budget, budgets, ws.I_hat, adaptive ? ws.pool : nullptr, pool->width,
                              pool->shift, p.spatial == RESTKV_SPATIAL_MAX, scores, indices, nullptr,
                              fuse_gather ? &p : nullptr, K, V, K_out, V_out, c.st), 1);
  if (!fuse_gather) {
    const int n_sel = budget < p.n_kv ? budget : p.n_kv;
    RESTKV_LAUNCH(c, RESTKV_KERNEL_COMPACT,
                  launch_compact(p, K, V, indices, n_sel, K_out, V_out, h->dev_status, c.st), 1);
  }
  return RESTKV_OK;
}

restkv_status restkv_evict(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                           const void* V, float ema_decay, const restkv_pool_params* pool, int budget,
                           float* scores_out, int32_t* indices, void* K_out, void* V_out, void* workspace,
                           size_t workspace_bytes, restkv_stream stream) {
  return evict_impl(h, shape, Q_obs, K, V, nullptr, nullptr, ema_decay, pool, budget, nullptr, scores_out, indices, K_out,
                    V_out, workspace, workspace_bytes, stream);
}

restkv_status restkv_evict_budgets(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                                   const void* V, float ema_decay, const restkv_pool_params* pool,
                                   const int32_t* budgets, int max_budget, float* scores_out, int32_t* indices,
                                   void* K_out, void* V_out, void* workspace, size_t workspace_bytes,
                                   restkv_stream stream) {
  if (!budgets) return RESTKV_ERR_INVALID_ARG;
  return evict_impl(h, shape, Q_obs, K, V, nullptr, nullptr, ema_decay, pool, max_budget, budgets, scores_out, indices,
                    K_out, V_out, workspace, workspace_bytes, stream);
}

restkv_status restkv_evict_from_lse(restkv_handle* h, const restkv_shape* shape, const void* Q_obs, const void* K,
                                    const void* V, const float* O_obs, const float* LSE_obs, float ema_decay,
                                    const restkv_pool_params* pool, int budget, float* scores_out, int32_t* indices,
                                    void* K_out, void* V_out, void* workspace, size_t workspace_bytes,
                                    restkv_stream stream) {
  if (!O_obs || !LSE_obs || !aligned16(O_obs)) return RESTKV_ERR_INVALID_ARG;
  return evict_impl(h, shape, Q_obs, K, V, O_obs, LSE_obs, ema_decay, pool, budget, nullptr, scores_out, indices, K_out,
                    V_out, workspace, workspace_bytes, stream);
}

restkv_status restkv_evict_host(restkv_handle* h, const restkv_shape* shape, const void* Q_host, const void* K_host,
                                const void* V_host, float ema_decay, const restkv_pool_params* pool, int budget,
                                int32_t* indices_host, void* K_out_host, void* V_out_host, void* d_Q, void* d_K,
                                void* d_V, int32_t* d_indices, void* d_K_out, void* d_V_out, void* workspace,
                                size_t workspace_bytes, restkv_stream stream) {
  if (!h || !Q_host || !K_host || !V_host || !indices_host || !K_out_host || !V_out_host) return RESTKV_ERR_INVALID_ARG;
  if (!d_Q || !d_K || !d_V || !d_indices || !d_K_out || !d_V_out) return RESTKV_ERR_INVALID_ARG;
  Problem p;
  restkv_status s = make_problem(shape, true, &p);
  if (s != RESTKV_OK) return s;
  if (shape->k_stride_b || shape->k_stride_h || shape->k_stride_n || shape->v_stride_b || shape->v_stride_h ||
      shape->v_stride_n)
    return RESTKV_ERR_INVALID_ARG;
  // everything restkv_evict would refuse is refused here, before the first copy is enqueued
  if (budget < 1 || !(ema_decay >= 0.f && ema_decay <= 1.f)) return RESTKV_ERR_INVALID_ARG;
  if (!aligned16(d_Q) || !aligned16(d_K) || !aligned16(d_V) || !aligned16(d_K_out) || !aligned16(d_V_out))
    return RESTKV_ERR_INVALID_ARG;
  if ((s = check_pool(pool, p)) != RESTKV_OK) return s;
  {
    Workspace ws_check;
    const bool adaptive = pool->mode == RESTKV_POOL_ADAPTIVE;
    const int ws_budget = adaptive ? (pool->budget > budget ? pool->budget : budget) : budget;
    if ((s = check_ws(p, ws_budget, h->sm_count, adaptive, workspace, workspace_bytes, &ws_check)) != RESTKV_OK)
      return s;
  }
  const size_t es = p.dtype == RESTKV_BF16 ? 2 : 4;
  const size_t q_bytes = (size_t)p.batch * p.Hq * p.w * p.d * es;
  const size_t kv_bytes = (size_t)p.BH * p.n_kv * p.d * es;
  const int n_sel = budget < p.n_kv ? budget : p.n_kv;
  const size_t out_bytes = (size_t)p.BH * n_sel * p.d * es;
  cudaStream_t st = (cudaStream_t)stream;
  Call c{h, st};
  cudaError_t e;
  if ((e = cudaMemcpyAsync(d_Q, Q_host, q_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return c.fail(e);
  if ((e = cudaMemcpyAsync(d_K, K_host, kv_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return c.fail(e);
  if ((e = cudaMemcpyAsync(d_V, V_host, kv_bytes, cudaMemcpyHostToDevice, st)) != cudaSuccess) return c.fail(e);
  s = restkv_evict(h, shape, d_Q, d_K, d_V, ema_decay, pool, budget, nullptr, d_indices, d_K_out, d_V_out, workspace,
                   workspace_bytes, stream);
  if (s != RESTKV_OK) return s;
  if ((e = cudaMemcpyAsync(indices_host, d_indices, (size_t)p.BH * n_sel * sizeof(int32_t), cudaMemcpyDeviceToHost,
                           st)) != cudaSuccess)
    return c.fail(e);
  if ((e = cudaMemcpyAsync(K_out_host, d_K_out, out_bytes, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return c.fail(e);
  if ((e = cudaMemcpyAsync(V_out_host, d_V_out, out_bytes, cudaMemcpyDeviceToHost, st)) != cudaSuccess) return c.fail(e);
  return RESTKV_OK;
}

restkv_status restkv_decode(restkv_handle* h, const restkv_shape* shape, const void* q, const void* Kc,
                            const void* Vc, int n_rows, float* out, float* lse, void* workspace,
                            size_t workspace_bytes, restkv_stream stream) {
  if (!h || !q || !Kc || !Vc || !out || n_rows < 1) return RESTKV_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(Kc) || !aligned16(Vc)) return RESTKV_ERR_INVALID_ARG;
  Problem p;
  restkv_status s = make_problem(shape, false, &p);
  if (s != RESTKV_OK) return s;
  if (!workspace || ((uintptr_t)workspace & 255u) != 0) return RESTKV_ERR_WORKSPACE;
  Call c{h, (cudaStream_t)stream};
  // bf16, head_dim 128: the decode step is plain attention of up to 128 query rows per KV head, i.e. phases A and B
  // of the tensor-core score kernel with the group's queries padded to its 128 rows.  It needs about 10 MB of
  // workspace (any restkv_workspace_bytes result has that); with less, or for other shapes, the SIMT kernels run.
  bool tc_ws_too_small = false;
  if (h->tc_state && h->kernel_path != 1 && p.dtype == RESTKV_BF16 && p.d == 128 && p.G <= 128 && n_rows > 1) {
    Problem pd = p;
    pd.G = 128; pd.Hq = p.Hkv * 128; pd.w = 1; pd.R = 128; pd.tail = 0; pd.n = pd.n_kv = n_rows;
    pd.ksn = pd.vsn = p.d;
    pd.ksh = pd.vsh = (long long)n_rows * p.d;
    pd.ksb = pd.vsb = (long long)p.Hkv * n_rows * p.d;
    Workspace ws;
    if (plan_decode_tc(pd.BH, h->sm_count, workspace, &ws) <= workspace_bytes) {
      RESTKV_LAUNCH(c, RESTKV_KERNEL_NONE, launch_decode_pad(p, q, ws.q_pad, c.st), 1);
      RESTKV_LAUNCH(c, RESTKV_KERNEL_NONE,
                    launch_tc_fused(h->tc_state, pd, ws, ws.q_pad, Kc, Vc, 0.f, h->sm_count, false, true, h->wait_limit,
                                    nullptr, nullptr, nullptr, h->dev_status, c.st), 1);
      RESTKV_LAUNCH(c, RESTKV_KERNEL_NONE, launch_decode_extract(p, ws.O_f32, ws.row_M2, out, lse, c.st), 1);
      return RESTKV_OK;
    }
    tc_ws_too_small = true;
  }
  // SIMT kernels: 1, 2, 4 or 8 query heads per KV head, rows of 2 to 64 sixteen-byte chunks
  if (p.G != 1 && p.G != 2 && p.G != 4 && p.G != 8)
    return tc_ws_too_small ? RESTKV_ERR_WORKSPACE : RESTKV_ERR_UNSUPPORTED;
  const int chunks = p.d * (p.dtype == RESTKV_BF16 ? 2 : 4) / 16;
  if (chunks != 2 && chunks != 4 && chunks != 8 && chunks != 16 && chunks != 32 && chunks != 64)
    return RESTKV_ERR_UNSUPPORTED;
  const size_t need = align256((size_t)p.BH * kDecodeMaxSplits * p.G * (p.d + 2) * sizeof(float));
  if (workspace_bytes < need) return RESTKV_ERR_WORKSPACE;
  int nl = 0;
  cudaError_t e = launch_decode(p, q, Kc, Vc, n_rows, out, lse, (float*)workspace,
                                decode_splits(p, n_rows, h->sm_count), c.st, &nl);
  if (e != cudaSuccess) return c.fail(e);
  h->launches += nl;
  return RESTKV_OK;
}

restkv_status restkv_poll_status(restkv_handle* h, restkv_stream stream) {
  if (!h) return RESTKV_ERR_INVALID_ARG;
  unsigned int word = 0;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(&word, h->dev_status, sizeof(word), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  if (e == cudaSuccess && word != 0) e = cudaMemsetAsync(h->dev_status, 0, sizeof(word), st);
  if (e != cudaSuccess) { h->last_cuda_error = (int)e; return RESTKV_ERR_CUDA; }
  if (word & kDevTimeout) return RESTKV_ERR_TIMEOUT;
  if (word & kDevBadIndex) return RESTKV_ERR_INVALID_ARG;
  return RESTKV_OK;
}

long long restkv_launch_count(const restkv_handle* h) { return h ? h->launches : 0; }
int restkv_last_cuda_error(const restkv_handle* h) { return h ? h->last_cuda_error : 0; }

const char* restkv_error_string(restkv_status s) {
  switch (s) {
    case RESTKV_OK: return "ok";
    case RESTKV_ERR_INVALID_ARG: return "invalid argument";
    case RESTKV_ERR_UNSUPPORTED: return "unsupported shape or mode";
    case RESTKV_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case RESTKV_ERR_CUDA: return "CUDA call failed";
    case RESTKV_ERR_TIMEOUT: return "a bounded device-side wait expired";
  }
  return "unknown status";
}

restkv_status restkv_set_profile_events(restkv_handle* h, int which, void* start, void* stop) {
  if (!h || which <= RESTKV_KERNEL_NONE || which > RESTKV_KERNEL_COMPACT) return RESTKV_ERR_INVALID_ARG;
  if ((start == nullptr) != (stop == nullptr)) return RESTKV_ERR_INVALID_ARG;
  h->prof_start[which] = (cudaEvent_t)start;
  h->prof_stop[which] = (cudaEvent_t)stop;
  return RESTKV_OK;
}

int restkv_last_evict_fused_select(const restkv_handle* h) { return h && h->last_evict_fused ? 1 : 0; }

restkv_status restkv_set_fused_select(restkv_handle* h, int on) {
  if (!h) return RESTKV_ERR_INVALID_ARG;
  h->fused_select = on != 0;
  return RESTKV_OK;
}

restkv_status restkv_set_wait_limit(restkv_handle* h, long long sm_clocks) {
  if (!h || sm_clocks < 1) return RESTKV_ERR_INVALID_ARG;
  h->wait_limit = sm_clocks;
  return RESTKV_OK;
}

restkv_status restkv_set_variant(restkv_handle* h, const restkv_variant* v) {
  if (!h) return RESTKV_ERR_INVALID_ARG;
  if (!v) {
    h->variant = restkv_variant{0, 0, 0, 0};
    return RESTKV_OK;
  }
  if (v->indicator < 0 || v->indicator > RESTKV_INDICATOR_ATTENTION_VNORM) return RESTKV_ERR_INVALID_ARG;
  if (v->temporal < 0 || v->temporal > RESTKV_TEMPORAL_NONE) return RESTKV_ERR_INVALID_ARG;
  if (v->spatial < 0 || v->spatial > RESTKV_SPATIAL_MAX) return RESTKV_ERR_INVALID_ARG;
  if (v->group < 0 || v->group > RESTKV_GROUP_MAX) return RESTKV_ERR_INVALID_ARG;
  h->variant = *v;
  return RESTKV_OK;
}

size_t restkv_output_projection_bytes(int n_q_heads, int head_dim) {
  if (n_q_heads < 1 || head_dim < 16 || head_dim > 128 || head_dim % 16 != 0) return 0;
  return projection_factor_bytes(n_q_heads, head_dim);
}

restkv_status restkv_prepare_output_projection(restkv_handle* h, int n_q_heads, int head_dim, int d_model,
                                               restkv_dtype dtype, const void* W_O, void* factor,
                                               size_t factor_bytes, restkv_stream stream) {
  if (!h || !W_O || !factor || n_q_heads < 1 || d_model < 1) return RESTKV_ERR_INVALID_ARG;
  if (dtype != RESTKV_BF16 && dtype != RESTKV_F32) return RESTKV_ERR_INVALID_ARG;
  if (head_dim < 16 || head_dim > 128 || head_dim % 16 != 0) return RESTKV_ERR_UNSUPPORTED;
  if (((uintptr_t)factor & 255u) != 0 || factor_bytes < projection_factor_bytes(n_q_heads, head_dim))
    return RESTKV_ERR_WORKSPACE;
  Call c{h, (cudaStream_t)stream};
  RESTKV_LAUNCH(c, RESTKV_KERNEL_NONE,
                launch_projection_prepare(n_q_heads, head_dim, d_model, dtype, W_O, factor, c.st), 2);
  return RESTKV_OK;
}

restkv_status restkv_set_output_projection(restkv_handle* h, const void* factor, int n_q_heads, int head_dim) {
  if (!h) return RESTKV_ERR_INVALID_ARG;
  if (!factor) {
    h->proj_factor = nullptr;
    h->proj_heads = h->proj_dim = 0;
    return RESTKV_OK;
  }
  if (n_q_heads < 1 || head_dim < 16 || head_dim > 128 || head_dim % 16 != 0 || ((uintptr_t)factor & 255u) != 0)
    return RESTKV_ERR_INVALID_ARG;
  h->proj_factor = factor;
  h->proj_heads = n_q_heads;
  h->proj_dim = head_dim;
  return RESTKV_OK;
}

restkv_status restkv_set_kernel_path(restkv_handle* h, int path) {
  if (!h || path < 0 || path > 3) return RESTKV_ERR_INVALID_ARG;
  h->kernel_path = path;
  return RESTKV_OK;
}

}  // extern "C"
