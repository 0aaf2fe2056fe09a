// Shared declarations of the CUDA library: handle, workspace plan, kernel launch prototypes.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "../../include/restkv.h"

namespace restkv {

// Device status block (one per handle).  word[0] is a sticky bit mask written by kernels.
enum : unsigned int {
  kDevTimeout = 1u,      // a bounded wait (mbarrier / flag) expired
  kDevBadIndex = 2u,     // an index outside [0, n_kv) reached the gather
};

// The output projection of Eq. 4 as quadratic forms, one per query head (all null: identity).
struct Projection {
  const float* M;            // [Hq, d, d]  W W^T
  const float* Mt;           // [Hq, d, d]  L L^T of the bf16-rounded Cholesky factor L of M
  const __nv_bfloat16* LT;   // [Hq, d, d]  that factor, transposed
};

struct Problem {
  int batch, Hq, Hkv, G, d;
  int n_kv, n, w, tail;   // n = scored prefix rows, tail = causal_tail
  int R;                  // w * G query rows per KV head
  int BH;                 // batch * Hkv
  float scale;            // softmax scale
  long long ksb, ksh, ksn, vsb, vsh, vsn;  // element strides
  restkv_dtype dtype;
  int indicator, temporal, spatial, group;   // restkv_variant; all 0 = the method as the paper prints it
  Projection proj;
};

// Workspace carve-up (all offsets 256-byte aligned).
struct Workspace {
  int splits;             // token splits (CTAs) of the score passes per (batch, KV head)
  float* part_m;          // [slots, R]     partial softmax results: one slot per (head, split) on the SIMT path,
  float* part_l;          // [slots, R]      one per CTA in the persistent tensor-core kernel
  float* part_O;          // [slots, R, d]
  float* vnorm;           // [BH, n_kv]  ||v_j||^2 (tensor-core path)
  unsigned int* counters; // [256] group barrier counters of the persistent score kernel
  float* tile_max;        // [BH, tiles, 128] per-tile row maxima of the persistent score kernel
  float* row_M2;          // [BH, 128] log2 normaliser of each query row
  unsigned int* sel_hist; // [BH, 4, 256] digit histograms of the selection inside the score kernel
  unsigned int* sel_sfx;  // [SMs, 4, 260] per-CTA suffix sums of those histograms
  __nv_bfloat16* q_pad;   // [BH, 128, 128] decode queries padded to the kernel's 128 rows
  float* fin_m;           // [BH, R]    row max of the scaled logits (natural units)
  float* fin_l;           // [BH, R]    sum of exp(s - m)
  float* O_f32;           // [BH, R, d]
  __nv_bfloat16* O_m2;    // [BH, R, d]   -2 * bf16(O)
  __nv_bfloat16* aug;     // [BH, R, 64]  per-row constants as bf16 pieces (see combine_kernel)
  float* I_hat;           // [BH, n]
  float* O_proj;          // [BH, R, d]   M o_r, with an output projection only
  float* vmv;             // [BH, G, n_kv] v_j^T Mt v_j, with an output projection on the tensor-core path only
  float* scores;          // [BH, n_kv] (used when the caller passes no scores buffer)
  int* pool;              // [BH, 2] (W, gamma)
  float* dec_part;        // decode partials
  float* I_raw;           // adaptive only: [batch, Hq, w, n]
  int32_t* adaptive_idx;  // adaptive only: [batch*Hq*w, B_p] per-query top-B_p indices
  unsigned long long* adaptive_sums;  // adaptive only: [BH, 2] index sums (front, rear)
  size_t bytes;
};

constexpr int kDecodeMaxSplits = 64;

// Pooling window, budget and outputs of the selection that the tensor-core score kernel can run itself.
struct FusedSelect {
  int keep, W, gamma;
  float* scores;          // [BH, n_kv] pooled scores
  int32_t* indices;       // [BH, keep]
  void* K_out;            // [BH, keep, d]
  void* V_out;
};

int pass1_splits(const Problem& p, int sm_count);
size_t plan_workspace(const Problem& p, int budget, int sm_count, bool adaptive, void* base, Workspace* ws);

// ---- launches (each returns the cudaError_t of the launch) -------------------------------------
cudaError_t launch_simt_pass1(const Problem& p, const Workspace& ws, const void* Q, const void* K, const void* V,
                              cudaStream_t st);
cudaError_t launch_combine(const Problem& p, const Workspace& ws, cudaStream_t st);
cudaError_t launch_simt_pass2(const Problem& p, const Workspace& ws, const void* Q, const void* K, const void* V,
                              float ema_decay, float* I_raw, cudaStream_t st);
cudaError_t launch_pool(const Problem& p, const Workspace& ws, const int* pool_dev, int W, int gamma, float* scores,
                        int32_t* pool_used, cudaStream_t st);
cudaError_t launch_select(int rows, int n, int n_kv, int budget, const int* keep_rows, const float* I_hat, const int* pool_dev, int W,
                          int gamma, bool pool_max, float* scores, int32_t* indices, int32_t* pool_used, const Problem* gather,
                          const void* K, const void* V, void* K_out, void* V_out, cudaStream_t st);
cudaError_t launch_compact(const Problem& p, const void* K, const void* V, const int32_t* indices, int n_sel,
                           void* K_out, void* V_out, unsigned int* dev_status, cudaStream_t st);
cudaError_t launch_decode(const Problem& p, const void* q, const void* Kc, const void* Vc, int n_rows, float* out,
                          float* lse, float* part, int splits, cudaStream_t st, int* n_launches);
cudaError_t launch_adaptive_params(const Problem& p, const Workspace& ws, int budget, float beta, int base_width,
                                   cudaStream_t st, int* n_launches);

// Output projection (Eq. 4): the caller-owned factor buffer and the per-call projected rows.
size_t projection_factor_bytes(int n_q_heads, int d);
Projection projection_view(const void* factor, int n_q_heads, int d);
cudaError_t launch_projection_prepare(int n_q_heads, int d, int d_model, restkv_dtype dtype, const void* W_O,
                                      void* factor, cudaStream_t st);
cudaError_t launch_projection_rows(const Problem& p, const float* O, float* O_proj, cudaStream_t st);

// Tensor-core (tcgen05 / TMEM / TMA) score kernels.  `supported` says whether the shape qualifies.
bool tc_supported(const Problem& p);
cudaError_t tc_init(void** state);   // resolves the driver entry point for tensor-map encoding
cudaError_t tc_fused_init();
cudaError_t launch_tc_fused(void* state, const Problem& p, const Workspace& ws, const void* Q, const void* K,
                            const void* V, float ema_decay, int sm_count, bool reuse_l2, bool attention_only,
                            long long wait_limit, const FusedSelect* sel, const float* O_given, float* I_raw,
                            unsigned int* dev_status, cudaStream_t st);
// Given the window rows' outputs O [BH, R, d] and log-sum-exps LSE [BH, R] (natural log): what the score kernels read
// instead of the results of pass 1 and the merge.  tensor_core: -2 bf16(O), the constant strip, the rows' log2
// normalisers; otherwise fin_m = LSE, fin_l = 1.
cudaError_t launch_from_lse_prep(const Problem& p, const Workspace& ws, const float* O, const float* LSE,
                                 bool tensor_core, cudaStream_t st);
// Output projection on the tensor-core path: the tokens' own terms v^T Mt v, [BH, G, n_kv], by a kernel of its own.
bool tc_vmv_supported(const Problem& p);
cudaError_t launch_tc_vmv(void* state, const Problem& p, const void* V, float* out, int sm_count, long long wait_limit,
                          unsigned int* dev_status, cudaStream_t st);
// Whether the tensor-core kernel's temporal chain can carry the variant's weights for this decay and window.
bool tc_variant_supported(const Problem& p, float ema_decay);
bool tc_fused_select_supported(const Problem& p, int sm_count, bool reuse_l2, int keep, int W, int gamma);
size_t tc_fused_select_sfx_words(int sm_count);
size_t tc_fused_select_hist_words(int BH);
cudaError_t launch_decode_pad(const Problem& p, const void* q, __nv_bfloat16* q_pad, cudaStream_t st);
cudaError_t launch_decode_extract(const Problem& p, const float* O_f32, const float* row_M2, float* out, float* lse,
                                  cudaStream_t st);

// ---- small device helpers ------------------------------------------------------------------------
template <typename T> __device__ __forceinline__ float to_f32(T x);
template <> __device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

}  // namespace restkv
