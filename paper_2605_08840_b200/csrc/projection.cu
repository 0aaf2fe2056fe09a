// The output projection of Eq. 4 inside Eq. 7's norm: || (o - v) W ||^2 = (o - v)^T M (o - v) with M = W W^T, one
// d x d matrix per query head (W = that head's d x d_model slice of the model's W_O).
//   restkv_prepare_output_projection:  M (fp32), a factor L of M (L L^T = M) rounded to bf16 (stored transposed, for
//     the tensor-core kernels) and Mt = L L^T of the rounded factor (fp32), so that every term the tensor-core path
//     forms belongs to one and the same quadratic form.
//   per call:  m_r = M o_r for the window rows (SIMT path; the tensor-core kernel does it in its merge).
#include "restkv_common.cuh"

namespace restkv {

namespace {

// M[hq] = W[hq] W[hq]^T.  grid (Hq), block 16 x 16; thread (ti, tk) owns the (d/16) x (d/16) outputs
// i = ti + 16 a, k = tk + 16 b.  d a multiple of 16, at most 128.
template <typename T>
__global__ void proj_gram_kernel(int d, int d_model, const T* __restrict__ W, float* __restrict__ M) {
  __shared__ float Ws[128][33];
  const int hq = blockIdx.x, ti = threadIdx.x, tk = threadIdx.y, per = d / 16;
  const T* Wh = W + (long long)hq * d * d_model;
  float acc[8][8];
#pragma unroll
  for (int a = 0; a < 8; ++a)
#pragma unroll
    for (int b = 0; b < 8; ++b) acc[a][b] = 0.f;
  const int tid = tk * 16 + ti;
  for (int m0 = 0; m0 < d_model; m0 += 32) {
    for (int e = tid; e < d * 32; e += 256) {
      const int row = e >> 5, c = e & 31;
      Ws[row][c] = (m0 + c < d_model) ? to_f32<T>(Wh[(long long)row * d_model + m0 + c]) : 0.f;
    }
    __syncthreads();
    for (int c = 0; c < 32; ++c) {
      float wi[8], wk[8];
#pragma unroll
      for (int a = 0; a < 8; ++a) {
        wi[a] = a < per ? Ws[ti + 16 * a][c] : 0.f;
        wk[a] = a < per ? Ws[tk + 16 * a][c] : 0.f;
      }
#pragma unroll
      for (int a = 0; a < 8; ++a)
#pragma unroll
        for (int b = 0; b < 8; ++b) acc[a][b] = fmaf(wi[a], wk[b], acc[a][b]);
    }
    __syncthreads();
  }
  float* Mh = M + (long long)hq * d * d;
  for (int a = 0; a < per; ++a)
    for (int b = 0; b < per; ++b) Mh[(ti + 16 * a) * d + tk + 16 * b] = acc[a][b];
}

// A factor L of M[hq] with L L^T = M, by Cholesky elimination with diagonal pivoting in shared memory, fp32: every
// step takes the row with the largest remaining diagonal entry, and the elimination stops once that entry has
// fallen to 1e-5 of the first one (M singular, d_model < d: what is left is rounding residue, and a column built
// on it would be noise divided by its square root); the remaining columns are zero.  The rows of L stay in their
// original order, its columns follow the pivots, so L is not triangular; nothing downstream needs that.  Then the
// factor is rounded to bf16 and written transposed (LT[c][i] = L[i][c]), and Mt = L L^T of the rounded factor.
// grid (Hq), block 128 threads (thread i < d owns row i), dynamic shared memory d * (d + 1) floats.
__global__ void proj_factor_kernel(int d, const float* __restrict__ M, float* __restrict__ Mt,
                                   __nv_bfloat16* __restrict__ LT) {
  extern __shared__ float Ls[];   // [d][d + 1]
  __shared__ float red_v[4];
  __shared__ int red_i[4];
  __shared__ float s_piv;
  __shared__ int s_row;
  const int hq = blockIdx.x, i = threadIdx.x, ld = d + 1, lane = i & 31, wid = i >> 5;
  const bool act = i < d;
  const float* Mh = M + (long long)hq * d * d;
  float dres = act ? Mh[i * d + i] : -1.f;   // what is left of the row's diagonal entry
  bool done = !act;
  float top = 0.f;
  for (int c = 0; c < d; ++c) {
    // the largest remaining diagonal entry (ties: the lower row)
    float bv = done ? -1.f : dres;
    int bi = i;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
      if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) { red_v[wid] = bv; red_i[wid] = bi; }
    __syncthreads();
    if (i == 0) {
      float v = red_v[0];
      int r = red_i[0];
      for (int w = 1; w < 4; ++w)
        if (red_v[w] > v) { v = red_v[w]; r = red_i[w]; }
      s_piv = v;
      s_row = r;
    }
    __syncthreads();
    const float piv = s_piv;
    const int pr = s_row;
    if (c == 0) top = piv;
    const bool stop = !(piv > 1e-5f * top) || !(piv > 1e-30f);   // uniform over the block
    if (stop) {
      if (act)
        for (int cc = c; cc < d; ++cc) Ls[i * ld + cc] = 0.f;
      break;
    }
    if (act) {
      // column c: (M[i][pr] - sum_{k<c} L[i][k] L[pr][k]) / sqrt(pivot); rows eliminated earlier get 0
      float v = Mh[i * d + pr];
      for (int k = 0; k < c; ++k) v = fmaf(-Ls[i * ld + k], Ls[pr * ld + k], v);
      const float sd = sqrtf(piv);
      const float l = done ? 0.f : (i == pr ? sd : v / sd);
      Ls[i * ld + c] = l;
      dres -= l * l;
      if (i == pr) done = true;
    }
    __syncthreads();
  }
  __syncthreads();
  __nv_bfloat16* LTh = LT + (long long)hq * d * d;
  if (act)
    for (int c = 0; c < d; ++c) {
      const __nv_bfloat16 r = __float2bfloat16_rn(Ls[i * ld + c]);
      LTh[c * d + i] = r;
      Ls[i * ld + c] = __bfloat162float(r);
    }
  __syncthreads();
  if (!act) return;
  float* Mth = Mt + (long long)hq * d * d;
  for (int k = 0; k < d; ++k) {
    float v = 0.f;
    for (int c = 0; c < d; ++c) v = fmaf(Ls[i * ld + c], Ls[k * ld + c], v);
    Mth[i * d + k] = v;
  }
}

// O_proj[bh, r, :] = M[hq(r)] O[bh, r, :].  grid (R, BH), block d threads (M is symmetric: column reads coalesce).
__global__ void proj_rows_kernel(int Hkv, int G, int w, int R, int d, const float* __restrict__ M,
                                 const float* __restrict__ O, float* __restrict__ O_proj) {
  extern __shared__ float orow[];
  const int r = blockIdx.x, bh = blockIdx.y, i = threadIdx.x;
  const int hq = (bh % Hkv) * G + r / w;
  const float* Mh = M + (long long)hq * d * d;
  const long long ri = ((long long)bh * R + r) * d;
  orow[i] = O[ri + i];
  __syncthreads();
  float v = 0.f;
  for (int k = 0; k < d; ++k) v = fmaf(Mh[k * d + i], orow[k], v);
  O_proj[ri + i] = v;
}

}  // namespace

size_t projection_factor_bytes(int n_q_heads, int d) {
  return (size_t)n_q_heads * d * d * (sizeof(float) + sizeof(float) + sizeof(__nv_bfloat16));
}

Projection projection_view(const void* factor, int n_q_heads, int d) {
  Projection pr{};
  if (!factor) return pr;
  const size_t dd = (size_t)n_q_heads * d * d;
  pr.M = (const float*)factor;
  pr.Mt = pr.M + dd;
  pr.LT = (const __nv_bfloat16*)(pr.Mt + dd);
  return pr;
}

cudaError_t launch_projection_prepare(int n_q_heads, int d, int d_model, restkv_dtype dtype, const void* W_O,
                                      void* factor, cudaStream_t st) {
  Projection pr = projection_view(factor, n_q_heads, d);
  float* M = const_cast<float*>(pr.M);
  if (dtype == RESTKV_BF16)
    proj_gram_kernel<__nv_bfloat16><<<n_q_heads, dim3(16, 16), 0, st>>>(d, d_model, (const __nv_bfloat16*)W_O, M);
  else
    proj_gram_kernel<float><<<n_q_heads, dim3(16, 16), 0, st>>>(d, d_model, (const float*)W_O, M);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const size_t smem = (size_t)d * (d + 1) * sizeof(float);
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(proj_factor_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  proj_factor_kernel<<<n_q_heads, 128, smem, st>>>(d, pr.M, const_cast<float*>(pr.Mt),
                                                 const_cast<__nv_bfloat16*>(pr.LT));
  return cudaGetLastError();
}

cudaError_t launch_projection_rows(const Problem& p, const float* O, float* O_proj, cudaStream_t st) {
  proj_rows_kernel<<<dim3(p.R, p.BH), p.d, p.d * sizeof(float), st>>>(p.Hkv, p.G, p.w, p.R, p.d, p.proj.M, O, O_proj);
  return cudaGetLastError();
}

}  // namespace restkv
