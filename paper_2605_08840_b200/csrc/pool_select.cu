// Spatial pooling (Eq. 13), top-B selection and row gather (Eq. 14).
#include "restkv_common.cuh"

namespace restkv {

namespace {

// ------------------------------------------------------------------------------------------------
__global__ void set_pool_kernel(int* pool, int BH, int W, int gamma) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < BH) { pool[2 * i] = W; pool[2 * i + 1] = gamma; }
}

// scores[j] = (1/W) * sum_{k=-W/2+gamma}^{W/2+gamma} I_hat[j+k], taps outside [0,n) are zero;
// rows n..n_kv-1 (the window's own tokens) get +inf.  grid (ceil(n_kv/256), BH).
__global__ void pool_kernel(int n, int n_kv, const float* __restrict__ I_hat, const int* __restrict__ pool,
                            float* __restrict__ scores, int32_t* __restrict__ pool_used) {
  const int bh = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  const int W = pool[2 * bh], gamma = pool[2 * bh + 1];
  if (pool_used && j == 0) { pool_used[2 * bh] = W; pool_used[2 * bh + 1] = gamma; }
  if (j >= n_kv) return;
  float out;
  if (j >= n) {
    out = INFINITY;
  } else {
    const float* src = I_hat + (long long)bh * n;
    const int half = W / 2;
    long long lo = (long long)j - half + gamma, hi = (long long)j + half + gamma;
    if (lo < 0) lo = 0;
    if (hi > n - 1) hi = n - 1;
    float s = 0.f;
    for (long long t = lo; t <= hi; ++t) s += src[t];
    out = s / (float)W;
  }
  scores[(long long)bh * n_kv + j] = out;
}

// ------------------------------------------------------------------------------------------------
// Radix select.  Scores map to unsigned keys whose order matches the float order.
__device__ __forceinline__ unsigned int float_key(float x) {
  const unsigned int u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kSelThreads = 1024;

// One block per row.  Four 8-bit passes from the most significant digit find the key T of the
// keep-th largest score and how many scores are strictly larger; a last ordered pass writes, in
// ascending index order, every index whose key is > T plus the first (keep - #larger) indices
// whose key equals T (lower index wins ties).
__global__ void __launch_bounds__(kSelThreads) select_kernel(int n_kv, int keep, const float* __restrict__ scores,
                                                             int32_t* __restrict__ indices) {
  __shared__ unsigned int hist[256];
  __shared__ unsigned int s_prefix, s_remaining;
  __shared__ unsigned int warp_sel[32], warp_eq[32];
  __shared__ unsigned int s_base_sel, s_base_eq;

  const int row = blockIdx.x;
  const float* src = scores + (long long)row * n_kv;
  int32_t* dst = indices + (long long)row * keep;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;

  if (keep >= n_kv) {   // budget covers everything: identity
    for (int j = tid; j < n_kv; j += kSelThreads) dst[j] = j;
    return;
  }

  unsigned int prefix = 0, remaining = keep;   // remaining: rank (1-based) still to find inside the prefix class
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    const unsigned int mask_hi = (pass == 0) ? 0u : (0xFFFFFFFFu << (shift + 8));
    if (tid < 256) hist[tid] = 0;
    __syncthreads();
    for (int j = tid; j < n_kv; j += kSelThreads) {
      const unsigned int key = float_key(src[j]);
      if ((key & mask_hi) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (tid == 0) {
      unsigned int acc = 0;
      int digit = 255;
      for (; digit > 0; --digit) {
        if (acc + hist[digit] >= remaining) break;
        acc += hist[digit];
      }
      s_prefix = prefix | ((unsigned int)digit << shift);
      s_remaining = remaining - acc;
    }
    __syncthreads();
    prefix = s_prefix;
    remaining = s_remaining;
    __syncthreads();
  }
  const unsigned int T = prefix;          // key of the keep-th largest score
  const unsigned int need_eq = remaining; // how many keys equal to T are kept (>= 1)

  if (tid == 0) { s_base_sel = 0; s_base_eq = 0; }
  __syncthreads();
  for (int j0 = 0; j0 < n_kv; j0 += kSelThreads) {
    const int j = j0 + tid;
    unsigned int key = 0;
    const bool in = j < n_kv;
    if (in) key = float_key(src[j]);
    const bool gt = in && key > T;
    const bool eq = in && key == T;
    // rank among equal keys, in index order
    const unsigned int eq_mask = __ballot_sync(0xffffffffu, eq);
    const unsigned int eq_before_in_warp = __popc(eq_mask & ((1u << lane) - 1u));
    if (lane == 0) warp_eq[wid] = __popc(eq_mask);
    __syncthreads();
    unsigned int eq_before = s_base_eq + eq_before_in_warp;
    for (int wv = 0; wv < wid; ++wv) eq_before += warp_eq[wv];
    const bool sel = gt || (eq && eq_before < need_eq);
    const unsigned int sel_mask = __ballot_sync(0xffffffffu, sel);
    const unsigned int sel_before_in_warp = __popc(sel_mask & ((1u << lane) - 1u));
    if (lane == 0) warp_sel[wid] = __popc(sel_mask);
    __syncthreads();
    unsigned int pos = s_base_sel + sel_before_in_warp;
    for (int wv = 0; wv < wid; ++wv) pos += warp_sel[wv];
    if (sel && pos < (unsigned int)keep) dst[pos] = j;
    __syncthreads();
    if (tid == 0) {
      unsigned int a = 0, c = 0;
      for (int wv = 0; wv < 32; ++wv) { a += warp_sel[wv]; c += warp_eq[wv]; }
      s_base_sel += a;
      s_base_eq += c;
    }
    __syncthreads();
  }
}

// ------------------------------------------------------------------------------------------------
// Gather: one 16-byte chunk per thread.  grid covers BH * n_sel rows for K then the same for V.
__global__ void compact_kernel(int Hkv, int n_kv, int n_sel, int row_chunks, long long ksb, long long ksh,
                               long long ksn, long long vsb, long long vsh, long long vsn, int esize,
                               const unsigned char* __restrict__ K, const unsigned char* __restrict__ V,
                               const int32_t* __restrict__ indices, unsigned char* __restrict__ K_out,
                               unsigned char* __restrict__ V_out, long long total_rows,
                               unsigned int* __restrict__ dev_status) {
  const long long gid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long row2 = gid / row_chunks;          // 0 .. 2*total_rows
  const int chunk = (int)(gid - row2 * row_chunks);
  if (row2 >= 2 * total_rows) return;
  const bool isV = row2 >= total_rows;
  const long long row = isV ? row2 - total_rows : row2;   // (bh, s)
  const long long bh = row / n_sel;
  const int b = (int)(bh / Hkv), h = (int)(bh % Hkv);
  const int j = indices[row];
  if (j < 0 || j >= n_kv) {
    if (chunk == 0) atomicOr(dev_status, kDevBadIndex);
    return;
  }
  const long long src_elem = isV ? ((long long)b * vsb + (long long)h * vsh + (long long)j * vsn)
                                 : ((long long)b * ksb + (long long)h * ksh + (long long)j * ksn);
  const uint4* src = reinterpret_cast<const uint4*>((isV ? V : K) + src_elem * esize) + chunk;
  uint4* dst = reinterpret_cast<uint4*>((isV ? V_out : K_out) + row * (long long)row_chunks * 16) + chunk;
  *dst = __ldg(src);
}

}  // namespace

cudaError_t launch_set_pool(const Problem& p, const Workspace& ws, int W, int gamma, cudaStream_t st) {
  set_pool_kernel<<<(p.BH + 127) / 128, 128, 0, st>>>(ws.pool, p.BH, W, gamma);
  return cudaGetLastError();
}

cudaError_t launch_pool(const Problem& p, const Workspace& ws, float* scores, int32_t* pool_used, cudaStream_t st) {
  dim3 grid((p.n_kv + 255) / 256, p.BH);
  pool_kernel<<<grid, 256, 0, st>>>(p.n, p.n_kv, ws.I_hat, ws.pool, scores, pool_used);
  return cudaGetLastError();
}

cudaError_t launch_select(int rows, int n_kv, int budget, const float* scores, int32_t* indices,
                          unsigned int* scratch, cudaStream_t st) {
  (void)scratch;
  const int keep = budget < n_kv ? budget : n_kv;
  select_kernel<<<rows, kSelThreads, 0, st>>>(n_kv, keep, scores, indices);
  return cudaGetLastError();
}

cudaError_t launch_compact(const Problem& p, const void* K, const void* V, const int32_t* indices, int n_sel,
                           void* K_out, void* V_out, unsigned int* dev_status, cudaStream_t st) {
  const int esize = p.dtype == RESTKV_BF16 ? 2 : 4;
  const int row_chunks = p.d * esize / 16;
  const long long total_rows = (long long)p.BH * n_sel;
  const long long threads = 2 * total_rows * row_chunks;
  if (threads == 0) return cudaSuccess;
  const int block = 256;
  const long long blocks = (threads + block - 1) / block;
  compact_kernel<<<(unsigned int)blocks, block, 0, st>>>(p.Hkv, p.n_kv, n_sel, row_chunks, p.ksb, p.ksh, p.ksn, p.vsb,
                                                         p.vsh, p.vsn, esize, (const unsigned char*)K,
                                                         (const unsigned char*)V, indices, (unsigned char*)K_out,
                                                         (unsigned char*)V_out, total_rows, dev_status);
  return cudaGetLastError();
}

}  // namespace restkv
