// Adaptive window parameters (Eq. 10-12): D_front / D_rear are the mean indices of the per-query
// top-B rows of the raw indicator over the first and second half of the window queries; the box
// width and shift follow from their difference.
#include "restkv_common.cuh"

namespace restkv {

namespace {

__global__ void zero_sums_kernel(unsigned long long* sums, int count) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < count) sums[i] = 0ull;
}

// grid = batch*Hq*w rows of idx [rows, Bp]; adds each row's index sum to its KV head's front or rear total.
__global__ void index_sum_kernel(int Hq, int G, int w, int Bp, const int32_t* __restrict__ idx,
                                 unsigned long long* __restrict__ sums) {
  const int row = blockIdx.x;            // (b, hq, i)
  const int i = row % w;
  const int bhq = row / w;
  const int b = bhq / Hq, hq = bhq % Hq;
  const int Hkv = Hq / G;
  const int bh = b * Hkv + hq / G;
  unsigned long long s = 0;
  for (int k = threadIdx.x; k < Bp; k += blockDim.x) s += (unsigned long long)idx[(long long)row * Bp + k];
  for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
  __shared__ unsigned long long red[32];
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned long long t = 0;
    for (int k = 0; k < (int)(blockDim.x >> 5); ++k) t += red[k];
    atomicAdd(&sums[2 * bh + (i < w / 2 ? 0 : 1)], t);
  }
}

__global__ void window_params_kernel(int BH, int G, int w, int Bp, double beta, int base_width,
                                     const unsigned long long* __restrict__ sums, int* __restrict__ pool) {
  const int bh = blockIdx.x * blockDim.x + threadIdx.x;
  if (bh >= BH) return;
  const long long cnt_front = (long long)G * (w / 2) * Bp;
  const long long cnt_rear = (long long)G * (w - w / 2) * Bp;
  const double D_rear = (double)sums[2 * bh + 1] / (double)cnt_rear;
  const double D_front = cnt_front ? (double)sums[2 * bh] / (double)cnt_front : D_rear;
  const double x = (D_front - D_rear) / beta;
  const int Ws = 2 * (int)floor(fabs(x)) + 1;   // Eq. 11
  const int gamma = (int)trunc(x);              // Eq. 12, truncating toward zero
  pool[2 * bh] = Ws + base_width - 1;
  pool[2 * bh + 1] = gamma;
}

}  // namespace

cudaError_t launch_adaptive_params(const Problem& p, const Workspace& ws, int budget, float beta, int base_width,
                                   cudaStream_t st, int* n_launches) {
  int Bp = budget - p.tail;
  if (Bp > p.n) Bp = p.n;
  const int rows = p.batch * p.Hq * p.w;
  *n_launches = 0;
  cudaError_t e = launch_select(rows, p.n, p.n, Bp, nullptr, nullptr, nullptr, 1, 0, false, ws.I_raw, ws.adaptive_idx, nullptr, nullptr, nullptr,
                                nullptr, nullptr, nullptr, st);
  if (e != cudaSuccess) return e;
  ++*n_launches;
  zero_sums_kernel<<<(2 * p.BH + 127) / 128, 128, 0, st>>>(ws.adaptive_sums, 2 * p.BH);
  index_sum_kernel<<<rows, 256, 0, st>>>(p.Hq, p.G, p.w, Bp, ws.adaptive_idx, ws.adaptive_sums);
  window_params_kernel<<<(p.BH + 127) / 128, 128, 0, st>>>(p.BH, p.G, p.w, Bp, (double)beta, base_width,
                                                           ws.adaptive_sums, ws.pool);
  *n_launches += 3;
  return cudaGetLastError();
}

}  // namespace restkv
