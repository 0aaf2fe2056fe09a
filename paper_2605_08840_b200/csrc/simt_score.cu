// fp32 SIMT kernels of the score path: used for RESTKV_F32 inputs and for every shape the
// tensor-core kernels do not cover.  Same two-pass structure as the tensor-core path:
//   pass 1   per (batch, KV head, token split): online softmax statistics (m, l) and the
//            unnormalised window outputs of all w*G query rows           (Eq. 3)
//   combine  merge the splits: m, l, O, plus the quantities the tensor-core pass 2 wants
//   pass 2   per token: A = exp(s - m) / l, I = A / (1 - A) * ||o - v||  (Eq. 7),
//            EMA recursion over the window queries                        (Eq. 8-9),
//            mean over the query heads of the group
#include "restkv_common.cuh"

namespace restkv {

namespace {

constexpr int kP1Tile = 32;   // tokens per shared-memory tile in pass 1
constexpr int kP2Tile = 64;   // tokens per block in pass 2

template <typename T>
__device__ __forceinline__ void load_tile_f32(float* dst, int dst_stride, const T* src, long long row_stride,
                                              int rows, int rows_valid, int d) {
  // rows x d elements, converted to fp32; rows >= rows_valid are zero-filled
  for (int e = threadIdx.x; e < rows * d; e += blockDim.x) {
    int r = e / d, k = e - r * d;
    dst[r * dst_stride + k] = (r < rows_valid) ? to_f32<T>(src[(long long)r * row_stride + k]) : 0.f;
  }
}

// ------------------------------------------------------------------------------------------------
// Pass 1.  grid (splits, BH), block = R rounded up to a warp multiple.  Thread r owns query row r.
// Shared memory: Qs [R][d+1], Os [R][d+1], Kt [32][d], Vt [32][d] (fp32).
template <typename T>
__global__ void simt_pass1_kernel(Problem p, const T* __restrict__ Q, const T* __restrict__ K,
                                  const T* __restrict__ V, float* __restrict__ part_m, float* __restrict__ part_l,
                                  float* __restrict__ part_O, int splits) {
  extern __shared__ float smem[];
  const int d = p.d, R = p.R, ld = d + 1;
  float* Qs = smem;
  float* Os = Qs + (size_t)R * ld;
  float* Kt = Os + (size_t)R * ld;
  float* Vt = Kt + (size_t)kP1Tile * d;

  const int split = blockIdx.x, bh = blockIdx.y;
  const int b = bh / p.Hkv, h = bh % p.Hkv;
  const int r = threadIdx.x;
  const bool active = r < R;
  const int i_q = active ? (r % p.w) : 0;   // window position of this row (row = g*w + i)

  const T* Qh = Q + ((long long)b * p.Hq + (long long)h * p.G) * p.w * d;   // [R, d] contiguous
  const T* Kh = K + (long long)b * p.ksb + (long long)h * p.ksh;
  const T* Vh = V + (long long)b * p.vsb + (long long)h * p.vsh;

  for (int e = threadIdx.x; e < R * d; e += blockDim.x) {
    int rr = e / d, k = e - rr * d;
    Qs[rr * ld + k] = to_f32<T>(Qh[(long long)rr * d + k]);
    Os[rr * ld + k] = 0.f;
  }

  // contiguous range of 32-token tiles for this split
  const int n_tiles = (p.n_kv + kP1Tile - 1) / kP1Tile;
  const int per = (n_tiles + splits - 1) / splits;
  const int tile0 = split * per;
  const int tile1 = min(n_tiles, tile0 + per);

  float m = -INFINITY, l = 0.f;
  for (int tile = tile0; tile < tile1; ++tile) {
    const int j0 = tile * kP1Tile;
    const int valid = min(kP1Tile, p.n_kv - j0);
    __syncthreads();
    load_tile_f32<T>(Kt, d, Kh + (long long)j0 * p.ksn, p.ksn, kP1Tile, valid, d);
    load_tile_f32<T>(Vt, d, Vh + (long long)j0 * p.vsn, p.vsn, kP1Tile, valid, d);
    __syncthreads();
    if (!active) continue;

    float s[kP1Tile];
#pragma unroll
    for (int t = 0; t < kP1Tile; ++t) s[t] = 0.f;
    for (int k = 0; k < d; ++k) {
      const float qv = Qs[r * ld + k];
#pragma unroll
      for (int t = 0; t < kP1Tile; ++t) s[t] = fmaf(qv, Kt[t * d + k], s[t]);
    }
    float tmax = -INFINITY;
#pragma unroll
    for (int t = 0; t < kP1Tile; ++t) {
      const int j = j0 + t;
      // visible: inside the cache, and for trailing (window) rows only those not after this query
      const bool vis = (t < valid) && (j < p.n || (j - p.n) <= i_q);
      s[t] = vis ? s[t] * p.scale : -INFINITY;
      tmax = fmaxf(tmax, s[t]);
    }
    const float m_new = fmaxf(m, tmax);
    if (m_new == -INFINITY) continue;   // nothing visible so far
    const float corr = expf(m - m_new);   // m = -inf gives 0
    float lsum = 0.f;
#pragma unroll
    for (int t = 0; t < kP1Tile; ++t) {
      s[t] = expf(s[t] - m_new);          // masked entries give 0
      lsum += s[t];
    }
    l = l * corr + lsum;
    m = m_new;
    for (int k = 0; k < d; ++k) {
      float acc = Os[r * ld + k] * corr;
#pragma unroll
      for (int t = 0; t < kP1Tile; ++t) acc = fmaf(s[t], Vt[t * d + k], acc);
      Os[r * ld + k] = acc;
    }
  }
  if (active) {
    const long long o = ((long long)bh * splits + split) * R + r;
    part_m[o] = m;
    part_l[o] = l;
    float* Op = part_O + o * d;
    for (int k = 0; k < d; ++k) Op[k] = Os[r * ld + k];
  }
}

// ------------------------------------------------------------------------------------------------
// Combine the token splits.  grid (R, BH), block 128: one block per query row.
__global__ void combine_kernel(int R, int d, int splits, const float* __restrict__ part_m,
                               const float* __restrict__ part_l, const float* __restrict__ part_O,
                               float* __restrict__ fin_m, float* __restrict__ fin_l, float* __restrict__ O_f32) {
  const int r = blockIdx.x, bh = blockIdx.y;
  const long long base = (long long)bh * splits * R + r;   // + s * R
  float m = -INFINITY;
  for (int s = 0; s < splits; ++s) m = fmaxf(m, part_m[base + (long long)s * R]);
  float l = 0.f;
  for (int s = 0; s < splits; ++s) {
    const float ms = part_m[base + (long long)s * R];
    if (ms != -INFINITY) l += part_l[base + (long long)s * R] * expf(ms - m);
  }
  const float inv_l = 1.f / l;
  for (int k = threadIdx.x; k < d; k += blockDim.x) {
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) {
      const float ms = part_m[base + (long long)s * R];
      if (ms != -INFINITY) acc += part_O[(base + (long long)s * R) * d + k] * expf(ms - m);
    }
    O_f32[((long long)bh * R + r) * d + k] = acc * inv_l;
  }
  if (threadIdx.x == 0) {
    fin_m[(long long)bh * R + r] = m;
    fin_l[(long long)bh * R + r] = l;
  }
}

// ------------------------------------------------------------------------------------------------
// Pass 2.  grid (token tiles of 64, BH), block 64 * GP threads: thread = (token, group slot).
// Shared memory: Kt [64][d+1], Vt [64][d+1], red [GP][64].
template <typename T>
__global__ void simt_pass2_kernel(Problem p, const T* __restrict__ Q, const T* __restrict__ K,
                                  const T* __restrict__ V, const float* __restrict__ fin_m,
                                  const float* __restrict__ fin_l, const float* __restrict__ O_f32,
                                  const float* __restrict__ O_proj, float ema_decay,
                                  float* __restrict__ I_hat, float* __restrict__ I_raw, int GP) {
  extern __shared__ float smem[];
  const int d = p.d, ld = d + 1;
  float* Kt = smem;
  float* Vt = Kt + (size_t)kP2Tile * ld;
  float* red = Vt + (size_t)kP2Tile * ld;
  float* MVs = red + (size_t)GP * kP2Tile;   // [GP * kP2Tile][ld]: M v_j of each thread, with a projection only

  const int bh = blockIdx.y, b = bh / p.Hkv, h = bh % p.Hkv;
  const int j0 = blockIdx.x * kP2Tile;
  const int valid = min(kP2Tile, p.n - j0);
  const T* Kh = K + (long long)b * p.ksb + (long long)h * p.ksh + (long long)j0 * p.ksn;
  const T* Vh = V + (long long)b * p.vsb + (long long)h * p.vsh + (long long)j0 * p.vsn;
  load_tile_f32<T>(Kt, ld, Kh, p.ksn, kP2Tile, valid, d);
  load_tile_f32<T>(Vt, ld, Vh, p.vsn, kP2Tile, valid, d);
  __syncthreads();

  const int t = threadIdx.x % kP2Tile, slot = threadIdx.x / kP2Tile;
  const int j = j0 + t;
  const float alpha = 1.f - ema_decay;
  const T* Qh = Q + ((long long)b * p.Hq + (long long)h * p.G) * p.w * d;
  const float* Oh = O_f32 + (long long)bh * p.R * d;
  const float* kr = Kt + t * ld;
  const float* vr = Vt + t * ld;

  // variants of Appendix G: p.indicator picks the per-query indicator, p.temporal the weights over the window
  // queries, p.group the reduction over the query heads of the group
  const bool gmax = p.group == RESTKV_GROUP_MAX;
  float group_red = 0.f;
  if (t < valid) {
    float vlen = 1.f;
    if (p.indicator == RESTKV_INDICATOR_ATTENTION_VNORM) {
      float vv = 0.f;
      for (int k = 0; k < d; ++k) vv = fmaf(vr[k], vr[k], vv);
      vlen = sqrtf(vv);
    }
    for (int g = slot; g < p.G; g += GP) {
      float ema = 0.f, pw = 1.f;   // pw = ema_decay^i for the inverted EMA
      // Eq. 7 with the projection of Eq. 4: (o - v)^T M (o - v) = (o - v) . (M o - M v); M v is formed once per
      // token and query head, M o comes in
      float* mv = MVs + (size_t)threadIdx.x * ld;
      if (p.proj.M && p.indicator == RESTKV_INDICATOR_RECONSTRUCTION) {
        const float* Mg = p.proj.M + (long long)(h * p.G + g) * d * d;
        for (int i = 0; i < d; ++i) {
          float acc = 0.f;
          for (int k = 0; k < d; ++k) acc = fmaf(Mg[i * d + k], vr[k], acc);
          mv[i] = acc;
        }
      }
      for (int i = 0; i < p.w; ++i) {
        // without temporal smoothing only the newest query counts (the raw indicators still want every query)
        if (p.temporal == RESTKV_TEMPORAL_NONE && i != p.w - 1 && !I_raw) continue;
        const int r = g * p.w + i;
        const T* qr = Qh + (long long)r * d;
        const float* orow = Oh + (long long)r * d;
        float s = 0.f, ss = 0.f;
        if (p.proj.M) {
          const float* oprow = O_proj + ((long long)bh * p.R + r) * d;
          for (int k = 0; k < d; ++k) {
            s = fmaf(to_f32<T>(qr[k]), kr[k], s);
            ss = fmaf(orow[k] - vr[k], oprow[k] - mv[k], ss);
          }
          ss = fmaxf(ss, 0.f);
        } else {
          for (int k = 0; k < d; ++k) {
            s = fmaf(to_f32<T>(qr[k]), kr[k], s);
            const float df = orow[k] - vr[k];
            ss = fmaf(df, df, ss);
          }
        }
        const long long ri = (long long)bh * p.R + r;
        const float l = fin_l[ri];
        const float e = expf(s * p.scale - fin_m[ri]);
        float I;
        if (p.indicator == RESTKV_INDICATOR_RECONSTRUCTION) {
          // 1 - A formed as (l - e) / l; clamped so that A -> 1 stays finite
          const float one_minus = fmaxf((l - e) / l, 5.9604645e-8f);
          I = (e / l) / one_minus * sqrtf(ss);
        } else {
          I = (e / l) * vlen;
        }
        if (I_raw) I_raw[(((long long)b * p.Hq + (long long)h * p.G + g) * p.w + i) * p.n + j] = I;
        switch (p.temporal) {
          case RESTKV_TEMPORAL_EMA:   // Eq. 9, oldest query first
            ema = (i == 0) ? I : fmaf(alpha, I, ema_decay * ema);
            break;
          case RESTKV_TEMPORAL_MEAN:
            ema += I;
            break;
          case RESTKV_TEMPORAL_INV_EMA:   // the recursion run backwards: weights alpha d^i, d^(w-1) for the newest
            ema = fmaf((i == p.w - 1) ? pw : alpha * pw, I, ema);
            pw *= ema_decay;
            break;
          default:
            if (i == p.w - 1) ema = I;
            break;
        }
      }
      if (p.temporal == RESTKV_TEMPORAL_MEAN) ema /= (float)p.w;
      group_red = gmax ? fmaxf(group_red, ema) : group_red + ema;
    }
  }
  red[slot * kP2Tile + t] = group_red;
  __syncthreads();
  if (slot == 0 && t < valid) {
    float tot = 0.f;
    for (int sl = 0; sl < GP; ++sl) tot = gmax ? fmaxf(tot, red[sl * kP2Tile + t]) : tot + red[sl * kP2Tile + t];
    I_hat[(long long)bh * p.n + j] = gmax ? tot : tot / (float)p.G;
  }
}

template <typename KernelT>
cudaError_t allow_smem(KernelT kernel, size_t bytes) {
  if (bytes <= 48 * 1024) return cudaSuccess;
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

}  // namespace

cudaError_t launch_simt_pass1(const Problem& p, const Workspace& ws, const void* Q, const void* K, const void* V,
                              cudaStream_t st) {
  const int threads = ((p.R + 31) / 32) * 32;
  const size_t smem = ((size_t)2 * p.R * (p.d + 1) + (size_t)2 * kP1Tile * p.d) * sizeof(float);
  dim3 grid(ws.splits, p.BH);
  cudaError_t e;
  if (p.dtype == RESTKV_BF16) {
    if ((e = allow_smem(simt_pass1_kernel<__nv_bfloat16>, smem)) != cudaSuccess) return e;
    simt_pass1_kernel<__nv_bfloat16><<<grid, threads, smem, st>>>(
        p, (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, (const __nv_bfloat16*)V, ws.part_m, ws.part_l,
        ws.part_O, ws.splits);
  } else {
    if ((e = allow_smem(simt_pass1_kernel<float>, smem)) != cudaSuccess) return e;
    simt_pass1_kernel<float><<<grid, threads, smem, st>>>(p, (const float*)Q, (const float*)K, (const float*)V,
                                                          ws.part_m, ws.part_l, ws.part_O, ws.splits);
  }
  return cudaGetLastError();
}

cudaError_t launch_combine(const Problem& p, const Workspace& ws, cudaStream_t st) {
  dim3 grid(p.R, p.BH);
  combine_kernel<<<grid, 128, 0, st>>>(p.R, p.d, ws.splits, ws.part_m, ws.part_l, ws.part_O, ws.fin_m, ws.fin_l,
                                       ws.O_f32);
  return cudaGetLastError();
}

cudaError_t launch_simt_pass2(const Problem& p, const Workspace& ws, const void* Q, const void* K, const void* V,
                              float ema_decay, float* I_raw, cudaStream_t st) {
  int GP = p.G < 4 ? p.G : 4;
  const int threads = kP2Tile * GP;
  size_t smem = ((size_t)2 * kP2Tile * (p.d + 1) + (size_t)GP * kP2Tile) * sizeof(float);
  if (p.proj.M) smem += (size_t)GP * kP2Tile * (p.d + 1) * sizeof(float);
  dim3 grid((p.n + kP2Tile - 1) / kP2Tile, p.BH);
  cudaError_t e;
  if (p.dtype == RESTKV_BF16) {
    if ((e = allow_smem(simt_pass2_kernel<__nv_bfloat16>, smem)) != cudaSuccess) return e;
    simt_pass2_kernel<__nv_bfloat16><<<grid, threads, smem, st>>>(
        p, (const __nv_bfloat16*)Q, (const __nv_bfloat16*)K, (const __nv_bfloat16*)V, ws.fin_m, ws.fin_l, ws.O_f32,
        ws.O_proj, ema_decay, ws.I_hat, I_raw, GP);
  } else {
    if ((e = allow_smem(simt_pass2_kernel<float>, smem)) != cudaSuccess) return e;
    simt_pass2_kernel<float><<<grid, threads, smem, st>>>(p, (const float*)Q, (const float*)K, (const float*)V,
                                                          ws.fin_m, ws.fin_l, ws.O_f32, ws.O_proj, ema_decay,
                                                          ws.I_hat, I_raw, GP);
  }
  return cudaGetLastError();
}

}  // namespace restkv
