// One decode step of every query head over a cache of n_rows rows (Eq. 3): split along the rows,
// partial softmax attention per split, log-sum-exp merge.  Memory-bound streaming of K and V; all
// G query heads of a KV head share each row that is loaded.
#include <math.h>

#include <mutex>

#include "restkv_common.cuh"

namespace restkv {

namespace {

constexpr int kDecThreads = 256;

template <typename T> struct Chunk;   // 16 bytes of a row
template <> struct Chunk<__nv_bfloat16> {
  static constexpr int kElems = 8;
  __device__ static void load(const __nv_bfloat16* p, float* out) {
    const uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
    const unsigned int w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      out[2 * i] = __uint_as_float(w[i] << 16);
      out[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
};
template <> struct Chunk<float> {
  static constexpr int kElems = 4;
  __device__ static void load(const float* p, float* out) {
    const float4 u = __ldg(reinterpret_cast<const float4*>(p));
    out[0] = u.x; out[1] = u.y; out[2] = u.z; out[3] = u.w;
  }
};

// grid (splits, batch*Hkv); block 256.  LPR lanes share one row (each owns CPL 16-byte chunks of it);
// a warp covers 32/LPR rows per step.  Every lane group keeps its own running (m, l, o) per query head
// and the groups are merged through shared memory at the end.
template <typename T, int G, int LPR, int CPL>
__global__ void __launch_bounds__(kDecThreads) decode_partial_kernel(
    int Hq, int Hkv, int d, int n_rows, float scale, const T* __restrict__ q, const T* __restrict__ Kc,
    const T* __restrict__ Vc, float* __restrict__ part, int splits) {
  constexpr int E = Chunk<T>::kElems;
  constexpr int EPL = E * CPL;                 // elements of a row owned by one lane
  constexpr int RPW = 32 / LPR;                // rows per warp step
  constexpr int kGroups = (kDecThreads / 32) * RPW;
  const int split = blockIdx.x, bh = blockIdx.y;
  const int b = bh / Hkv, h = bh % Hkv;
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
  const int sub = lane % LPR, grp = wid * RPW + lane / LPR;

  float qf[G][EPL];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    const T* qr = q + ((long long)b * Hq + (long long)h * G + g) * d;
#pragma unroll
    for (int c = 0; c < CPL; ++c) Chunk<T>::load(qr + (c * LPR + sub) * E, &qf[g][c * E]);
  }
  float m[G], l[G], o[G][EPL];
#pragma unroll
  for (int g = 0; g < G; ++g) {
    m[g] = -INFINITY; l[g] = 0.f;
#pragma unroll
    for (int e = 0; e < EPL; ++e) o[g][e] = 0.f;
  }

  const long long per = ((long long)n_rows + splits - 1) / splits;
  const long long r0 = (long long)split * per;
  const long long r1 = (r0 + per < n_rows) ? r0 + per : n_rows;
  const T* Kh = Kc + (long long)bh * n_rows * d;
  const T* Vh = Vc + (long long)bh * n_rows * d;

  for (long long base = r0; base < r1; base += kGroups) {
    const long long row = base + grp;
    const bool in = row < r1;
    float kf[EPL], vf[EPL];
    if (in) {
#pragma unroll
      for (int c = 0; c < CPL; ++c) {
        Chunk<T>::load(Kh + row * d + (c * LPR + sub) * E, &kf[c * E]);
        Chunk<T>::load(Vh + row * d + (c * LPR + sub) * E, &vf[c * E]);
      }
    } else {
#pragma unroll
      for (int e = 0; e < EPL; ++e) { kf[e] = 0.f; vf[e] = 0.f; }
    }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float s = 0.f;
#pragma unroll
      for (int e = 0; e < EPL; ++e) s = fmaf(qf[g][e], kf[e], s);
#pragma unroll
      for (int off = LPR / 2; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
      s = in ? s * scale : -INFINITY;
      if (s > m[g]) {                         // new running maximum: rescale what was accumulated
        const float corr = __expf(m[g] - s);  // m = -inf gives 0
        l[g] *= corr;
#pragma unroll
        for (int e = 0; e < EPL; ++e) o[g][e] *= corr;
        m[g] = s;
      }
      const float pexp = in ? __expf(s - m[g]) : 0.f;
      l[g] += pexp;
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[g][e] = fmaf(pexp, vf[e], o[g][e]);
    }
  }

  // ---- merge, in a fixed order (no atomics: the result is bit-reproducible) ----
  // 1. the lane groups of a warp, by butterfly exchange: afterwards every group holds the warp's result
#pragma unroll
  for (int off = LPR; off < 32; off <<= 1) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      const float m_o = __shfl_xor_sync(0xffffffffu, m[g], off);
      const float l_o = __shfl_xor_sync(0xffffffffu, l[g], off);
      const float mm = fmaxf(m[g], m_o);
      const float sa = (m[g] == -INFINITY) ? 0.f : __expf(m[g] - mm);
      const float sb = (m_o == -INFINITY) ? 0.f : __expf(m_o - mm);
      l[g] = l[g] * sa + l_o * sb;
#pragma unroll
      for (int e = 0; e < EPL; ++e) o[g][e] = o[g][e] * sa + __shfl_xor_sync(0xffffffffu, o[g][e], off) * sb;
      m[g] = mm;
    }
  }
  // 2. the warps, through shared memory: w_ml [warps][G][2], w_o [warps][G][d]
  extern __shared__ float dec_smem[];
  constexpr int kWarps = kDecThreads / 32;
  float* w_ml = dec_smem;
  float* w_o = dec_smem + kWarps * G * 2;
  if (lane < LPR) {
#pragma unroll
    for (int g = 0; g < G; ++g) {
      if (sub == 0) { w_ml[(wid * G + g) * 2] = m[g]; w_ml[(wid * G + g) * 2 + 1] = l[g]; }
#pragma unroll
      for (int c = 0; c < CPL; ++c)
#pragma unroll
        for (int e = 0; e < E; ++e) w_o[((long long)wid * G + g) * d + (c * LPR + sub) * E + e] = o[g][c * E + e];
    }
  }
  __syncthreads();
  float* my_part = part + ((long long)bh * splits + split) * G * (d + 2);
  for (int e = threadIdx.x; e < G * d; e += kDecThreads) {
    const int g = e / d, k = e - g * d;
    float mm = -INFINITY;
#pragma unroll
    for (int wv = 0; wv < kWarps; ++wv) mm = fmaxf(mm, w_ml[(wv * G + g) * 2]);
    float acc = 0.f, ll = 0.f;
#pragma unroll
    for (int wv = 0; wv < kWarps; ++wv) {
      const float mw = w_ml[(wv * G + g) * 2];
      const float sc = (mw == -INFINITY) ? 0.f : __expf(mw - mm);
      acc = fmaf(w_o[((long long)wv * G + g) * d + k], sc, acc);
      ll = fmaf(w_ml[(wv * G + g) * 2 + 1], sc, ll);
    }
    my_part[g * (d + 2) + 2 + k] = acc;
    if (k == 0) { my_part[g * (d + 2)] = mm; my_part[g * (d + 2) + 1] = ll; }
  }
}

// grid (Hq, batch); block d threads (rounded to a warp).  Merges the splits.
__global__ void decode_combine_kernel(int Hq, int G, int d, int splits, const float* __restrict__ part,
                                      float* __restrict__ out, float* __restrict__ lse) {
  const int hq = blockIdx.x, b = blockIdx.y;
  const int Hkv = Hq / G, h = hq / G, g = hq % G;
  const float* base = part + (((long long)b * Hkv + h) * splits) * G * (d + 2) + (long long)g * (d + 2);
  const long long stride = (long long)G * (d + 2);
  float mm = -INFINITY;
  for (int s = 0; s < splits; ++s) mm = fmaxf(mm, base[s * stride]);
  float ll = 0.f;
  for (int s = 0; s < splits; ++s) {
    const float ms = base[s * stride];
    if (ms != -INFINITY) ll += base[s * stride + 1] * __expf(ms - mm);
  }
  for (int k = threadIdx.x; k < d; k += blockDim.x) {
    float acc = 0.f;
    for (int s = 0; s < splits; ++s) {
      const float ms = base[s * stride];
      if (ms != -INFINITY) acc += base[s * stride + 2 + k] * __expf(ms - mm);
    }
    out[((long long)b * Hq + hq) * d + k] = acc / ll;
  }
  if (lse && threadIdx.x == 0) lse[(long long)b * Hq + hq] = mm + logf(ll);
}

template <typename T, int G>
cudaError_t launch_partial(const Problem& p, const void* q, const void* Kc, const void* Vc, int n_rows, float* part,
                           int splits, cudaStream_t st) {
  constexpr int E = Chunk<T>::kElems;
  dim3 grid(splits, p.BH);
  const int chunks = p.d / E;   // 16-byte chunks per row
  const size_t smem = (size_t)(kDecThreads / 32) * G * (p.d + 2) * sizeof(float);
#define RESTKV_DEC(LPR, CPL)                                                                                    \
  do {                                                                                                          \
    if (smem > 48 * 1024) {                                                                                     \
      cudaError_t e_ = cudaFuncSetAttribute(decode_partial_kernel<T, G, LPR, CPL>,                              \
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);            \
      if (e_ != cudaSuccess) return e_;                                                                         \
    }                                                                                                           \
    decode_partial_kernel<T, G, LPR, CPL><<<grid, kDecThreads, smem, st>>>(                                     \
        p.Hq, p.Hkv, p.d, n_rows, p.scale, (const T*)q, (const T*)Kc, (const T*)Vc, part, splits);              \
  } while (0)
  // one 16-byte chunk per lane where the row allows it: few registers per thread, several CTAs per SM
  if (chunks == 8) RESTKV_DEC(8, 1);
  else if (chunks == 16) RESTKV_DEC(16, 1);
  else if (chunks == 32) RESTKV_DEC(32, 1);
  else if (chunks == 64) RESTKV_DEC(32, 2);
  else if (chunks == 4) RESTKV_DEC(4, 1);
  else if (chunks == 2) RESTKV_DEC(2, 1);
  else return cudaErrorInvalidValue;
#undef RESTKV_DEC
  return cudaGetLastError();
}

template <typename T>
cudaError_t launch_partial_g(const Problem& p, const void* q, const void* Kc, const void* Vc, int n_rows, float* part,
                             int splits, cudaStream_t st) {
  switch (p.G) {
    case 1: return launch_partial<T, 1>(p, q, Kc, Vc, n_rows, part, splits, st);
    case 2: return launch_partial<T, 2>(p, q, Kc, Vc, n_rows, part, splits, st);
    case 4: return launch_partial<T, 4>(p, q, Kc, Vc, n_rows, part, splits, st);
    case 8: return launch_partial<T, 8>(p, q, Kc, Vc, n_rows, part, splits, st);
    default: return cudaErrorInvalidValue;
  }
}

}  // namespace

cudaError_t launch_decode(const Problem& p, const void* q, const void* Kc, const void* Vc, int n_rows, float* out,
                          float* lse, float* part, int splits, cudaStream_t st, int* n_launches) {
  cudaError_t e = (p.dtype == RESTKV_BF16)
                      ? launch_partial_g<__nv_bfloat16>(p, q, Kc, Vc, n_rows, part, splits, st)
                      : launch_partial_g<float>(p, q, Kc, Vc, n_rows, part, splits, st);
  if (e != cudaSuccess) return e;
  const int threads = ((p.d + 31) / 32) * 32;
  dim3 grid(p.Hq, p.batch);
  decode_combine_kernel<<<grid, threads, 0, st>>>(p.Hq, p.G, p.d, splits, part, out, lse);
  *n_launches = 2;
  return cudaGetLastError();
}

}  // namespace restkv

// ------------------------------------------------------------------------------------------------
// Decode through the tensor-core attention phases: the G queries of a KV head are padded with zero rows to the
// kernel's 128 query rows, and afterwards the G real rows are copied out.
namespace restkv {
namespace {

// grid (128, BH), block 64: q_pad[bh, r, :] = q[b, h*G + r, :] for r < G, else 0 (bf16, head_dim 128).
__global__ void decode_pad_kernel(int Hq, int Hkv, int G, const __nv_bfloat16* __restrict__ q,
                                  __nv_bfloat16* __restrict__ q_pad) {
  const int r = blockIdx.x, bh = blockIdx.y, b = bh / Hkv, h = bh % Hkv;
  const unsigned int* src = reinterpret_cast<const unsigned int*>(q + ((long long)b * Hq + (long long)h * G + r) * 128);
  unsigned int* dst = reinterpret_cast<unsigned int*>(q_pad + ((long long)bh * 128 + r) * 128);
  dst[threadIdx.x] = r < G ? src[threadIdx.x] : 0u;
}

// grid (G, BH), block 128: out[b, h*G + g, :] = O[bh, g, :]; lse = M2 * ln 2 (M2 is in log2 units).
__global__ void decode_extract_kernel(int Hq, int Hkv, int G, const float* __restrict__ O_f32,
                                      const float* __restrict__ row_M2, float* __restrict__ out,
                                      float* __restrict__ lse) {
  const int g = blockIdx.x, bh = blockIdx.y, b = bh / Hkv, h = bh % Hkv;
  const long long hq = (long long)b * Hq + (long long)h * G + g;
  out[hq * 128 + threadIdx.x] = O_f32[((long long)bh * 128 + g) * 128 + threadIdx.x];
  if (lse && threadIdx.x == 0) lse[hq] = row_M2[(long long)bh * 128 + g] * 0.6931471805599453f;
}

}  // namespace

cudaError_t launch_decode_pad(const Problem& p, const void* q, __nv_bfloat16* q_pad, cudaStream_t st) {
  decode_pad_kernel<<<dim3(128, p.BH), 64, 0, st>>>(p.Hq, p.Hkv, p.G, (const __nv_bfloat16*)q, q_pad);
  return cudaGetLastError();
}

cudaError_t launch_decode_extract(const Problem& p, const float* O_f32, const float* row_M2, float* out, float* lse,
                                  cudaStream_t st) {
  decode_extract_kernel<<<dim3(p.G, p.BH), 128, 0, st>>>(p.Hq, p.Hkv, p.G, O_f32, row_M2, out, lse);
  return cudaGetLastError();
}

}  // namespace restkv

// ================================================================================================
// restkv_decode_static: the decode step with its split partials in memory that ships with the library.
// ================================================================================================
namespace restkv {
namespace {

// Room for the per-split partial results (m, l, o[head_dim]) of one call.  The array is part of the loaded module:
// every GPU that loads the library holds these 2 MiB until the process exits, whether the entry point is used or not.
constexpr size_t kStaticScratchFloats = 512 * 1024;
static __device__ __align__(256) float g_static_decode_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
float* g_static_scratch_addr[kMaxDevices];   // device address of the array, per device ordinal (null: not looked up yet)
int g_static_sm_count[kMaxDevices];
int g_static_last_cuda_error = 0;

// In host code `g_static_decode_scratch` only names the symbol; the address a kernel can use comes from the
// runtime, for the device that is current.
cudaError_t static_scratch_for_current_device(float** ptr, int* sm_count) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (!g_static_scratch_addr[dev]) {
    void* addr = nullptr;
    e = cudaGetSymbolAddress(&addr, g_static_decode_scratch);
    if (e != cudaSuccess) return e;
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    g_static_sm_count[dev] = sms > 0 ? sms : 1;
    g_static_scratch_addr[dev] = (float*)addr;
  }
  *ptr = g_static_scratch_addr[dev];
  *sm_count = g_static_sm_count[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace restkv

extern "C" restkv_status restkv_decode_static(const restkv_shape* shape, const void* q, const void* Kc, const void* Vc,
                                              int n_rows, float* out, float* lse, restkv_stream stream) {
  using namespace restkv;
  if (!shape || !q || !Kc || !Vc || !out || n_rows < 1) return RESTKV_ERR_INVALID_ARG;
  if ((((uintptr_t)q) | ((uintptr_t)Kc) | ((uintptr_t)Vc)) & 15u) return RESTKV_ERR_INVALID_ARG;
  if (shape->batch < 1 || shape->n_q_heads < 1 || shape->n_kv_heads < 1 || shape->head_dim < 1)
    return RESTKV_ERR_INVALID_ARG;
  if (shape->n_q_heads % shape->n_kv_heads != 0) return RESTKV_ERR_INVALID_ARG;
  if (shape->dtype != RESTKV_BF16 && shape->dtype != RESTKV_F32) return RESTKV_ERR_INVALID_ARG;
  Problem p{};
  p.batch = shape->batch; p.Hq = shape->n_q_heads; p.Hkv = shape->n_kv_heads; p.G = p.Hq / p.Hkv;
  p.d = shape->head_dim; p.dtype = shape->dtype; p.BH = p.batch * p.Hkv;
  p.scale = shape->softmax_scale != 0.f ? shape->softmax_scale : 1.0f / sqrtf((float)p.d);
  if (!(p.scale > 0.f) || !isfinite(p.scale)) return RESTKV_ERR_INVALID_ARG;
  if (p.d % 8 != 0 || p.d > 256) return RESTKV_ERR_UNSUPPORTED;
  if (p.G != 1 && p.G != 2 && p.G != 4 && p.G != 8) return RESTKV_ERR_UNSUPPORTED;
  const int chunks = p.d * (p.dtype == RESTKV_BF16 ? 2 : 4) / 16;
  if (chunks != 2 && chunks != 4 && chunks != 8 && chunks != 16 && chunks != 32 && chunks != 64)
    return RESTKV_ERR_UNSUPPORTED;
  // one split's partials for every query head must fit; more splits are used only while they fit
  const size_t per_split = (size_t)p.BH * p.G * (p.d + 2);
  if (per_split > kStaticScratchFloats) return RESTKV_ERR_WORKSPACE;
  float* scratch = nullptr;
  int sm_count = 0;
  if (const cudaError_t es = static_scratch_for_current_device(&scratch, &sm_count); es != cudaSuccess) {
    g_static_last_cuda_error = (int)es;
    return RESTKV_ERR_CUDA;
  }
  int splits = (2 * sm_count + p.BH - 1) / p.BH;
  const int by_rows = (n_rows + 255) / 256;
  if (splits > by_rows) splits = by_rows;
  if (splits > kDecodeMaxSplits) splits = kDecodeMaxSplits;
  if ((size_t)splits > kStaticScratchFloats / per_split) splits = (int)(kStaticScratchFloats / per_split);
  if (splits < 1) splits = 1;
  int n_launches = 0;
  // Every (head, split) slot that the merge kernel reads is written by the partial kernel of the same call, so
  // nothing left in the array by an earlier call is ever read and nothing has to be cleared first.
  const cudaError_t e = launch_decode(p, q, Kc, Vc, n_rows, out, lse, scratch, splits, (cudaStream_t)stream,
                                      &n_launches);
  if (e != cudaSuccess) g_static_last_cuda_error = (int)e;
  return e == cudaSuccess ? RESTKV_OK : RESTKV_ERR_CUDA;
}

extern "C" int restkv_decode_static_last_cuda_error(void) { return restkv::g_static_last_cuda_error; }
