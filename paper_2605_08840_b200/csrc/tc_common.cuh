// Shared pieces of the tensor-core score kernels: tile geometry, UMMA descriptors, tensor-map builders.
#pragma once

#include <cuda.h>

#include "restkv_common.cuh"
#include "sm100_ptx.cuh"

namespace restkv {
namespace {

using namespace ptx;

constexpr int kTile = 128;                       // tokens per tile
constexpr int kHeadDim = 128;
constexpr int kRows = 128;                       // query rows per KV head (w * G)
constexpr uint32_t kBoxBytes = 128 * 64 * 2;     // one [128 rows x 64 bf16] TMA box
constexpr uint32_t kTileBytes = 2 * kBoxBytes;   // a [128 x 128] bf16 operand tile
constexpr uint32_t kStageBytes = 2 * kTileBytes; // K tile + V tile
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kRescaleThreshold = 8.0f;        // log2 units the running maximum may exceed the reference by

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TcState {
  EncodeTiledFn encode;
};

constexpr uint32_t kIdescKK = make_idesc_bf16(128, 128, false);   // both operands K-major
constexpr uint32_t kIdescKMN = make_idesc_bf16(128, 128, true);   // B operand MN-major (V in O += P V)

__device__ __forceinline__ uint64_t kmajor_desc(uint32_t addr) { return make_smem_desc(addr, 16, 1024); }

// D[128 x 128] (+)= A[128 x 128] * B[128 x 128]^T, both operands K-major 128B-swizzled [128 x 128] bf16 tiles
// made of two [128 x 64] boxes.  One thread issues the eight K = 16 steps.
// (The issuing thread's own instruction stream is what bounds a run of small products: the two descriptors are built
// once and stepped by adding to their address field, which counts 16-byte units.)
__device__ __forceinline__ void mma_tile_kk(uint32_t tmem_d, uint32_t a_smem, uint32_t b_smem, bool accumulate) {
  const uint64_t a0 = kmajor_desc(a_smem), b0 = kmajor_desc(b_smem);
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint64_t step = (uint64_t)(((uint32_t)(k >> 2) * kBoxBytes + (uint32_t)(k & 3) * 32u) >> 4);
    umma_ss(tmem_d, a0 + step, b0 + step, kIdescKK, accumulate || k > 0);
  }
}

// Exact ||o - v||^2 for the rare entries whose attention weight is large (the expansion ||o||^2 + ||v||^2 - 2 o.v
// cancels when o approaches v).  Computed by a whole warp: lane L takes elements 4L .. 4L+3, the partial sums meet by butterfly exchange (every
// lane returns the full sum).
__device__ __forceinline__ float exact_dist2_warp(const float* __restrict__ o_row, const __nv_bfloat16* __restrict__ v_row,
                                                  int lane) {
  const float4 o = *reinterpret_cast<const float4*>(o_row + lane * 4);
  const uint2 vv = *reinterpret_cast<const uint2*>(v_row + lane * 4);
  const float d0 = o.x - __uint_as_float(vv.x << 16), d1 = o.y - __uint_as_float(vv.x & 0xFFFF0000u);
  const float d2 = o.z - __uint_as_float(vv.y << 16), d3 = o.w - __uint_as_float(vv.y & 0xFFFF0000u);
  float ss = (d0 * d0 + d1 * d1) + (d2 * d2 + d3 * d3);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
  return ss;
}

// The same under the output projection: (o - v)^T Mt (o - v) = (o - v) . (Mt o - Mt v), Mt symmetric [128 x 128] fp32,
// Mt o given (op_row).  Row k of Mt is read by the whole warp (coalesced) and weighted with v_k, which lane k / 4 holds.
__device__ __forceinline__ float exact_proj_dist2_warp(const float* __restrict__ o_row, const float* __restrict__ op_row,
                                                       const __nv_bfloat16* __restrict__ v_row,
                                                       const float* __restrict__ Mt, int lane) {
  const float4 o = *reinterpret_cast<const float4*>(o_row + lane * 4);
  const float4 op = *reinterpret_cast<const float4*>(op_row + lane * 4);
  const uint2 vv = *reinterpret_cast<const uint2*>(v_row + lane * 4);
  const float v[4] = {__uint_as_float(vv.x << 16), __uint_as_float(vv.x & 0xFFFF0000u), __uint_as_float(vv.y << 16),
                      __uint_as_float(vv.y & 0xFFFF0000u)};
  float4 mv = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
  for (int src = 0; src < 32; ++src) {
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float vk = __shfl_sync(0xffffffffu, v[e], src);
      const float4 m = __ldg(reinterpret_cast<const float4*>(Mt + (src * 4 + e) * kHeadDim + lane * 4));
      mv.x = fmaf(m.x, vk, mv.x); mv.y = fmaf(m.y, vk, mv.y); mv.z = fmaf(m.z, vk, mv.z); mv.w = fmaf(m.w, vk, mv.w);
    }
  }
  float ss = ((o.x - v[0]) * (op.x - mv.x) + (o.y - v[1]) * (op.y - mv.y)) +
             ((o.z - v[2]) * (op.z - mv.z) + (o.w - v[3]) * (op.w - mv.w));
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
  return fmaxf(ss, 0.f);
}

// The expansion o^T Mt o - 2 (Mt o) . v + v^T Mt v in fp32 with exact dot products (vmv = v^T Mt v given): accurate
// as long as the three terms do not nearly cancel, i.e. while o stays away from v.
__device__ __forceinline__ float expanded_proj_dist2_warp(const float* __restrict__ o_row, const float* __restrict__ op_row,
                                                          const __nv_bfloat16* __restrict__ v_row, float vmv, int lane) {
  const float4 o = *reinterpret_cast<const float4*>(o_row + lane * 4);
  const float4 op = *reinterpret_cast<const float4*>(op_row + lane * 4);
  const uint2 vv = *reinterpret_cast<const uint2*>(v_row + lane * 4);
  const float v0 = __uint_as_float(vv.x << 16), v1 = __uint_as_float(vv.x & 0xFFFF0000u);
  const float v2 = __uint_as_float(vv.y << 16), v3 = __uint_as_float(vv.y & 0xFFFF0000u);
  // o . (Mt o) - 2 v . (Mt o) = (o - 2 v) . (Mt o)
  float ss = ((o.x - 2.f * v0) * op.x + (o.y - 2.f * v1) * op.y) + ((o.z - 2.f * v2) * op.z + (o.w - 2.f * v3) * op.w);
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
  return fmaxf(ss + vmv, 0.f);
}

// After a wait has failed: wait (bounded, whatever the abort flag says) for a bulk copy or an MMA that this thread
// itself set in motion, so that nothing is still writing this CTA's shared or tensor memory when it returns.
__device__ __forceinline__ void wait_issued(uint64_t* bar, uint32_t parity) {
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity & 1u))
    if (clock64() - t0 > 4000000000ll) return;
}

constexpr uint32_t kAugBytes = kBoxBytes;     // [128 rows x 64 bf16], only K steps 0 (S') and 1 (C') are used
constexpr uint32_t kOnesBytes = 1024;         // one 8-row group of ones, shared by all 16 groups (stride 0)
constexpr float kHeavyA = 0.125f;             // attention weight above which ||o - v||^2 is recomputed exactly

// ------------------------------------------------------------------------------------------------
inline CUresult encode_tiles(TcState* st, CUtensorMap* map, const void* base, int rank, const cuuint64_t* dims,
                      const cuuint64_t* strides_bytes) {
  cuuint32_t box[4] = {64, 128, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return st->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), dims,
                    strides_bytes, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

inline bool make_rows_map(TcState* st, CUtensorMap* map, const void* base, int BH) {   // [BH, 128, 128] contiguous
  cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)kRows, (cuuint64_t)BH};
  cuuint64_t str[2] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)kRows * kHeadDim * 2};
  return encode_tiles(st, map, base, 3, dims, str) == CUDA_SUCCESS;
}

inline bool make_aug_map(TcState* st, CUtensorMap* map, const void* base, int BH) {   // [BH, 128, 64] contiguous
  cuuint64_t dims[3] = {64, (cuuint64_t)kRows, (cuuint64_t)BH};
  cuuint64_t str[2] = {64 * 2, (cuuint64_t)kRows * 64 * 2};
  return encode_tiles(st, map, base, 3, dims, str) == CUDA_SUCCESS;
}

inline bool make_kv_map(TcState* st, CUtensorMap* map, const void* base, const Problem& p, long long sb, long long sh,
                 long long sn) {
  cuuint64_t dims[4] = {(cuuint64_t)p.d, (cuuint64_t)p.n_kv, (cuuint64_t)p.Hkv, (cuuint64_t)p.batch};
  // a dimension of extent 1 may carry any stride; give it a valid one
  cuuint64_t str[3] = {(cuuint64_t)sn * 2, (cuuint64_t)(p.Hkv > 1 ? sh : sn) * 2,
                       (cuuint64_t)(p.batch > 1 ? sb : sn) * 2};
  return encode_tiles(st, map, base, 4, dims, str) == CUDA_SUCCESS;
}


}  // namespace
}  // namespace restkv
