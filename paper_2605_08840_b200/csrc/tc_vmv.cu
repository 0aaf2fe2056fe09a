// q[bh, g, j] = v_j^T Mt_g v_j = || L_g^T v_j ||^2 for every token j of a KV head and each of the G query heads that
// share it: the token's own term of Eq. 7's norm under the output projection of Eq. 4 (the counterpart of ||v_j||^2
// without one).  It does not depend on the queries.
//
// Per 128-token tile: Y_g = V_tile L_g on the tensor cores (tcgen05, fp32 accumulators in tensor memory, one
// 128-column accumulator per query head; two query heads share one product of N = 256, their factor tiles lying
// behind one another in shared memory), then the row sums of squares.  One CTA per SM over an equal, contiguous
// share of the (head, tile) pairs; CTAs do not wait for one another.
//   warp 0     TMA: the head's G factor tiles L_g^T [128 x 128] bf16 (reloaded when the share enters a new head),
//              then the V tiles through a ring that takes the rest of shared memory (three to six tiles: the loads
//              are latency-bound, so every tile in flight counts)
//   warp 1     MMA issue: for each tile one product per pair of query heads (eight K = 16 steps of N = 256; N = 128
//              with a single head), each committed to the pair's barrier.  A step costs the issuing thread and the
//              tensor pipe about as much at N = 64 as at N = 128, so fewer, wider steps are what pays (narrowing
//              the steps to the triangular factor's non-zero columns did not)
//   warps 2-17 read-out: thread = token (tensor-memory lane), 128 columns squared and summed; each of the four warps
//              of a lane quarter takes one query head
// Every wait is bounded; after a failed wait the roles stop, wait for what they issued and the CTA returns.
#include "tc_common.cuh"

namespace restkv {

namespace {

constexpr int kVThreads = 576;
constexpr int kVMaxG = 4;
constexpr int kVTiles = 7;                 // factor tiles + ring slots: 224 KB
constexpr int kVMaxRing = kVTiles - 1;
constexpr size_t kVSmem = (size_t)kVTiles * kTileBytes + 1024;

struct VmvBars {
  uint64_t lt_full, v_full[kVMaxRing], v_empty[kVMaxRing], acc_full[kVMaxG], acc_empty[kVMaxG], drain;
};

struct VmvArgs {
  int Hkv, BH, G, n_kv, tiles;
  float* out;                // [BH, G, n_kv]
  unsigned int* dev_status;
  long long wait_limit;
};

__global__ void __launch_bounds__(kVThreads, 1)
vmv_kernel(const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmLT, const VmvArgs a) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) VmvBars bars;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const long long total = (long long)a.BH * a.tiles;
  const long long per = (total + gridDim.x - 1) / gridDim.x;
  const long long first = (long long)blockIdx.x * per;
  const int cnt = (int)max(0ll, min(total, first + per) - first);
  if (cnt == 0) return;   // uniform over the CTA

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  const uint32_t off_v = (uint32_t)a.G * kTileBytes;   // the ring follows the factor tiles
  const int kVRing = kVTiles - a.G;
  const uint32_t half_stride = a.G >= 2 ? kTileBytes : kBoxBytes;   // distance of a factor operand's two K halves
  const int pairs = (a.G + 1) / 2;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  VmvBars* B = &bars;
  unsigned int* dev_status = a.dev_status;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&B->lt_full, 1);
    for (int i = 0; i < kVMaxRing; ++i) {
      mbar_init(&B->v_full[i], 1);
      mbar_init(&B->v_empty[i], 1);
    }
    for (int g = 0; g < kVMaxG; ++g) {
      mbar_init(&B->acc_full[g], 1);    // indexed by pair of query heads
      mbar_init(&B->acc_empty[g], a.G >= 2 ? 8 : 4);   // the read-out warps of the pair: four lane quarters per head
    }
    mbar_init(&B->drain, 1);
    fence_mbar_init();
    prefetch_tensormap(&tmV);
    prefetch_tensormap(&tmLT);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      int prev_bh = -1, heads_seen = 0, issued = 0;
      bool ok = true;
      for (int it = 0; it < cnt && ok; ++it) {
        const long long idx = first + it;
        const int bh = (int)(idx / a.tiles), tile = (int)(idx % a.tiles);
        const int s = it % kVRing;
        if (it >= kVRing)
          ok = mbar_wait(&B->v_empty[s], (uint32_t)(it / kVRing - 1) & 1u, &abort_flag, dev_status, kDevTimeout, a.wait_limit);
        if (ok && bh != prev_bh) {
          // the products of every earlier tile read the previous head's factor tiles: they must be complete
          if (it > 0)
            ok = mbar_wait(&B->v_empty[(it - 1) % kVRing], (uint32_t)((it - 1) / kVRing) & 1u, &abort_flag, dev_status,
                           kDevTimeout, a.wait_limit);
          if (ok) {
            mbar_arrive_expect_tx(&B->lt_full, (uint32_t)a.G * kTileBytes);
            for (int g = 0; g < a.G; ++g) {
              // a pair's tiles interleave by K half: [half 0: head 2p, head 2p+1][half 1: head 2p, head 2p+1], so
              // that each half is one K-major operand of 256 rows
              const int hq = (bh % a.Hkv) * a.G + g;
              uint8_t* dst = gen_base + (uint32_t)(g >> 1) * 2u * kTileBytes + (uint32_t)(g & 1) * kBoxBytes;
              tma_load_3d(dst, &tmLT, &B->lt_full, 0, 0, hq);
              tma_load_3d(dst + half_stride, &tmLT, &B->lt_full, 64, 0, hq);
            }
            ++heads_seen;
            prev_bh = bh;
          }
        }
        if (!ok) break;
        uint8_t* dv = gen_base + off_v + (uint32_t)s * kTileBytes;
        mbar_arrive_expect_tx(&B->v_full[s], kTileBytes);
        tma_load_4d(dv, &tmV, &B->v_full[s], 0, tile * kTile, bh % a.Hkv, bh / a.Hkv);
        tma_load_4d(dv + kBoxBytes, &tmV, &B->v_full[s], 64, tile * kTile, bh % a.Hkv, bh / a.Hkv);
        issued = it + 1;
      }
      if (*(volatile int*)&abort_flag) {
        // the tiles requested last may still be on their way into shared memory
        if (heads_seen > 0) wait_issued(&B->lt_full, (uint32_t)(heads_seen - 1));
        for (int i = max(0, issued - kVRing); i < issued; ++i) wait_issued(&B->v_full[i % kVRing], (uint32_t)(i / kVRing));
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      int prev_bh = -1, heads_seen = 0;
      bool ok = true;
      for (int it = 0; it < cnt && ok; ++it) {
        const long long idx = first + it;
        const int bh = (int)(idx / a.tiles);
        const int s = it % kVRing;
        if (bh != prev_bh) {
          ok = mbar_wait(&B->lt_full, (uint32_t)heads_seen & 1u, &abort_flag, dev_status, kDevTimeout, a.wait_limit);
          ++heads_seen;
          prev_bh = bh;
        }
        ok = ok && mbar_wait(&B->v_full[s], (uint32_t)(it / kVRing) & 1u, &abort_flag, dev_status, kDevTimeout, a.wait_limit);
        for (int pr = 0; pr < pairs && ok; ++pr) {
          if (it > 0)
            ok = mbar_wait(&B->acc_empty[pr], (uint32_t)(it - 1) & 1u, &abort_flag, dev_status, kDevTimeout, a.wait_limit);
          if (!ok) break;
          tc_fence_after();
          const uint32_t a_smem = smem_base + off_v + (uint32_t)s * kTileBytes;
          const uint32_t b_smem = smem_base + (uint32_t)pr * 2u * kTileBytes;
          // the descriptors are built once and stepped by adding to their address field (16-byte units)
          const uint64_t a0 = kmajor_desc(a_smem), b0 = kmajor_desc(b_smem);
          const uint32_t idesc = a.G >= 2 ? make_idesc_bf16(128, 256, false) : make_idesc_bf16(128, 128, false);
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint64_t a_step = (uint64_t)(((uint32_t)(k >> 2) * kBoxBytes + (uint32_t)(k & 3) * 32u) >> 4);
            const uint64_t b_step = (uint64_t)(((uint32_t)(k >> 2) * half_stride + (uint32_t)(k & 3) * 32u) >> 4);
            umma_ss(tmem + (uint32_t)pr * 256u, a0 + a_step, b0 + b_step, idesc, k > 0);
          }
          umma_commit(&B->acc_full[pr]);
        }
        if (ok) umma_commit(&B->v_empty[s]);   // the tile's slot is free once its last product has read it
      }
      if (*(volatile int*)&abort_flag) {   // let the products already issued finish before the CTA returns
        umma_commit(&B->drain);
        wait_issued(&B->drain, 0);
      }
    }
  } else {
    const int quad = warp & 3;   // the tensor-memory lane quarter this warp may touch
    const int g_first = (warp - 2) >> 2;
    const int t = quad * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    bool ok = true;
    for (int it = 0; it < cnt && ok; ++it) {
      const long long idx = first + it;
      const int bh = (int)(idx / a.tiles), tile = (int)(idx % a.tiles);
      const int j = tile * kTile + t;
      for (int g = g_first; g < a.G && ok; g += 4) {
        ok = mbar_wait(&B->acc_full[g >> 1], (uint32_t)it & 1u, &abort_flag, dev_status, kDevTimeout, a.wait_limit);
        float sum = 0.f;
        if (ok) {
          tc_fence_after();
          const uint32_t tY = tmem + lane_base + (uint32_t)g * 128u;
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            float y0[32], y1[32];
            tmem_ld32(tY + (uint32_t)c * 64u, y0);
            tmem_ld32(tY + (uint32_t)c * 64u + 32u, y1);
            tmem_wait_ld();
            float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
            for (int u = 0; u < 32; u += 2) {
              s0 = fmaf(y0[u], y0[u], s0); s1 = fmaf(y0[u + 1], y0[u + 1], s1);
              s2 = fmaf(y1[u], y1[u], s2); s3 = fmaf(y1[u + 1], y1[u + 1], s3);
            }
            sum += (s0 + s1) + (s2 + s3);
          }
          tc_fence_before();
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&B->acc_empty[g >> 1]);
        if (ok && j < a.n_kv) a.out[((long long)bh * a.G + g) * a.n_kv + j] = sum;
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

bool tc_vmv_supported(const Problem& p) {
  return tc_supported(p) && p.G <= kVMaxG && p.proj.LT != nullptr;
}

cudaError_t launch_tc_vmv(void* state, const Problem& p, const void* V, float* out, int sm_count, long long wait_limit,
                          unsigned int* dev_status, cudaStream_t st) {
  TcState* ts = (TcState*)state;
  CUtensorMap tmV, tmLT;
  if (!make_kv_map(ts, &tmV, V, p, p.vsb, p.vsh, p.vsn) || !make_rows_map(ts, &tmLT, p.proj.LT, p.Hq))
    return cudaErrorInvalidValue;
  static bool attr_set = false;
  if (!attr_set) {
    cudaError_t e = cudaFuncSetAttribute(vmv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kVSmem);
    if (e != cudaSuccess) return e;
    attr_set = true;
  }
  VmvArgs a{};
  a.Hkv = p.Hkv; a.BH = p.BH; a.G = p.G; a.n_kv = p.n_kv; a.tiles = (p.n_kv + kTile - 1) / kTile;
  a.out = out; a.dev_status = dev_status; a.wait_limit = wait_limit;
  const long long total = (long long)a.BH * a.tiles;
  const int grid = (int)(total < sm_count ? total : sm_count);
  vmv_kernel<<<grid, kVThreads, kVSmem, st>>>(tmV, tmLT, a);
  return cudaGetLastError();
}

}  // namespace restkv
