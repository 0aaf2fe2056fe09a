// Tensor-core score kernels for sm_100a: bf16 inputs, head_dim 128, w * group = 128 query rows per KV head.
//
// Both kernels work on tiles of 128 tokens.  K and V tiles arrive in shared memory through TMA
// (128-byte swizzle, two [128 x 64] boxes per tile), the contractions run on tcgen05.mma with fp32
// accumulators in tensor memory, and warp-specialised CTAs (one TMA warp, one MMA warp, epilogue
// warpgroups) overlap the three.
//
//   pass 1  (Eq. 3)   S = Q K^T per tile (queries in TMEM lanes), online softmax statistics with a lazily
//                     updated reference maximum, P = exp2(.) written to TMEM as bf16 and used as the A operand
//                     of O += P V.  One partial (m, l, O) per (batch, head, token split).
//   pass 2  (Eq. 7-9) S^T = K Q^T and C^T = V O^T per tile (tokens in TMEM lanes, one thread per token):
//                     A = exp2(s*c - M), ||o - v||^2 = ||o||^2 + ||v||^2 - 2 o.v, I = A/(1-A) * ||o - v||,
//                     EMA over the window queries as a Horner chain down the accumulator columns,
//                     mean over the query heads of the group.
// Every mbarrier wait is bounded; a wait that runs out sets the sticky timeout bit and the CTA unwinds.
#include <cuda.h>

#include "tc_common.cuh"

namespace restkv {

namespace {

// ================================================================================================
// Pass 1
// ================================================================================================
// Warp 0: TMA producer.  Warp 1: MMA issuer.  Warps 2-5 and 6-9: two softmax warpgroups (thread = query row);
// warpgroup g owns the tiles it = g, g + 2, ... of the CTA with its own running (m, l) and its own output
// accumulator, so the CTA writes two partials.  Tensor memory: S_g at g*128 (the bf16 P_g overwrites its first
// 64 columns once the logits are in registers), O_g at 256 + g*128.  K and V travel in separate rings (3 slots
// of 32 KB each): a K slot is free as soon as S = Q K^T has run, a V slot after O += P V.
// The warpgroup that owns a tile also computes ||v_j||^2 of its 128 tokens from the V tile in shared memory
// and stores them for pass 2.
constexpr int kP1SoftWarps = 8;
constexpr int kP1Threads = 64 + kP1SoftWarps * 32;
constexpr int kP1KSlots = 3, kP1VSlots = 3;

__global__ void __launch_bounds__(kP1Threads, 1)
tc_pass1_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, int Hkv, int n, int n_kv, int w, float scale, int splits,
                float* __restrict__ part_m, float* __restrict__ part_l, float* __restrict__ part_O,
                float* __restrict__ vnorm, unsigned int* __restrict__ dev_status) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_q_full, bar_k_full[kP1KSlots], bar_k_empty[kP1KSlots], bar_v_full[kP1VSlots],
      bar_v_empty[kP1VSlots], bar_s_full[2], bar_p_full[2], bar_pv_done[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem_base;
  const uint32_t sK = sQ + kTileBytes;                       // K slot i at sK + i*kTileBytes
  const uint32_t sV = sK + kP1KSlots * kTileBytes;           // V slot i at sV + i*kTileBytes
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, bh = blockIdx.y;
  const int b = bh / Hkv, h = bh % Hkv;

  const int n_tiles = (n_kv + kTile - 1) / kTile;
  const int per = (n_tiles + splits - 1) / splits;
  const int tile0 = split * per;
  const int T = max(0, min(n_tiles, tile0 + per) - tile0);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&bar_q_full, 1);
    for (int i = 0; i < kP1KSlots; ++i) { mbar_init(&bar_k_full[i], 1); mbar_init(&bar_k_empty[i], 1); }
    for (int i = 0; i < kP1VSlots; ++i) { mbar_init(&bar_v_full[i], 1); mbar_init(&bar_v_empty[i], 1 + 4); }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar_s_full[i], 1);
      mbar_init(&bar_p_full[i], 128);
      mbar_init(&bar_pv_done[i], 1);
    }
    fence_mbar_init();
    prefetch_tensormap(&tmQ);
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
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
    // ---------------- TMA producer ----------------
    if (lane == 0 && T > 0) {
      mbar_arrive_expect_tx(&bar_q_full, kTileBytes);
      tma_load_3d(gen_base, &tmQ, &bar_q_full, 0, 0, bh);
      tma_load_3d(gen_base + kBoxBytes, &tmQ, &bar_q_full, 64, 0, bh);
      for (int it = 0; it < T; ++it) {
        const int ks = it % kP1KSlots, vs = it % kP1VSlots;
        const int j0 = (tile0 + it) * kTile;
        if (it >= kP1KSlots &&
            !mbar_wait(&bar_k_empty[ks], (it / kP1KSlots - 1) & 1, &abort_flag, dev_status, kDevTimeout))
          break;
        uint8_t* dK = gen_base + kTileBytes + (size_t)ks * kTileBytes;
        mbar_arrive_expect_tx(&bar_k_full[ks], kTileBytes);
        tma_load_4d(dK, &tmK, &bar_k_full[ks], 0, j0, h, b);
        tma_load_4d(dK + kBoxBytes, &tmK, &bar_k_full[ks], 64, j0, h, b);
        if (it >= kP1VSlots &&
            !mbar_wait(&bar_v_empty[vs], (it / kP1VSlots - 1) & 1, &abort_flag, dev_status, kDevTimeout))
          break;
        uint8_t* dV = gen_base + (1 + kP1KSlots) * kTileBytes + (size_t)vs * kTileBytes;
        mbar_arrive_expect_tx(&bar_v_full[vs], kTileBytes);
        tma_load_4d(dV, &tmV, &bar_v_full[vs], 0, j0, h, b);
        tma_load_4d(dV + kBoxBytes, &tmV, &bar_v_full[vs], 64, j0, h, b);
      }
    }
  } else if (warp == 1) {
    // ---------------- MMA issuer: S(it), then O += P V of tile it - 1 ----------------
    if (lane == 0 && T > 0) {
      bool ok = mbar_wait(&bar_q_full, 0, &abort_flag, dev_status, kDevTimeout);
      for (int it = 0; ok && it <= T; ++it) {
        if (it < T) {
          const int ks = it % kP1KSlots, g = it & 1;
          if (!mbar_wait(&bar_k_full[ks], (it / kP1KSlots) & 1, &abort_flag, dev_status, kDevTimeout)) break;
          tc_fence_after();
          // S_g may be overwritten: O += P V of tile it - 2 (which read P_g) was issued earlier and MMAs run in order
          mma_tile_kk(tmem + (uint32_t)g * 128u, sQ, sK + (uint32_t)ks * kTileBytes, false);
          umma_commit(&bar_s_full[g]);
          umma_commit(&bar_k_empty[ks]);
        }
        if (it >= 1) {
          const int pt = it - 1, g = pt & 1, vs = pt % kP1VSlots;
          if (!mbar_wait(&bar_p_full[g], (pt >> 1) & 1, &abort_flag, dev_status, kDevTimeout)) break;
          if (!mbar_wait(&bar_v_full[vs], (pt / kP1VSlots) & 1, &abort_flag, dev_status, kDevTimeout)) break;
          tc_fence_after();
          // A = P_g in TMEM (16 tokens = 8 packed columns per K step), B = V tile, MN-major
          const uint32_t vaddr = sV + (uint32_t)vs * kTileBytes;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint64_t bdesc = make_smem_desc(vaddr + (uint32_t)k * 2048u, kBoxBytes, 1024);
            umma_ts(tmem + 256u + (uint32_t)g * 128u, tmem + (uint32_t)g * 128u + (uint32_t)k * 8u, bdesc, kIdescKMN,
                    pt >= 2 || k > 0);
          }
          umma_commit(&bar_pv_done[g]);
          umma_commit(&bar_v_empty[vs]);
        }
      }
    }
  } else {
    // ---------------- softmax warpgroups: thread = query row ----------------
    const int g = (warp - 2) >> 2;
    const int quad = warp & 3;
    const int row = quad * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const uint32_t tS = tmem + (uint32_t)g * 128u + lane_base, tO = tmem + 256u + (uint32_t)g * 128u + lane_base;
    const int i_q = row % w;                  // window position of this row (row = group * w + i)
    const float c2 = scale * kLog2e;
    float m_ref = -INFINITY;
    float2 l2 = make_float2(0.f, 0.f);
    bool ok = true;
    int uses = 0;                             // tiles this warpgroup has processed
    for (int it = g; it < T; it += 2, ++uses) {
      const uint32_t par = (uint32_t)uses & 1u;
      ok = ok && mbar_wait(&bar_s_full[g], par, &abort_flag, dev_status, kDevTimeout);
      if (!ok) break;
      tc_fence_after();
      const int j0 = (tile0 + it) * kTile;
      const bool ragged = j0 + kTile > n;   // rows past the scored prefix: window rows (causal) or padding
      // ---- sweep 1: row maximum of the tile ----
      float tmax = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float s[32];
        tmem_ld32(tS + c * 32, s);
        tmem_wait_ld();
        if (ragged) {
#pragma unroll
          for (int u = 0; u < 32; ++u) {
            const int j = j0 + c * 32 + u;
            const bool vis = (j < n_kv) && (j < n || (j - n) <= i_q);
            s[u] = vis ? s[u] : -INFINITY;
          }
        }
#pragma unroll
        for (int u = 0; u < 32; ++u) tmax = fmaxf(tmax, s[u]);
      }
      const float m_tile = tmax * c2;
      const bool need = m_tile > m_ref + kRescaleThreshold;   // also true for the first visible entries (m_ref = -inf)
      float factor = 1.f;
      if (need) {
        factor = ex2_approx(m_ref - m_tile);   // 0 when m_ref = -inf
        l2.x *= factor;
        l2.y *= factor;
        m_ref = m_tile;
      }
      // S(it) has landed, so O += P V of this warpgroup's previous tile (issued before it) is complete
      if (uses > 0 && __any_sync(0xffffffffu, need)) {
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          float o[32];
          tmem_ld32(tO + c * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int u = 0; u < 32; ++u) o[u] *= factor;
          tmem_st32(tO + c * 32, o);
        }
      }
      // ---- sweep 2: P = exp2(s*c2 - m_ref) as bf16 over the first 64 columns of S_g.  Chunk c of P lands on
      //      columns [16c, 16c + 16), which belong to a chunk of S that is already in registers. ----
      const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
      const float2 c22 = make_float2(c2, c2), nm2 = make_float2(-m_use, -m_use);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float s[32];
        tmem_ld32(tS + c * 32, s);
        tmem_wait_ld();
        if (ragged) {
#pragma unroll
          for (int u = 0; u < 32; ++u) {
            const int j = j0 + c * 32 + u;
            const bool vis = (j < n_kv) && (j < n || (j - n) <= i_q);
            s[u] = vis ? s[u] : -INFINITY;
          }
        }
        uint32_t packed[16];
#pragma unroll
        for (int u = 0; u < 16; ++u) {
          const float2 a = ffma2(make_float2(s[2 * u], s[2 * u + 1]), c22, nm2);
          const float2 pp = make_float2(ex2_approx(a.x), ex2_approx(a.y));
          l2 = fadd2(l2, pp);
          packed[u] = pack_bf16x2(pp.x, pp.y);
        }
        tmem_st16(tS + c * 16, packed);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bar_p_full[g]);

      // ---- ||v||^2 of token j0 + row from the swizzled V tile (chunk c of row r sits at chunk c ^ (r & 7)) ----
      const int vs = it % kP1VSlots;
      ok = ok && mbar_wait(&bar_v_full[vs], (it / kP1VSlots) & 1, &abort_flag, dev_status, kDevTimeout);
      if (!ok) break;
      {
        const uint8_t* vt = gen_base + (1 + kP1KSlots) * kTileBytes + (size_t)vs * kTileBytes;
        float2 acc = make_float2(0.f, 0.f);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const uint8_t* rowp = vt + half * kBoxBytes + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint4 u = *reinterpret_cast<const uint4*>(rowp + ((c ^ (row & 7)) << 4));
            const unsigned int wv[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const float2 e = make_float2(__uint_as_float(wv[q] << 16), __uint_as_float(wv[q] & 0xFFFF0000u));
              acc = ffma2(e, e, acc);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&bar_v_empty[vs]);
        const int j = j0 + row;
        if (j < n_kv) vnorm[(long long)bh * n_kv + j] = acc.x + acc.y;
      }
    }
    // ---- write this warpgroup's partial (m, l, O) ----
    const long long o_idx = (((long long)bh * splits + split) * 2 + g) * kRows + row;
    float* Op = part_O + o_idx * kHeadDim;
    if (uses > 0 && ok) ok = mbar_wait(&bar_pv_done[g], (uint32_t)(uses - 1) & 1u, &abort_flag, dev_status, kDevTimeout);
    if (uses > 0 && ok) {
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float o[32];
        tmem_ld32(tO + c * 32, o);
        tmem_wait_ld();
#pragma unroll
        for (int u = 0; u < 32; u += 4)
          *reinterpret_cast<float4*>(Op + c * 32 + u) = make_float4(o[u], o[u + 1], o[u + 2], o[u + 3]);
      }
      part_m[o_idx] = (m_ref == -INFINITY) ? -INFINITY : m_ref * kLn2;   // natural-log units
      part_l[o_idx] = l2.x + l2.y;
    } else {
      for (int u = 0; u < kHeadDim; u += 4) *reinterpret_cast<float4*>(Op + u) = make_float4(0.f, 0.f, 0.f, 0.f);
      part_m[o_idx] = -INFINITY;
      part_l[o_idx] = 0.f;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ================================================================================================
// Pass 2
// ================================================================================================
// Warp 0: TMA producer.  Warp 1: MMA issuer.  Warps 2-17: four epilogue warpgroups; all of them work on the same
// tile, warpgroup c on accumulator columns [32c, 32c + 32) (one thread per token and 32 query rows).
//
// The per-query-row constants ride through the tensor core: one extra K = 16 step against a block of ones adds
//   -(m*log2e + log2 l)/(scale*log2e)  to  S^T = K Q^T      (so that exp2(-scale*log2e * S') = 1/A), and
//   ||o||^2                            to  C^T = V (-2 O)^T (so that C' + ||v||^2 = ||o - v||^2),
// which leaves the epilogue without any per-column operand.  With u = 1/A and x = ||o - v||^2 the indicator is
//   A/(1-A) * sqrt(x) = sqrt(x)/(u - 1) = x * rsqrt(x * (u-1)^2).
constexpr int kP2EpiWarps = 16;
constexpr int kP2EpiThreads = kP2EpiWarps * 32;
constexpr int kP2Threads = 64 + kP2EpiThreads;
template <int kW>
__global__ void __launch_bounds__(kP2Threads, 1)
tc_pass2_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmO,
                const __grid_constant__ CUtensorMap tmAug, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, int Hkv, int n, float scale, float ema_decay, int splits,
                const float* __restrict__ O_f32, const __nv_bfloat16* __restrict__ V, long long vsb, long long vsh,
                long long vsn, const float* __restrict__ vnorm, int n_kv, float* __restrict__ I_hat,
                unsigned int* __restrict__ dev_status) {
  constexpr int kG = kRows / kW;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_const_full, bar_kv_full[2], bar_kv_empty[2], bar_acc_full[2], bar_acc_empty[2],
      bar_red_full[4];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ float red[4][4][kTile];       // [tile & 3][warpgroup][token]: each warpgroup's share of the score

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t sQ = smem_base, sO = sQ + kTileBytes, sAug = sO + kTileBytes, sOnes = sAug + kAugBytes;
  const uint32_t sKV = sOnes + kOnesBytes;
  uint8_t* gen_base = smem_raw + (smem_base - smem_u32(smem_raw));
  uint8_t* gen_kv = gen_base + (sKV - smem_base);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int split = blockIdx.x, bh = blockIdx.y;
  const int b = bh / Hkv, h = bh % Hkv;

  const int n_tiles = (n + kTile - 1) / kTile;   // only the scored prefix rows
  const int per = (n_tiles + splits - 1) / splits;
  const int tile0 = split * per;
  const int T = max(0, min(n_tiles, tile0 + per) - tile0);

  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(&bar_const_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bar_kv_full[i], 1);
      mbar_init(&bar_kv_empty[i], 1);                 // MMA commit
      mbar_init(&bar_acc_full[i], 1);
      mbar_init(&bar_acc_empty[i], kP2EpiWarps);
    }
    for (int i = 0; i < 4; ++i) mbar_init(&bar_red_full[i], kP2EpiWarps);
    fence_mbar_init();
    prefetch_tensormap(&tmQ);
    prefetch_tensormap(&tmO);
    prefetch_tensormap(&tmAug);
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
  }
  if (warp == 1) {
    tmem_alloc(&tmem_slot, 512);
    tmem_relinquish();
  }
  if (threadIdx.x >= 64 && threadIdx.x < 64 + (int)(kOnesBytes / 4))   // the block of ones (bf16 1.0 = 0x3F80)
    reinterpret_cast<uint32_t*>(gen_base + (sOnes - smem_base))[threadIdx.x - 64] = 0x3F803F80u;
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = tmem_slot;   // buffer b: S' at b*256, C' at b*256 + 128

  if (warp == 0) {
    if (lane == 0 && T > 0) {
      mbar_arrive_expect_tx(&bar_const_full, 2 * kTileBytes + kAugBytes);
      tma_load_3d(gen_base, &tmQ, &bar_const_full, 0, 0, bh);
      tma_load_3d(gen_base + kBoxBytes, &tmQ, &bar_const_full, 64, 0, bh);
      tma_load_3d(gen_base + kTileBytes, &tmO, &bar_const_full, 0, 0, bh);
      tma_load_3d(gen_base + kTileBytes + kBoxBytes, &tmO, &bar_const_full, 64, 0, bh);
      tma_load_3d(gen_base + 2 * kTileBytes, &tmAug, &bar_const_full, 0, 0, bh);
      for (int it = 0; it < T; ++it) {
        const int s = it & 1;
        if (it >= 2 && !mbar_wait(&bar_kv_empty[s], ((it >> 1) - 1) & 1, &abort_flag, dev_status, kDevTimeout)) break;
        uint8_t* dK = gen_kv + (size_t)s * kStageBytes;
        uint8_t* dV = dK + kTileBytes;
        const int j0 = (tile0 + it) * kTile;
        mbar_arrive_expect_tx(&bar_kv_full[s], kStageBytes);
        tma_load_4d(dK, &tmK, &bar_kv_full[s], 0, j0, h, b);
        tma_load_4d(dK + kBoxBytes, &tmK, &bar_kv_full[s], 64, j0, h, b);
        tma_load_4d(dV, &tmV, &bar_kv_full[s], 0, j0, h, b);
        tma_load_4d(dV + kBoxBytes, &tmV, &bar_kv_full[s], 64, j0, h, b);
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && T > 0) {
      bool ok = mbar_wait(&bar_const_full, 0, &abort_flag, dev_status, kDevTimeout);
      const uint64_t ones_desc = make_smem_desc(sOnes, 16, 0);   // every 8-row group reads the same block
      const uint64_t aug_s = kmajor_desc(sAug), aug_c = kmajor_desc(sAug + 32u);
      for (int it = 0; ok && it < T; ++it) {
        const int s = it & 1;
        if (!mbar_wait(&bar_kv_full[s], (it >> 1) & 1, &abort_flag, dev_status, kDevTimeout)) break;
        if (it >= 2 && !mbar_wait(&bar_acc_empty[s], ((it >> 1) - 1) & 1, &abort_flag, dev_status, kDevTimeout)) break;
        tc_fence_after();
        const uint32_t sK = sKV + (uint32_t)s * kStageBytes, sV = sK + kTileBytes;
        const uint32_t tS = tmem + (uint32_t)s * 256u, tC = tS + 128u;
        mma_tile_kk(tS, sK, sQ, false);                       // S^T = K Q^T
        umma_ss(tS, ones_desc, aug_s, kIdescKK, true);        //   + row constant
        mma_tile_kk(tC, sV, sO, false);                       // C^T = V (-2 O)^T
        umma_ss(tC, ones_desc, aug_c, kIdescKK, true);        //   + ||o||^2
        umma_commit(&bar_acc_full[s]);
        umma_commit(&bar_kv_empty[s]);
      }
    }
  } else {
    // ---------------- epilogue: thread = token, warpgroup = 32 query rows ----------------
    const int cgp = (warp - 2) >> 2;                 // column group 0..3
    const int quad = warp & 3;                       // TMEM lane quarter this warp may touch
    const int t = quad * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
    const float neg_c2 = -scale * kLog2e;
    const float heavy_thr = log2f(1.f / kHeavyA) / neg_c2;   // S' above this <=> A > kHeavyA
    const float alpha = 1.f - ema_decay;                     // > 0 on this path
    // Eq. 9 over a run of consecutive window positions i_a..i_b as a Horner chain H = sum c_i I_i decay^(i_b - i),
    // c_0 = 1/alpha (the seed), c_i = 1: the run contributes alpha * decay^(w-1-i_b) * H.  Even and odd columns
    // of a run are chained separately in decay^2 (one packed FMA per column pair): H = decay * H_even + H_odd.
    constexpr int kRun = kW < 32 ? kW : 32;                  // columns of one run inside this warpgroup
    const int i_first = (cgp * 32) % kW;
    const float seed_coef = (i_first == 0) ? 1.f / alpha : 1.f;
    const float fin_scale = alpha * powf(ema_decay, (float)(kW - 1 - (i_first + kRun - 1))) / (float)kG;
    const f32x2 d2 = f2_make(ema_decay * ema_decay, ema_decay * ema_decay);
    const f32x2 nc2 = f2_make(neg_c2, neg_c2), m1 = f2_make(-1.f, -1.f), tiny2 = f2_make(1e-36f, 1e-36f);
    const float* O_head = O_f32 + (long long)bh * kRows * kHeadDim;
    const __nv_bfloat16* V_head = V + (long long)b * vsb + (long long)h * vsh;
    const float* vn_head = vnorm + (long long)bh * n_kv;
    float* I_head = I_hat + (long long)bh * n;
    bool ok = true;
    float vn_next = 0.f;
    if (T > 0) {
      const int j = tile0 * kTile + t;
      vn_next = (j < n) ? vn_head[j] : 1.f;
    }

    for (int it = 0; it < T; ++it) {
      const int s = it & 1;
      const uint32_t par = (uint32_t)(it >> 1) & 1u;
      const float vn = vn_next;
      if (it + 1 < T) {   // next tile's ||v||^2, well ahead of its use
        const int jn = (tile0 + it + 1) * kTile + t;
        vn_next = (jn < n) ? vn_head[jn] : 1.f;
      }
      // The shares of the previous tile are summed in a fixed order by warpgroup 0 once all sixteen warps have
      // stored theirs.  A slot of `red` is rewritten four tiles later, which the two accumulator buffers only
      // allow after every warp has moved past this point.
      if (it > 0 && cgp == 0) {
        const int rs = (it - 1) & 3;
        ok = ok && mbar_wait(&bar_red_full[rs], (uint32_t)((it - 1) >> 2) & 1u, &abort_flag, dev_status, kDevTimeout);
        const int jp = (tile0 + it - 1) * kTile + t;
        if (ok && jp < n) I_head[jp] = (red[rs][0][t] + red[rs][1][t]) + (red[rs][2][t] + red[rs][3][t]);
      }
      ok = ok && mbar_wait(&bar_acc_full[s], par, &abort_flag, dev_status, kDevTimeout);
      float tot = 0.f;
      if (ok) {
        tc_fence_after();
        const int j = (tile0 + it) * kTile + t;
        const uint32_t tS = tmem + (uint32_t)s * 256u + lane_base + (uint32_t)cgp * 32u, tC = tS + 128u;
        // ||o - v||^2 = C' + ||v||^2 is formed with ||v||^2 raised by 2^-16 of itself: a bias of ~1e-5 that keeps
        // the sum positive when the expansion cancels, so that no clamp is needed.
        const float vnb = vn * 1.0000152587890625f;
        const f32x2 vn2 = f2_make(vnb, vnb);
        f32x2 h2 = f2_make(0.f, 0.f);
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          float sv[16], cv[16];
          float I[16];
          tmem_ld16(tS + c * 16, sv);
          tmem_ld16(tC + c * 16, cv);
          tmem_wait_ld();
          float smax = sv[0];
#pragma unroll
          for (int u = 1; u < 16; ++u) smax = fmaxf(smax, sv[u]);
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const f32x2 nt = f2_mul(f2_make(sv[2 * q], sv[2 * q + 1]), nc2);
            const f32x2 um = f2_add(f2_make(ex2_approx(f2_lo(nt)), ex2_approx(f2_hi(nt))), m1);   // 1/A - 1
            const f32x2 x = f2_add(f2_make(cv[2 * q], cv[2 * q + 1]), vn2);                       // ||o - v||^2
            const f32x2 bq = f2_fma(f2_mul(x, um), um, tiny2);                                    // x (1/A - 1)^2
            const f32x2 Iq = f2_mul(x, f2_make(rsqrt_approx(f2_lo(bq)), rsqrt_approx(f2_hi(bq))));
            I[2 * q] = f2_lo(Iq);
            I[2 * q + 1] = f2_hi(Iq);
          }
          if (smax > heavy_thr && j < n) {   // rare: exact distance where the attention weight is large
#pragma unroll
            for (int u = 0; u < 16; ++u) {
              if (sv[u] > heavy_thr) {
                const float um = ex2_approx(sv[u] * neg_c2) - 1.f;
                const float x = exact_dist2(O_head + (cgp * 32 + c * 16 + u) * kHeadDim, V_head + (long long)j * vsn);
                I[u] = x * rsqrt_approx(fmaf(x * um, um, 1e-36f));
              }
            }
          }
          if ((c * 16) % kRun == 0) I[0] *= seed_coef;
#pragma unroll
          for (int q = 0; q < 8; ++q) h2 = f2_fma(h2, d2, f2_make(I[2 * q], I[2 * q + 1]));
          if ((c * 16 + 16) % kRun == 0) {   // end of a run
            tot += fmaf(f2_lo(h2), ema_decay, f2_hi(h2));
            h2 = f2_make(0.f, 0.f);
          }
        }
        tc_fence_before();
      }
      red[it & 3][cgp][t] = tot * fin_scale;
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&bar_acc_empty[s]);
        mbar_arrive(&bar_red_full[it & 3]);
      }
    }
    if (T > 0 && cgp == 0) {
      const int rs = (T - 1) & 3;
      ok = ok && mbar_wait(&bar_red_full[rs], (uint32_t)((T - 1) >> 2) & 1u, &abort_flag, dev_status, kDevTimeout);
      const int jl = (tile0 + T - 1) * kTile + t;
      if (ok && jl < n) I_head[jl] = (red[rs][0][t] + red[rs][1][t]) + (red[rs][2][t] + red[rs][3][t]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

constexpr size_t kP1Smem = (1 + kP1KSlots + kP1VSlots) * kTileBytes + 1024;   // Q + K ring + V ring + slack
constexpr size_t kP2Smem = 2 * kTileBytes + kAugBytes + kOnesBytes + 2 * kStageBytes + 1024;   // + alignment slack

}  // namespace

bool tc_supported(const Problem& p) {
  if (p.dtype != RESTKV_BF16 || p.d != kHeadDim || p.R != kRows) return false;
  if (p.w != 16 && p.w != 32 && p.w != 64 && p.w != 128) return false;
  return true;
}

cudaError_t tc_init(void** state) {
  *state = nullptr;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
  e = cudaFuncSetAttribute(tc_pass1_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kP1Smem);
  if (e != cudaSuccess) return e;
  cudaFuncSetAttribute(tc_pass2_kernel<16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kP2Smem);
  cudaFuncSetAttribute(tc_pass2_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kP2Smem);
  cudaFuncSetAttribute(tc_pass2_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kP2Smem);
  e = cudaFuncSetAttribute(tc_pass2_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kP2Smem);
  if (e != cudaSuccess) return e;
  static TcState the_state;
  the_state.encode = (EncodeTiledFn)fn;
  *state = &the_state;
  return cudaSuccess;
}

cudaError_t launch_tc_pass1(void* state, const Problem& p, const Workspace& ws, const void* Q, const void* K,
                            const void* V, unsigned int* dev_status, cudaStream_t st) {
  TcState* ts = (TcState*)state;
  CUtensorMap tmQ, tmK, tmV;
  if (!make_rows_map(ts, &tmQ, Q, p.BH) || !make_kv_map(ts, &tmK, K, p, p.ksb, p.ksh, p.ksn) ||
      !make_kv_map(ts, &tmV, V, p, p.vsb, p.vsh, p.vsn))
    return cudaErrorInvalidValue;
  dim3 grid(ws.splits, p.BH);
  tc_pass1_kernel<<<grid, kP1Threads, kP1Smem, st>>>(tmQ, tmK, tmV, p.Hkv, p.n, p.n_kv, p.w, p.scale, ws.splits,
                                                     ws.part_m, ws.part_l, ws.part_O, ws.vnorm, dev_status);
  return cudaGetLastError();
}

cudaError_t launch_tc_pass2(void* state, const Problem& p, const Workspace& ws, const void* Q, const void* K,
                            const void* V, float ema_decay, unsigned int* dev_status, cudaStream_t st) {
  TcState* ts = (TcState*)state;
  CUtensorMap tmQ, tmO, tmAug, tmK, tmV;
  if (!make_rows_map(ts, &tmQ, Q, p.BH) || !make_rows_map(ts, &tmO, ws.O_m2, p.BH) ||
      !make_aug_map(ts, &tmAug, ws.aug, p.BH) || !make_kv_map(ts, &tmK, K, p, p.ksb, p.ksh, p.ksn) ||
      !make_kv_map(ts, &tmV, V, p, p.vsb, p.vsh, p.vsn))
    return cudaErrorInvalidValue;
  dim3 grid(ws.splits, p.BH);
#define RESTKV_P2(W)                                                                                              \
  tc_pass2_kernel<W><<<grid, kP2Threads, kP2Smem, st>>>(tmQ, tmO, tmAug, tmK, tmV, p.Hkv, p.n, p.scale, ema_decay, \
                                                        ws.splits, ws.O_f32, (const __nv_bfloat16*)V, p.vsb,      \
                                                        p.vsh, p.vsn, ws.vnorm, p.n_kv, ws.I_hat, dev_status)
  switch (p.w) {
    case 16: RESTKV_P2(16); break;
    case 32: RESTKV_P2(32); break;
    case 64: RESTKV_P2(64); break;
    case 128: RESTKV_P2(128); break;
    default: return cudaErrorInvalidValue;
  }
#undef RESTKV_P2
  return cudaGetLastError();
}

}  // namespace restkv
