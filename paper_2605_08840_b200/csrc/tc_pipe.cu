// Head-pipelined tensor-core score kernel for sm_100a (bf16, head_dim 128, w * group = 128 query rows).
//
// One persistent CTA per SM.  The CTAs of a group walk through the group's (batch, KV head) pairs one after the
// other, every CTA owning the same share of the 64-token sub-tiles of every head.  Inside a CTA two teams run side
// by side, each a small warp-specialised pipeline of its own (a TMA thread, an MMA thread, worker warps):
//
//   team A (Eq. 3)     head h+1:  S = Q K^T, online softmax, O += P V over the CTA's sub-tiles, read from DRAM;
//                                 ||v_j||^2 and the per-sub-tile row maxima as side outputs; the CTA's partial
//                                 (m, l, O) goes to global memory at the end of the head
//   team C (Eq. 7-9)   head h:    waits until every CTA of the group has written its partial of head h, merges a
//                                 share of them, waits for the other CTAs' shares, then S' = Q K^T and
//                                 C' = (-2 O) V^T over the same sub-tiles (now served by L2), the indicator, the
//                                 temporal weights of Eq. 9, the mean over the query heads of the group
//
// so K and V cross DRAM once, and the exp2 / rsqrt work of the indicator runs under the DRAM time of the next
// head.  Both teams keep the query rows in the tensor-memory lanes.  Team C holds Q and -2 bf16(O) in tensor memory
// (A operands); its per-row constants live in registers, and the sum over the 128 query rows is taken with the
// 16x256b tensor-memory load shape (four rows per thread) followed by three shuffle rounds.
//
// Tensor memory (512 columns): Q_C | O'_C | O_A (128) | S_A (2 x 64) | S'_C | C'_C.
// Shared memory: Q_A (32 KB), team A's K ring (3 x 16 KB) and V ring (4 x 16 KB), team C's K and V rings (2 x 16 KB
// each).  mbarrier phases and ring positions run on from head to head; nothing is re-initialised between heads.
// Every wait is bounded: one that runs out sets the sticky timeout bit, every role of the CTA stops issuing work,
// waits (bounded) for what it already issued, and the CTA releases its tensor memory and returns.
#include "tc_common.cuh"

namespace restkv {

namespace {

constexpr int kSub = 64;                          // tokens per sub-tile
constexpr uint32_t kSubBox = 64 * 64 * 2;         // one [64 rows x 64 bf16] TMA box
constexpr uint32_t kSubBytes = 2 * kSubBox;       // a [64 x 128] bf16 sub-tile
constexpr int kKRing = 3, kVRing = 4, kCRing = 2;
constexpr int kCtrlWarps = 8;                     // 0 TMA A, 1 MMA A, 2-3 ||v||^2, 4 TMA C, 5 MMA C, 6-7 idle
constexpr int kAWarps = 4, kCWarps = 8;
constexpr int kFirstA = kCtrlWarps, kFirstC = kCtrlWarps + kAWarps;
constexpr int kPThreads = (kCtrlWarps + kAWarps + kCWarps) * 32;
// registers: 96 per thread at launch (640 threads); the control warps shrink to 32, the workers grow to 136
constexpr int kPRegsLaunch = 96, kPRegsControl = 32, kPRegsWorker = 136;
static_assert(kCtrlWarps * kPRegsControl + (kAWarps + kCWarps) * kPRegsWorker <=
                  (kCtrlWarps + kAWarps + kCWarps) * kPRegsLaunch,
              "the register split must fit the pool the CTA is launched with");
static_assert(kFirstC % 4 == 0 && kFirstA % 4 == 0, "worker warps must line up with the tensor-memory lane quarters");

// tensor-memory columns
constexpr uint32_t kTQc = 0, kTOc = 64, kTOa = 128, kTSa = 256, kTSc = 384, kTCc = 448;
// shared memory (offsets from the 1024-aligned base)
constexpr uint32_t kOffQa = 0, kOffKa = kTileBytes, kOffVa = kOffKa + kKRing * kSubBytes,
                   kOffKc = kOffVa + kVRing * kSubBytes, kOffVc = kOffKc + kCRing * kSubBytes,
                   kPipeSmem = kOffVc + kCRing * kSubBytes;
constexpr size_t kPSmem = kPipeSmem + 1024;

constexpr uint32_t kIdesc64KK = make_idesc_bf16(128, 64, false);   // [128 x 64] += A B^T, both K-major
constexpr float kShift = 32.f;          // the epilogue works on (1/A - 1) / (c * 2^32): keeps x (1/A - 1)^2 in range
constexpr long long kDrainCycles = 4000000000ll;   // bound of the waits for work already issued, at exit

struct PipeArgs {
  int Hkv, BH, n, n_kv, w;
  float scale, ema_decay;
  int groups, cpg;                   // CTA groups and CTAs per group
  int vn_stride;                     // floats per head in vnorm (n_kv rounded up to whole sub-tiles)
  long long wait_limit;              // SM clocks a wait may last
  const __nv_bfloat16* Q;            // [BH, 128, 128]
  const __nv_bfloat16* V;
  long long vsb, vsh, vsn;
  float* part_m;                     // [2, CTA, 128]       partial softmax results, two slots used in turn
  float* part_l;                     // [2, CTA, 128]
  float* part_O;                     // [2, CTA, 128 (dim), 128 (row)]
  float* O_f32;                      // [BH, 128, 128]
  float* row_M2;                     // [BH, 128]  m * log2e + log2 l
  float* vnorm;                      // [BH, vn_stride]
  float* tile_max;                   // [BH, sub-tiles, 128]
  float* I_hat;                      // [BH, n]
  unsigned int* counters;            // [groups, 64]: word 0 = partials written, word 32 = merge shares done
  unsigned int* dev_status;
};

struct PipeBars {
  // team A
  uint64_t q_full, q_empty, k_full[kKRing], k_empty[kKRing], v_full[kVRing], v_empty[kVRing], s_full[2], p_full[2],
      pv_done, o_free, drain_a;
  // team C
  uint64_t kc_full[kCRing], kc_empty[kCRing], vc_full[kCRing], vc_empty[kCRing], acc_full, acc_empty, opr_ready,
      red_full[4], drain_c;
};

struct PCtx {
  uint32_t smem_base;
  uint8_t* gen;
  uint32_t tmem;
  PipeBars* B;
  int* abort_flag;
  unsigned int* dev_status;
  long long limit;
  int warp, lane;
};

__device__ __forceinline__ void named_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ unsigned int ld_acquire(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void red_release(unsigned int* p) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(1u) : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
// 16 lanes x (4 x 256 bits): thread t receives, for each group k of eight columns, rows t/4 and t/4 + 8 at columns
// 8k + 2(t%4) and 8k + 2(t%4) + 1: v[4k + 0..1] = row t/4, v[4k + 2..3] = row t/4 + 8.
__device__ __forceinline__ void tmem_ld_16x256b_x4(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.16x256b.x4.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Wait for something this thread itself set in motion (a bulk copy, an MMA), whatever the abort flag says: used
// on the way out, so that nothing is still in flight when the CTA returns.  Bounded.
__device__ __forceinline__ void wait_issued(uint64_t* bar, long long completion) {
  const uint32_t parity = (uint32_t)completion & 1u;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity))
    if (clock64() - t0 > kDrainCycles) return;
}
// Index of the last of `count` ring items (0, 1, ...) that went to slot `s` of a ring of `ring` slots; -1: none.
__device__ __forceinline__ long long last_in_slot(long long count, int s, int ring) {
  if (count <= s) return -1;
  return (count - 1) - (count - 1 - s) % ring;
}

#define PWAIT(bar, par) mbar_wait((bar), (uint32_t)(par)&1u, cx.abort_flag, cx.dev_status, kDevTimeout, cx.limit)

// Waits until *counter reaches `target`.  One thread calls it; bounded.
__device__ bool poll_counter(const PCtx& cx, const unsigned int* counter, unsigned int target) {
  const long long t0 = clock64();
  while (ld_acquire(counter) < target) {
    if (*(volatile int*)cx.abort_flag) return false;
    if (clock64() - t0 > cx.limit) {
      *(volatile int*)cx.abort_flag = 1;
      atomicOr(cx.dev_status, kDevTimeout);
      return false;
    }
  }
  return true;
}

// Temporal weight of Eq. 9 (closed form of the recursion seeded with the oldest query) of window position i,
// divided by the group size: c_0 = decay^(w-1), c_i = (1 - decay) decay^(w-1-i).
__device__ __forceinline__ float row_weight(int row, int w, float decay) {
  const int i = row % w;
  const float p = powf(decay, (float)(w - 1 - i));   // powf(0, 0) = 1
  return (i == 0 ? p : (1.f - decay) * p) * ((float)w / (float)kRows);
}

struct Share {
  int group, rank, tile0, T1, T2;
};

// ------------------------------------------------------------------------------------------------
// Team A, warp 0: K and V sub-tiles of every head of the group into the rings, Q of each head into Q_A.
__device__ void tma_a_main(const PCtx& cx, const PipeArgs& a, const Share& sh, const CUtensorMap* tmQ,
                           const CUtensorMap* tmK, const CUtensorMap* tmV) {
  PipeBars* B = cx.B;
  long long kN = 0, vN = 0, qN = 0;   // K sub-tiles, V sub-tiles and Q tiles requested so far
  bool ok = true;
  for (int bh = sh.group; bh < a.BH && ok && sh.T1 > 0; bh += a.groups) {
    const int b = bh / a.Hkv, h = bh % a.Hkv;
    // Q_A may be overwritten once every S MMA of the previous head has read it
    if (qN > 0 && !PWAIT(&B->q_empty, qN - 1)) break;
    mbar_arrive_expect_tx(&B->q_full, kTileBytes);
    tma_load_3d(cx.gen + kOffQa, tmQ, &B->q_full, 0, 0, bh);
    tma_load_3d(cx.gen + kOffQa + kBoxBytes, tmQ, &B->q_full, 64, 0, bh);
    ++qN;
    for (int t = 0; t < sh.T1; ++t) {
      const int j0 = (sh.tile0 + t) * kSub;
      const int ks = (int)(kN % kKRing), vs = (int)(vN % kVRing);
      if (kN >= kKRing && !PWAIT(&B->k_empty[ks], kN / kKRing - 1)) { ok = false; break; }
      uint8_t* dK = cx.gen + kOffKa + (uint32_t)ks * kSubBytes;
      mbar_arrive_expect_tx(&B->k_full[ks], kSubBytes);
      tma_load_4d(dK, tmK, &B->k_full[ks], 0, j0, h, b);
      tma_load_4d(dK + kSubBox, tmK, &B->k_full[ks], 64, j0, h, b);
      ++kN;
      if (vN >= kVRing && !PWAIT(&B->v_empty[vs], vN / kVRing - 1)) { ok = false; break; }
      uint8_t* dV = cx.gen + kOffVa + (uint32_t)vs * kSubBytes;
      mbar_arrive_expect_tx(&B->v_full[vs], kSubBytes);
      tma_load_4d(dV, tmV, &B->v_full[vs], 0, j0, h, b);
      tma_load_4d(dV + kSubBox, tmV, &B->v_full[vs], 64, j0, h, b);
      ++vN;
    }
  }
  // nothing this thread requested may still be on its way into shared memory when the CTA returns
  for (int s = 0; s < kKRing; ++s) {
    const long long last = last_in_slot(kN, s, kKRing);
    if (last >= 0) wait_issued(&B->k_full[s], last / kKRing);
  }
  for (int s = 0; s < kVRing; ++s) {
    const long long last = last_in_slot(vN, s, kVRing);
    if (last >= 0) wait_issued(&B->v_full[s], last / kVRing);
  }
  if (qN > 0) wait_issued(&B->q_full, qN - 1);
}

// Team A, warp 1: S(t) = Q K_t^T into S_A[t & 1], then O += P(t-1) V_{t-1}.
__device__ void mma_a_main(const PCtx& cx, const PipeArgs& a, const Share& sh) {
  PipeBars* B = cx.B;
  const uint32_t tmem = cx.tmem;
  long long sI = 0;   // sub-tiles whose S has been issued (all heads)
  int hk = 0;
  bool ok = true;
  for (int bh = sh.group; bh < a.BH && ok; bh += a.groups, ++hk) {
    if (sh.T1 == 0) continue;
    if (!PWAIT(&B->q_full, hk)) break;
    const long long s0 = sI;
    for (int t = 0; t <= sh.T1 && ok; ++t) {
      if (t < sh.T1) {
        const long long it = s0 + t;
        const int ks = (int)(it % kKRing), buf = (int)(it & 1);
        if (!PWAIT(&B->k_full[ks], it / kKRing)) { ok = false; break; }
        tc_fence_after();
        // S_A[buf] held P of sub-tile it - 2, whose O += P V was issued earlier: MMAs execute in issue order
        const uint32_t sQ = cx.smem_base + kOffQa, sK = cx.smem_base + kOffKa + (uint32_t)ks * kSubBytes;
#pragma unroll
        for (int k = 0; k < 8; ++k)
          umma_ss(tmem + kTSa + (uint32_t)buf * 64u, kmajor_desc(sQ + (uint32_t)(k >> 2) * kBoxBytes + (uint32_t)(k & 3) * 32u),
                  kmajor_desc(sK + (uint32_t)(k >> 2) * kSubBox + (uint32_t)(k & 3) * 32u), kIdesc64KK, k > 0);
        umma_commit(&B->s_full[buf]);
        umma_commit(&B->k_empty[ks]);
        if (t == sh.T1 - 1) umma_commit(&B->q_empty);
        ++sI;
      }
      if (t >= 1) {
        const long long pt = s0 + t - 1;
        const int vs = (int)(pt % kVRing), buf = (int)(pt & 1);
        if (!PWAIT(&B->p_full[buf], pt >> 1)) { ok = false; break; }
        if (!PWAIT(&B->v_full[vs], pt / kVRing)) { ok = false; break; }
        // the first O += P V of a head overwrites O_A: the previous head's must have been read out
        if (t == 1 && hk > 0 && !PWAIT(&B->o_free, hk - 1)) { ok = false; break; }
        tc_fence_after();
        const uint32_t vaddr = cx.smem_base + kOffVa + (uint32_t)vs * kSubBytes;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          // A = P in tensor memory (16 tokens = 8 packed columns per K step), B = V sub-tile, MN-major
          const uint64_t bdesc = make_smem_desc(vaddr + (uint32_t)k * 2048u, kSubBox, 1024);
          umma_ts(tmem + kTOa, tmem + kTSa + (uint32_t)buf * 64u + (uint32_t)k * 8u, bdesc, kIdescKMN, t > 1 || k > 0);
        }
        umma_commit(&B->pv_done);
        umma_commit(&B->v_empty[vs]);
      }
    }
  }
  umma_commit(&B->drain_a);
  wait_issued(&B->drain_a, 0);
}

// Team A, warps 2 and 3: ||v_j||^2 of every token from the V sub-tiles in shared memory (even / odd sub-tiles;
// a lane takes two rows).
__device__ void vnorm_main(const PCtx& cx, const PipeArgs& a, const Share& sh) {
  PipeBars* B = cx.B;
  const int vg = cx.warp - 2, lane = cx.lane;
  long long vI = 0;
  bool ok = true;
  for (int bh = sh.group; bh < a.BH && ok; bh += a.groups) {
    float* vn_head = a.vnorm + (long long)bh * a.vn_stride;
    for (int t = 0; t < sh.T1 && ok; ++t, ++vI) {
      const int vs = (int)(vI % kVRing);
      // both warps wait for every sub-tile, so that neither can fall a whole phase behind a slot's barrier
      ok = PWAIT(&B->v_full[vs], vI / kVRing);
      if (!ok || (int)(vI & 1) != vg) continue;
      const uint8_t* vt = cx.gen + kOffVa + (uint32_t)vs * kSubBytes;
      float vn[2];
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int row = rr * 32 + lane;
        float2 acc = make_float2(0.f, 0.f);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          // 16-byte chunk c of row r of a 128-byte-swizzled box sits at chunk c ^ (r & 7)
          const uint8_t* rowp = vt + half * kSubBox + (row >> 3) * 1024 + (row & 7) * 128;
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
        vn[rr] = acc.x + acc.y;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&B->v_empty[vs]);
      const int j0 = (sh.tile0 + t) * kSub;
      vn_head[j0 + lane] = vn[0];          // rows past n_kv are zero-filled by TMA: the padded array takes zeros
      vn_head[j0 + 32 + lane] = vn[1];
    }
  }
}

// Team A, warps 8-11: online softmax, thread = query row, 64 tokens per sub-tile.
__device__ void softmax_main(const PCtx& cx, const PipeArgs& a, const Share& sh) {
  PipeBars* B = cx.B;
  const int lane = cx.lane, quad = cx.warp & 3;
  const int row = quad * 32 + lane;
  const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
  const uint32_t tO = cx.tmem + kTOa + lane_base;
  const int i_q = row % a.w;
  const float c2 = a.scale * kLog2e;
  const int n = a.n, n_kv = a.n_kv;
  const int nt_all = (n_kv + kSub - 1) / kSub;
  const int cta = sh.group * a.cpg + sh.rank, n_cta = a.groups * a.cpg;
  unsigned int* counter_a = a.counters + (size_t)sh.group * 64;
  const unsigned int* counter_b = counter_a + 32;
  long long sI = 0;
  int hk = 0;
  bool ok = true;
  for (int bh = sh.group; bh < a.BH; bh += a.groups, ++hk) {
    float m_ref = -INFINITY;
    float2 l2 = make_float2(0.f, 0.f);
    for (int t = 0; t < sh.T1; ++t, ++sI) {
      const int buf = (int)(sI & 1);
      ok = ok && PWAIT(&B->s_full[buf], sI >> 1);
      if (!ok) continue;
      tc_fence_after();
      const uint32_t tS = cx.tmem + kTSa + (uint32_t)buf * 64u + lane_base;
      const int j0 = (sh.tile0 + t) * kSub;
      float s[64];
      tmem_ld16(tS, s);
      tmem_ld16(tS + 16, s + 16);
      tmem_ld16(tS + 32, s + 32);
      tmem_ld16(tS + 48, s + 48);
      tmem_wait_ld();
      if (j0 + kSub > n) {   // rows past the scored prefix: the window's own rows (causal) or padding
#pragma unroll
        for (int u = 0; u < 64; ++u) {
          const int j = j0 + u;
          const bool vis = (j < n_kv) && (j < n || (j - n) <= i_q);
          s[u] = vis ? s[u] : -INFINITY;
        }
      }
      float tmax = s[0];
#pragma unroll
      for (int u = 1; u < 64; ++u) tmax = fmaxf(tmax, s[u]);
      const float m_tile = tmax * c2;
      a.tile_max[((long long)bh * nt_all + sh.tile0 + t) * kRows + row] = m_tile;
      const bool need = m_tile > m_ref + kRescaleThreshold;   // also true for the first visible entries
      float factor = 1.f;
      if (need) {
        factor = ex2_approx(m_ref - m_tile);   // 0 when m_ref = -inf
        l2.x *= factor;
        l2.y *= factor;
        m_ref = m_tile;
      }
      if (t > 0 && __any_sync(0xffffffffu, need)) {
        // O_A is rescaled between O += P V of the previous sub-tile (awaited here) and that of this one (which
        // needs the P this thread has yet to write)
        ok = PWAIT(&B->pv_done, sI - 1);
        if (!ok) continue;
        tc_fence_after();
#pragma unroll
        for (int c = 0; c < 8; ++c) {
          float o[16];
          tmem_ld16(tO + c * 16, o);
          tmem_wait_ld();
#pragma unroll
          for (int u = 0; u < 16; ++u) o[u] *= factor;
          tmem_st16(tO + c * 16, reinterpret_cast<const uint32_t*>(o));
        }
      }
      const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
      const float2 c22 = make_float2(c2, c2), nm2 = make_float2(-m_use, -m_use);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t packed[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float2 e = ffma2(make_float2(s[c * 16 + 2 * u], s[c * 16 + 2 * u + 1]), c22, nm2);
          const float2 pp = make_float2(ex2_approx(e.x), ex2_approx(e.y));
          l2 = fadd2(l2, pp);
          packed[u] = pack_bf16x2(pp.x, pp.y);
        }
        tmem_st8(tS + c * 8, packed);   // P overwrites the first 32 columns of S (all of S is in registers)
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&B->p_full[buf]);
    }
    // ---- end of the head: this CTA's partial (m, l, O) ----
    if (sh.T1 > 0 && ok) {
      ok = PWAIT(&B->pv_done, sI - 1);
      if (ok) tc_fence_after();
    }
    // the slot was last read by the merge of the head two before this one
    if (hk >= 2) {
      if (threadIdx.x == kFirstA * 32) {
        if (ok && !poll_counter(cx, counter_b, (unsigned int)(hk - 1) * (unsigned int)a.cpg)) { /* abort flag set */ }
      }
      named_sync(1, kAWarps * 32);
      ok = ok && (*(volatile int*)cx.abort_flag == 0);
    }
    const long long slot = (long long)(hk & 1) * n_cta + cta;
    const bool have = ok && sh.T1 > 0;
    if (ok) {
      a.part_m[slot * kRows + row] = have ? m_ref : -INFINITY;
      a.part_l[slot * kRows + row] = have ? l2.x + l2.y : 0.f;
      float* Op = a.part_O + slot * kRows * kHeadDim + row;
#pragma unroll
      for (int c = 0; c < 8; ++c) {
        float o[16];
        if (have) {
          tmem_ld16(tO + c * 16, o);
          tmem_wait_ld();
        } else {
#pragma unroll
          for (int u = 0; u < 16; ++u) o[u] = 0.f;
        }
#pragma unroll
        for (int u = 0; u < 16; ++u) Op[(c * 16 + u) * kRows] = o[u];
      }
    }
    tc_fence_before();
    mbar_arrive(&B->o_free);
    named_sync(1, kAWarps * 32);
    if (threadIdx.x == kFirstA * 32) red_release(counter_a);   // arrives even after a failure: peers must not wait for it
  }
}

// ------------------------------------------------------------------------------------------------
// Team C, warp 4: K and V sub-tiles of the scored rows of every head, in the order team A read them.
__device__ void tma_c_main(const PCtx& cx, const PipeArgs& a, const Share& sh, const CUtensorMap* tmK,
                           const CUtensorMap* tmV) {
  PipeBars* B = cx.B;
  const uint64_t pol = policy_evict_first();   // the second and last read of these lines
  long long kN = 0, vN = 0;
  bool ok = true;
  for (int bh = sh.group; bh < a.BH && ok; bh += a.groups) {
    const int b = bh / a.Hkv, h = bh % a.Hkv;
    for (int t = 0; t < sh.T2; ++t) {
      const int j0 = (sh.tile0 + t) * kSub;
      const int s = (int)(kN % kCRing);
      if (kN >= kCRing && !PWAIT(&B->kc_empty[s], kN / kCRing - 1)) { ok = false; break; }
      uint8_t* dK = cx.gen + kOffKc + (uint32_t)s * kSubBytes;
      mbar_arrive_expect_tx(&B->kc_full[s], kSubBytes);
      tma_load_4d_hint(dK, tmK, &B->kc_full[s], 0, j0, h, b, pol);
      tma_load_4d_hint(dK + kSubBox, tmK, &B->kc_full[s], 64, j0, h, b, pol);
      ++kN;
      if (vN >= kCRing && !PWAIT(&B->vc_empty[s], vN / kCRing - 1)) { ok = false; break; }
      uint8_t* dV = cx.gen + kOffVc + (uint32_t)s * kSubBytes;
      mbar_arrive_expect_tx(&B->vc_full[s], kSubBytes);
      tma_load_4d_hint(dV, tmV, &B->vc_full[s], 0, j0, h, b, pol);
      tma_load_4d_hint(dV + kSubBox, tmV, &B->vc_full[s], 64, j0, h, b, pol);
      ++vN;
    }
  }
  for (int s = 0; s < kCRing; ++s) {
    const long long lk = last_in_slot(kN, s, kCRing), lv = last_in_slot(vN, s, kCRing);
    if (lk >= 0) wait_issued(&B->kc_full[s], lk / kCRing);
    if (lv >= 0) wait_issued(&B->vc_full[s], lv / kCRing);
  }
}

// Team C, warp 5: S' = Q K^T and C' = (-2 O) V^T of one sub-tile, operands A from tensor memory.
__device__ void mma_c_main(const PCtx& cx, const PipeArgs& a, const Share& sh) {
  PipeBars* B = cx.B;
  const uint32_t tmem = cx.tmem;
  long long cI = 0;
  int hk = 0;
  bool ok = true;
  for (int bh = sh.group; bh < a.BH && ok; bh += a.groups, ++hk) {
    if (!PWAIT(&B->opr_ready, hk)) break;
    for (int t = 0; t < sh.T2; ++t, ++cI) {
      const int s = (int)(cI % kCRing);
      if (!PWAIT(&B->kc_full[s], cI / kCRing)) { ok = false; break; }
      if (cI > 0 && !PWAIT(&B->acc_empty, cI - 1)) { ok = false; break; }
      tc_fence_after();
      const uint32_t sK = cx.smem_base + kOffKc + (uint32_t)s * kSubBytes, sV = cx.smem_base + kOffVc + (uint32_t)s * kSubBytes;
#pragma unroll
      for (int k = 0; k < 8; ++k)
        umma_ts(tmem + kTSc, tmem + kTQc + (uint32_t)k * 8u,
                kmajor_desc(sK + (uint32_t)(k >> 2) * kSubBox + (uint32_t)(k & 3) * 32u), kIdesc64KK, k > 0);
      umma_commit(&B->kc_empty[s]);
      if (!PWAIT(&B->vc_full[s], cI / kCRing)) { ok = false; break; }
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < 8; ++k)
        umma_ts(tmem + kTCc, tmem + kTOc + (uint32_t)k * 8u,
                kmajor_desc(sV + (uint32_t)(k >> 2) * kSubBox + (uint32_t)(k & 3) * 32u), kIdesc64KK, k > 0);
      umma_commit(&B->vc_empty[s]);
      umma_commit(&B->acc_full);
    }
  }
  umma_commit(&B->drain_c);
  wait_issued(&B->drain_c, 0);
}

// The partials of one (lane quarter, group of four output dims) pair are merged by `s` warps (warp `sub` of the pair
// takes partials sub, sub + s, ...; lane = row of the quarter), whose results meet in shared memory and are added in
// a fixed order.  pair < 0: this warp has none (it still takes part in the synchronisation).
__device__ void merge_pair(const PCtx& cx, const PipeArgs& a, int bh, int group, int slot_base, int pair, int sub, int s,
                           int cw, float (*xch)[32][6]) {
  const int lane = cx.lane;
  float m = -INFINITY, l = 0.f;
  float acc[4] = {0.f, 0.f, 0.f, 0.f};
  const int q = pair >> 5, d4 = pair & 31, row = q * 32 + lane;
  if (pair >= 0) {
    constexpr int kBatch = 8;
#pragma unroll 1
    for (int p0 = sub; p0 < a.cpg; p0 += kBatch * s) {
      float mp[kBatch], lp[kBatch], v[kBatch][4];
#pragma unroll
      for (int k = 0; k < kBatch; ++k) {
        const int p = p0 + k * s;
        const bool in = p < a.cpg;
        const long long ci = (long long)slot_base + (long long)group * a.cpg + (in ? p : p0);
        mp[k] = in ? __ldcg(a.part_m + ci * kRows + row) : -INFINITY;
        lp[k] = __ldcg(a.part_l + ci * kRows + row);
        const float* Op = a.part_O + ci * kRows * kHeadDim + (long long)(d4 * 4) * kRows + row;
#pragma unroll
        for (int e = 0; e < 4; ++e) v[k][e] = __ldcg(Op + e * kRows);
      }
#pragma unroll
      for (int k = 0; k < kBatch; ++k) {
        const float m_new = fmaxf(m, mp[k]);
        const float s_old = (m == -INFINITY) ? 0.f : ex2_approx(m - m_new);
        const float s_p = (mp[k] == -INFINITY) ? 0.f : ex2_approx(mp[k] - m_new);   // an empty partial weighs 0
        l = l * s_old + lp[k] * s_p;
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[e] = acc[e] * s_old + v[k][e] * s_p;
        m = m_new;
      }
    }
    if (s > 1) {
#pragma unroll
      for (int e = 0; e < 4; ++e) xch[cw][lane][e] = acc[e];
      xch[cw][lane][4] = l;
      xch[cw][lane][5] = m;
    }
  }
  named_sync(2, kCWarps * 32);
  if (pair < 0 || sub != 0) return;
  if (s > 1) {
    float mm = m;
    for (int k = 1; k < s; ++k) mm = fmaxf(mm, xch[cw + k][lane][5]);
    const float s0 = (m == -INFINITY) ? 0.f : ex2_approx(m - mm);
#pragma unroll
    for (int e = 0; e < 4; ++e) acc[e] *= s0;
    l *= s0;
    for (int k = 1; k < s; ++k) {
      const float mk = xch[cw + k][lane][5];
      const float sk = (mk == -INFINITY) ? 0.f : ex2_approx(mk - mm);
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[e] = fmaf(xch[cw + k][lane][e], sk, acc[e]);
      l = fmaf(xch[cw + k][lane][4], sk, l);
    }
    m = mm;
  }
  const float inv_l = 1.f / l;
  const long long ri = (long long)bh * kRows + row;
  *reinterpret_cast<float4*>(a.O_f32 + ri * kHeadDim + d4 * 4) =
      make_float4(acc[0] * inv_l, acc[1] * inv_l, acc[2] * inv_l, acc[3] * inv_l);
  if (d4 == 0) a.row_M2[ri] = m + log2f(l);   // A = exp2(s * scale * log2e - M2)
}

struct RowConst {
  float Mr, Dr, on, hthr;   // exponent offset, 2^-shift / c, ||bf16(o)||^2, heavy threshold on the exponent
};

// Team C, warps 12-19.
__device__ void epilogue_main(const PCtx& cx, const PipeArgs& a, const Share& sh, RowConst* rowc, float (*onp)[kRows],
                              float (*red)[4][kSub], float (*xch)[32][6]) {
  PipeBars* B = cx.B;
  const int lane = cx.lane, cw = cx.warp - kFirstC;
  const int q = cw & 3, hf = cw >> 2;
  const uint32_t quarter = (uint32_t)(q * 32) << 16;
  const int n = a.n;
  const int nt_all = (a.n_kv + kSub - 1) / kSub;
  const float neg_c2 = -a.scale * kLog2e;
  const f32x2 nc2 = f2_make(neg_c2, neg_c2), tiny2 = f2_make(1e-36f, 1e-36f);
  unsigned int* counter_a = a.counters + (size_t)sh.group * 64;
  unsigned int* counter_b = counter_a + 32;
  const int n_cta = a.groups * a.cpg;
  const bool leader = threadIdx.x == kFirstC * 32;
  const int col0 = 2 * (lane & 3);                       // this thread's two columns inside a group of eight
  const int my_col = 16 * ((lane >> 4) & 1) + 8 * ((lane >> 3) & 1) + col0 + ((lane >> 2) & 1);   // after the reduction
  const int r0 = q * 32 + (lane >> 2);                   // rows r0, r0 + 8, r0 + 16, r0 + 24
  long long cI = 0;
  int hk = 0;
  bool ok = true;
  for (int bh = sh.group; bh < a.BH; bh += a.groups, ++hk) {
    const int b = bh / a.Hkv, h = bh % a.Hkv;
    // ---- every CTA of the group has written its partial of this head ----
    if (leader && ok) poll_counter(cx, counter_a, (unsigned int)(hk + 1) * (unsigned int)a.cpg);
    named_sync(2, kCWarps * 32);
    ok = ok && (*(volatile int*)cx.abort_flag == 0);
    // ---- this CTA's share of the merge ----
    {
      const int P = sh.rank < 128 ? (127 - sh.rank) / a.cpg + 1 : 0;   // pairs rank, rank + cpg, ... below 128
      int P_max = (127) / a.cpg + 1;                                    // the busiest CTA's count (rank 0)
      int s = kCWarps;
      while (s > 1 && kCWarps / s < P_max) s >>= 1;
      const int at_once = kCWarps / s;
      for (int i0 = 0; i0 < P_max; i0 += at_once) {
        const int pi = i0 + cw / s;
        const int pair = (ok && pi < P) ? sh.rank + pi * a.cpg : -1;
        merge_pair(cx, a, bh, sh.group, (hk & 1) * n_cta, pair, cw % s, s, cw, xch);
        named_sync(2, kCWarps * 32);   // the exchange buffer is reused by the next batch of pairs
      }
    }
    if (leader) {
      red_release(counter_b);
      if (ok) poll_counter(cx, counter_b, (unsigned int)(hk + 1) * (unsigned int)a.cpg);
    }
    named_sync(2, kCWarps * 32);
    ok = ok && (*(volatile int*)cx.abort_flag == 0);
    // ---- operands of this head into tensor memory: Q and -2 bf16(O), thread = (row, half of the dims) ----
    {
      const int row = q * 32 + lane;
      const long long ri = (long long)bh * kRows + row;
      float on = 0.f;
      if (ok) {
        const float4* orow = reinterpret_cast<const float4*>(a.O_f32 + ri * kHeadDim + hf * 64);
        uint32_t pk[32];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float4 o = __ldcg(orow + i);
          const float f0 = __bfloat162float(__float2bfloat16_rn(o.x)), f1 = __bfloat162float(__float2bfloat16_rn(o.y));
          const float f2 = __bfloat162float(__float2bfloat16_rn(o.z)), f3 = __bfloat162float(__float2bfloat16_rn(o.w));
          on += (f0 * f0 + f1 * f1) + (f2 * f2 + f3 * f3);
          pk[2 * i] = pack_bf16x2(-2.f * f0, -2.f * f1);       // exact: a bf16 times two
          pk[2 * i + 1] = pack_bf16x2(-2.f * f2, -2.f * f3);
        }
        tmem_st16(cx.tmem + kTOc + quarter + (uint32_t)hf * 32u, pk);
        tmem_st16(cx.tmem + kTOc + quarter + (uint32_t)hf * 32u + 16u, pk + 16);
        const uint4* qrow = reinterpret_cast<const uint4*>(a.Q + ri * kHeadDim + hf * 64);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const uint4 u = __ldg(qrow + i);
          pk[4 * i] = u.x; pk[4 * i + 1] = u.y; pk[4 * i + 2] = u.z; pk[4 * i + 3] = u.w;
        }
        tmem_st16(cx.tmem + kTQc + quarter + (uint32_t)hf * 32u, pk);
        tmem_st16(cx.tmem + kTQc + quarter + (uint32_t)hf * 32u + 16u, pk + 16);
        tmem_wait_st();
      }
      onp[hf][row] = on;
      named_sync(2, kCWarps * 32);
      if (hf == 0) {
        const float c = row_weight(row, a.w, a.ema_decay);
        const float M2 = ok ? __ldcg(a.row_M2 + ri) : 0.f;
        RowConst rc;
        if (c > 0.f) {
          const float lc = log2f(c);
          rc.Mr = M2 - lc - kShift;
          rc.Dr = exp2f(-kShift) / c;
          rc.hthr = 3.f - lc - kShift;              // exponent below this <=> A > 1/8
        } else {                                     // weight zero: the exponent saturates and the entry adds 0
          rc.Mr = 200.f;
          rc.Dr = 0.f;
          rc.hthr = -INFINITY;
        }
        rc.on = onp[0][row] + onp[1][row];
        rowc[row] = rc;
      }
      tc_fence_before();
      named_sync(2, kCWarps * 32);
      if (lane == 0) mbar_arrive(&B->opr_ready);
    }
    // ---- per-thread constants of its four rows; the heavy test of this warp's 32 rows ----
    f32x2 Mr2[4], nDr2[4], on2[4];
    float hthr[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const RowConst rc = rowc[r0 + 8 * i];
      Mr2[i] = f2_make(rc.Mr, rc.Mr);
      nDr2[i] = f2_make(-rc.Dr, -rc.Dr);
      on2[i] = f2_make(rc.on, rc.on);
      hthr[i] = rc.hthr;
    }
    // a sub-tile needs exact distances iff some row's largest logit in it reaches M2 - 3 (A > 1/8)
    const float my_M2m3 = (ok ? __ldcg(a.row_M2 + (long long)bh * kRows + q * 32 + lane) : 0.f) - 3.f;
    const float* tm_head = a.tile_max + (long long)bh * nt_all * kRows + q * 32 + lane;
    const float* vn_head = a.vnorm + (long long)bh * a.vn_stride + hf * 32 + col0;
    const float* O_head = a.O_f32 + (long long)bh * kRows * kHeadDim;
    const __nv_bfloat16* V_head = a.V + (long long)b * a.vsb + (long long)h * a.vsh;
    float* I_head = a.I_hat + (long long)bh * n;
    float2 vn_next[4];
    float tm_next = -INFINITY;
    if (sh.T2 > 0 && ok) {
      const int j0 = sh.tile0 * kSub;
#pragma unroll
      for (int k = 0; k < 4; ++k) vn_next[k] = __ldcg(reinterpret_cast<const float2*>(vn_head + j0 + 8 * k));
      tm_next = __ldcg(tm_head + (long long)sh.tile0 * kRows);
    }
    for (int t = 0; t < sh.T2; ++t, ++cI) {
      const int j0 = (sh.tile0 + t) * kSub;
      float2 vn[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) vn[k] = vn_next[k];
      const bool heavy = __any_sync(0xffffffffu, tm_next > my_M2m3);
      if (t + 1 < sh.T2 && ok) {
#pragma unroll
        for (int k = 0; k < 4; ++k) vn_next[k] = __ldcg(reinterpret_cast<const float2*>(vn_head + j0 + kSub + 8 * k));
        tm_next = __ldcg(tm_head + (long long)(sh.tile0 + t + 1) * kRows);
      }
      // the four lane quarters' sums of the previous sub-tile, added in a fixed order
      if (t > 0 && q == 0) {
        const int rs = (int)((cI - 1) & 3);
        ok = ok && PWAIT(&B->red_full[rs], (cI - 1) >> 2);
        const int jp = j0 - kSub + hf * 32 + lane;
        if (ok && jp < n)
          I_head[jp] = ((red[rs][0][hf * 32 + lane] + red[rs][1][hf * 32 + lane]) +
                        (red[rs][2][hf * 32 + lane] + red[rs][3][hf * 32 + lane])) * exp2f(-kShift);
      }
      ok = ok && PWAIT(&B->acc_full, cI);
      f32x2 acc[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) acc[k] = f2_make(0.f, 0.f);
      if (ok) {
        tc_fence_after();
        float sv[32], cv[32];
        const uint32_t tS = cx.tmem + kTSc + quarter + (uint32_t)hf * 32u, tC = cx.tmem + kTCc + quarter + (uint32_t)hf * 32u;
        tmem_ld_16x256b_x4(tS, sv);
        tmem_ld_16x256b_x4(tS + (16u << 16), sv + 16);
        tmem_ld_16x256b_x4(tC, cv);
        tmem_ld_16x256b_x4(tC + (16u << 16), cv + 16);
        tmem_wait_ld();
        // every tensor-memory read of this sub-tile is done: the MMA thread may refill the accumulators
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&B->acc_empty);
        // ||o - v||^2 = C' + ||o||^2 + ||v||^2 with ||v||^2 raised by 2^-16 of itself: a bias of ~1e-5 that keeps
        // the sum positive when the expansion cancels, so that no clamp is needed
        f32x2 vnb[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) vnb[k] = f2_make(vn[k].x * 1.0000152587890625f, vn[k].y * 1.0000152587890625f);
        if (!heavy) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {        // row r0 + 8 i: registers 16 (i / 2) + 4 k + 2 (i % 2) + {0, 1}
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const int r = 16 * (i >> 1) + 4 * k + 2 * (i & 1);
              const f32x2 te = f2_fma(f2_make(sv[r], sv[r + 1]), nc2, Mr2[i]);
              const f32x2 um = f2_add(f2_make(ex2_approx(f2_lo(te)), ex2_approx(f2_hi(te))), nDr2[i]);
              const f32x2 x = f2_add(f2_add(f2_make(cv[r], cv[r + 1]), on2[i]), vnb[k]);
              const f32x2 bq = f2_fma(f2_mul(x, um), um, tiny2);
              const f32x2 Iq = f2_mul(x, f2_make(rsqrt_approx(f2_lo(bq)), rsqrt_approx(f2_hi(bq))));
              acc[k] = f2_add(acc[k], Iq);
            }
          }
        } else {
          // rare: some weight of this warp's rows may exceed 1/8 here; those entries take the exact distance
#pragma unroll
          for (int i = 0; i < 4; ++i) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
#pragma unroll
              for (int e = 0; e < 2; ++e) {
                const int r = 16 * (i >> 1) + 4 * k + 2 * (i & 1) + e;
                const float te = fmaf(sv[r], neg_c2, f2_lo(Mr2[i]));
                const float um = ex2_approx(te) + f2_lo(nDr2[i]);
                float x = (cv[r] + f2_lo(on2[i])) + (e == 0 ? f2_lo(vnb[k]) : f2_hi(vnb[k]));
                const int j = j0 + hf * 32 + 8 * k + col0 + e;
                unsigned int todo = __ballot_sync(0xffffffffu, te < hthr[i] && j < n);
                while (todo) {
                  const int src = __ffs(todo) - 1;
                  todo &= todo - 1;
                  const int js = __shfl_sync(0xffffffffu, j, src);
                  const int rs = __shfl_sync(0xffffffffu, r0 + 8 * i, src);
                  const float d2x = exact_dist2_warp(O_head + rs * kHeadDim, V_head + (long long)js * a.vsn, lane);
                  if (lane == src) x = d2x;
                }
                const float Iv = x * rsqrt_approx(fmaf(x * um, um, 1e-36f));
                acc[k] = f2_add(acc[k], e == 0 ? f2_make(Iv, 0.f) : f2_make(0.f, Iv));
              }
            }
          }
        }
      } else {
        __syncwarp();
        if (lane == 0) mbar_arrive(&B->acc_empty);
      }
      // ---- sum over the eight lanes that hold the same columns (rows differ): three exchange rounds, each
      //      halving what a lane keeps; lane L ends with the column my_col ----
      {
        const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
        const f32x2 s0 = b4 ? acc[0] : acc[2], s1 = b4 ? acc[1] : acc[3];
        const f32x2 k0 = b4 ? acc[2] : acc[0], k1 = b4 ? acc[3] : acc[1];
        const f32x2 a0 = f2_add(k0, f2_make(__shfl_xor_sync(0xffffffffu, f2_lo(s0), 16), __shfl_xor_sync(0xffffffffu, f2_hi(s0), 16)));
        const f32x2 a1 = f2_add(k1, f2_make(__shfl_xor_sync(0xffffffffu, f2_lo(s1), 16), __shfl_xor_sync(0xffffffffu, f2_hi(s1), 16)));
        const f32x2 sB = b3 ? a0 : a1, kB = b3 ? a1 : a0;
        const f32x2 c0 = f2_add(kB, f2_make(__shfl_xor_sync(0xffffffffu, f2_lo(sB), 8), __shfl_xor_sync(0xffffffffu, f2_hi(sB), 8)));
        const float sC = b2 ? f2_lo(c0) : f2_hi(c0), kC = b2 ? f2_hi(c0) : f2_lo(c0);
        const float tot = kC + __shfl_xor_sync(0xffffffffu, sC, 4);
        red[cI & 3][q][hf * 32 + my_col] = tot;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&B->red_full[cI & 3]);
    }
    if (sh.T2 > 0 && q == 0) {
      const int rs = (int)((cI - 1) & 3);
      ok = ok && PWAIT(&B->red_full[rs], (cI - 1) >> 2);
      const int jl = (sh.tile0 + sh.T2 - 1) * kSub + hf * 32 + lane;
      if (ok && jl < n)
        I_head[jl] = ((red[rs][0][hf * 32 + lane] + red[rs][1][hf * 32 + lane]) +
                      (red[rs][2][hf * 32 + lane] + red[rs][3][hf * 32 + lane])) * exp2f(-kShift);
    }
  }
}

// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kPThreads, 1)
tc_pipe_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const PipeArgs a) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) PipeBars bars;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;
  __shared__ RowConst rowc[kRows];
  __shared__ float onp[2][kRows];
  __shared__ float red[4][4][kSub];     // [sub-tile & 3][lane quarter][token]
  __shared__ float xch[kCWarps][32][6];
  const int group = blockIdx.x / a.cpg, rank = blockIdx.x % a.cpg;
  if (group >= a.groups) return;   // uniform per CTA

  PCtx cx;
  cx.smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  cx.gen = smem_raw + (cx.smem_base - smem_u32(smem_raw));
  cx.B = &bars;
  cx.abort_flag = &abort_flag;
  cx.dev_status = a.dev_status;
  cx.limit = a.wait_limit;
  cx.warp = threadIdx.x >> 5;
  cx.lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    PipeBars* B = &bars;
    mbar_init(&B->q_full, 1);
    mbar_init(&B->q_empty, 1);
    for (int i = 0; i < kKRing; ++i) { mbar_init(&B->k_full[i], 1); mbar_init(&B->k_empty[i], 1); }
    for (int i = 0; i < kVRing; ++i) { mbar_init(&B->v_full[i], 1); mbar_init(&B->v_empty[i], 2); }   // MMA + ||v||^2 warp
    for (int i = 0; i < 2; ++i) { mbar_init(&B->s_full[i], 1); mbar_init(&B->p_full[i], kAWarps * 32); }
    mbar_init(&B->pv_done, 1);
    mbar_init(&B->o_free, kAWarps * 32);
    mbar_init(&B->drain_a, 1);
    for (int i = 0; i < kCRing; ++i) {
      mbar_init(&B->kc_full[i], 1); mbar_init(&B->kc_empty[i], 1);
      mbar_init(&B->vc_full[i], 1); mbar_init(&B->vc_empty[i], 1);
    }
    mbar_init(&B->acc_full, 1);
    mbar_init(&B->acc_empty, kCWarps);
    mbar_init(&B->opr_ready, kCWarps);
    for (int i = 0; i < 4; ++i) mbar_init(&B->red_full[i], kCWarps);
    mbar_init(&B->drain_c, 1);
    fence_mbar_init();
    prefetch_tensormap(&tmQ);
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
  }
  if (cx.warp == 1) {
    tmem_alloc(&tmem_slot, 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  cx.tmem = tmem_slot;

  // the same split of the sub-tiles for both teams and every head (team C covers only the scored rows)
  Share sh;
  sh.group = group;
  sh.rank = rank;
  const int nt1 = (a.n_kv + kSub - 1) / kSub, nt2 = (a.n + kSub - 1) / kSub;
  const int per = (nt1 + a.cpg - 1) / a.cpg;
  sh.tile0 = rank * per;
  sh.T1 = max(0, min(nt1, sh.tile0 + per) - sh.tile0);
  sh.T2 = max(0, min(nt2, sh.tile0 + per) - sh.tile0);

  if (cx.warp < kCtrlWarps) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kPRegsControl));
    if (cx.warp == 0) {
      if (cx.lane == 0) tma_a_main(cx, a, sh, &tmQ, &tmK, &tmV);
    } else if (cx.warp == 1) {
      if (cx.lane == 0) mma_a_main(cx, a, sh);
    } else if (cx.warp < 4) {
      vnorm_main(cx, a, sh);
    } else if (cx.warp == 4) {
      if (cx.lane == 0) tma_c_main(cx, a, sh, &tmK, &tmV);
    } else if (cx.warp == 5) {
      if (cx.lane == 0) mma_c_main(cx, a, sh);
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kPRegsWorker));
    if (cx.warp < kFirstC) softmax_main(cx, a, sh);
    else epilogue_main(cx, a, sh, rowc, onp, red, xch);
  }

  tc_fence_before();
  __syncthreads();
  if (cx.warp == 1) {
    tc_fence_after();
    tmem_dealloc(cx.tmem, 512);
  }
}

inline bool make_kv_sub_map(TcState* st, CUtensorMap* map, const void* base, const Problem& p, long long sb, long long sh,
                            long long sn) {
  cuuint64_t dims[4] = {(cuuint64_t)p.d, (cuuint64_t)p.n_kv, (cuuint64_t)p.Hkv, (cuuint64_t)p.batch};
  cuuint64_t str[3] = {(cuuint64_t)sn * 2, (cuuint64_t)(p.Hkv > 1 ? sh : sn) * 2, (cuuint64_t)(p.batch > 1 ? sb : sn) * 2};
  cuuint32_t box[4] = {64, kSub, 1, 1};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  return st->encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, str, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Groups of CTAs: each group has two heads in flight (one per team), so at most as many groups as keep twice their
// heads inside a 96 MB share of L2 (one group if even that does not fit).  Among the allowed counts the cheapest
// wins: a group runs its heads back to back, each costing its sub-tiles per CTA plus a fixed part (merge, barriers),
// and the last head's second phase is not hidden.
void pipe_plan(const Problem& p, int sm_count, int* groups, int* cpg) {
  const long long head_bytes = 2ll * p.n_kv * p.d * 2;
  long long limit = (96ll << 20) / (2 * (head_bytes > 0 ? head_bytes : 1));
  if (limit < 1) limit = 1;
  const int tiles = (p.n_kv + kSub - 1) / kSub;
  constexpr int kHeadOverheadTiles = 4;
  int best_g = 1;
  long long best_cost = -1;
  for (int g = 1; g <= p.BH && g <= limit && g <= sm_count && g <= 128; ++g) {
    const int c = sm_count / g;
    const long long per = (tiles + c - 1) / c;
    const long long heads = (p.BH + g - 1) / g;
    const long long cost = heads * (per + kHeadOverheadTiles) + per / 2 + kHeadOverheadTiles;
    if (best_cost < 0 || cost <= best_cost) { best_cost = cost; best_g = g; }
  }
  *groups = best_g;
  *cpg = sm_count / best_g;
}

bool tc_pipe_supported(const Problem& p) {
  return p.dtype == RESTKV_BF16 && p.d == kHeadDim && p.R == kRows && p.w >= 1 && kRows % p.w == 0;
}

cudaError_t tc_pipe_init() {
  cudaFuncAttributes fa;
  cudaError_t e = cudaFuncGetAttributes(&fa, tc_pipe_kernel);
  if (e != cudaSuccess) return e;
  if (fa.numRegs != kPRegsLaunch) return cudaErrorInvalidConfiguration;   // the register split assumes this pool
  return cudaFuncSetAttribute(tc_pipe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPSmem);
}

// One launch for every head: team A's pass, the merge and team C's pass.  The CTAs of a group wait for one another,
// so all of them must be resident: the grid never exceeds the SM count and a CTA fills an SM (shared memory), which
// holds as long as the device is not shared with another kernel at that moment; if it is, the bounded waits give up
// with the timeout status instead of hanging.
cudaError_t launch_tc_pipe(void* state, const Problem& p, const Workspace& ws, const void* Q, const void* K,
                           const void* V, float ema_decay, int sm_count, long long wait_limit,
                           unsigned int* dev_status, cudaStream_t st) {
  TcState* ts = (TcState*)state;
  CUtensorMap tmQ, tmK, tmV;
  if (!make_rows_map(ts, &tmQ, Q, p.BH) || !make_kv_sub_map(ts, &tmK, K, p, p.ksb, p.ksh, p.ksn) ||
      !make_kv_sub_map(ts, &tmV, V, p, p.vsb, p.vsh, p.vsn))
    return cudaErrorInvalidValue;
  PipeArgs a{};
  a.Hkv = p.Hkv; a.BH = p.BH; a.n = p.n; a.n_kv = p.n_kv; a.w = p.w;
  a.scale = p.scale; a.ema_decay = ema_decay;
  pipe_plan(p, sm_count, &a.groups, &a.cpg);
  a.vn_stride = ws.vn_stride;
  a.wait_limit = wait_limit;
  a.Q = (const __nv_bfloat16*)Q;
  a.V = (const __nv_bfloat16*)V; a.vsb = p.vsb; a.vsh = p.vsh; a.vsn = p.vsn;
  a.part_m = ws.part_m; a.part_l = ws.part_l; a.part_O = ws.part_O;
  a.O_f32 = ws.O_f32; a.row_M2 = ws.row_M2; a.vnorm = ws.vnorm; a.tile_max = ws.tile_max; a.I_hat = ws.I_hat;
  a.counters = ws.pipe_counters; a.dev_status = dev_status;
  cudaError_t e = cudaMemsetAsync(ws.pipe_counters, 0, kPipeCounterBytes, st);
  if (e != cudaSuccess) return e;
  tc_pipe_kernel<<<dim3(a.groups * a.cpg), dim3(kPThreads), kPSmem, st>>>(tmQ, tmK, tmV, a);
  return cudaGetLastError();
}

}  // namespace restkv
