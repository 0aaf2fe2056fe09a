// Persistent tensor-core score kernel for sm_100a (bf16, head_dim 128, w * group = 128 query rows).
//
// One CTA per SM.  The CTAs are divided into groups; a group takes one (batch, KV head) at a time and runs, back
// to back,
//   phase A  (Eq. 3)    every CTA of the group: S = Q K^T, online softmax, O += P V over its share of the tiles
//   phase B             the group's partial (m, l, O) are merged row by row
//   phase C  (Eq. 7-9)  every CTA: S^T = K Q^T, C^T = V (-2 O)^T over its share of the tiles, indicator, EMA,
//                       group mean
// The CTAs of a group meet at two counter barriers per head (after A and after B); different groups never wait
// for one another.  By default there are as many groups as heads (every head in flight, one round); with
// reuse_l2 only as many heads are in flight as fit in L2, so that phase C re-reads K and V from there.
// Every wait on data is bounded: a wait that runs out sets the sticky timeout bit, and the CTA skips the rest of
// its work and still releases its tensor memory.
#include "tc_common.cuh"

namespace restkv {

namespace {

constexpr int kFFirstWorker = 4;                  // warp 0: TMA producer, 1: MMA issuer, 2-3: ||v||^2 during phase A
constexpr int kFWorkerWarps = 16;                 // warps 4..19
constexpr int kFThreads = (kFFirstWorker + kFWorkerWarps) * 32;
// Registers per thread: 96 at launch (640 threads), i.e. a pool of 20 warps x 32 x 96 = 61440 for the CTA.  The control
// warpgroup then shrinks to 32 and the sixteen worker warps grow to 112: 4*32*32 + 16*32*112 = 61440, exactly the pool
// (a larger request would block for ever: the pool is what the CTA was launched with, not the SM's register file).
constexpr int kFRegsLaunch = 96, kFRegsControl = 32, kFRegsWorker = 112;
static_assert(kFFirstWorker * kFRegsControl + kFWorkerWarps * kFRegsWorker <= (kFFirstWorker + kFWorkerWarps) * kFRegsLaunch,
              "the register split must fit the pool the CTA is launched with");
constexpr int kFRing = 4;                         // 32 KB tile slots after Q | O' | aug | ones
constexpr size_t kFSmem = 2 * kTileBytes + kAugBytes + kOnesBytes + kFRing * kTileBytes + 1024;
constexpr int kFVSlots = 3;                       // phase A: V slots = ring 2, ring 3 and the (then unused) O' tile

struct FusedArgs {
  int Hkv, BH, n, n_kv, w;
  float scale;
  // Temporal weights (Eq. 9 and the variants of Appendix G.2) as a Horner chain: the score of a token is
  // t_scale * sum_i c_i I_i t_decay^(w-1-i) with c_0 = t_seed_first, c_(w-1) = t_seed_last, c_i = 1 otherwise (w >= 16 here).
  float t_decay, t_seed_first, t_seed_last, t_scale;
  int group_max;                     // 1: maximum over the query heads of a group instead of their mean
  int pool_max;                      // 1: the selection phase takes the maximum over the box instead of the mean
  int groups, cpg;                   // CTA groups and CTAs per group
  int attention_only;                // 1: stop after the merge (phases A and B): plain attention of the 128 rows
  int from_lse;                      // 1: O and the rows' log-sum-exp are given: phases A and B are skipped, phase C
                                     //    computes ||v||^2 and finds the tiles with large weights by itself
  float* part_m;                     // [CTA, 128]       running maximum, log2 units (one slot per CTA, reused
  float* part_l;                     // [CTA, 128]        from head to head: a group is past phase B of a head
  float* part_O;                     // [CTA, 128, 128]   before any of its CTAs writes the next head's partial)
  float* O_f32;                      // [BH, 128, 128]
  __nv_bfloat16* O_m2;               // [BH, 128, 128]  -2 * bf16(O)
  __nv_bfloat16* aug;                // [BH, 128, 64]
  float* vnorm;                      // [BH, n_kv]
  float* tile_max;                   // [BH, tiles, 128] largest scaled logit (log2 units) of each query row in each tile
  float* row_M2;                     // [BH, 128] m*log2e + log2 l of each query row (written by the merge)
  float* I_hat;                      // [BH, n]
  float* I_raw;                      // [BH, 128, n] or null: the per-query indicators, for the adaptive window of
                                     //  Eq. 10-12; every tile then takes the slower epilogue that holds them
  const __nv_bfloat16* V;
  long long vsb, vsh, vsn;
  // Output projection of Eq. 4 (all null without one): Eq. 7's squared norm becomes the quadratic form of Mt, the
  // per-head matrices [Hq, 128, 128]; vmv [BH, G, n_kv] holds the tokens' own terms v^T Mt v (in place of ||v||^2),
  // O_proj [BH, 128, 128] receives Mt o of the window rows.
  const float* proj_Mt;
  const float* vmv;
  float* O_proj;
  unsigned int* counters;            // [groups] (at most 256), zero at launch
  unsigned int* dev_status;
  long long wait_limit;              // SM clocks a wait may last
  // Pooling (Eq. 13), top-B selection and row gather (Eq. 14) of every head right after its phase C, by the head's own
  // group of CTAs (sel_keep = 0: not done here).
  int sel_keep, sel_W, sel_gamma;
  float* sel_scores;                 // [BH, n_kv] pooled scores
  int32_t* sel_indices;              // [BH, keep]
  unsigned int* sel_hist;            // [BH, 4, 256] digit histograms of the group, zero at launch
  unsigned int* sel_sfx;             // [CTA, 4, kSfxStride] per CTA: suffix sums of its own digit histograms
  const __nv_bfloat16* K;
  long long ksb, ksh, ksn;
  __nv_bfloat16* K_out;              // [BH, keep, 128]
  __nv_bfloat16* V_out;
};

constexpr int kSelPasses = 4;                     // 8-bit digits of the 32-bit keys, from the top
constexpr int kSfxStride = 260;                   // 257 suffix sums per (CTA, pass), padded
constexpr int kSelMaxKeys = 20480;                // scores of one CTA's share of a head kept in shared memory
constexpr int kSelHalo = 64;                      // widest reach of the pooling window beyond the share
constexpr int kSelBarriers = 2 + kSelPasses;      // group barriers of the selection phase

struct FusedBars {
  // phase A
  uint64_t q_full, k_full[2], k_empty[2], v_full[kFVSlots], v_empty[kFVSlots], s_full[2], p_full[2], pv_done[2];
  // phase C
  uint64_t const_full, kv_full[2], kv_empty[2], acc_full[2], acc_empty[2], red_full[4];
  uint64_t drain;   // only after a failed wait: completion of the MMAs issued so far
  uint64_t vn_full[4];   // from_lse: ||v||^2 of a tile is in shared memory (ring of four tiles)
};

__device__ __forceinline__ void mbar_inval(uint64_t* bar) {
  asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void named_barrier_sync(int id, int count) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(count) : "memory");
}
__device__ __forceinline__ unsigned int ld_acquire_gpu(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// (Re)initialises every mbarrier of the CTA for one phase.  Called by one thread between two __syncthreads.
__device__ void init_bars(FusedBars* B, bool first, bool from_lse) {
  uint64_t* all = reinterpret_cast<uint64_t*>(B);
  constexpr int kCount = sizeof(FusedBars) / sizeof(uint64_t);
  if (!first)
    for (int i = 0; i < kCount; ++i) mbar_inval(all + i);
  mbar_init(&B->q_full, 1);
  for (int i = 0; i < 2; ++i) {
    mbar_init(&B->k_full[i], 1);
    mbar_init(&B->k_empty[i], 1);
    mbar_init(&B->s_full[i], 1);
    mbar_init(&B->p_full[i], 256);
    mbar_init(&B->pv_done[i], 1);
    mbar_init(&B->kv_full[i], 1);
    mbar_init(&B->kv_empty[i], from_lse ? 3 : 1);   // MMA commit (+ the two ||v||^2 warps, which read the V tile)
    mbar_init(&B->acc_full[i], 1);
    mbar_init(&B->acc_empty[i], kFWorkerWarps);
  }
  for (int i = 0; i < kFVSlots; ++i) {
    mbar_init(&B->v_full[i], 1);
    mbar_init(&B->v_empty[i], 1 + 1);   // MMA commit + the warp that reduces ||v||^2
  }
  mbar_init(&B->const_full, 1);
  mbar_init(&B->drain, 1);
  for (int i = 0; i < 4; ++i) mbar_init(&B->red_full[i], kFWorkerWarps);
  for (int i = 0; i < 4; ++i) mbar_init(&B->vn_full[i], 2);
  fence_mbar_init();
}

// All CTAs of a group arrive and wait until `target` arrivals have been counted.  Bounded.  Thread 0 runs the
// counter; every other thread calls group_barrier_follow at the same point.  Both return the same verdict (one
// shared word written between the two synchronisations): false once any wait of the CTA has run out.
__device__ bool group_barrier(unsigned int* counter, unsigned int target, volatile int* abort_flag, volatile int* go,
                              unsigned int* dev_status, long long wait_limit) {
  __syncthreads();
  if (threadIdx.x == 0) {
    // release: everything the CTA wrote before the __syncthreads is visible to whoever acquires the count
    asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(counter), "r"(1u) : "memory");
    const long long t0 = clock64();
    while (ld_acquire_gpu(counter) < target) {
      if (*abort_flag) break;
      if (clock64() - t0 > wait_limit) {
        *abort_flag = 1;
        atomicOr(dev_status, kDevTimeout);
        break;
      }
    }
    *go = (*abort_flag == 0);
  }
  __syncthreads();
  return *go != 0;
}
__device__ bool group_barrier_follow(volatile int* go) {
  __syncthreads();
  __syncthreads();
  return *go != 0;
}

struct Ctx {
  uint32_t smem_base;      // shared-window address of the 1024-aligned dynamic region
  uint8_t* gen_base;       // the same location as a generic pointer
  uint32_t tmem;
  FusedBars* B;
  int* abort_flag;
  float* sm_stats;         // [6][128] floats: row maxima of the column halves [slot][half], then (m, l) hand-over
  float* vn_s;             // [4][128] ||v||^2 of the last four tiles of phase C (from_lse only)
  int warp, lane;
};

constexpr uint32_t kOffQ = 0, kOffO = kTileBytes, kOffAug = 2 * kTileBytes, kOffOnes = kOffAug + kAugBytes,
                   kOffRing = kOffOnes + kOnesBytes;
__device__ __forceinline__ uint32_t k_slot_off(int i) { return kOffRing + (uint32_t)i * kTileBytes; }
__device__ __forceinline__ uint32_t v_slot_off(int i) { return i < 2 ? kOffRing + (uint32_t)(2 + i) * kTileBytes : kOffO; }

// ------------------------------------------------------------------------------------------------
// Phase A: this CTA's share [tile0, tile0 + T) of one head.
// Control warps: warp 0 loads (K ring of 2 slots, V ring of 3), warp 1 issues the MMAs (S(it), then O += P V of tile
// it - 1), warps 2 and 3 reduce ||v_j||^2 of the tokens from the V tiles (even / odd tiles).
// Tensor memory: tile slot g = it & 1 holds S_g at g*128 (the bf16 P_g overwrites columns [0,32) and [64,96) of
// it) and O_g at 256 + g*128.
__device__ void phase_a_control(const Ctx& cx, const FusedArgs& a, const CUtensorMap* tmQ, const CUtensorMap* tmK,
                        const CUtensorMap* tmV, int bh, int rank, int tile0, int T) {
  FusedBars* B = cx.B;
  int* abort_flag = cx.abort_flag;
  unsigned int* dev_status = a.dev_status;
  const int b = bh / a.Hkv, h = bh % a.Hkv;
  const int warp = cx.warp, lane = cx.lane;
  const uint32_t tmem = cx.tmem;

  if (warp == 0) {
    if (lane == 0 && T > 0) {
      mbar_arrive_expect_tx(&B->q_full, kTileBytes);
      tma_load_3d(cx.gen_base + kOffQ, tmQ, &B->q_full, 0, 0, bh);
      tma_load_3d(cx.gen_base + kOffQ + kBoxBytes, tmQ, &B->q_full, 64, 0, bh);
      int nK = 0, nV = 0;   // K and V tiles requested so far
      for (int it = 0; it < T; ++it) {
        const int ks = it & 1, vs = it % kFVSlots;
        const int j0 = (tile0 + it) * kTile;
        if (it >= 2 && !mbar_wait(&B->k_empty[ks], ((it >> 1) - 1) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit)) break;
        uint8_t* dK = cx.gen_base + k_slot_off(ks);
        mbar_arrive_expect_tx(&B->k_full[ks], kTileBytes);
        tma_load_4d(dK, tmK, &B->k_full[ks], 0, j0, h, b);
        tma_load_4d(dK + kBoxBytes, tmK, &B->k_full[ks], 64, j0, h, b);
        ++nK;
        if (it >= kFVSlots &&
            !mbar_wait(&B->v_empty[vs], (it / kFVSlots - 1) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit))
          break;
        uint8_t* dV = cx.gen_base + v_slot_off(vs);
        mbar_arrive_expect_tx(&B->v_full[vs], kTileBytes);
        tma_load_4d(dV, tmV, &B->v_full[vs], 0, j0, h, b);
        tma_load_4d(dV + kBoxBytes, tmV, &B->v_full[vs], 64, j0, h, b);
        ++nV;
      }
      if (*(volatile int*)abort_flag) {
        // a wait of this CTA has failed: the tiles requested last may still be on their way into shared memory
        wait_issued(&B->q_full, 0);
        for (int i = max(0, nK - 2); i < nK; ++i) wait_issued(&B->k_full[i & 1], (uint32_t)(i >> 1));
        for (int i = max(0, nV - kFVSlots); i < nV; ++i) wait_issued(&B->v_full[i % kFVSlots], (uint32_t)(i / kFVSlots));
      }
    }
  } else if (warp == 1) {
    // S(it), then O += P V of tile it - 1
    if (lane == 0 && T > 0) {
      bool ok = mbar_wait(&B->q_full, 0, abort_flag, dev_status, kDevTimeout, a.wait_limit);
      for (int it = 0; ok && it <= T; ++it) {
        if (it < T) {
          const int ks = it & 1, g = it & 1;
          if (!mbar_wait(&B->k_full[ks], (it >> 1) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit)) break;
          tc_fence_after();
          // S_g may be overwritten: O += P V of tile it - 2 (which read P_g) was issued earlier and MMAs run in order
          mma_tile_kk(tmem + (uint32_t)g * 128u, cx.smem_base + kOffQ, cx.smem_base + k_slot_off(ks), false);
          umma_commit(&B->s_full[g]);
          umma_commit(&B->k_empty[ks]);
        }
        if (it >= 1) {
          const int pt = it - 1, g = pt & 1, vs = pt % kFVSlots;
          if (!mbar_wait(&B->p_full[g], (pt >> 1) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit)) break;
          if (!mbar_wait(&B->v_full[vs], (pt / kFVSlots) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit)) break;
          tc_fence_after();
          // A = P_g in TMEM (16 tokens = 8 packed columns per K step), B = V tile, MN-major
          const uint32_t vaddr = cx.smem_base + v_slot_off(vs);
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const uint64_t bdesc = make_smem_desc(vaddr + (uint32_t)k * 2048u, kBoxBytes, 1024);
            // tokens 0-63 of P_g sit in columns [0, 32) of S_g, tokens 64-127 in columns [64, 96)
            const uint32_t pcol = (uint32_t)(k < 4 ? k * 8 : 64 + (k - 4) * 8);
            umma_ts(tmem + 256u + (uint32_t)g * 128u, tmem + (uint32_t)g * 128u + pcol, bdesc, kIdescKMN,
                    pt >= 2 || k > 0);
          }
          umma_commit(&B->pv_done[g]);
          umma_commit(&B->v_empty[vs]);
        }
      }
      if (*(volatile int*)abort_flag) {   // let the MMAs already issued finish before the CTA goes on to return
        umma_commit(&B->drain);
        wait_issued(&B->drain, 0);
      }
    }
  } else if (warp < kFFirstWorker) {
    // ---------------- ||v||^2: one warp takes the even tiles, the other the odd ones; lane = 4 tokens ----------------
    const int vg = warp - 2;
    bool ok = true;
    for (int it = 0; it < T && ok; ++it) {
      const int vs = it % kFVSlots;
      // both warps wait for every tile so that neither falls a whole phase behind a slot's barrier
      ok = mbar_wait(&B->v_full[vs], (it / kFVSlots) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit);
      if (!ok || (it & 1) != vg) continue;
      const uint8_t* vt = cx.gen_base + v_slot_off(vs);
      float vn[4];
#pragma unroll
      for (int rr = 0; rr < 4; ++rr) {
        const int row = rr * 32 + lane;
        float2 acc = make_float2(0.f, 0.f);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          // 16-byte chunk c of row r of a 128-byte-swizzled box sits at chunk c ^ (r & 7)
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
        vn[rr] = acc.x + acc.y;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&B->v_empty[vs]);
#pragma unroll
      for (int rr = 0; rr < 4; ++rr) {
        const int j = (tile0 + it) * kTile + rr * 32 + lane;
        if (j < a.n_kv && !a.attention_only) a.vnorm[(long long)bh * a.n_kv + j] = vn[rr];
      }
    }
  }
}

// Worker warps in phase A: four softmax warpgroups, thread = query row; warpgroups g and g + 2 share tile slot g
// (tokens 0-63 and 64-127 of the tile).  At the end the two slots' (m, l, O) are merged and written as the CTA's
// partial.
__device__ void phase_a_worker(const Ctx& cx, const FusedArgs& a, const CUtensorMap* tmQ, const CUtensorMap* tmK,
                        const CUtensorMap* tmV, int bh, int rank, int tile0, int T) {
  FusedBars* B = cx.B;
  int* abort_flag = cx.abort_flag;
  unsigned int* dev_status = a.dev_status;
  const int b = bh / a.Hkv, h = bh % a.Hkv;
  const int warp = cx.warp, lane = cx.lane;
  const uint32_t tmem = cx.tmem;

  // ---------------- four softmax warpgroups: thread = query row; warpgroups g and g + 2 share tile slot g,
  //                  the first takes tokens 0-63 of the tile, the second tokens 64-127 ----------------
  const int wgi = (warp - kFFirstWorker) >> 2;
  const int g = wgi & 1, hf = wgi >> 1;
  const int quad = warp & 3;
  const int row = quad * 32 + lane;
  const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
  const uint32_t tS = tmem + (uint32_t)g * 128u + lane_base + (uint32_t)hf * 64u;   // this half's 64 logits
  const uint32_t tP = tS;                                                           // and where its P goes
  const uint32_t tO = tmem + 256u + (uint32_t)g * 128u + lane_base + (uint32_t)hf * 64u;
  const int i_q = row % a.w;                // window position of this row (row = group * w + i)
  const float c2 = a.scale * kLog2e;
  const int n = a.n, n_kv = a.n_kv;
  const int nt_all = (n_kv + kTile - 1) / kTile;
  float* my_max = cx.sm_stats + (g * 2 + hf) * kRows;
  const float* other_max = cx.sm_stats + (g * 2 + (hf ^ 1)) * kRows;
  float m_ref = -INFINITY;
  float2 l2 = make_float2(0.f, 0.f);
  bool ok = true;
  int uses = 0;                             // tiles this warpgroup has processed
  for (int it = g; it < T; it += 2, ++uses) {
    ok = ok && mbar_wait(&B->s_full[g], (uint32_t)uses & 1u, abort_flag, dev_status, kDevTimeout, a.wait_limit);
    if (ok) tc_fence_after();
    const int j0 = (tile0 + it) * kTile + hf * 64;
    const bool ragged = j0 + 64 > n;   // rows past the scored prefix: window rows (causal) or padding
    auto mask = [&](float* s, int c) {
#pragma unroll
      for (int u = 0; u < 16; ++u) {
        const int j = j0 + c * 16 + u;
        const bool vis = (j < n_kv) && (j < n || (j - n) <= i_q);
        s[u] = vis ? s[u] : -INFINITY;
      }
    };
    float sa[16], sb[16];
    // ---- sweep 1: row maximum of this half of the tile; the next 16 columns travel while 16 are reduced ----
    float tmax = -INFINITY;
    if (ok) {
      tmem_ld16(tS, sa);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float* cur = (c & 1) ? sb : sa;
        float* nxt = (c & 1) ? sa : sb;
        tmem_wait_ld();
        tmem_ld16(tS + ((c + 1) & 3) * 16, nxt);   // after the last chunk: chunk 0 again, for sweep 2
        if (ragged) mask(cur, c);
#pragma unroll
        for (int u = 0; u < 16; ++u) tmax = fmaxf(tmax, cur[u]);
      }
    }
    my_max[row] = tmax;
    named_barrier_sync(3 + g, 256);            // the two halves of the slot exchange their row maxima
    tmax = fmaxf(tmax, other_max[row]);
    named_barrier_sync(3 + g, 256);            // both have read before the next tile overwrites
    if (!ok) continue;
    const float m_tile = tmax * c2;
    // phase C takes the exact distance only in tiles where some weight can exceed kHeavyA: it compares this
    // maximum with the row's final normaliser
    if (hf == 0 && !a.attention_only) a.tile_max[((long long)bh * nt_all + tile0 + it) * kRows + row] = m_tile;
    const bool need = m_tile > m_ref + kRescaleThreshold;   // also true for the first visible entries (m_ref = -inf)
    float factor = 1.f;
    if (need) {
      factor = ex2_approx(m_ref - m_tile);   // 0 when m_ref = -inf
      l2.x *= factor;
      l2.y *= factor;
      m_ref = m_tile;
    }
    // S(it) has landed, so O += P V of this slot's previous tile (issued before it) is complete; each half
    // rescales its 64 columns of O_g
    if (uses > 0 && __any_sync(0xffffffffu, need)) {
      tmem_wait_ld();
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float o[16];
        tmem_ld16(tO + c * 16, o);
        tmem_wait_ld();
#pragma unroll
        for (int u = 0; u < 16; ++u) o[u] *= factor;
        tmem_st16(tO + c * 16, reinterpret_cast<const uint32_t*>(o));
      }
    }
    // ---- sweep 2: P = exp2(s*c2 - m_ref) as bf16 over the first 32 columns of this half.  Chunk c of P lands
    //      on columns [8c, 8c + 8) of the half, which belong to a chunk of S that is already in registers. ----
    const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
    const float2 c22 = make_float2(c2, c2), nm2 = make_float2(-m_use, -m_use);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float* cur = (c & 1) ? sb : sa;     // chunk 0 sits in sa (loaded at the end of sweep 1)
      float* nxt = (c & 1) ? sa : sb;
      tmem_wait_ld();
      if (c < 3) tmem_ld16(tS + (c + 1) * 16, nxt);
      if (ragged) mask(cur, c);
      uint32_t packed[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const float2 e = ffma2(make_float2(cur[2 * u], cur[2 * u + 1]), c22, nm2);
        const float2 pp = make_float2(ex2_approx(e.x), ex2_approx(e.y));
        l2 = fadd2(l2, pp);
        packed[u] = pack_bf16x2(pp.x, pp.y);
      }
      tmem_st8(tP + c * 8, packed);
    }
    tmem_wait_st();
    tc_fence_before();
    mbar_arrive(&B->p_full[g]);
  }
  if (uses > 0 && ok) ok = mbar_wait(&B->pv_done[g], (uint32_t)(uses - 1) & 1u, abort_flag, dev_status, kDevTimeout, a.wait_limit);
  if (ok && uses > 0) tc_fence_after();
  const bool have = ok && uses > 0;
  const float m_mine = have ? m_ref : -INFINITY, l_mine = have ? l2.x + l2.y : 0.f;

  // ---- merge: the halves add their l, then slot 1 hands (m, l, O) to slot 0 through shared memory (the K
  //      slots are idle: every MMA of this phase has completed once all warpgroups have seen their last
  //      O += P V).  Each thread moves the 64 columns of O of its half. ----
  float* xO = reinterpret_cast<float*>(cx.gen_base + k_slot_off(0));   // [128 cols][128 rows] floats, 64 KB
  float* st_l = cx.sm_stats + 4 * kRows;   // [slot][row]: l of the second half
  float* st_m1 = cx.sm_stats;              // slot 1's m     (the row-maxima exchange is over)
  float* st_l1 = cx.sm_stats + kRows;      // slot 1's l
  named_barrier_sync(1, kFWorkerWarps * 32);
  if (hf == 1) st_l[g * kRows + row] = l_mine;
  named_barrier_sync(1, kFWorkerWarps * 32);
  const float l_slot = l_mine + (hf == 0 ? st_l[g * kRows + row] : 0.f);   // meaningful in the first half only
  if (g == 1) {
    if (hf == 0) { st_m1[row] = m_mine; st_l1[row] = l_slot; }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float o[16];
      if (have) {
        tmem_ld16(tO + c * 16, o);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int u = 0; u < 16; ++u) o[u] = 0.f;
      }
#pragma unroll
      for (int u = 0; u < 16; ++u) xO[(hf * 64 + c * 16 + u) * 128 + row] = o[u];
    }
  }
  named_barrier_sync(1, kFWorkerWarps * 32);
  if (g == 0) {
    const float m1 = st_m1[row], l1 = st_l1[row];
    const float m = fmaxf(m_mine, m1);
    const float a0 = (m_mine == -INFINITY) ? 0.f : ex2_approx(m_mine - m);
    const float a1 = (m1 == -INFINITY) ? 0.f : ex2_approx(m1 - m);
    const long long o_idx = (long long)blockIdx.x * kRows + row;
    float* Op = a.part_O + o_idx * kHeadDim + hf * 64;
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float o[16];
      if (have) {
        tmem_ld16(tO + c * 16, o);
        tmem_wait_ld();
      } else {
#pragma unroll
        for (int u = 0; u < 16; ++u) o[u] = 0.f;
      }
#pragma unroll
      for (int u = 0; u < 16; ++u) o[u] = o[u] * a0 + xO[(hf * 64 + c * 16 + u) * 128 + row] * a1;
#pragma unroll
      for (int u = 0; u < 16; u += 4)
        *reinterpret_cast<float4*>(Op + c * 16 + u) = make_float4(o[u], o[u + 1], o[u + 2], o[u + 3]);
    }
    if (hf == 0) {
      a.part_m[o_idx] = m;
      a.part_l[o_idx] = l_slot * a0 + l1 * a1;
    }
  }
  fence_proxy_async_smem();   // the hand-over buffer lies in the tile ring, which TMA loads refill next
  tc_fence_before();
}

// (Mt x) for a 128-vector x held in shared memory, Mt symmetric [128 x 128] fp32 in global memory: lane L returns
// elements 4L .. 4L+3 (row k of Mt is read as a whole by the warp: coalesced).
__device__ __forceinline__ float4 project_row_warp(const float* __restrict__ Mt, const float* x, int lane) {
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 8
  for (int k = 0; k < kHeadDim; ++k) {
    const float4 m = __ldg(reinterpret_cast<const float4*>(Mt + k * kHeadDim + lane * 4));
    const float xk = x[k];
    acc.x = fmaf(m.x, xk, acc.x); acc.y = fmaf(m.y, xk, acc.y); acc.z = fmaf(m.z, xk, acc.z); acc.w = fmaf(m.w, xk, acc.w);
  }
  return acc;
}

// x = hi + mid + lo with three bf16 pieces (24 significant bits).
__device__ __forceinline__ void split3(float x, __nv_bfloat16* out) {
  const __nv_bfloat16 hi = __float2bfloat16_rn(x);
  const float r1 = x - __bfloat162float(hi);
  const __nv_bfloat16 mid = __float2bfloat16_rn(r1);
  out[0] = hi;
  out[1] = mid;
  out[2] = __float2bfloat16_rn(r1 - __bfloat162float(mid));
}

// ------------------------------------------------------------------------------------------------
// Phase B: the group's `cpg` partials of one query row are merged by `wpr` warps (lane = four output dims; warp
// `sub` of the row takes partials sub, sub + wpr, ...), whose sums meet in shared memory and are added in a fixed
// order: the result does not depend on timing.  Written for phase C: O (fp32), -2 bf16(O), and the row's strip
// of bf16 constant pieces.  Called by all sixteen worker warps; r < 0 means this warp has no row.
template <bool kProj>
__device__ void combine_rows(const FusedArgs& a, int bh, int group, int r, int sub, int wpr, int wq, int lane,
                             float (*xch)[kHeadDim + 4]) {
  float m = -INFINITY, l = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  if (r >= 0) {
    const long long base = (long long)group * a.cpg * kRows + r;   // + p * kRows
    // running merge of this warp's partials (all loads of a batch are issued before any is used)
    constexpr int kBatch = 10;   // loads in flight per lane
#pragma unroll 1
    for (int p0 = sub; p0 < a.cpg; p0 += kBatch * wpr) {
      float mp[kBatch], lp[kBatch];
      float4 v[kBatch];
#pragma unroll
      for (int k = 0; k < kBatch; ++k) {
        const int p = p0 + k * wpr;
        const bool in = p < a.cpg;
        const long long pi = base + (long long)(in ? p : p0) * kRows;
        mp[k] = in ? a.part_m[pi] : -INFINITY;
        lp[k] = a.part_l[pi];
        v[k] = *reinterpret_cast<const float4*>(a.part_O + pi * kHeadDim + lane * 4);
      }
#pragma unroll
      for (int k = 0; k < kBatch; ++k) {
        const float m_new = fmaxf(m, mp[k]);
        const float s_old = (m == -INFINITY) ? 0.f : ex2_approx(m - m_new);
        const float s_p = (mp[k] == -INFINITY) ? 0.f : ex2_approx(mp[k] - m_new);   // an empty partial weighs 0
        l = l * s_old + lp[k] * s_p;
        acc.x = acc.x * s_old + v[k].x * s_p;
        acc.y = acc.y * s_old + v[k].y * s_p;
        acc.z = acc.z * s_old + v[k].z * s_p;
        acc.w = acc.w * s_old + v[k].w * s_p;
        m = m_new;
      }
    }
    *reinterpret_cast<float4*>(&xch[wq][lane * 4]) = acc;
    if (lane == 0) { xch[wq][kHeadDim] = l; xch[wq][kHeadDim + 1] = m; }
  }
  named_barrier_sync(2, kFWorkerWarps * 32);
  if (r < 0 || sub != 0) return;
  {
    // the row's wpr warp results, merged in a fixed order
    float mm = m;
    for (int k = 1; k < wpr; ++k) mm = fmaxf(mm, xch[wq + k][kHeadDim + 1]);
    const float s0 = (m == -INFINITY) ? 0.f : ex2_approx(m - mm);
    acc.x *= s0; acc.y *= s0; acc.z *= s0; acc.w *= s0;
    l *= s0;
    for (int k = 1; k < wpr; ++k) {
      const float mk = xch[wq + k][kHeadDim + 1];
      const float sk = (mk == -INFINITY) ? 0.f : ex2_approx(mk - mm);
      const float4 v = *reinterpret_cast<const float4*>(&xch[wq + k][lane * 4]);
      acc.x = fmaf(v.x, sk, acc.x); acc.y = fmaf(v.y, sk, acc.y); acc.z = fmaf(v.z, sk, acc.z); acc.w = fmaf(v.w, sk, acc.w);
      l = fmaf(xch[wq + k][kHeadDim], sk, l);
    }
    m = mm;
  }
  const float inv_l = 1.f / l;
  const float4 o = make_float4(acc.x * inv_l, acc.y * inv_l, acc.z * inv_l, acc.w * inv_l);
  const long long ri = (long long)bh * kRows + r;
  *reinterpret_cast<float4*>(a.O_f32 + ri * kHeadDim + lane * 4) = o;
  __nv_bfloat16* om = a.O_m2 + ri * kHeadDim + lane * 4;
  float on;
  if (kProj) {
    // with the output projection: the row of the third contraction is -2 bf16(Mt o), its constant o^T Mt o
    __syncwarp();
    *reinterpret_cast<float4*>(&xch[wq][lane * 4]) = o;   // the warp's own slot: its partials were merged above
    __syncwarp();
    const float4 mo = project_row_warp(a.proj_Mt + (long long)((bh % a.Hkv) * (kRows / a.w) + r / a.w) * kHeadDim * kHeadDim,
                                       xch[wq], lane);
    *reinterpret_cast<float4*>(a.O_proj + ri * kHeadDim + lane * 4) = mo;
    om[0] = __float2bfloat16_rn(-2.f * mo.x);
    om[1] = __float2bfloat16_rn(-2.f * mo.y);
    om[2] = __float2bfloat16_rn(-2.f * mo.z);
    om[3] = __float2bfloat16_rn(-2.f * mo.w);
    on = (o.x * mo.x + o.y * mo.y) + (o.z * mo.z + o.w * mo.w);
  } else {
    const __nv_bfloat16 b0 = __float2bfloat16_rn(o.x), b1 = __float2bfloat16_rn(o.y), b2 = __float2bfloat16_rn(o.z),
                        b3 = __float2bfloat16_rn(o.w);
    const float f0 = __bfloat162float(b0), f1 = __bfloat162float(b1), f2 = __bfloat162float(b2),
                f3 = __bfloat162float(b3);
    om[0] = __float2bfloat16_rn(-2.f * f0);   // -2 x is exact for a bf16 x
    om[1] = __float2bfloat16_rn(-2.f * f1);
    om[2] = __float2bfloat16_rn(-2.f * f2);
    om[3] = __float2bfloat16_rn(-2.f * f3);
    on = (f0 * f0 + f1 * f1) + (f2 * f2 + f3 * f3);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) on += __shfl_xor_sync(0xffffffffu, on, off);
  __nv_bfloat16* arow = a.aug + ri * 64;
  arow[2 * lane] = __float2bfloat16_rn(0.f);
  arow[2 * lane + 1] = __float2bfloat16_rn(0.f);
  __syncwarp();
  if (lane == 0) {
    const float c2 = a.scale * kLog2e;
    const float M2 = m + log2f(l);        // A = exp2(s * c2 - M2)
    a.row_M2[ri] = M2;
    split3(-M2 / c2, arow);
    split3(on, arow + 16);
  }
}

// One K tile and one V tile of phase C into stage s (ring slots 2s and 2s + 1).
__device__ __forceinline__ void load_stage_c(const Ctx& cx, const CUtensorMap* tmK, const CUtensorMap* tmV, int b, int h,
                                             int j0, int s) {
  uint8_t* dK = cx.gen_base + k_slot_off(2 * s);
  uint8_t* dV = dK + kTileBytes;
  uint64_t* bar = &cx.B->kv_full[s];
  mbar_arrive_expect_tx(bar, kStageBytes);
  tma_load_4d(dK, tmK, bar, 0, j0, h, b);
  tma_load_4d(dK + kBoxBytes, tmK, bar, 64, j0, h, b);
  tma_load_4d(dV, tmV, bar, 0, j0, h, b);
  tma_load_4d(dV + kBoxBytes, tmV, bar, 64, j0, h, b);
}

// ------------------------------------------------------------------------------------------------
// Phase C: this CTA's share [tile0, tile0 + T) of the scored rows of one head, walked from the last tile to the
// first (the tiles phase A read last are the likeliest to still be in L2).  Warp 0 loads, warp 1 issues the
// MMAs, the sixteen worker warps are four epilogue warpgroups (thread = token, warpgroup c = accumulator columns
// [32c, 32c + 32)).  Q is still in shared memory from phase A.  The per-query-row constants ride through the
// tensor core (one extra K = 16 step against a block of ones), so with u = exp2(-scale*log2e * S') = 1/A and
// x = C' + ||v||^2 = ||o - v||^2 the indicator is x * rsqrt(x * (u - 1)^2).
template <int kW, bool kLse>
__device__ void phase_c_control(const Ctx& cx, const FusedArgs& a, const CUtensorMap* tmQ, const CUtensorMap* tmO,
                                const CUtensorMap* tmAug, const CUtensorMap* tmK, const CUtensorMap* tmV, int bh,
                                int tile0, int T, int pre) {
  constexpr int kG = kRows / kW;
  FusedBars* B = cx.B;
  int* abort_flag = cx.abort_flag;
  unsigned int* dev_status = a.dev_status;
  const int b = bh / a.Hkv, h = bh % a.Hkv;
  const int warp = cx.warp, lane = cx.lane;
  const uint32_t tmem = cx.tmem;   // buffer s: S' at s*256, C' at s*256 + 128
  const int n = a.n;

  if (warp == 0) {
    if (lane == 0 && T > 0) {
      fence_proxy_async_all();   // O' and the constant strip were written with ordinary stores by other CTAs
      mbar_arrive_expect_tx(&B->const_full, kTileBytes + kAugBytes + (kLse ? kTileBytes : 0u));
      if (kLse) {   // no phase A has brought Q in
        tma_load_3d(cx.gen_base + kOffQ, tmQ, &B->const_full, 0, 0, bh);
        tma_load_3d(cx.gen_base + kOffQ + kBoxBytes, tmQ, &B->const_full, 64, 0, bh);
      }
      tma_load_3d(cx.gen_base + kOffO, tmO, &B->const_full, 0, 0, bh);
      tma_load_3d(cx.gen_base + kOffO + kBoxBytes, tmO, &B->const_full, 64, 0, bh);
      tma_load_3d(cx.gen_base + kOffAug, tmAug, &B->const_full, 0, 0, bh);
      int nS = pre;   // stages requested so far
      for (int it = pre; it < T; ++it) {   // the first `pre` tiles were requested before the group barriers
        const int s = it & 1;
        if (it >= 2 && !mbar_wait(&B->kv_empty[s], ((it >> 1) - 1) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit)) break;
        load_stage_c(cx, tmK, tmV, b, h, (tile0 + T - 1 - it) * kTile, s);
        ++nS;
      }
      if (*(volatile int*)abort_flag) {
        wait_issued(&B->const_full, 0);
        for (int i = max(0, nS - 2); i < nS; ++i) wait_issued(&B->kv_full[i & 1], (uint32_t)(i >> 1));
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && T > 0) {
      bool ok = mbar_wait(&B->const_full, 0, abort_flag, dev_status, kDevTimeout, a.wait_limit);
      const uint32_t sQ = cx.smem_base + kOffQ, sO = cx.smem_base + kOffO, sAug = cx.smem_base + kOffAug;
      const uint64_t ones_desc = make_smem_desc(cx.smem_base + kOffOnes, 16, 0);   // every 8-row group reads the same block
      const uint64_t aug_s = kmajor_desc(sAug), aug_c = kmajor_desc(sAug + 32u);
      for (int it = 0; ok && it < T; ++it) {
        const int s = it & 1;
        if (!mbar_wait(&B->kv_full[s], (it >> 1) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit)) break;
        if (it >= 2 && !mbar_wait(&B->acc_empty[s], ((it >> 1) - 1) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit)) break;
        tc_fence_after();
        const uint32_t sK = cx.smem_base + k_slot_off(2 * s), sV = sK + kTileBytes;
        const uint32_t tS = tmem + (uint32_t)s * 256u, tC = tS + 128u;
        mma_tile_kk(tS, sK, sQ, false);                       // S^T = K Q^T
        umma_ss(tS, ones_desc, aug_s, kIdescKK, true);        //   + row constant
        mma_tile_kk(tC, sV, sO, false);                       // C^T = V (-2 O)^T
        umma_ss(tC, ones_desc, aug_c, kIdescKK, true);        //   + ||o||^2
        umma_commit(&B->acc_full[s]);
        umma_commit(&B->kv_empty[s]);
      }
      if (*(volatile int*)abort_flag) {
        umma_commit(&B->drain);
        wait_issued(&B->drain, 0);
      }
    }
  } else if (kLse) {
    // ---- ||v||^2 of the tile's tokens from the V tile in shared memory (phase A, which computes it otherwise, does
    //      not run): warp 2 takes tokens 0-63, warp 3 tokens 64-127, a lane two rows; ring of four tiles ----
    bool ok = true;
    for (int it = 0; it < T && ok; ++it) {
      const int s = it & 1;
      ok = mbar_wait(&B->kv_full[s], (it >> 1) & 1, abort_flag, dev_status, kDevTimeout, a.wait_limit);
      if (!ok) break;
      const uint8_t* vt = cx.gen_base + k_slot_off(2 * s) + kTileBytes;
#pragma unroll
      for (int rr = 0; rr < 2; ++rr) {
        const int row = (warp - 2) * 64 + rr * 32 + lane;
        f32x2 acc[4] = {f2_make(0.f, 0.f), f2_make(0.f, 0.f), f2_make(0.f, 0.f), f2_make(0.f, 0.f)};
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          const uint8_t* rowp = vt + half * kBoxBytes + (row >> 3) * 1024 + (row & 7) * 128;
#pragma unroll
          for (int c = 0; c < 8; ++c) {
            const uint4 u = *reinterpret_cast<const uint4*>(rowp + ((c ^ (row & 7)) << 4));
            const unsigned int wv[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const f32x2 e = f2_make(__uint_as_float(wv[q] << 16), __uint_as_float(wv[q] & 0xFFFF0000u));
              acc[q] = f2_fma(e, e, acc[q]);
            }
          }
        }
        const f32x2 t2 = f2_add(f2_add(acc[0], acc[1]), f2_add(acc[2], acc[3]));
        cx.vn_s[(it & 3) * kTile + row] = f2_lo(t2) + f2_hi(t2);
      }
      __syncwarp();
      if (lane == 0) {
        mbar_arrive(&B->vn_full[it & 3]);
        mbar_arrive(&B->kv_empty[s]);
      }
    }
  }
}

// kInd: 0 = Eq. 7; 1 = the attention weight alone; 2 = attention weight times ||v|| (Appendix G.1); 3 = Eq. 7 with
// the output projection of Eq. 4 inside its norm.
template <int kW, bool kLse, int kInd>
__device__ void phase_c_worker(const Ctx& cx, const FusedArgs& a, const CUtensorMap* tmO, const CUtensorMap* tmAug,
                        const CUtensorMap* tmK, const CUtensorMap* tmV, int bh, int tile0, int T, int pre,
                        float (*red)[4][kTile]) {
  constexpr int kG = kRows / kW;
  constexpr bool kEq7 = kInd == 0 || kInd == 3, kProj = kInd == 3;
  FusedBars* B = cx.B;
  int* abort_flag = cx.abort_flag;
  unsigned int* dev_status = a.dev_status;
  const int b = bh / a.Hkv, h = bh % a.Hkv;
  const int warp = cx.warp, lane = cx.lane;
  const uint32_t tmem = cx.tmem;   // buffer s: S' at s*256, C' at s*256 + 128
  const int n = a.n;

  const int cgp = (warp - kFFirstWorker) >> 2;     // column group 0..3
  const int quad = warp & 3;                       // TMEM lane quarter this warp may touch
  const int t = quad * 32 + lane;
  const uint32_t lane_base = (uint32_t)(quad * 32) << 16;
  const float ema_decay = a.t_decay;
  const float neg_c2 = -a.scale * kLog2e;
  const float heavy_thr = log2f(1.f / kHeavyA) / neg_c2;   // S' above this <=> A > kHeavyA
  // The temporal weights over a run of consecutive window positions i_a..i_b as a Horner chain
  // H = sum c_i I_i decay^(i_b - i): the run contributes t_scale * decay^(w-1-i_b) * H.  For Eq. 9 decay = 1 - alpha,
  // c_0 = 1/alpha (the seed), t_scale = alpha.  Even and odd columns of a run are chained separately in decay^2
  // (one packed FMA per column pair): H = decay * H_even + H_odd.
  constexpr int kRun = kW < 32 ? kW : 32;                  // columns of one run inside this warpgroup
  const int i_first = (cgp * 32) % kW;
  const float seed_coef = (i_first == 0) ? a.t_seed_first : 1.f;
  const float last_coef = (i_first + kRun == kW) ? a.t_seed_last : 1.f;
  const bool group_max = a.group_max != 0;
  const float fin_scale = a.t_scale * powf(ema_decay, (float)(kW - 1 - (i_first + kRun - 1))) / (group_max ? 1.f : (float)kG);
  const f32x2 d2 = f2_make(ema_decay * ema_decay, ema_decay * ema_decay);
  const f32x2 nc2 = f2_make(neg_c2, neg_c2), m1 = f2_make(-1.f, -1.f), tiny2 = f2_make(1e-36f, 1e-36f);
  const f32x2 seed2 = f2_make(seed_coef, 1.f), last2 = f2_make(1.f, last_coef);
  // the shares of the four warpgroups: every 32 columns are one query head's window when w = 32, several whole
  // windows when w < 32, half a window when w = 64 and a quarter when w = 128
  auto join_shares = [group_max](float r0, float r1, float r2, float r3) {
    if (!group_max || kW == 128) return (r0 + r1) + (r2 + r3);
    if (kW == 64) return fmaxf(r0 + r1, r2 + r3);
    return fmaxf(fmaxf(r0, r1), fmaxf(r2, r3));
  };
  const float* O_head = a.O_f32 + (long long)bh * kRows * kHeadDim;
  const __nv_bfloat16* V_head = a.V + (long long)b * a.vsb + (long long)h * a.vsh;
  // with the output projection the token's own term is v^T Mt v of the query head that this warpgroup's 32 columns
  // belong to (w >= 32 there), and the exact distances go through that head's Mt
  const int g_cols = (cgp * 32) / kW;
  const float* vn_head = kProj ? a.vmv + ((long long)bh * kG + g_cols) * a.n_kv : a.vnorm + (long long)bh * a.n_kv;
  const float* Mt_g = kProj ? a.proj_Mt + (long long)(h * kG + g_cols) * kHeadDim * kHeadDim : nullptr;
  const float* Op_head = kProj ? a.O_proj + (long long)bh * kRows * kHeadDim : nullptr;
  // S' above this <=> A > 0.9: under the projection only those entries take the exact quadratic form; the others
  // above kHeavyA take its expansion in fp32 from exact dot products, which is accurate while 1 - A is not small
  const float extreme_thr = log2f(1.f / 0.9f) / neg_c2;
  auto exact_dist2 = [&](int row, int js, bool extreme) {
    const __nv_bfloat16* v_row = V_head + (long long)js * a.vsn;
    if (!kProj) return exact_dist2_warp(O_head + row * kHeadDim, v_row, lane);
    if (extreme) return exact_proj_dist2_warp(O_head + row * kHeadDim, Op_head + row * kHeadDim, v_row, Mt_g, lane);
    return expanded_proj_dist2_warp(O_head + row * kHeadDim, Op_head + row * kHeadDim, v_row, vn_head[js], lane);
  };
  float* I_head = a.I_hat + (long long)bh * n;
  float* raw_head = (a.I_raw && !kLse) ? a.I_raw + (long long)bh * kRows * n : nullptr;
  bool ok = true;
  const int nt_all = (a.n_kv + kTile - 1) / kTile;
  // a tile needs exact distances iff some row's largest logit in it reaches that row's M2 - log2(1 / kHeavyA);
  // every warp checks all 128 rows (lane = rows lane, lane + 32, ...) so that no synchronisation is needed
  const float* tm_head = a.tile_max + (long long)bh * nt_all * kRows;
  float m2r[4], tm_next[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    m2r[k] = a.row_M2[(long long)bh * kRows + k * 32 + lane] - log2f(1.f / kHeavyA);
    tm_next[k] = -INFINITY;
  }
  float vn_next = 0.f;
  // from_lse: no phase A has left ||v||^2 and the tiles' row maxima behind; ||v||^2 comes from the control warps
  // through shared memory and a warp finds out from the logits themselves whether its part of a tile is heavy
  constexpr bool from_lse = kLse;
  const bool vn_global = !from_lse || kProj;   // the token's own term is read from global memory
  if (T > 0 && vn_global) {
    const int j = (tile0 + T - 1) * kTile + t;
    vn_next = (j < n) ? vn_head[j] : 1.f;
  }
  if (T > 0 && !from_lse) {
#pragma unroll
    for (int k = 0; k < 4; ++k) tm_next[k] = tm_head[(long long)(tile0 + T - 1) * kRows + k * 32 + lane];
  }

  for (int it = 0; it < T; ++it) {
    const int s = it & 1;
    const uint32_t par = (uint32_t)(it >> 1) & 1u;
    float vn = vn_next;
    // only Eq. 7 has the factor 1 / (1 - A) and the distance that need the exact form near A = 1
    const bool tile_heavy = raw_head != nullptr ||
                            (kEq7 && __any_sync(0xffffffffu, tm_next[0] > m2r[0] || tm_next[1] > m2r[1] ||
                                                                      tm_next[2] > m2r[2] || tm_next[3] > m2r[3]));
    if (from_lse) {
      ok = ok && mbar_wait(&B->vn_full[it & 3], (uint32_t)(it >> 2) & 1u, abort_flag, dev_status, kDevTimeout, a.wait_limit);
      const int jv = (tile0 + T - 1 - it) * kTile + t;
      if (!vn_global) vn = (ok && jv < n) ? cx.vn_s[(it & 3) * kTile + t] : 1.f;
    }
    if (it + 1 < T && vn_global) {   // next tile's ||v||^2 (or v^T Mt v), well ahead of its use
      const int jn = (tile0 + T - 2 - it) * kTile + t;
      vn_next = (jn < n) ? vn_head[jn] : 1.f;
    }
    if (it + 1 < T && !from_lse) {   // next tile's row maxima
#pragma unroll
      for (int k = 0; k < 4; ++k) tm_next[k] = tm_head[(long long)(tile0 + T - 2 - it) * kRows + k * 32 + lane];
    }
    // The shares of the previous tile are summed in a fixed order by warpgroup 0 once all sixteen warps have
    // stored theirs.  A slot of `red` is rewritten four tiles later, which the two accumulator buffers only
    // allow after every warp has moved past this point.
    if (it > 0 && cgp == 0) {
      const int rs = (it - 1) & 3;
      ok = ok && mbar_wait(&B->red_full[rs], (uint32_t)((it - 1) >> 2) & 1u, abort_flag, dev_status, kDevTimeout, a.wait_limit);
      const int jp = (tile0 + T - it) * kTile + t;
      if (ok && jp < n) I_head[jp] = join_shares(red[rs][0][t], red[rs][1][t], red[rs][2][t], red[rs][3][t]);
    }
    ok = ok && mbar_wait(&B->acc_full[s], par, abort_flag, dev_status, kDevTimeout, a.wait_limit);
    float tot = 0.f;
    if (ok) {
      tc_fence_after();
      const int j = (tile0 + T - 1 - it) * kTile + t;
      const uint32_t tS = tmem + (uint32_t)s * 256u + lane_base + (uint32_t)cgp * 32u, tC = tS + 128u;
      // ||o - v||^2 = C' + ||v||^2 is formed with ||v||^2 raised by 2^-16 of itself: a bias of ~1e-5 that keeps
      // the sum positive when the expansion cancels, so that no clamp is needed.
      const float vnb = vn * 1.0000152587890625f;
      const f32x2 vn2 = f2_make(vnb, vnb);
      const float vlen = kInd == 2 ? sqrtf(vn) : 1.f;          // ||v_j||
      const f32x2 vlen2 = f2_make(vlen, vlen);
      f32x2 h2 = f2_make(0.f, 0.f);
      float sv0[16], cv0[16], sv1[16], cv1[16];
      if (!tile_heavy) {
        tmem_ld16(tS, sv0);
        if (kEq7) tmem_ld16(tC, cv0);
        tmem_wait_ld();
        tmem_ld16(tS + 16, sv1);   // the second half of the columns travels while the first is worked on
        if (kEq7) tmem_ld16(tC + 16, cv1);
      }
      bool redo_heavy = false;   // from_lse: this warp found a weight above kHeavyA among the logits it holds
      if (!tile_heavy) {
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const float* sv = c == 0 ? sv0 : sv1;
          const float* cv = c == 0 ? cv0 : cv1;
          if (c == 1) {
            tmem_wait_ld();
            // every tensor-memory read of this tile is done: the MMA warp may refill the accumulators
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&B->acc_empty[s]);
            if (from_lse && kEq7) {
              // no pass 1 has flagged the tiles with large weights: the warp looks at the logits it now holds in
              // registers (S' above heavy_thr <=> A > kHeavyA) and, if it finds one, does its part of the tile again
              // below with exact distances, from those registers (the accumulators are already released)
              float mx = fmaxf(sv0[0], sv1[0]);
#pragma unroll
              for (int u = 1; u < 16; ++u) mx = fmaxf(mx, fmaxf(sv0[u], sv1[u]));
              redo_heavy = __any_sync(0xffffffffu, mx > heavy_thr && j < n);
              if (redo_heavy) break;
            }
          }
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const f32x2 nt = f2_mul(f2_make(sv[2 * q], sv[2 * q + 1]), nc2);
            f32x2 Iq;
            if (kEq7) {
              const f32x2 um = f2_add(f2_make(ex2_approx(f2_lo(nt)), ex2_approx(f2_hi(nt))), m1);   // 1/A - 1
              const f32x2 x = f2_add(f2_make(cv[2 * q], cv[2 * q + 1]), vn2);                       // ||o - v||^2
              const f32x2 bq = f2_fma(f2_mul(x, um), um, tiny2);                                    // x (1/A - 1)^2
              Iq = f2_mul(x, f2_make(rsqrt_approx(f2_lo(bq)), rsqrt_approx(f2_hi(bq))));
            } else {
              Iq = f2_make(ex2_approx(-f2_lo(nt)), ex2_approx(-f2_hi(nt)));                         // A
              if (kInd == 2) Iq = f2_mul(Iq, vlen2);
            }
            if (q == 0 && (c * 16) % kRun == 0) Iq = f2_mul(Iq, seed2);
            if (q == 7 && (c * 16 + 16) % kRun == 0) Iq = f2_mul(Iq, last2);
            h2 = f2_fma(h2, d2, Iq);
          }
          if ((c * 16 + 16) % kRun == 0) {   // end of a run
            const float run = fmaf(f2_lo(h2), ema_decay, f2_hi(h2));
            tot = group_max ? fmaxf(tot, run) : tot + run;
            h2 = f2_make(0.f, 0.f);
          }
        }
        if (from_lse && kEq7 && redo_heavy) {
          tot = 0.f;
          h2 = f2_make(0.f, 0.f);
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            const float* sv = (c < 2 ? sv0 : sv1) + (c & 1) * 8;
            const float* cv = (c < 2 ? cv0 : cv1) + (c & 1) * 8;
            float I[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
              const float um = ex2_approx(sv[u] * neg_c2) - 1.f;
              float x = cv[u] + vnb;
              unsigned int todo = __ballot_sync(0xffffffffu, sv[u] > heavy_thr && j < n);
              while (todo) {
                const int src = __ffs(todo) - 1;
                todo &= todo - 1;
                const int js = __shfl_sync(0xffffffffu, j, src);
                const float d2x = exact_dist2(cgp * 32 + c * 8 + u, js, __shfl_sync(0xffffffffu, sv[u] > extreme_thr, src) != 0);
                if (lane == src) x = d2x;
              }
              I[u] = x * rsqrt_approx(fmaf(x * um, um, 1e-36f));
            }
            if ((c * 8) % kRun == 0) I[0] *= seed_coef;
            if ((c * 8 + 8) % kRun == 0) I[7] *= last_coef;
#pragma unroll
            for (int q = 0; q < 4; ++q) h2 = f2_fma(h2, d2, f2_make(I[2 * q], I[2 * q + 1]));
            if ((c * 8 + 8) % kRun == 0) {   // end of a run
              const float run = fmaf(f2_lo(h2), ema_decay, f2_hi(h2));
              tot = group_max ? fmaxf(tot, run) : tot + run;
              h2 = f2_make(0.f, 0.f);
            }
          }
        }
      } else {
        // rare: the tile may hold large attention weights; those entries take the exact distance.  Also the
        // epilogue of every tile when the per-query indicators are wanted.
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float sv[8], cv[8], I[8];
          tmem_ld8(tS + c * 8, sv);
          tmem_ld8(tC + c * 8, cv);
          tmem_wait_ld();
#pragma unroll
          for (int u = 0; u < 8; ++u) {
            if (kEq7) {
              const float um = ex2_approx(sv[u] * neg_c2) - 1.f;
              float x = cv[u] + vnb;
              // the whole warp computes the exact distance of each of its lanes' heavy entries in turn
              unsigned int todo = __ballot_sync(0xffffffffu, sv[u] > heavy_thr && j < n);
              while (todo) {
                const int src = __ffs(todo) - 1;
                todo &= todo - 1;
                const int js = __shfl_sync(0xffffffffu, j, src);
                const float d2x = exact_dist2(cgp * 32 + c * 8 + u, js, __shfl_sync(0xffffffffu, sv[u] > extreme_thr, src) != 0);
                if (lane == src) x = d2x;
              }
              I[u] = x * rsqrt_approx(fmaf(x * um, um, 1e-36f));
            } else {
              I[u] = ex2_approx(-sv[u] * neg_c2) * vlen;
            }
          }
          if (raw_head && j < n) {
#pragma unroll
            for (int u = 0; u < 8; ++u) raw_head[(long long)(cgp * 32 + c * 8 + u) * n + j] = I[u];
          }
          if ((c * 8) % kRun == 0) I[0] *= seed_coef;
          if ((c * 8 + 8) % kRun == 0) I[7] *= last_coef;
#pragma unroll
          for (int q = 0; q < 4; ++q) h2 = f2_fma(h2, d2, f2_make(I[2 * q], I[2 * q + 1]));
          if ((c * 8 + 8) % kRun == 0) {   // end of a run
            const float run = fmaf(f2_lo(h2), ema_decay, f2_hi(h2));
            tot = group_max ? fmaxf(tot, run) : tot + run;
            h2 = f2_make(0.f, 0.f);
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&B->acc_empty[s]);
      }
    } else {
      __syncwarp();
      if (lane == 0) mbar_arrive(&B->acc_empty[s]);
    }
    red[it & 3][cgp][t] = tot * fin_scale;
    __syncwarp();
    if (lane == 0) mbar_arrive(&B->red_full[it & 3]);
  }
  if (T > 0 && cgp == 0) {
    const int rs = (T - 1) & 3;
    ok = ok && mbar_wait(&B->red_full[rs], (uint32_t)((T - 1) >> 2) & 1u, abort_flag, dev_status, kDevTimeout, a.wait_limit);
    const int jl = tile0 * kTile + t;   // the last tile processed is the first of the share
    if (ok && jl < n) I_head[jl] = join_shares(red[rs][0][t], red[rs][1][t], red[rs][2][t], red[rs][3][t]);
  }
}

// ------------------------------------------------------------------------------------------------
struct Plan {
  int group, rank, tile0, T1, T2;
};

// Scores map to unsigned keys whose order matches the float order.
__device__ __forceinline__ unsigned int sel_key(float x) {
  const unsigned int u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// ------------------------------------------------------------------------------------------------
// Pooling, selection and gather of one head by its group of CTAs, run by the sixteen worker warps right after the
// head's phase C (the control warps run the matching group barriers).  CTA `rank` owns the tokens of its tiles, a
// contiguous run [j_first, j_first + cnt) of the head; lower ranks own lower tokens.
//   1. after a group barrier (every I_hat of the head is written): box mean of Eq. 13 over the own run (taps staged
//      in shared memory, summed in ascending order), pooled scores to global memory, their keys kept in shared memory;
//   2. four radix passes over 8-bit digits from the top: per-warp histograms of the keys that match the digits
//      chosen so far, summed per CTA, added to the group's histogram in global memory; the CTA also publishes the
//      suffix sums of its own histogram.  After the pass's group barrier every CTA finds the digit that holds the
//      keep-th largest key and adds up, from the suffix sums of the lower ranks, how many keys above it they hold;
//   3. ordered emit: indices ascending, every key above the threshold key T plus the first ones equal to it (the
//      lower index wins ties), at positions that continue the lower ranks' counts;
//   4. after a last group barrier the rows of the head's `keep` indices are copied, an equal share per CTA.
// Returns false once a wait of the CTA has run out.
__device__ bool select_worker(const Ctx& cx, const FusedArgs& a, const Plan& pl, int bh, volatile int* go) {
  const int tid = (int)threadIdx.x - kFFirstWorker * 32, lane = cx.lane, wq = cx.warp - kFFirstWorker;
  constexpr int kT = kFWorkerWarps * 32;
  const int n = a.n, n_kv = a.n_kv, keep = a.sel_keep;
  const int j_first = pl.tile0 * kTile;
  const int cnt = max(0, min(n_kv, (pl.tile0 + pl.T1) * kTile) - j_first);
  unsigned int* wh = reinterpret_cast<unsigned int*>(cx.gen_base + kOffQ);   // [16 warps][256]
  unsigned int* hist_s = wh + kFWorkerWarps * 256;                            // [256]
  unsigned int* misc = hist_s + 256;                                          // digit, remaining, gt/eq of lower ranks, warp sums
  unsigned int* keys = misc + 64;                                             // [kSelMaxKeys]
  float* staged = reinterpret_cast<float*>(keys + kSelMaxKeys);               // [kSelMaxKeys + 2 * kSelHalo]
  static_assert((kFWorkerWarps * 256 + 256 + 64 + 2 * kSelMaxKeys + 2 * kSelHalo) * 4 <= kOffRing + kFRing * kTileBytes,
                "the selection's buffers must fit the operand tiles and the ring");

  if (!group_barrier_follow(go)) return false;   // every CTA of the group has written its I_hat of this head
  // ---- 1. pooling ----
  {
    const int W = a.sel_W, gamma = a.sel_gamma, half = W / 2;
    const float* src = a.I_hat + (long long)bh * n;
    const long long lo64 = (long long)j_first - half + gamma, hi64 = (long long)j_first + cnt - 1 + half + gamma;
    const int s_lo = lo64 < 0 ? 0 : (int)(lo64 < n ? lo64 : n), s_hi = hi64 > n - 1 ? n - 1 : (int)(hi64 > -1 ? hi64 : -1);
    for (int t0 = s_lo + tid; t0 <= s_hi; t0 += 8 * kT) {   // several loads in flight per thread
      float v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int t = t0 + k * kT;
        v[k] = t <= s_hi ? __ldcg(src + t) : 0.f;
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int t = t0 + k * kT;
        if (t <= s_hi) staged[t - s_lo] = v[k];
      }
    }
    named_barrier_sync(1, kT);
    float* srow = a.sel_scores + (long long)bh * n_kv + j_first;
    const float fw = (float)W;
    for (int jj = tid; jj < cnt; jj += kT) {
      const int j = j_first + jj;
      float out = INFINITY;
      if (j < n) {
        const long long a64 = (long long)j - half + gamma, b64 = (long long)j + half + gamma;
        const int ta = a64 < s_lo ? s_lo : (int)(a64 <= s_hi ? a64 : s_hi + 1), tb = b64 > s_hi ? s_hi : (int)(b64 >= s_lo ? b64 : s_lo - 1);
        float acc = 0.f;
        if (a.pool_max) {   // Appendix G.2: maximum over the box, taps outside the scored rows count as 0
          for (int t = ta; t <= tb; ++t) acc = fmaxf(acc, staged[t - s_lo]);
          out = acc;
        } else {
          for (int t = ta; t <= tb; ++t) acc += staged[t - s_lo];
          out = acc / fw;
        }
      }
      srow[jj] = out;
      keys[jj] = sel_key(out);
    }
    if (tid < 4) misc[2 + tid] = 0u;
    named_barrier_sync(1, kT);
  }
  // ---- 2. radix passes ----
  unsigned int prefix = 0, remaining = (unsigned int)keep;
  // one slot per CTA, reused from head to head: a CTA has read its peers' sums of a head before it passes that
  // head's last group barrier, and the peers write the next head's only after it
  unsigned int* sfx_mine = a.sel_sfx + ((long long)pl.group * a.cpg + pl.rank) * kSelPasses * kSfxStride;
#pragma unroll 1
  for (int p = 0; p < kSelPasses; ++p) {
    const int lo = 24 - 8 * p;
    for (int b = tid; b < kFWorkerWarps * 256; b += kT) wh[b] = 0u;
    named_barrier_sync(1, kT);
    for (int jj = tid; jj < cnt; jj += kT) {
      const unsigned int key = keys[jj];
      if (p == 0 || ((key ^ prefix) >> (lo + 8)) == 0u) atomicAdd(&wh[wq * 256 + ((key >> lo) & 255u)], 1u);
    }
    named_barrier_sync(1, kT);
    if (tid < 256) {
      unsigned int h = 0;
#pragma unroll 4
      for (int w = 0; w < kFWorkerWarps; ++w) h += wh[w * 256 + tid];
      hist_s[tid] = h;
      if (h) atomicAdd(a.sel_hist + ((long long)bh * kSelPasses + p) * 256 + tid, h);
    }
    named_barrier_sync(1, kT);
    if (wq == 0) {
      // suffix sums of the CTA's histogram: sfx[b] = keys of this CTA, matching the digits so far, with digit >= b
      unsigned int mine[8], sum = 0;
#pragma unroll
      for (int k = 7; k >= 0; --k) { sum += hist_s[8 * lane + k]; mine[k] = sum; }   // within the lane's eight bins
      unsigned int above = sum;                                                      // inclusive over lanes >= this one
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const unsigned int t = __shfl_down_sync(0xffffffffu, above, off);
        if (lane + off < 32) above += t;
      }
      above -= sum;                                                                  // lanes above this one
      unsigned int* dst = sfx_mine + p * kSfxStride + 8 * lane;
#pragma unroll
      for (int k = 0; k < 8; ++k) dst[k] = mine[k] + above;
      if (lane == 31) dst[8] = 0u;   // sfx[256]
    }
    if (!group_barrier_follow(go)) return false;
    if (wq == 0) {
      // lane L owns bins 255-8L .. 248-8L of the group's histogram, so that the lanes walk the bins from the top
      const unsigned int* gh = a.sel_hist + ((long long)bh * kSelPasses + p) * 256;
      unsigned int mine[8], sum = 0;
#pragma unroll
      for (int k = 0; k < 8; ++k) { mine[k] = __ldcg(gh + 255 - 8 * lane - k); sum += mine[k]; }
      unsigned int incl = sum;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const unsigned int t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
      }
      unsigned int acc = incl - sum;
      if (acc < remaining && remaining <= incl) {   // exactly one lane
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          if (acc < remaining && remaining <= acc + mine[k]) {
            misc[0] = (unsigned int)(255 - 8 * lane - k);
            misc[1] = remaining - acc;
          }
          acc += mine[k];
        }
      }
    }
    named_barrier_sync(1, kT);
    const unsigned int d = misc[0];
    remaining = misc[1];
    prefix |= d << lo;
    if (wq == 1) {
      // keys of the lower ranks above the chosen digit (and, in the last pass, equal to the threshold key)
      unsigned int g = 0, e = 0;
      for (int r = lane; r < pl.rank; r += 32) {
        const unsigned int* sr = a.sel_sfx + (((long long)pl.group * a.cpg + r) * kSelPasses + p) * kSfxStride;
        const unsigned int above = __ldcg(sr + d + 1);
        g += above;
        if (p == kSelPasses - 1) e += __ldcg(sr + d) - above;
      }
      g = __reduce_add_sync(0xffffffffu, g);
      e = __reduce_add_sync(0xffffffffu, e);
      if (lane == 0) { misc[2] += g; misc[3] += e; }
    }
    named_barrier_sync(1, kT);   // misc[0..1] may be rewritten, misc[2..3] are final after the last pass
  }
  const unsigned int T = prefix, need_eq = remaining;
  // ---- 3. ordered emit: warp wq owns a contiguous run of the CTA's tokens ----
  {
    int32_t* dst = a.sel_indices + (long long)bh * keep;
    unsigned int* warp_a = misc + 8;
    unsigned int* warp_b = misc + 8 + kFWorkerWarps;
    const int cw = (((cnt + kFWorkerWarps - 1) / kFWorkerWarps) + 31) & ~31;
    const int wbeg = min(cnt, wq * cw), wend = min(cnt, wbeg + cw);
    const unsigned int lt_mask = (1u << lane) - 1u;
    unsigned int cgt = 0, ceq = 0;
    for (int base = wbeg; base < wend; base += 32) {
      const int jj = base + lane;
      const bool valid = jj < wend;
      const unsigned int key = valid ? keys[jj] : 0u;
      cgt += __popc(__ballot_sync(0xffffffffu, valid && key > T));
      ceq += __popc(__ballot_sync(0xffffffffu, valid && key == T));
    }
    if (lane == 0) { warp_a[wq] = cgt; warp_b[wq] = ceq; }
    named_barrier_sync(1, kT);
    unsigned int run_gt = misc[2], run_eq = misc[3];
    for (int w = 0; w < wq; ++w) { run_gt += warp_a[w]; run_eq += warp_b[w]; }
    for (int base = wbeg; base < wend; base += 32) {
      const int jj = base + lane;
      const bool valid = jj < wend;
      const unsigned int key = valid ? keys[jj] : 0u;
      const bool gt = valid && key > T, eq = valid && key == T;
      const unsigned int mgt = __ballot_sync(0xffffffffu, gt), meq = __ballot_sync(0xffffffffu, eq);
      const unsigned int gt_before = run_gt + __popc(mgt & lt_mask);
      const unsigned int eq_before = run_eq + __popc(meq & lt_mask);
      if (gt || (eq && eq_before < need_eq)) {
        const unsigned int pos = gt_before + min(eq_before, need_eq);
        if (pos < (unsigned int)keep) dst[pos] = (int32_t)(j_first + jj);
      }
      run_gt += __popc(mgt);
      run_eq += __popc(meq);
    }
  }
  if (!group_barrier_follow(go)) return false;   // all indices of the head are written
  // ---- 4. gather: an equal share of the head's rows per CTA, eight 16-byte chunks in flight per thread ----
  {
    const int b = bh / a.Hkv, h = bh % a.Hkv;
    const int share = (keep + a.cpg - 1) / a.cpg;
    const int first = min(keep, pl.rank * share), mine = min(keep, first + share) - first;
    const int32_t* idx = a.sel_indices + (long long)bh * keep + first;
    const __nv_bfloat16* Kh = a.K + (long long)b * a.ksb + (long long)h * a.ksh;
    const __nv_bfloat16* Vh = a.V + (long long)b * a.vsb + (long long)h * a.vsh;
    constexpr int kRC = kHeadDim * 2 / 16;   // 16-byte chunks per row
    const int total = mine * 2 * kRC;
    for (int e0 = tid; e0 < total; e0 += 8 * kT) {
      long long jj[8];
      uint4 val[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int e = e0 + k * kT;
        jj[k] = e < total ? __ldcg(idx + e / (2 * kRC)) : 0;
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int e = e0 + k * kT;
        const int c = e % (2 * kRC);
        const bool isV = c >= kRC;
        const uint4* srcp = reinterpret_cast<const uint4*>(isV ? Vh + jj[k] * a.vsn : Kh + jj[k] * a.ksn) + (isV ? c - kRC : c);
        if (e < total) val[k] = __ldg(srcp);
      }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int e = e0 + k * kT;
        if (e >= total) continue;
        const int r = e / (2 * kRC), c = e % (2 * kRC);
        const bool isV = c >= kRC;
        uint4* outp = reinterpret_cast<uint4*>((isV ? a.V_out : a.K_out) + ((long long)bh * keep + first + r) * kHeadDim) + (isV ? c - kRC : c);
        *outp = val[k];
      }
    }
  }
  // the buffers lie where the operand tiles of the next head land, and they covered the block of ones
  named_barrier_sync(1, kT);
  if (tid < (int)(kOnesBytes / 4)) reinterpret_cast<uint32_t*>(cx.gen_base + kOffOnes)[tid] = 0x3F803F80u;
  fence_proxy_async_smem();
  return true;
}



// The two role loops below run through the same sequence of CTA-wide synchronisations: per head a barrier
// re-initialisation (from the second head on), phase A, the prefetch point, group barrier, phase B, group
// barrier, phase C, and a closing __syncthreads.

// Warps 0-3: TMA producer, MMA issuer, the two ||v||^2 warps; thread 0 also runs the group barriers.
template <int kW, bool kLse>
__device__ void control_main(const Ctx& cx, const FusedArgs& a, const Plan& pl, const CUtensorMap* tmQ,
                             const CUtensorMap* tmK, const CUtensorMap* tmV, const CUtensorMap* tmO,
                             const CUtensorMap* tmAug, FusedBars* bars, int* abort_flag, int* go) {
  unsigned int* counter = a.counters + pl.group;
  unsigned int epoch = 0;
  for (int bh = pl.group; bh < a.BH; bh += a.groups) {
    if (bh != pl.group) {   // fresh barriers for every head: nothing is in flight between two __syncthreads
      if (threadIdx.x == 0) init_bars(bars, false, kLse);
      __syncthreads();
    }
    if (kLse) {
      // O and the rows' normalisers are given: phase C only, and no CTA waits for another
      phase_c_control<kW, kLse>(cx, a, tmQ, tmO, tmAug, tmK, tmV, bh, pl.tile0, pl.T2, 0);
      tc_fence_before();
      __syncthreads();
      tc_fence_after();
      if (a.sel_keep > 0) {   // as below: the worker warps pool, select and gather; this side runs the group barriers
        bool sel_ok = true;
        for (int i = 0; i < kSelBarriers && sel_ok; ++i)
          sel_ok = group_barrier(counter, (++epoch) * (unsigned int)a.cpg, abort_flag, go, a.dev_status, a.wait_limit);
        if (!sel_ok) break;
        __syncthreads();
      }
      continue;
    }
    phase_a_control(cx, a, tmQ, tmK, tmV, bh, pl.rank, pl.tile0, pl.T1);
    // Phase A no longer needs the tile ring: request phase C's first two K/V stages now, so that they arrive
    // while the group merges its partials (K and V are inputs; only O' depends on the merge).
    __syncthreads();
    const int pre = pl.T2 < 2 ? pl.T2 : 2;
    if (threadIdx.x == 0)
      for (int it = 0; it < pre; ++it)
        load_stage_c(cx, tmK, tmV, bh / a.Hkv, bh % a.Hkv, (pl.tile0 + pl.T2 - 1 - it) * kTile, it);
    bool through = group_barrier(counter, (++epoch) * (unsigned int)a.cpg, abort_flag, go, a.dev_status, a.wait_limit);
    // phase B belongs to the worker warps
    through = through && group_barrier(counter, (++epoch) * (unsigned int)a.cpg, abort_flag, go, a.dev_status, a.wait_limit);
    if (!through) {
      // a barrier gave up: the stages requested above must have landed before this CTA may return
      if (threadIdx.x == 0)
        for (int it = 0; it < pre; ++it) wait_issued(&bars->kv_full[it], 0);
      break;
    }
    tc_fence_after();
    phase_c_control<kW, kLse>(cx, a, tmQ, tmO, tmAug, tmK, tmV, bh, pl.tile0, pl.T2, pre);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (a.sel_keep > 0) {   // the worker warps pool, select and gather; this side runs the group barriers
      bool sel_ok = true;
      for (int i = 0; i < kSelBarriers && sel_ok; ++i)
        sel_ok = group_barrier(counter, (++epoch) * (unsigned int)a.cpg, abort_flag, go, a.dev_status, a.wait_limit);
      if (!sel_ok) break;
      __syncthreads();      // the selection's buffers are free for the next head
    }
  }
}

// Warps 4-19: softmax in phase A, the merge of the partials in phase B, the indicator epilogue in phase C.
template <int kW, bool kLse, int kInd>
__device__ void worker_main(const Ctx& cx, const FusedArgs& a, const Plan& pl, const CUtensorMap* tmQ,
                            const CUtensorMap* tmK, const CUtensorMap* tmV, const CUtensorMap* tmO,
                            const CUtensorMap* tmAug, int* go, float (*red)[4][kTile]) {
  for (int bh = pl.group; bh < a.BH; bh += a.groups) {
    if (bh != pl.group) __syncthreads();
    if (kLse) {
      phase_c_worker<kW, kLse, kInd>(cx, a, tmO, tmAug, tmK, tmV, bh, pl.tile0, pl.T2, 0, red);
      tc_fence_before();
      __syncthreads();
      tc_fence_after();
      if (a.sel_keep > 0) {
        if (!select_worker(cx, a, pl, bh, go)) break;
        __syncthreads();
      }
      continue;
    }
    phase_a_worker(cx, a, tmQ, tmK, tmV, bh, pl.rank, pl.tile0, pl.T1);
    __syncthreads();
    if (!group_barrier_follow(go)) break;
    {
      const int wq = cx.warp - kFFirstWorker;
      const int rows_max = (kRows + a.cpg - 1) / a.cpg;          // rows of the busiest CTA of the group
      int wpr = kFWorkerWarps;                                    // warps per row: 16, 8, 4, 2 or 1
      while (wpr > 1 && kFWorkerWarps / wpr < rows_max) wpr >>= 1;
      const int rows_at_once = kFWorkerWarps / wpr;
      float (*xch)[kHeadDim + 4] = reinterpret_cast<float (*)[kHeadDim + 4]>(cx.gen_base + kOffAug);
      for (int k0 = 0; k0 < rows_max; k0 += rows_at_once) {
        const int r = pl.rank + (k0 + wq / wpr) * a.cpg;
        combine_rows<kInd == 3>(a, bh, pl.group, r < kRows ? r : -1, wq % wpr, wpr, wq, cx.lane, xch);
        named_barrier_sync(2, kFWorkerWarps * 32);   // the exchange buffer is reused by the next batch of rows
      }
      fence_proxy_async_smem();   // the exchange buffer is overwritten by a TMA load in phase C
    }
    if (!group_barrier_follow(go)) break;
    tc_fence_after();
    phase_c_worker<kW, kLse, kInd>(cx, a, tmO, tmAug, tmK, tmV, bh, pl.tile0, pl.T2, 0, red);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (a.sel_keep > 0) {
      if (!select_worker(cx, a, pl, bh, go)) break;
      __syncthreads();
    }
  }
}

// ------------------------------------------------------------------------------------------------
template <int kW, bool kLse, int kInd>
__global__ void __launch_bounds__(kFThreads, 1)
tc_fused_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO,
                const __grid_constant__ CUtensorMap tmAug, const FusedArgs a) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) FusedBars bars;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag, go_flag;
  __shared__ float sm_stats[6 * kRows];
  __shared__ float vn_ring[4 * kTile];
  __shared__ float red[4][4][kTile];   // [tile & 3][warpgroup][token]: each warpgroup's share of the score

  const int group = blockIdx.x / a.cpg, rank = blockIdx.x % a.cpg;
  if (group >= a.groups) return;   // CTAs beyond groups * cpg have no work (uniform per CTA)

  Ctx cx;
  cx.smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  cx.gen_base = smem_raw + (cx.smem_base - smem_u32(smem_raw));
  cx.B = &bars;
  cx.abort_flag = &abort_flag;
  cx.sm_stats = sm_stats;
  cx.vn_s = vn_ring;
  cx.warp = threadIdx.x >> 5;
  cx.lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    init_bars(&bars, true, kLse);
    prefetch_tensormap(&tmQ);
    prefetch_tensormap(&tmK);
    prefetch_tensormap(&tmV);
    prefetch_tensormap(&tmO);
    prefetch_tensormap(&tmAug);
  }
  if (cx.warp == 1) {
    tmem_alloc(&tmem_slot, 512);
    tmem_relinquish();
  }
  if (threadIdx.x >= 128 && threadIdx.x < 128 + (int)(kOnesBytes / 4))   // the block of ones (bf16 1.0 = 0x3F80)
    reinterpret_cast<uint32_t*>(cx.gen_base + kOffOnes)[threadIdx.x - 128] = 0x3F803F80u;
  fence_proxy_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  cx.tmem = tmem_slot;
  // the same split of the token tiles in both phases (phase C covers only the scored rows)
  Plan pl;
  pl.group = group;
  pl.rank = rank;
  const int nt1 = (a.n_kv + kTile - 1) / kTile, nt2 = (a.n + kTile - 1) / kTile;
  const int per = (nt1 + a.cpg - 1) / a.cpg;
  pl.tile0 = rank * per;
  pl.T1 = max(0, min(nt1, pl.tile0 + per) - pl.tile0);
  pl.T2 = a.attention_only ? 0 : max(0, min(nt2, pl.tile0 + per) - pl.tile0);

  // Each role's code sits behind its own register-budget change, so that the sixteen worker warps can be
  // compiled for more registers than the launch gives every thread.
  if (cx.warp < kFFirstWorker) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kFRegsControl));
    control_main<kW, kLse>(cx, a, pl, &tmQ, &tmK, &tmV, &tmO, &tmAug, &bars, &abort_flag, &go_flag);
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kFRegsWorker));
    worker_main<kW, kLse, kInd>(cx, a, pl, &tmQ, &tmK, &tmV, &tmO, &tmAug, &go_flag, red);
  }

  tc_fence_before();
  __syncthreads();
  if (cx.warp == 1) {
    tc_fence_after();
    tmem_dealloc(cx.tmem, 512);
  }
}

// ------------------------------------------------------------------------------------------------
// The window rows' outputs O and log-sum-exps given by the caller (the prefill attention has them): what phase B
// would have written for phase C.  One warp per query row, lane = four output dims.
// With the output projection (proj_Mt non-null): the row becomes -2 bf16(Mt o), the constant o^T Mt o, and Mt o is
// kept in O_proj.
__global__ void from_lse_prep_kernel(int rows, float scale, const float* __restrict__ O, const float* __restrict__ LSE,
                                     __nv_bfloat16* __restrict__ O_m2, __nv_bfloat16* __restrict__ aug,
                                     float* __restrict__ row_M2, const float* __restrict__ proj_Mt,
                                     float* __restrict__ O_proj, int Hkv, int w) {
  __shared__ float xs[8][kHeadDim];
  const int wi = threadIdx.x >> 5;
  const int ri = blockIdx.x * (blockDim.x >> 5) + wi, lane = threadIdx.x & 31;
  if (ri >= rows) return;
  const float4 o = *reinterpret_cast<const float4*>(O + (long long)ri * kHeadDim + lane * 4);
  __nv_bfloat16* om = O_m2 + (long long)ri * kHeadDim + lane * 4;
  float on;
  if (proj_Mt) {
    *reinterpret_cast<float4*>(&xs[wi][lane * 4]) = o;
    __syncwarp();
    const int bh = ri / kRows, r = ri % kRows;
    const float4 mo = project_row_warp(proj_Mt + (long long)((bh % Hkv) * (kRows / w) + r / w) * kHeadDim * kHeadDim,
                                       xs[wi], lane);
    *reinterpret_cast<float4*>(O_proj + (long long)ri * kHeadDim + lane * 4) = mo;
    om[0] = __float2bfloat16_rn(-2.f * mo.x);
    om[1] = __float2bfloat16_rn(-2.f * mo.y);
    om[2] = __float2bfloat16_rn(-2.f * mo.z);
    om[3] = __float2bfloat16_rn(-2.f * mo.w);
    on = (o.x * mo.x + o.y * mo.y) + (o.z * mo.z + o.w * mo.w);
  } else {
    const float f0 = __bfloat162float(__float2bfloat16_rn(o.x)), f1 = __bfloat162float(__float2bfloat16_rn(o.y));
    const float f2 = __bfloat162float(__float2bfloat16_rn(o.z)), f3 = __bfloat162float(__float2bfloat16_rn(o.w));
    om[0] = __float2bfloat16_rn(-2.f * f0);   // -2 x is exact for a bf16 x
    om[1] = __float2bfloat16_rn(-2.f * f1);
    om[2] = __float2bfloat16_rn(-2.f * f2);
    om[3] = __float2bfloat16_rn(-2.f * f3);
    on = (f0 * f0 + f1 * f1) + (f2 * f2 + f3 * f3);
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) on += __shfl_xor_sync(0xffffffffu, on, off);
  __nv_bfloat16* arow = aug + (long long)ri * 64;
  arow[2 * lane] = __float2bfloat16_rn(0.f);
  arow[2 * lane + 1] = __float2bfloat16_rn(0.f);
  __syncwarp();
  if (lane == 0) {
    const float c2 = scale * kLog2e;
    const float M2 = LSE[ri] * kLog2e;     // A = exp2(s * c2 - M2)
    row_M2[ri] = M2;
    split3(-M2 / c2, arow);
    split3(on, arow + 16);
  }
}

// SIMT kernels: A = exp(s * scale - fin_m) / fin_l with fin_m = LSE and fin_l = 1.
__global__ void from_lse_prep_simt_kernel(int rows, const float* __restrict__ LSE, float* __restrict__ fin_m,
                                          float* __restrict__ fin_l) {
  const int ri = blockIdx.x * blockDim.x + threadIdx.x;
  if (ri >= rows) return;
  fin_m[ri] = LSE[ri];
  fin_l[ri] = 1.f;
}

}  // namespace

// Number of CTA groups = heads in flight.  With `reuse_l2` only as many as fit a 72 MB share of L2 (phase C then
// re-reads the heads from there); otherwise as many as there are heads.  Among the allowed counts the cheapest wins,
// where a round costs its tiles per CTA plus about eight tiles' worth of pipeline fill, merge and barriers
// (measured); ties go to more groups.
void fused_plan(const Problem& p, int sm_count, bool reuse_l2, int* groups, int* cpg) {
  const long long head_bytes = 2ll * p.n_kv * p.d * 2;
  long long limit = reuse_l2 ? (72ll << 20) / (head_bytes > 0 ? head_bytes : 1) : p.BH;
  if (limit < 1) limit = 1;
  const int tiles = (p.n_kv + kTile - 1) / kTile;
  constexpr int kRoundOverheadTiles = 8;
  int best_g = 1;
  long long best_cost = -1;
  for (int g = 1; g <= p.BH && g <= limit && g <= sm_count && g <= 256; ++g) {
    const int c = sm_count / g;
    const long long cost = (long long)((p.BH + g - 1) / g) * ((tiles + c - 1) / c + kRoundOverheadTiles);
    if (best_cost < 0 || cost <= best_cost) { best_cost = cost; best_g = g; }
  }
  *groups = best_g;
  *cpg = sm_count / best_g;
}

// Whether the score kernel can also pool, select and gather (fixed window): every CTA's share of a head must fit the
// shared-memory buffers, the window must stay within the staged halo, and the budget must leave something out.
bool tc_fused_select_supported(const Problem& p, int sm_count, bool reuse_l2, int keep, int W, int gamma) {
  if (keep < 1 || keep >= p.n_kv) return false;
  if (W / 2 + (gamma < 0 ? -gamma : gamma) > kSelHalo) return false;
  int groups, cpg;
  fused_plan(p, sm_count, reuse_l2, &groups, &cpg);
  // with only a few CTAs per head the separate selection kernel, which puts a cluster of eight on every head, is faster
  if (cpg < 8) return false;
  const int tiles = (p.n_kv + kTile - 1) / kTile, per = (tiles + cpg - 1) / cpg;
  return (long long)per * kTile <= kSelMaxKeys;
}
size_t tc_fused_select_sfx_words(int sm_count) { return (size_t)sm_count * kSelPasses * kSfxStride; }
size_t tc_fused_select_hist_words(int BH) { return (size_t)BH * kSelPasses * 256; }

cudaError_t launch_from_lse_prep(const Problem& p, const Workspace& ws, const float* O, const float* LSE,
                                 bool tensor_core, cudaStream_t st) {
  const int rows = p.BH * p.R;
  if (tensor_core)
    from_lse_prep_kernel<<<(rows + 7) / 8, 256, 0, st>>>(rows, p.scale, O, LSE, ws.O_m2, ws.aug, ws.row_M2, p.proj.Mt,
                                                         ws.O_proj, p.Hkv, p.w);
  else
    from_lse_prep_simt_kernel<<<(rows + 255) / 256, 256, 0, st>>>(rows, LSE, ws.fin_m, ws.fin_l);
  return cudaGetLastError();
}

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
  static TcState the_state;
  the_state.encode = (EncodeTiledFn)fn;
  *state = &the_state;
  return cudaSuccess;
}

// The register split inside the kernel assumes that it was compiled for exactly kFRegsLaunch registers per thread.
template <typename K>
static cudaError_t check_launch_regs(K kernel) {
  cudaFuncAttributes fa;
  cudaError_t e = cudaFuncGetAttributes(&fa, kernel);
  if (e != cudaSuccess) return e;
  return fa.numRegs == kFRegsLaunch ? cudaSuccess : cudaErrorInvalidConfiguration;
}

using FusedKernel = void (*)(CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, CUtensorMap, FusedArgs);

template <int kW>
static FusedKernel pick_fused_w(bool from_lse, int indicator) {
  if (from_lse) {
    if (indicator == 0) return tc_fused_kernel<kW, true, 0>;
    if (indicator == 3) return tc_fused_kernel<kW, true, 3>;
    return indicator == 1 ? tc_fused_kernel<kW, true, 1> : tc_fused_kernel<kW, true, 2>;
  }
  if (indicator == 0) return tc_fused_kernel<kW, false, 0>;
  if (indicator == 3) return tc_fused_kernel<kW, false, 3>;
  return indicator == 1 ? tc_fused_kernel<kW, false, 1> : tc_fused_kernel<kW, false, 2>;
}

// The instantiation for a window length (it only matters to phase C), input form and indicator (3: Eq. 7 under the
// output projection); null if there is none.
static FusedKernel pick_fused(int w, bool from_lse, int indicator) {
  if (indicator < 0 || indicator > 3) return nullptr;
  switch (w) {
    case 16: return pick_fused_w<16>(from_lse, indicator);
    case 32: return pick_fused_w<32>(from_lse, indicator);
    case 64: return pick_fused_w<64>(from_lse, indicator);
    case 128: return pick_fused_w<128>(from_lse, indicator);
    default: return nullptr;
  }
}

cudaError_t tc_fused_init() {
  cudaError_t e = cudaSuccess;
  const int widths[4] = {16, 32, 64, 128};
  for (int w : widths)
    for (int lse = 0; lse < 2; ++lse)
      for (int ind = 0; ind < 4; ++ind) {
        FusedKernel kernel = pick_fused(w, lse != 0, ind);
        if (e == cudaSuccess) e = check_launch_regs(kernel);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kFSmem);
      }
  return e;
}

// Temporal weights of the variant as the kernel's Horner chain (see FusedArgs).  False when the chain cannot carry
// them in fp32: Eq. 9 with alpha = 0, or the inverted EMA when its growth factor (1 / decay)^(w-1) is too large.
static bool temporal_chain(int mode, float ema_decay, int w, float* decay, float* seed_first, float* seed_last,
                           float* scale) {
  const float alpha = 1.f - ema_decay;
  *seed_first = 1.f; *seed_last = 1.f;
  switch (mode) {
    case RESTKV_TEMPORAL_EMA:        // weights alpha * d^(w-1-i), d^(w-1) for the oldest query
      if (!(alpha > 0.f)) return false;
      *decay = ema_decay; *seed_first = 1.f / alpha; *scale = alpha;
      return true;
    case RESTKV_TEMPORAL_MEAN:
      *decay = 1.f; *scale = 1.f / (float)w;
      return true;
    case RESTKV_TEMPORAL_NONE:       // the newest query alone
      *decay = 0.f; *scale = 1.f;
      return true;
    case RESTKV_TEMPORAL_INV_EMA:    // weights alpha * d^i, d^(w-1) for the newest query: a chain in 1 / d
      if (!(alpha > 0.f) || !(ema_decay > 0.f)) return false;
      if ((float)(w - 1) * log2f(1.f / ema_decay) > 40.f) return false;
      *decay = 1.f / ema_decay; *seed_last = 1.f / alpha; *scale = alpha * powf(ema_decay, (float)(w - 1));
      return true;
    default: return false;
  }
}

bool tc_variant_supported(const Problem& p, float ema_decay) {
  float d, sf, sl, sc;
  return temporal_chain(p.temporal, ema_decay, p.w, &d, &sf, &sl, &sc);
}

// One launch for pass 1, the merge and pass 2 of every head.  The CTAs of a group wait for one another, so all of
// them must be resident: the grid never exceeds the SM count and a CTA fills an SM (shared memory), which holds as
// long as the device is not shared with another kernel at that moment; if it is, the bounded group barrier gives up
// with the timeout status instead of hanging.  (A cooperative launch would guarantee residency but costs ~25 us.)
cudaError_t launch_tc_fused(void* state, const Problem& p, const Workspace& ws, const void* Q, const void* K,
                            const void* V, float ema_decay, int sm_count, bool reuse_l2, bool attention_only,
                            long long wait_limit, const FusedSelect* sel, const float* O_given, float* I_raw,
                            unsigned int* dev_status, cudaStream_t st) {
  TcState* ts = (TcState*)state;
  CUtensorMap tmQ, tmK, tmV, tmO, tmAug;
  if (!make_rows_map(ts, &tmQ, Q, p.BH) || !make_rows_map(ts, &tmO, ws.O_m2, p.BH) ||
      !make_aug_map(ts, &tmAug, ws.aug, p.BH) || !make_kv_map(ts, &tmK, K, p, p.ksb, p.ksh, p.ksn) ||
      !make_kv_map(ts, &tmV, V, p, p.vsb, p.vsh, p.vsn))
    return cudaErrorInvalidValue;
  FusedArgs a{};
  a.Hkv = p.Hkv; a.BH = p.BH; a.n = p.n; a.n_kv = p.n_kv; a.w = p.w;
  a.scale = p.scale;
  if (attention_only) {
    a.t_decay = 0.f; a.t_seed_first = a.t_seed_last = a.t_scale = 1.f;
  } else if (!temporal_chain(p.temporal, ema_decay, p.w, &a.t_decay, &a.t_seed_first, &a.t_seed_last, &a.t_scale)) {
    return cudaErrorInvalidValue;
  }
  if (p.proj.Mt && !attention_only) {
    a.proj_Mt = p.proj.Mt; a.vmv = ws.vmv; a.O_proj = ws.O_proj;
  }
  a.group_max = p.group == RESTKV_GROUP_MAX ? 1 : 0;
  a.pool_max = p.spatial == RESTKV_SPATIAL_MAX ? 1 : 0;
  a.attention_only = attention_only ? 1 : 0;
  a.from_lse = O_given ? 1 : 0;
  fused_plan(p, sm_count, reuse_l2, &a.groups, &a.cpg);
  a.part_m = ws.part_m; a.part_l = ws.part_l; a.part_O = ws.part_O;
  a.O_f32 = ws.O_f32; a.O_m2 = ws.O_m2; a.aug = ws.aug; a.vnorm = ws.vnorm; a.I_hat = ws.I_hat;
  a.V = (const __nv_bfloat16*)V; a.vsb = p.vsb; a.vsh = p.vsh; a.vsn = p.vsn;
  a.counters = ws.counters; a.tile_max = ws.tile_max; a.row_M2 = ws.row_M2; a.dev_status = dev_status;
  a.wait_limit = wait_limit;
  a.I_raw = O_given ? nullptr : I_raw;
  if (O_given) a.O_f32 = const_cast<float*>(O_given);   // read only in this mode
  cudaError_t e = cudaMemsetAsync(ws.counters, 0, 1024, st);
  if (e != cudaSuccess) return e;
  if (sel) {
    a.sel_keep = sel->keep; a.sel_W = sel->W; a.sel_gamma = sel->gamma;
    a.sel_scores = sel->scores; a.sel_indices = sel->indices;
    a.sel_hist = ws.sel_hist; a.sel_sfx = ws.sel_sfx;
    a.K = (const __nv_bfloat16*)K; a.ksb = p.ksb; a.ksh = p.ksh; a.ksn = p.ksn;
    a.K_out = (__nv_bfloat16*)sel->K_out; a.V_out = (__nv_bfloat16*)sel->V_out;
    e = cudaMemsetAsync(ws.sel_hist, 0, (size_t)p.BH * kSelPasses * 256 * sizeof(unsigned int), st);
    if (e != cudaSuccess) return e;
  }
  const dim3 grid(a.groups * a.cpg), block(kFThreads);
  FusedKernel kernel = attention_only ? pick_fused(32, false, 0) : pick_fused(p.w, a.from_lse != 0, a.proj_Mt ? 3 : p.indicator);
  if (!kernel) return cudaErrorInvalidValue;
  kernel<<<grid, block, kFSmem, st>>>(tmQ, tmK, tmV, tmO, tmAug, a);
  return cudaGetLastError();
}

}  // namespace restkv
