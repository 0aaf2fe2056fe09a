// Spatial pooling (Eq. 13), top-B selection and row gather (Eq. 14).
#include <cooperative_groups.h>

#include "restkv_common.cuh"

namespace restkv {

namespace {

namespace cg = cooperative_groups;

// ------------------------------------------------------------------------------------------------
// Box mean of Eq. 13 at row j of one head: (1/W) * sum_{k=-W/2+gamma}^{W/2+gamma} I_hat[j+k], taps outside
// [0,n) are zero; rows n..n_kv-1 (the window's own tokens) get +inf.
// pool_max (Appendix G.2): the maximum over the same taps instead, taps outside counting as 0 as well.
__device__ __forceinline__ float box_mean(const float* __restrict__ src, int n, int j, int W, int gamma, bool pool_max) {
  if (j >= n) return INFINITY;
  const int half = W / 2;
  const long long lo64 = (long long)j - half + gamma, hi64 = (long long)j + half + gamma;
  const int lo = lo64 < 0 ? 0 : (int)(lo64 < n ? lo64 : n), hi = hi64 > n - 1 ? n - 1 : (int)(hi64 > -1 ? hi64 : -1);
  float s = 0.f;
  if (pool_max) {
    for (int t = lo; t <= hi; ++t) s = fmaxf(s, src[t]);
    return s;
  }
  for (int t = lo; t <= hi; ++t) s += src[t];
  return s / (float)W;
}

// grid (ceil(n_kv/256), BH).  The window (W, gamma) comes from `pool` (per head, device) when it is non-null.
__global__ void pool_kernel(int n, int n_kv, const float* __restrict__ I_hat, const int* __restrict__ pool, int W,
                            int gamma, bool pool_max, float* __restrict__ scores, int32_t* __restrict__ pool_used) {
  const int bh = blockIdx.y;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (pool) { W = pool[2 * bh]; gamma = pool[2 * bh + 1]; }
  if (pool_used && j == 0) { pool_used[2 * bh] = W; pool_used[2 * bh + 1] = gamma; }
  if (j >= n_kv) return;
  scores[(long long)bh * n_kv + j] = box_mean(I_hat + (long long)bh * n, n, j, W, gamma, pool_max);
}

// ------------------------------------------------------------------------------------------------
// Radix select.  Scores map to unsigned keys whose order matches the float order.
__device__ __forceinline__ unsigned int float_key(float x) {
  const unsigned int u = __float_as_uint(x);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Optional gather fused into the select kernel (all pointers null: indices only).  K, V addressed by element strides;
// K_out, V_out [rows, keep, row_chunks * 16 bytes] contiguous.
struct GatherArgs {
  const unsigned char* K;
  const unsigned char* V;
  unsigned char* K_out;
  unsigned char* V_out;
  long long ksb, ksh, ksn, vsb, vsh, vsn;   // element strides
  int Hkv, esize, row_chunks;
};

constexpr int kSelThreads = 1024;
constexpr int kSelBins = 256;                // 8-bit digits
constexpr int kSelMaxSmemKeys = 44 * 1024;   // keys of one CTA's slice kept in shared memory (176 KB)
constexpr int kSelMaxStagedWidth = 65;       // widest box whose taps are staged in shared memory

// Inclusive scan over the 1024 threads of the block, in thread order.
__device__ __forceinline__ unsigned int block_inclusive_scan(unsigned int v, unsigned int* warp_sums) {
  const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const unsigned int t = __shfl_up_sync(0xffffffffu, v, off);
    if (lane >= off) v += t;
  }
  if (lane == 31) warp_sums[wid] = v;
  __syncthreads();
  if (wid == 0) {
    unsigned int w = warp_sums[lane];
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const unsigned int t = __shfl_up_sync(0xffffffffu, w, off);
      if (lane >= off) w += t;
    }
    warp_sums[lane] = w;   // inclusive over warps
  }
  __syncthreads();
  if (wid > 0) v += warp_sums[wid - 1];
  __syncthreads();   // warp_sums may be reused by the caller
  return v;
}

// Box means of one CTA's slice from its staged taps (staged[t - s_lo] = I_hat[t] for t in [s_lo, s_hi]), summed in
// the same order as box_mean; writes the pooled scores and their keys.  kWidth = 0: width known only at run time.
template <int kWidth>
__device__ __forceinline__ void pool_staged(const float* __restrict__ staged, int s_lo, int s_hi, int n, int j0, int cnt,
                                            int W, int gamma, float* __restrict__ srow, unsigned int* __restrict__ skeys) {
  const int width = kWidth ? kWidth : W;
  const int half = width / 2;
  const float fw = (float)width;
  for (int jj = threadIdx.x; jj < cnt; jj += kSelThreads) {
    const int j = j0 + jj;
    float out = INFINITY;
    if (j < n) {
      const long long a64 = (long long)j - half + gamma, b64 = (long long)j + half + gamma;
      float acc = 0.f;
      if (a64 >= s_lo && b64 <= s_hi) {   // the whole window is staged: fixed trip count
        const float* p = staged + (int)(a64 - s_lo);
        if (kWidth) {
#pragma unroll
          for (int k = 0; k < kWidth; ++k) acc += p[k];
        } else {
          for (int k = 0; k < width; ++k) acc += p[k];
        }
      } else {
        const int a = a64 < s_lo ? s_lo : (int)(a64 <= s_hi ? a64 : s_hi + 1), b = b64 > s_hi ? s_hi : (int)(b64 >= s_lo ? b64 : s_lo - 1);
        for (int t = a; t <= b; ++t) acc += staged[t - s_lo];
      }
      out = acc / fw;
    }
    srow[jj] = out;
    skeys[jj] = float_key(out);
  }
}

// One thread-block cluster per row; CTA `rank` of the cluster owns the contiguous slice [rank*per, (rank+1)*per)
// of the row.  With I_hat non-null the kernel first applies the box mean of Eq. 13 and writes the pooled scores;
// otherwise it reads `scores`.  The keys of the slice stay in shared memory (use_smem) or are re-read from
// `scores`.  The cluster first agrees on the smallest and largest key: the bits they share are common to every
// key and are skipped.  The remaining bits are resolved 8 at a time from the top: every warp counts into its own
// 256-bin histogram (no contention between warps), the CTA sums them, the cluster sums the CTAs' histograms
// through distributed shared memory, and one warp finds the bin that holds the keep-th largest key.  That yields
// the key T of the keep-th largest score and how many scores equal to T are kept; an ordered pass then writes,
// in ascending index order, every index whose key is > T plus the first kept ones whose key equals T (lower
// index wins ties).
// keep_rows non-null: row r keeps min(max(keep_rows[r], 1), keep) entries instead of `keep` (non-uniform budgets);
// its outputs still have a row stride of `keep`, the unused tail of its indices is set to -1.
__global__ void __launch_bounds__(kSelThreads, 1)
select_kernel(int n, int n_kv, int keep, const int* __restrict__ keep_rows, const float* __restrict__ I_hat, const int* __restrict__ pool, int W,
              int gamma, int pool_max, float* scores, int32_t* __restrict__ indices, int32_t* __restrict__ pool_used,
              int per, int use_smem, int stage_taps, GatherArgs ga) {
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned int CS = cluster.num_blocks(), rank = cluster.block_rank();
  const int row = blockIdx.x / CS;
  extern __shared__ unsigned int skeys[];
  __shared__ unsigned int wh[32][kSelBins];    // per-warp histograms
  __shared__ unsigned int hist[2][kSelBins];   // the CTA's histogram of the current pass (double-buffered)
  __shared__ unsigned int tot[kSelBins];       // the cluster's histogram
  __shared__ unsigned int warp_a[32], warp_b[32];
  __shared__ unsigned int s_digit, s_remaining;
  __shared__ unsigned int cta_counts[2];
  __shared__ unsigned int cta_minmax[2];

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const long long j0 = (long long)rank * per;
  const int cnt = (int)max(0ll, min((long long)n_kv, j0 + per) - j0);
  float* srow = scores + (long long)row * n_kv;
  const int out_stride = keep;
  int32_t* dst = indices + (long long)row * out_stride;
  if (keep_rows) {
    keep = min(max(keep_rows[row], 1), out_stride);
    if (rank == 0)
      for (int pos = keep + tid; pos < out_stride; pos += kSelThreads) dst[pos] = -1;
  }

  // ---- keys of the slice ----
  if (I_hat) {
    if (pool) { W = pool[2 * row]; gamma = pool[2 * row + 1]; }
    if (pool_used && rank == 0 && tid == 0) { pool_used[2 * row] = W; pool_used[2 * row + 1] = gamma; }
    const float* src = I_hat + (long long)row * n;
    if (stage_taps && !pool_max && W <= kSelMaxStagedWidth && cnt > 0) {
      // the taps of the whole slice (slice + halo) are staged in shared memory once, then summed from there in
      // the same order as box_mean does
      float* staged = reinterpret_cast<float*>(skeys + per);
      const int half = W / 2;
      const long long lo64 = j0 - half + gamma, hi64 = j0 + cnt - 1 + half + gamma;
      const int s_lo = lo64 < 0 ? 0 : (int)(lo64 < n ? lo64 : n), s_hi = hi64 > n - 1 ? n - 1 : (int)(hi64 > -1 ? hi64 : -1);
      // several loads in flight per thread
      for (int t0 = s_lo + tid; t0 <= s_hi; t0 += 8 * kSelThreads) {
        float v[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int t = t0 + k * kSelThreads;
          v[k] = t <= s_hi ? src[t] : 0.f;
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int t = t0 + k * kSelThreads;
          if (t <= s_hi) staged[t - s_lo] = v[k];
        }
      }
      __syncthreads();
      switch (W) {   // the common widths get a compile-time trip count
        case 1: pool_staged<1>(staged, s_lo, s_hi, n, (int)j0, cnt, W, gamma, srow + j0, skeys); break;
        case 3: pool_staged<3>(staged, s_lo, s_hi, n, (int)j0, cnt, W, gamma, srow + j0, skeys); break;
        case 5: pool_staged<5>(staged, s_lo, s_hi, n, (int)j0, cnt, W, gamma, srow + j0, skeys); break;
        case 7: pool_staged<7>(staged, s_lo, s_hi, n, (int)j0, cnt, W, gamma, srow + j0, skeys); break;
        case 21: pool_staged<21>(staged, s_lo, s_hi, n, (int)j0, cnt, W, gamma, srow + j0, skeys); break;
        case 31: pool_staged<31>(staged, s_lo, s_hi, n, (int)j0, cnt, W, gamma, srow + j0, skeys); break;
        default: pool_staged<0>(staged, s_lo, s_hi, n, (int)j0, cnt, W, gamma, srow + j0, skeys); break;
      }
    } else {
      for (int jj = tid; jj < cnt; jj += kSelThreads) {
        const float out = box_mean(src, n, (int)(j0 + jj), W, gamma, pool_max != 0);
        srow[j0 + jj] = out;
        if (use_smem) skeys[jj] = float_key(out);
      }
    }
  } else if (use_smem) {
    for (int jj = tid; jj < cnt; jj += kSelThreads) skeys[jj] = float_key(srow[j0 + jj]);
  }
  __syncthreads();
  auto key_at = [&](int jj) -> unsigned int { return use_smem ? skeys[jj] : float_key(srow[j0 + jj]); };

  if (keep >= n_kv) {   // budget covers everything: identity (uniform over the cluster)
    for (int jj = tid; jj < cnt; jj += kSelThreads) dst[j0 + jj] = (int32_t)(j0 + jj);
    if (ga.K) {
      const int b = row / ga.Hkv, h = row % ga.Hkv;
      const unsigned char* Kh = ga.K + ((long long)b * ga.ksb + (long long)h * ga.ksh) * ga.esize;
      const unsigned char* Vh = ga.V + ((long long)b * ga.vsb + (long long)h * ga.vsh) * ga.esize;
      const int rc2 = 2 * ga.row_chunks;
      for (long long e = tid; e < (long long)cnt * rc2; e += kSelThreads) {
        const long long r = e / rc2;
        const int c = (int)(e - r * rc2);
        const bool isV = c >= ga.row_chunks;
        const int chunk = isV ? c - ga.row_chunks : c;
        const long long j = j0 + r;
        const uint4* src = reinterpret_cast<const uint4*>((isV ? Vh + j * ga.vsn * ga.esize : Kh + j * ga.ksn * ga.esize)) + chunk;
        uint4* out = reinterpret_cast<uint4*>((isV ? ga.V_out : ga.K_out) + ((long long)row * out_stride + j) * ga.row_chunks * 16) + chunk;
        *out = __ldg(src);
      }
    }
    return;
  }

  // ---- smallest and largest key of the row ----
  unsigned int kmin = 0xFFFFFFFFu, kmax = 0u;
  for (int jj = tid; jj < cnt; jj += kSelThreads) {
    const unsigned int key = key_at(jj);
    kmin = min(kmin, key);
    kmax = max(kmax, key);
  }
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if (lane == 0) { warp_a[wid] = kmin; warp_b[wid] = kmax; }
  __syncthreads();
  if (wid == 0) {
    kmin = __reduce_min_sync(0xffffffffu, warp_a[lane]);
    kmax = __reduce_max_sync(0xffffffffu, warp_b[lane]);
    if (lane == 0) { cta_minmax[0] = kmin; cta_minmax[1] = kmax; }
  }
  cluster.sync();
  kmin = 0xFFFFFFFFu;
  kmax = 0u;
  for (unsigned int r = 0; r < CS; ++r) {
    const unsigned int* mm = cluster.map_shared_rank(cta_minmax, r);
    kmin = min(kmin, mm[0]);
    kmax = max(kmax, mm[1]);
  }

  // ---- radix passes over the bits in which the keys differ ----
  const unsigned int diff = kmin ^ kmax;
  int hi = diff ? 32 - __clz(diff) : 0;                                  // bits [hi-1 .. 0] vary
  unsigned int prefix = hi >= 32 ? 0u : (kmax >> hi) << hi;              // the bits every key shares
  unsigned int remaining = (unsigned int)keep;
  int pb = 0;
#pragma unroll 1
  while (hi > 0) {
    const int lo = hi > 8 ? hi - 8 : 0;
    const unsigned int dmask = (1u << (hi - lo)) - 1u;
    for (int b = tid; b < 32 * kSelBins; b += kSelThreads) (&wh[0][0])[b] = 0;
    __syncthreads();
    for (int jj = tid; jj < cnt; jj += kSelThreads) {
      const unsigned int key = key_at(jj);
      if (hi >= 32 || ((key ^ prefix) >> hi) == 0) atomicAdd(&wh[wid][(key >> lo) & dmask], 1u);
    }
    __syncthreads();
    if (tid < kSelBins) {
      unsigned int h = 0;
#pragma unroll 8
      for (int wv = 0; wv < 32; ++wv) h += wh[wv][tid];
      hist[pb][tid] = h;
    }
    cluster.sync();
    if (tid < kSelBins) {
      unsigned int h = 0;
      for (unsigned int r = 0; r < CS; ++r) h += cluster.map_shared_rank(&hist[pb][0], r)[tid];
      tot[tid] = h;
    }
    __syncthreads();
    if (wid == 0) {
      // lane L owns bins 255-8L .. 248-8L, so that the lanes walk the bins from the top
      unsigned int mine[8], sum = 0;
#pragma unroll
      for (int k = 0; k < 8; ++k) { mine[k] = tot[kSelBins - 1 - 8 * lane - k]; sum += mine[k]; }
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
            s_digit = (unsigned int)(kSelBins - 1 - 8 * lane - k);
            s_remaining = remaining - acc;
          }
          acc += mine[k];
        }
      }
    }
    __syncthreads();
    prefix |= s_digit << lo;
    remaining = s_remaining;
    hi = lo;
    pb ^= 1;
    // hist[pb] is rewritten two passes later, after another cluster.sync that every peer reaches only once it
    // has finished reading this pass's histograms
  }
  const unsigned int T = prefix;            // key of the keep-th largest score
  const unsigned int need_eq = remaining;   // how many keys equal to T are kept (>= 1)

  // ---- ordered emit: warp `wid` owns a contiguous run of the slice ----
  const int cw = (((cnt + 31) / 32) + 31) & ~31;
  const int wbeg = min(cnt, wid * cw), wend = min(cnt, wbeg + cw);
  const unsigned int lt_mask = (1u << lane) - 1u;
  unsigned int cgt = 0, ceq = 0;
  for (int base = wbeg; base < wend; base += 32) {
    const int jj = base + lane;
    const bool valid = jj < wend;
    const unsigned int key = valid ? key_at(jj) : 0u;
    cgt += __popc(__ballot_sync(0xffffffffu, valid && key > T));
    ceq += __popc(__ballot_sync(0xffffffffu, valid && key == T));
  }
  if (lane == 0) { warp_a[wid] = cgt; warp_b[wid] = ceq; }
  __syncthreads();
  if (wid == 0) {
    unsigned int a = warp_a[lane], b = warp_b[lane];
    const unsigned int a_own = a, b_own = b;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const unsigned int ta = __shfl_up_sync(0xffffffffu, a, off), tb = __shfl_up_sync(0xffffffffu, b, off);
      if (lane >= off) { a += ta; b += tb; }
    }
    warp_a[lane] = a - a_own;   // exclusive over the warps
    warp_b[lane] = b - b_own;
    if (lane == 31) { cta_counts[0] = a; cta_counts[1] = b; }
  }
  __syncthreads();
  cluster.sync();
  unsigned int g_before = 0, e_before = 0;   // totals of the lower ranks of the cluster
  for (unsigned int r = 0; r < rank; ++r) {
    const unsigned int* rc = cluster.map_shared_rank(cta_counts, r);
    g_before += rc[0];
    e_before += rc[1];
  }
  unsigned int run_gt = warp_a[wid] + g_before, run_eq = warp_b[wid] + e_before;
  for (int base = wbeg; base < wend; base += 32) {
    const int jj = base + lane;
    const bool valid = jj < wend;
    const unsigned int key = valid ? key_at(jj) : 0u;
    const bool gt = valid && key > T, eq = valid && key == T;
    const unsigned int mgt = __ballot_sync(0xffffffffu, gt), meq = __ballot_sync(0xffffffffu, eq);
    const unsigned int gt_before = run_gt + __popc(mgt & lt_mask);
    const unsigned int eq_before = run_eq + __popc(meq & lt_mask);
    if (gt || (eq && eq_before < need_eq)) {
      const unsigned int pos = gt_before + min(eq_before, need_eq);
      if (pos < (unsigned int)keep) dst[pos] = (int32_t)(j0 + jj);
    }
    run_gt += __popc(mgt);
    run_eq += __popc(meq);
  }
  if (ga.K) {
    // ---- gather: every CTA of the cluster takes an equal share of the row's `keep` indices, whoever emitted them
    //      (the selected rows may all lie in one CTA's slice) ----
    cluster.sync();   // all indices of the row are written and visible to the cluster
    const unsigned int share = ((unsigned int)keep + CS - 1) / CS;
    const unsigned int first = min((unsigned int)keep, rank * share);
    const unsigned int mine = min((unsigned int)keep, first + share) - first;
    const int b = row / ga.Hkv, h = row % ga.Hkv;
    const unsigned char* Kh = ga.K + ((long long)b * ga.ksb + (long long)h * ga.ksh) * ga.esize;
    const unsigned char* Vh = ga.V + ((long long)b * ga.vsb + (long long)h * ga.vsh) * ga.esize;
    const long long out_row0 = (long long)row * out_stride;
    const int rc2 = 2 * ga.row_chunks;
    // four chunks per thread and round, the index loads first and then the row loads, so that they overlap
    const unsigned int total = mine * (unsigned int)rc2;
    for (unsigned int e0 = tid; e0 < total; e0 += 4 * kSelThreads) {
      long long jj[4];
      uint4 val[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const unsigned int e = e0 + k * kSelThreads;
        jj[k] = e < total ? dst[first + e / rc2] : 0;
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const unsigned int e = e0 + k * kSelThreads;
        const int c = (int)(e % rc2);
        const bool isV = c >= ga.row_chunks;
        const int chunk = isV ? c - ga.row_chunks : c;
        const uint4* src = reinterpret_cast<const uint4*>((isV ? Vh + jj[k] * ga.vsn * ga.esize : Kh + jj[k] * ga.ksn * ga.esize)) + chunk;
        if (e < total) val[k] = __ldg(src);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const unsigned int e = e0 + k * kSelThreads;
        if (e >= total) continue;
        const unsigned int r = e / rc2;
        const int c = (int)(e - r * rc2);
        const bool isV = c >= ga.row_chunks;
        const int chunk = isV ? c - ga.row_chunks : c;
        uint4* out = reinterpret_cast<uint4*>((isV ? ga.V_out : ga.K_out) + (out_row0 + first + r) * ga.row_chunks * 16) + chunk;
        *out = val[k];
      }
    }
  }
  cluster.sync();   // shared memory stays alive until every peer has read cta_counts
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

cudaError_t launch_pool(const Problem& p, const Workspace& ws, const int* pool_dev, int W, int gamma, float* scores,
                        int32_t* pool_used, cudaStream_t st) {
  dim3 grid((p.n_kv + 255) / 256, p.BH);
  pool_kernel<<<grid, 256, 0, st>>>(p.n, p.n_kv, ws.I_hat, pool_dev, W, gamma, p.spatial == RESTKV_SPATIAL_MAX, scores,
                                    pool_used);
  return cudaGetLastError();
}

// rows x n_kv scores -> rows x min(budget, n_kv) indices.  I_hat non-null: pool first (n scored rows per row of
// I_hat, window from pool_dev or (W, gamma)) and write the pooled scores.
cudaError_t launch_select(int rows, int n, int n_kv, int budget, const int* keep_rows, const float* I_hat, const int* pool_dev, int W,
                          int gamma, bool pool_max, float* scores, int32_t* indices, int32_t* pool_used, const Problem* gather,
                          const void* K, const void* V, void* K_out, void* V_out, cudaStream_t st) {
  GatherArgs ga{};
  if (gather) {
    ga.K = (const unsigned char*)K; ga.V = (const unsigned char*)V;
    ga.K_out = (unsigned char*)K_out; ga.V_out = (unsigned char*)V_out;
    ga.ksb = gather->ksb; ga.ksh = gather->ksh; ga.ksn = gather->ksn;
    ga.vsb = gather->vsb; ga.vsh = gather->vsh; ga.vsn = gather->vsn;
    ga.Hkv = gather->Hkv; ga.esize = gather->dtype == RESTKV_BF16 ? 2 : 4; ga.row_chunks = gather->d * ga.esize / 16;
  }
  const int keep = budget < n_kv ? budget : n_kv;
  // CTAs per row: 8 for long rows, fewer when there are so many rows that all clusters would not be resident at
  // once (two 1024-thread CTAs per SM) and the slices still fit in shared memory
  int CS = n_kv > 4096 ? 8 : 1;
  int sms = 148;
  {
    int dev = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  }
  while (CS > 1 && (long long)rows * CS > 2ll * sms && (n_kv + CS / 2 - 1) / (CS / 2) <= kSelMaxSmemKeys / 2) CS >>= 1;
  cudaError_t e = cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       kSelMaxSmemKeys * (int)sizeof(unsigned int));
  if (e != cudaSuccess) return e;
  int per = (n_kv + CS - 1) / CS;
  per = (per + 3) & ~3;
  const int use_smem = per <= kSelMaxSmemKeys ? 1 : 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned int)(rows * CS));
  cfg.blockDim = dim3(kSelThreads);
  // with room for it, the pooling taps of the slice (slice + halo) are staged behind the keys
  const int stage_taps = (I_hat && use_smem && 2 * per + kSelMaxStagedWidth <= kSelMaxSmemKeys) ? 1 : 0;
  cfg.dynamicSmemBytes = use_smem ? (size_t)(stage_taps ? 2 * per + kSelMaxStagedWidth : per) * sizeof(unsigned int) : 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, select_kernel, n, n_kv, keep, keep_rows, I_hat, pool_dev, W, gamma, pool_max ? 1 : 0, scores, indices,
                            pool_used, per, use_smem, stage_taps, ga);
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
