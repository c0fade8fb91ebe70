// Step 2b of VMoBA: global (per head) threshold selection of (query, key-block) pairs
// (Eq. 3 TopkMask, Eq. 4 threshold k), and emission of the work lists the attention
// kernels consume.
//
// Sorting the head's pool and accumulating normalised similarity until tau is reached is
// equivalent to finding the weighted quantile of the scores under the softmax weights:
// the cutoff is the largest score c with mass{score >= c} >= tau * Z.  That is found without
// a sort by three histogram refinements (2048 bins each, linear in the score, fp64 bin
// masses), after which the mask is one comparison per pair.  Every kernel streams the score
// matrix with 16-byte loads; the stage is bound by HBM bandwidth.
//
//   init (+ minmax, unless the caller hands over each head's score range)
//           -> hist level 0 -> scan -> hist level 1 -> scan -> hist level 2 -> scan (cutoff)
//   (level 1 copies the pairs of the level-0 crossing bin aside, and level 2 reads that short list instead of the
//    score matrix: three traversals of the matrix, levels 0 and 1 and mark)
//   mark    : mask bits + per (segment, block) counts + per-segment pair totals
//   offsets : CSR offsets by key block (kb_ptr) and by query (q_ptr)
//   fill    : q_idx (queries of each key block, ascending) and q_pairs (pairs of each query)
#include <algorithm>
#include <type_traits>

#include "common.cuh"

namespace vmoba {

constexpr int kBins = 2048;
constexpr int kBins0 = 512;    // level 0 uses fewer bins, each replicated once per lane
constexpr int kSegThreads = 512;

struct HeadState {
  uint32_t min_key, max_key;   // order-preserving keys of the head's extreme scores
  float anchor[3];             // lower edge of the interval refined at each level
  float inv[3];                // bins per unit score at each level
  int bin[3];                  // crossing bin found at each level
  int resolved;                // the level-1 crossing bin held a single distinct score: level 2 is skipped
  double Z;                    // sum of all weights
  double target;               // tau * Z
  double mass_above;           // weight of everything above the crossing bin so far
  unsigned long long cnt_above;
  uint32_t cutoff_key;
  unsigned int cand_cnt;       // pairs of the level-0 crossing bin, copied aside by the level-1 pass
  int cand_ok;                 // every one of them found room in the list: level 2 reads the list
  float bin0_off;              // -anchor[0] * inv[0]: the level-0 bin of s is floor(s * inv[0] + bin0_off)
  uint32_t pad;
};

// bin of a score at refinement level L given the state; monotone non-decreasing in s.
// Unnormalised softmax weight of a pair relative to the head's largest score (Eq. 4 accumulates these
// in descending score order).  One definition for every histogram level and for the final exact
// steps, so that the masses they hand to each other are sums of the same numbers; the fast
// exponential (one multiply, one ex2) is within a few ulp of expf over the range that carries mass.
// One fused multiply-add and one ex2 per pair: exp(sigma (s - smax)) = 2^(s c - smax c) with c = sigma log2(e);
// c and smax c do not depend on the pair and leave the loops.
__device__ __forceinline__ float pair_weight(float sigma, float s, float smax) {
  const float c = sigma * 1.4426950408889634f;
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(fmaf(s, c, -smax * c)));
  return y;
}

// Level 0 sees every pair: its bin is one fused multiply-add (bin0_off = -anchor[0] * inv[0], a number of bins, so
// its rounding moves a bin edge by a few millionths of a bin) and an integer clamp.  The finer levels keep the
// subtraction first: their inv is so large that the product form would cancel.
__device__ __forceinline__ int bin_at(const HeadState& hs, int L, float s) {
  if (L == 0) return min(max(__float2int_rd(fmaf(s, hs.inv[0], hs.bin0_off)), 0), kBins0 - 1);
  float t = (s - hs.anchor[L]) * hs.inv[L];
  int b = t > 0.f ? (int)fminf(t, (float)(kBins - 1)) : 0;
  return b;
}

// Streams the P scores of one head through f(value); blockIdx.x strides over chunks.
template <typename F>
__device__ __forceinline__ void for_each_score(const float* __restrict__ base, long long P, F f) {
  const long long tid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long nth = (long long)gridDim.x * blockDim.x;
  if ((reinterpret_cast<uintptr_t>(base) & 15u) == 0) {
    long long P4 = P >> 2;
    const float4* b4 = reinterpret_cast<const float4*>(base);
    long long i = tid;
    for (; i + 3 * nth < P4; i += 4 * nth) {     // four independent 16-byte loads in flight
      float4 x[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) x[j] = __ldg(b4 + i + j * nth);
#pragma unroll
      for (int j = 0; j < 4; ++j) { f(x[j].x); f(x[j].y); f(x[j].z); f(x[j].w); }
    }
    for (; i < P4; i += nth) {
      float4 x = __ldg(b4 + i);
      f(x.x); f(x.y); f(x.z); f(x.w);
    }
    for (long long i = (P4 << 2) + tid; i < P; i += nth) f(__ldg(base + i));
  } else {
    for (long long i = tid; i < P; i += nth) f(__ldg(base + i));
  }
}

__global__ void __launch_bounds__(256)
minmax_kernel(const float* __restrict__ scores, long long P, HeadState* __restrict__ st) {
  const int bh = blockIdx.y;
  uint32_t kmin = 0xffffffffu, kmax = 0u;
  for_each_score(scores + (long long)bh * P, P, [&](float s) {
    uint32_t k = float_key(s);
    kmin = min(kmin, k);
    kmax = max(kmax, k);
  });
  kmin = __reduce_min_sync(0xffffffffu, kmin);
  kmax = __reduce_max_sync(0xffffffffu, kmax);
  if ((threadIdx.x & 31) == 0) {
    atomicMin(&st[bh].min_key, kmin);
    atomicMax(&st[bh].max_key, kmax);
  }
}

// Start of a call: the per-head state and, for the head-wide rules, the histogram arrays (one kernel instead of
// a memset per array).  If the caller knows each head's score range (range: [BH][2] = minimum, maximum, as
// vmoba_block_scores_range writes them), the level-0 bins are laid over it here and no pass of the selection's
// own has to look for it.
__global__ void init_state_kernel(HeadState* st, int BH, const float* __restrict__ range, unsigned int* __restrict__ g_cnt,
                                  double* __restrict__ g_w, uint32_t* __restrict__ g_minkey,
                                  uint32_t* __restrict__ g_maxkey) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (g_cnt && i < (long long)BH * kBins) { g_cnt[i] = 0u; g_w[i] = 0.0; g_minkey[i] = 0xffffffffu; g_maxkey[i] = 0u; }
  if (i >= BH) return;
  HeadState h;
  memset(&h, 0, sizeof(h));
  h.min_key = 0xffffffffu;
  h.max_key = 0u;
  h.cutoff_key = 0xffffffffu;      // the per-query rules take the minimum of their row cutoffs into it
  if (range) {
    const float lo = range[2 * i], hi = range[2 * i + 1];
    h.min_key = float_key(lo);
    h.max_key = float_key(hi);
    const float span = hi - lo;
    h.anchor[0] = lo;
    h.inv[0] = span > 0.f ? (float)kBins0 / span : 0.f;
    h.bin0_off = -lo * h.inv[0];
  }
  st[i] = h;
}

// Level L >= 1 histogram: pairs that fall in the crossing bins of all earlier levels add
// (1, exp(sigma * (s - max))) to their level-L bin.  The smallest key of each bin is tracked too,
// which turns the last crossing bin into an exact fp32 cutoff; at level 1 also the largest, so that
// a crossing bin with a single distinct score ends the search there.
template <int L>
__global__ void __launch_bounds__(256)
hist_kernel(const float* __restrict__ scores, long long P, const HeadState* __restrict__ st, float sigma, int unit_w,
            unsigned int* __restrict__ g_cnt, double* __restrict__ g_w, uint32_t* __restrict__ g_minkey,
            uint32_t* __restrict__ g_maxkey, float* __restrict__ cand, long long ccap, unsigned int* __restrict__ cand_cnt) {
  __shared__ unsigned int s_cnt[kBins];
  __shared__ float s_w[kBins];
  __shared__ uint32_t s_min[kBins];
  __shared__ uint32_t s_max[L == 1 ? kBins : 1];
  const int bh = blockIdx.y;
  const HeadState hs = st[bh];
  if (L == 2 && hs.resolved) return;     // level 1 already pinned the cutoff: nothing to refine
  for (int i = threadIdx.x; i < kBins; i += blockDim.x) {
    s_cnt[i] = 0; s_w[i] = 0.f;
    s_min[i] = 0xffffffffu;
    if (L == 1) s_max[i] = 0u;
  }
  __syncthreads();
  const float smax = key_float(hs.max_key);
  // level 1 copies the pairs of the level-0 crossing bin (one bin of 512: few) to the head's list; level 2 reads
  // the list instead of the matrix if all of them found room
  float* list = cand ? cand + (long long)bh * ccap : nullptr;
  const bool from_list = L == 2 && hs.cand_ok;
  const float* src = from_list ? list : scores + (long long)bh * P;
  const long long n_src = from_list ? (long long)hs.cand_cnt : P;
  for_each_score(src, n_src, [&](float s) {
    if (L >= 1 && bin_at(hs, 0, s) != hs.bin[0]) return;
    if (L == 1 && list) {
      const unsigned int pos = atomicAdd(cand_cnt + bh * (sizeof(HeadState) / sizeof(unsigned int)), 1u);
      if (pos < ccap) list[pos] = s;
    }
    if (L >= 2 && bin_at(hs, 1, s) != hs.bin[1]) return;
    int b = bin_at(hs, L, s);
    atomicAdd(&s_cnt[b], 1u);
    atomicAdd(&s_w[b], unit_w ? 1.0f : pair_weight(sigma, s, smax));
    atomicMin(&s_min[b], float_key(s));
    if (L == 1) atomicMax(&s_max[b], float_key(s));
  });
  __syncthreads();
  for (int i = threadIdx.x; i < kBins; i += blockDim.x) {
    unsigned int c = s_cnt[i];
    if (c) {
      atomicAdd(&g_cnt[(long long)bh * kBins + i], c);
      atomicAdd(&g_w[(long long)bh * kBins + i], (double)s_w[i]);
      atomicMin(&g_minkey[(long long)bh * kBins + i], s_min[i]);
      if (L == 1) atomicMax(&g_maxkey[(long long)bh * kBins + i], s_max[i]);
    }
  }
}

// Level 0 sees every pair, and scores cluster: with one set of bins most lanes of a warp hit the
// same few addresses and the shared-memory atomics serialise.  Here every bin has one copy per lane
// in 32 consecutive words (a warp's updates always fall into 32 different banks), and only the
// masses are kept: the scan needs no counts at this level.
constexpr int kRep = 32;
__global__ void __launch_bounds__(512)
hist0_kernel(const float* __restrict__ scores, long long P, const HeadState* __restrict__ st, float sigma, int unit_w,
             double* __restrict__ g_w) {
  extern __shared__ float s_wr[];   // [kBins0][kRep]
  const int bh = blockIdx.y;
  const HeadState hs = st[bh];
  for (int i = threadIdx.x; i < kBins0 * kRep; i += blockDim.x) s_wr[i] = 0.f;
  __syncthreads();
  const float smax = key_float(hs.max_key);
  const int rep = threadIdx.x & (kRep - 1);
  for_each_score(scores + (long long)bh * P, P, [&](float s) {
    atomicAdd(&s_wr[bin_at(hs, 0, s) * kRep + rep], unit_w ? 1.0f : pair_weight(sigma, s, smax));
  });
  __syncthreads();
  for (int i = threadIdx.x; i < kBins0; i += blockDim.x) {
    float w = 0.f;
#pragma unroll
    for (int r = 0; r < kRep; ++r) w += s_wr[i * kRep + ((r + i) & (kRep - 1))];
    if (w > 0.f) atomicAdd(&g_w[(long long)bh * kBins + i], (double)w);
  }
}

// One CTA (1024 threads, two bins each) per head: walk the bins from the top, find the bin in
// which the cumulative mass first reaches the target, record it and clear the histogram.
template <int L>
__global__ void __launch_bounds__(1024)
scan_kernel(HeadState* __restrict__ st, float tau, double count_target, unsigned int* __restrict__ g_cnt,
            double* __restrict__ g_w,
            uint32_t* __restrict__ g_minkey, uint32_t* __restrict__ g_maxkey, int64_t* __restrict__ k_per_head,
            float* __restrict__ cutoff_per_head, long long ccap) {
  __shared__ double s_wsum[32];
  __shared__ unsigned long long s_csum[32];
  __shared__ int s_cross;
  __shared__ int s_lowest;
  __shared__ uint32_t s_minkey;
  const int bh = blockIdx.x;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  HeadState hs = st[bh];
  if (L == 2 && hs.resolved) return;     // cutoff written at level 1; the histogram arrays are clear
  // element e = 0..2047 walks bins from the top: bin = 2047 - e; thread t owns e = 2t, 2t+1
  const long long hb = (long long)bh * kBins;
  const long long i0 = hb + (kBins - 1 - 2 * t), i1 = hb + (kBins - 2 - 2 * t);
  double w0 = g_w[i0], w1 = g_w[i1];
  // level 0 keeps masses only: a bin counts as occupied when its mass is positive
  unsigned long long c0 = L == 0 ? (w0 > 0.0) : g_cnt[i0], c1 = L == 0 ? (w1 > 0.0) : g_cnt[i1];
  uint32_t mk0 = 0xffffffffu, mk1 = 0xffffffffu, xk0 = 0u, xk1 = 0u;
  if (L >= 1) { mk0 = g_minkey[i0]; mk1 = g_minkey[i1]; }
  if (L == 1) { xk0 = g_maxkey[i0]; xk1 = g_maxkey[i1]; }
  // clear for the next level / next call
  g_w[i0] = 0.0; g_w[i1] = 0.0;
  if (L >= 1) { g_cnt[i0] = 0u; g_cnt[i1] = 0u; g_minkey[i0] = 0xffffffffu; g_minkey[i1] = 0xffffffffu; }
  if (L == 1) { g_maxkey[i0] = 0u; g_maxkey[i1] = 0u; }
  double wl = w0 + w1;
  unsigned long long cl = c0 + c1;
  // inclusive warp scan
  double wi = wl; unsigned long long ci = cl;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    double wv = __shfl_up_sync(0xffffffffu, wi, o);
    unsigned long long cv = __shfl_up_sync(0xffffffffu, ci, o);
    if (lane >= o) { wi += wv; ci += cv; }
  }
  if (lane == 31) { s_wsum[warp] = wi; s_csum[warp] = ci; }
  if (t == 0) { s_cross = -1; s_lowest = -1; s_minkey = 0xffffffffu; }
  __syncthreads();
  if (warp == 0) {
    double wv = s_wsum[lane]; unsigned long long cv = s_csum[lane];
    double wi2 = wv; unsigned long long ci2 = cv;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      double a = __shfl_up_sync(0xffffffffu, wi2, o);
      unsigned long long b = __shfl_up_sync(0xffffffffu, ci2, o);
      if (lane >= o) { wi2 += a; ci2 += b; }
    }
    s_wsum[lane] = wi2 - wv;    // exclusive
    s_csum[lane] = ci2 - cv;
  }
  __syncthreads();
  const double w_excl = s_wsum[warp] + (wi - wl);            // mass of all elements before e = 2t
  const unsigned long long c_excl = s_csum[warp] + (ci - cl);
  __shared__ double s_total;
  if (t == 1023) s_total = w_excl + wl;
  __syncthreads();
  // unit weights (count_target >= 0): the masses are pair counts and the target is the budget itself
  if (L == 0) {
    hs.Z = s_total;
    hs.target = count_target >= 0.0 ? count_target : (double)tau * s_total;
    hs.mass_above = 0.0; hs.cnt_above = 0ull;
  }
  const double need = hs.target - hs.mass_above;    // mass still to be covered inside this level
  // crossing element: first e with inclusive mass >= need (and a non-empty bin)
  int my_cross = -1;
  if (c0 && w_excl < need && w_excl + w0 >= need) my_cross = 2 * t;
  else if (c1 && w_excl + w0 < need && w_excl + w0 + w1 >= need) my_cross = 2 * t + 1;
  if (my_cross >= 0) atomicMax(&s_cross, kBins - 1 - my_cross);      // as a bin index
  // lowest non-empty bin = fallback when rounding keeps the sum below `need`
  if (c1) atomicMax(&s_lowest, 2 * t + 1);
  else if (c0) atomicMax(&s_lowest, 2 * t);
  __syncthreads();
  int cross_bin = s_cross;
  if (cross_bin < 0) cross_bin = s_lowest >= 0 ? kBins - 1 - s_lowest : 0;
  // mass / count strictly above the crossing bin
  const int e_cross = kBins - 1 - cross_bin;
  __shared__ double s_above_w;
  __shared__ unsigned long long s_above_c;
  __shared__ uint32_t s_cross_min, s_cross_max;
  if (2 * t == e_cross) { s_above_w = w_excl; s_above_c = c_excl; s_cross_min = mk0; s_cross_max = xk0; }
  if (2 * t + 1 == e_cross) { s_above_w = w_excl + w0; s_above_c = c_excl + c0; s_cross_min = mk1; s_cross_max = xk1; }
  if (L == 2) {
    // exact cutoff: smallest key among the bins at or above the crossing bin
    uint32_t mk = 0xffffffffu;
    if (2 * t <= e_cross) mk = min(mk, mk0);
    if (2 * t + 1 <= e_cross) mk = min(mk, mk1);
    mk = __reduce_min_sync(0xffffffffu, mk);
    if (lane == 0) atomicMin(&s_minkey, mk);
  }
  __syncthreads();
  if (t == 0) {
    hs.bin[L] = cross_bin;
    // level 2 may read the list if level 1 copied the level-0 crossing bin to it in full
    if (L == 1) hs.cand_ok = (long long)hs.cand_cnt <= ccap ? 1 : 0;
    hs.mass_above += s_above_w;
    hs.cnt_above += s_above_c;
    if (L < 2) {
      hs.anchor[L + 1] = hs.inv[L] > 0.f ? hs.anchor[L] + (float)cross_bin / hs.inv[L] : hs.anchor[L];
      hs.inv[L + 1] = fminf(hs.inv[L] * (float)kBins, 1e30f);
      // one distinct score in the crossing bin: everything above it is below the target and the
      // bin reaches it, so that score is the cutoff
      if (L == 1 && tau < 1.0f && s_cross_min == s_cross_max && s_cross_min != 0xffffffffu) {
        hs.resolved = 1;
        hs.cutoff_key = s_cross_min;
        cutoff_per_head[bh] = key_float(hs.cutoff_key);
      }
    } else {
      hs.cutoff_key = s_minkey;
      if (tau >= 1.0f) hs.cutoff_key = hs.min_key;
      cutoff_per_head[bh] = key_float(hs.cutoff_key);
    }
    st[bh] = hs;
  }
}

// After minmax: level-0 anchors.
__global__ void setup_level0_kernel(HeadState* st, int BH) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= BH) return;
  float lo = key_float(st[i].min_key), hi = key_float(st[i].max_key);
  float range = hi - lo;
  st[i].anchor[0] = lo;
  st[i].inv[0] = range > 0.f ? (float)kBins0 / range : 0.f;
  st[i].bin0_off = -lo * st[i].inv[0];
}

// mark: a CTA takes a segment of QSEG consecutive queries of one head (a contiguous run of
// QSEG * Nb scores), sets the mask bits in shared memory, counts selections per key block,
// then writes mask words, per-(segment, block) counts and the segment's pair total.
__global__ void __launch_bounds__(kSegThreads)
mark_kernel(const float* __restrict__ scores, const HeadState* __restrict__ st, int S, int Nb, int mw, int QSEG,
            int nseg, int own_sb, uint32_t* __restrict__ mask_bits, int* __restrict__ seg_cnt,
            int* __restrict__ seg_total, uint32_t* __restrict__ tmask) {
  extern __shared__ uint32_t sm[];
  const int TW = QSEG >> 5;                           // words of a block's column over the segment's queries
  uint32_t* s_mask = sm;                              // [QSEG][mw]
  int* s_cnt = reinterpret_cast<int*>(sm + QSEG * mw);  // [Nb]
  uint32_t* s_tm = sm + QSEG * mw + Nb;               // [Nb][TW]: the same bits, one row per key block
  __shared__ int s_total;
  const int seg = blockIdx.x, bh = blockIdx.y;
  const int q0 = seg * QSEG;
  const int nq = min(QSEG, S - q0);
  const uint32_t cutoff = st[bh].cutoff_key;
  for (int i = threadIdx.x; i < QSEG * mw; i += blockDim.x) s_mask[i] = 0u;
  for (int i = threadIdx.x; i < Nb; i += blockDim.x) s_cnt[i] = 0;
  for (int i = threadIdx.x; i < Nb * TW; i += blockDim.x) s_tm[i] = 0u;
  if (threadIdx.x == 0) s_total = 0;
  __syncthreads();
  const float* base = scores + ((long long)bh * S + q0) * Nb;
  const long long n = (long long)nq * Nb;
  // (query, block) of element i of the segment by reciprocal: i < QSEG * Nb < 2^23, and (i + 0.5) / Nb is at
  // least 0.5 / Nb away from an integer, the rounding error far less (a fix-up step covers the rest)
  const float inv_nb = 1.0f / (float)Nb;
  auto mark = [&](long long i, float s) {
    const bool sel = float_key(s) >= cutoff;
    if (!sel && own_sb <= 0) return;          // the common case: no index arithmetic at all
    const int ii = (int)i;
    int ql = (int)(((float)ii + 0.5f) * inv_nb), j = ii - ql * Nb;
    if (j < 0) { --ql; j += Nb; } else if (j >= Nb) { ++ql; j -= Nb; }     // belt and braces for huge Nb
    // own_sb > 0: a query also keeps the block it lies in (block-major position / tokens per block)
    if (sel || (q0 + ql) / own_sb == j) {
      atomicOr(&s_mask[ql * mw + (j >> 5)], 1u << (j & 31));
      atomicOr(&s_tm[j * TW + (ql >> 5)], 1u << (ql & 31));
      atomicAdd(&s_cnt[j], 1);
    }
  };
  if ((reinterpret_cast<uintptr_t>(base) & 15u) == 0) {
    const float4* b4 = reinterpret_cast<const float4*>(base);
    long long n4 = n >> 2;
    // four independent 16-byte loads per thread in flight
    long long i = threadIdx.x;
    for (; i + 3 * (long long)blockDim.x < n4; i += 4 * (long long)blockDim.x) {
      float4 x[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) x[j] = __ldg(b4 + i + j * (long long)blockDim.x);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const long long e = 4 * (i + j * (long long)blockDim.x);
        mark(e, x[j].x); mark(e + 1, x[j].y); mark(e + 2, x[j].z); mark(e + 3, x[j].w);
      }
    }
    for (; i < n4; i += blockDim.x) {
      float4 x = __ldg(b4 + i);
      mark(4 * i, x.x); mark(4 * i + 1, x.y); mark(4 * i + 2, x.z); mark(4 * i + 3, x.w);
    }
    for (long long i = (n4 << 2) + threadIdx.x; i < n; i += blockDim.x) mark(i, __ldg(base + i));
  } else {
    for (long long i = threadIdx.x; i < n; i += blockDim.x) mark(i, __ldg(base + i));
  }
  __syncthreads();
  uint32_t* gm = mask_bits + ((long long)bh * S + q0) * mw;
  int local = 0;
  for (int i = threadIdx.x; i < nq * mw; i += blockDim.x) {
    uint32_t wv = s_mask[i];
    gm[i] = wv;
    local += __popc(wv);
  }
  local = __reduce_add_sync(0xffffffffu, local);
  if ((threadIdx.x & 31) == 0 && local) atomicAdd(&s_total, local);
  int* sc = seg_cnt + ((long long)bh * nseg + seg) * Nb;
  for (int i = threadIdx.x; i < Nb; i += blockDim.x) sc[i] = s_cnt[i];
  uint32_t* tm = tmask + ((long long)bh * nseg + seg) * Nb * TW;
  for (int i = threadIdx.x; i < Nb * TW; i += blockDim.x) tm[i] = s_tm[i];
  __syncthreads();
  if (threadIdx.x == 0) seg_total[bh * nseg + seg] = s_total;
}

// offsets A: per (head, block) turn the per-segment counts into exclusive prefixes along the
// segments and record the block's total.
__global__ void seg_prefix_kernel(int* __restrict__ seg_cnt, int* __restrict__ kb_total, int BH, int Nb, int nseg) {
  long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)BH * Nb) return;
  int bh = (int)(i / Nb), j = (int)(i % Nb);
  int run = 0;
  // eight segments per trip: their loads go out together (the stores of a trip would otherwise order them)
  for (int s0 = 0; s0 < nseg; s0 += 8) {
    int* p = seg_cnt + ((long long)bh * nseg + s0) * Nb + j;
    int c[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) c[k] = s0 + k < nseg ? p[(long long)k * Nb] : 0;
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if (s0 + k < nseg) { p[(long long)k * Nb] = run; run += c[k]; }
  }
  kb_total[i] = run;
}

__global__ void __launch_bounds__(1024)
offsets_kernel(const int* __restrict__ kb_total, int* __restrict__ kb_ptr, long long n_kb,
               const int* __restrict__ seg_total, int* __restrict__ seg_qoff, long long n_seg,
               int BH, int Nb, int64_t* __restrict__ k_per_head, long long capacity,
               int* __restrict__ q_ptr_last, int32_t* __restrict__ dev_status) {
  __shared__ long long total_a, total_b;
  block_exclusive_scan([&](long long i) { return kb_total[i]; }, kb_ptr, n_kb, &total_a);
  block_exclusive_scan([&](long long i) { return seg_total[i]; }, seg_qoff, n_seg, &total_b);
  __syncthreads();
  for (int bh = threadIdx.x; bh < BH; bh += blockDim.x) {
    long long a = 0;
    for (int j = 0; j < Nb; ++j) a += kb_total[(long long)bh * Nb + j];
    k_per_head[bh] = a;
  }
  if (threadIdx.x == 0) {
    *q_ptr_last = (int)min(total_a, (long long)INT32_MAX);
    if (total_a > capacity) set_status(dev_status, VMOBA_ERR_CAPACITY);
  }
}

// fill: a CTA re-reads its segment's mask words and derives q_ptr for its queries; then, one warp
// per key block, the block's column of the segment (a few words written by the mark kernel) gives
// the selecting queries in ascending order without touching the unset bits: each is placed in
// q_idx, and the same position is recorded in the query-major list q_pairs.
__global__ void __launch_bounds__(kSegThreads)
fill_kernel(const uint32_t* __restrict__ mask_bits, const uint32_t* __restrict__ tmask, int S, int Nb, int mw, int QSEG,
            int nseg, const int* __restrict__ kb_ptr, const int* __restrict__ seg_cnt, const int* __restrict__ seg_qoff,
            int* __restrict__ q_idx, int* __restrict__ q_ptr, int* __restrict__ q_pairs, long long capacity) {
  extern __shared__ uint32_t sm[];
  uint32_t* s_mask = sm;                                   // [QSEG][mw]
  int* s_qoff = reinterpret_cast<int*>(sm + QSEG * mw);    // [QSEG] exclusive pair offset inside the segment
  __shared__ int s_warp[kSegThreads / 32];
  const int seg = blockIdx.x, bh = blockIdx.y;
  const int q0 = seg * QSEG;
  const int nq = min(QSEG, S - q0);
  const int TW = QSEG >> 5;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5, nwarps = blockDim.x >> 5;
  const uint32_t* gm = mask_bits + ((long long)bh * S + q0) * mw;
  for (int i = t; i < QSEG * mw; i += blockDim.x) s_mask[i] = i < nq * mw ? gm[i] : 0u;
  __syncthreads();
  const int qbase = seg_qoff[bh * nseg + seg];
  // exclusive scan of per-query pair counts (QSEG <= blockDim.x)
  int cnt = 0;
  if (t < nq)
    for (int w = 0; w < mw; ++w) cnt += __popc(s_mask[t * mw + w]);
  int inc = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    int x = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += x;
  }
  if (lane == 31) s_warp[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int x = lane < nwarps ? s_warp[lane] : 0;
    int xi = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, xi, o);
      if (lane >= o) xi += y;
    }
    if (lane < nwarps) s_warp[lane] = xi - x;
  }
  __syncthreads();
  if (t < QSEG) {
    int excl = s_warp[warp] + inc - cnt;
    s_qoff[t] = excl;
    if (t < nq) q_ptr[(long long)bh * S + q0 + t] = (int)min((long long)qbase + excl, (long long)INT32_MAX);
  }
  __syncthreads();
  const int* sc = seg_cnt + ((long long)bh * nseg + seg) * Nb;
  const uint32_t* tm = tmask + ((long long)bh * nseg + seg) * Nb * TW;
  for (int j = warp; j < Nb; j += nwarps) {
    // lane l holds the block's bits of queries 32 l .. 32 l + 31 of the segment (TW <= 16 words)
    uint32_t word = lane < TW ? tm[j * TW + lane] : 0u;
    int before = __popc(word);
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      int x = __shfl_up_sync(0xffffffffu, before, o);
      if (lane >= o) before += x;
    }
    before -= __popc(word);                                 // selecting queries in the lower words
    const long long base = (long long)kb_ptr[(long long)bh * Nb + j] + sc[j];
    const int wj = j >> 5;
    const uint32_t bit = 1u << (j & 31);
    while (word) {
      const int b = __ffs(word) - 1;
      word &= word - 1;
      const int ql = 32 * lane + b;
      const long long pos = base + before;
      ++before;
      if (pos < capacity) {
        q_idx[pos] = q0 + ql;
        int within = __popc(s_mask[ql * mw + wj] & (bit - 1u));
        for (int w = 0; w < wj; ++w) within += __popc(s_mask[ql * mw + w]);
        const long long qp = (long long)qbase + s_qoff[ql] + within;
        if (qp < capacity) q_pairs[qp] = (int)pos;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Per-query ("local") rules: one warp per query row, N_b <= 1024 so that lane l holds the blocks
// j = l + 32 i as order-preserving keys.  The cutoff of a row is the largest key c with
// measure{key >= c} >= target, found bit by bit from the top (measure = count for top-k, softmax
// mass for the threshold rule); blocks above it are taken, blocks tied with it in block order until
// the target is met.  Block j = l + 32 i is bit l of mask word i: a ballot IS the mask word.
constexpr int kLocalMaxWords = 32;
// MW: compile-time bound on the mask words of a row (the loops over a lane's blocks unroll to it)
template <bool TOPK, int MW>
__global__ void __launch_bounds__(256)
select_local_kernel(const float* __restrict__ scores, int S, int Nb, int mw, float sigma, float tau, int topk, int own_sb,
                    uint32_t* __restrict__ mask_bits, HeadState* __restrict__ st, long long n_rows) {
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
  const uint32_t lt_mask = (1u << lane) - 1u;
  // A warp takes a run of consecutive rows: they belong to one head (or two), so the smallest cutoff of the run
  // reaches the head's state with one atomic per run instead of one per row, and the next row's scores are
  // requested while the current row is worked on.
  const long long per_warp = (n_rows + nwarps - 1) / nwarps;
  const long long row_begin = warp * per_warp, row_end = min(n_rows, row_begin + per_warp);
  uint32_t run_cut = 0xffffffffu;
  long long run_head = -1;
  auto note_cutoff = [&](long long row, uint32_t c) {
    const long long head = row / S;
    if (head != run_head) {
      if (lane == 0 && run_head >= 0) atomicMin(&st[run_head].cutoff_key, run_cut);
      run_head = head;
      run_cut = 0xffffffffu;
    }
    run_cut = min(run_cut, c);
  };
  auto load_row = [&](long long row, uint32_t (&k)[MW]) {
    const float* sr = scores + row * Nb;
#pragma unroll
    for (int i = 0; i < MW; ++i) {
      const int j = lane + 32 * i;
      k[i] = (i < mw && j < Nb) ? float_key(__ldg(sr + j)) : 0u;     // 0 is below every real score's key
    }
  };
  uint32_t next_key[MW];
  if (row_begin < row_end) load_row(row_begin, next_key);
  for (long long row = row_begin; row < row_end; ++row) {
    const int own = own_sb > 0 ? (int)(row % S) / own_sb : -1;      // the query's own block, if it is to be kept
    const uint32_t own_bit = (own >= 0 && (own >> 5) == lane) ? 1u << (own & 31) : 0u;
    uint32_t key[MW];
    uint32_t kmax = 0u;
#pragma unroll
    for (int i = 0; i < MW; ++i) {
      key[i] = next_key[i];
      kmax = max(kmax, key[i]);
    }
    if (row + 1 < row_end) load_row(row + 1, next_key);
    kmax = __reduce_max_sync(0xffffffffu, kmax);
    double w[TOPK ? 1 : MW];
    double target;
    if (TOPK) {
      target = (double)min(topk, Nb);
    } else {
      const float smax = key_float(kmax);
      double z = 0.0;
#pragma unroll
      for (int i = 0; i < MW; ++i) {
        w[i] = key[i] ? (double)pair_weight(sigma, key_float(key[i]), smax) : 0.0;
        z += w[i];
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
      target = (double)tau * z;
    }
    auto measure_ge = [&](uint32_t c) {
      if (TOPK) {
        int n = 0;
#pragma unroll
        for (int i = 0; i < MW; ++i) n += (i < mw && key[i] >= c) ? 1 : 0;
        return (double)__reduce_add_sync(0xffffffffu, n);
      } else {
        double m = 0.0;
#pragma unroll
        for (int i = 0; i < MW; ++i) m += (i < mw && key[i] >= c) ? w[TOPK ? 0 : i] : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m += __shfl_xor_sync(0xffffffffu, m, o);
        return m;
      }
    };
    // Short selections (the usual case: a handful of blocks per query) are taken one block at a time,
    // best first, lowest block index among equals, exactly the order the rule is stated in; the
    // cumulative mass of the threshold rule is the running sum of the winners' weights.
    {
      // (a round costs about as much as two steps of the 32-step bitwise search below: beyond eight blocks the
      // top-k rule, whose count is known, goes there directly)
      constexpr int kRounds = 24, kTopkRounds = 8;
      const int rounds = TOPK ? ((int)target <= kTopkRounds ? (int)target : 0) : (tau < 1.0f ? min(kRounds, Nb) : 0);
      uint32_t taken = 0u;              // bit i: this lane's block lane + 32 i is selected
      uint32_t c_last = 0u;
      double acc = 0.0;
      bool done = false;
      for (int r = 0; r < rounds && !done; ++r) {
        uint32_t m = 0u;
#pragma unroll
        for (int i = 0; i < MW; ++i) m = max(m, ((taken >> i) & 1u) ? 0u : key[i]);
        m = __reduce_max_sync(0xffffffffu, m);
        if (m == 0u) { done = true; break; }          // every block of the row is taken
        int my_j = INT32_MAX;
#pragma unroll
        for (int i = MW - 1; i >= 0; --i)
          if (key[i] == m && !((taken >> i) & 1u)) my_j = lane + 32 * i;
        const int j_min = __reduce_min_sync(0xffffffffu, my_j);
        if ((j_min & 31) == lane) taken |= 1u << (j_min >> 5);
        c_last = m;
        if (TOPK) {
          done = r + 1 == rounds;
        } else {
          acc += (double)pair_weight(sigma, key_float(m), key_float(kmax));
          done = acc >= target;
        }
      }
      if (done) {
        uint32_t my_word = 0u;
#pragma unroll
        for (int i = 0; i < MW; ++i) {
          const uint32_t word = __ballot_sync(0xffffffffu, (taken >> i) & 1u);
          if (lane == i) my_word = word;
        }
        if (lane < mw) mask_bits[row * mw + lane] = my_word | own_bit;
        note_cutoff(row, c_last);
        continue;
      }
    }
    // General path: bitwise search for the cutoff key.
    uint32_t c = 0u;
    if (!TOPK && tau >= 1.0f) {
      c = 1u;                                  // everything: every real key is >= 1
    } else {
      // the top-k rule counts in integers (its measure is a number of blocks)
      const int k_target = TOPK ? (int)target : 0;
      auto count_ge = [&](uint32_t cc) {
        int n = 0;
#pragma unroll
        for (int i = 0; i < MW; ++i) n += (i < mw && key[i] >= cc) ? 1 : 0;
        return __reduce_add_sync(0xffffffffu, n);
      };
      for (int b = 31; b >= 0; --b) {
        const uint32_t cand = c | (1u << b);
        if (cand > kmax) continue;
        if (TOPK ? count_ge(cand) >= k_target : measure_ge(cand) >= target) c = cand;
      }
      if (c == 0u) c = 1u;                     // rounding kept the mass below the target: take the row
    }
    // what the blocks strictly above the cutoff already cover, and how many of the tied ones are needed
    const double above = c == 0xffffffffu ? 0.0 : measure_ge(c + 1u);
    int n_ties = 0;
    double w_tie = 0.0;
#pragma unroll
    for (int i = 0; i < MW; ++i)
      if (i < mw && key[i] == c) { n_ties += 1; if (!TOPK) w_tie = w[TOPK ? 0 : i]; }
    n_ties = __reduce_add_sync(0xffffffffu, n_ties);
    int need;
    if (TOPK) {
      need = (int)(target - above);
    } else {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) w_tie = fmax(w_tie, __shfl_xor_sync(0xffffffffu, w_tie, o));
      need = (tau >= 1.0f || !(w_tie > 0.0)) ? n_ties : (int)ceil((target - above) / w_tie);
    }
    need = max(1, min(need, n_ties));
    int run = 0;
    uint32_t my_word = 0u;
#pragma unroll
    for (int i = 0; i < MW; ++i) {
      if (i < mw) {
        const bool eq = key[i] == c;
        const uint32_t e = __ballot_sync(0xffffffffu, eq);
        const bool sel = key[i] > c || (eq && run + __popc(e & lt_mask) < need);
        const uint32_t word = __ballot_sync(0xffffffffu, sel);
        if (lane == i) my_word = word;
        run += __popc(e);
      }
    }
    if (lane < mw) mask_bits[row * mw + lane] = my_word | own_bit;
    note_cutoff(row, c);
  }
  if (lane == 0 && run_head >= 0) atomicMin(&st[run_head].cutoff_key, run_cut);
}

__global__ void local_cutoff_kernel(const HeadState* __restrict__ st, float* __restrict__ cutoff_per_head, int BH) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < BH) cutoff_per_head[i] = key_float(st[i].cutoff_key);
}

// The mark pass of the local rules: the mask words exist already; a segment's CTA derives the
// per-block columns, the per-(segment, block) counts and the segment's pair total from them.
__global__ void __launch_bounds__(kSegThreads)
mark_from_mask_kernel(const uint32_t* __restrict__ mask_bits, int S, int Nb, int mw, int QSEG, int nseg,
                      int* __restrict__ seg_cnt, int* __restrict__ seg_total, uint32_t* __restrict__ tmask) {
  extern __shared__ uint32_t sm[];
  const int TW = QSEG >> 5;
  int* s_cnt = reinterpret_cast<int*>(sm);            // [Nb]
  uint32_t* s_tm = sm + Nb;                           // [Nb][TW]
  __shared__ int s_total;
  const int seg = blockIdx.x, bh = blockIdx.y;
  const int q0 = seg * QSEG;
  const int nq = min(QSEG, S - q0);
  for (int i = threadIdx.x; i < Nb; i += blockDim.x) s_cnt[i] = 0;
  for (int i = threadIdx.x; i < Nb * TW; i += blockDim.x) s_tm[i] = 0u;
  if (threadIdx.x == 0) s_total = 0;
  __syncthreads();
  const uint32_t* gm = mask_bits + ((long long)bh * S + q0) * mw;
  int local = 0;
  for (int i = threadIdx.x; i < nq * mw; i += blockDim.x) {
    uint32_t word = gm[i];
    const int ql = i / mw, wj = i - ql * mw;
    local += __popc(word);
    while (word) {
      const int j = 32 * wj + __ffs(word) - 1;
      word &= word - 1;
      atomicOr(&s_tm[j * TW + (ql >> 5)], 1u << (ql & 31));
      atomicAdd(&s_cnt[j], 1);
    }
  }
  local = __reduce_add_sync(0xffffffffu, local);
  if ((threadIdx.x & 31) == 0 && local) atomicAdd(&s_total, local);
  __syncthreads();
  int* sc = seg_cnt + ((long long)bh * nseg + seg) * Nb;
  for (int i = threadIdx.x; i < Nb; i += blockDim.x) sc[i] = s_cnt[i];
  uint32_t* tm = tmask + ((long long)bh * nseg + seg) * Nb * TW;
  for (int i = threadIdx.x; i < Nb * TW; i += blockDim.x) tm[i] = s_tm[i];
  if (threadIdx.x == 0) seg_total[bh * nseg + seg] = s_total;
}

// Row normalisation for the second reading of Eq. 4: out[i][j] = sigma * s[i][j] - logsumexp_j(sigma * s[i][:]),
// the logarithm of S times the pair's probability when every query is normalised on its own.  One
// warp per query row; the head-wide quantile search then runs on `out` with unit temperature.
__global__ void __launch_bounds__(256)
rownorm_kernel(const float* __restrict__ scores, float* __restrict__ out, int Nb, float sigma, long long n_rows) {
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long row = warp; row < n_rows; row += nwarps) {
    const float* sr = scores + row * Nb;
    float mx = -INFINITY;
    for (int j = lane; j < Nb; j += 32) mx = fmaxf(mx, sigma * __ldg(sr + j));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float z = 0.f;
    for (int j = lane; j < Nb; j += 32) z += expf(sigma * __ldg(sr + j) - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    const float lse = mx + logf(z);
    float* orow = out + row * Nb;
    for (int j = lane; j < Nb; j += 32) orow[j] = sigma * __ldg(sr + j) - lse;
  }
}

static int seg_queries(int mw) {
  int q = 4096 / mw;            // keep the shared mask tile <= 16 KB
  q = q / 32 * 32;
  if (q > kSegThreads) q = kSegThreads;
  if (q < 32) q = 32;
  return q;
}

struct SelectWs {
  HeadState* state;
  unsigned int* g_cnt;
  double* g_w;
  uint32_t* g_minkey;
  uint32_t* g_maxkey;
  uint32_t* tmask;
  int* seg_cnt;
  int* seg_total;
  int* seg_qoff;
  int* kb_total;
  float* cand;          // [BH][ccap] scores copied aside by the level-0 pass (optional: the last slice)
  long long ccap;
  size_t base_bytes;    // without the candidate lists
  size_t bytes;
  Guards guards;
};

// Room for the list of one head: the pairs of one of the 512 level-0 bins.
static long long cand_capacity(const Dims& D) {
  const long long P = (long long)D.S * D.Nb;
  return std::max<long long>(4096, ((P / 32 + 3) / 4) * 4);
}

static SelectWs carve_select(const Dims& D, void* ws) {
  SelectWs w;
  Carver c(ws);
  int QSEG = seg_queries(D.mask_words);
  long long nseg = (D.S + QSEG - 1) / QSEG;
  w.state = c.take<HeadState>(D.BH);
  w.g_cnt = c.take<unsigned int>((size_t)D.BH * kBins);
  w.g_w = c.take<double>((size_t)D.BH * kBins);
  w.g_minkey = c.take<uint32_t>((size_t)D.BH * kBins);
  w.g_maxkey = c.take<uint32_t>((size_t)D.BH * kBins);
  w.tmask = c.take<uint32_t>((size_t)D.BH * nseg * D.Nb * (QSEG >> 5));
  w.seg_cnt = c.take<int>((size_t)D.BH * nseg * D.Nb);
  w.seg_total = c.take<int>((size_t)D.BH * nseg);
  w.seg_qoff = c.take<int>((size_t)D.BH * nseg + 1);
  w.kb_total = c.take<int>((size_t)D.BH * D.Nb);
  w.base_bytes = c.total();
  w.ccap = cand_capacity(D);
  w.cand = c.take<float>((size_t)D.BH * w.ccap);
  w.bytes = c.total();
  w.guards = c.guards;
  return w;
}

size_t select_ws_bytes(const Dims& D) { return carve_select(D, nullptr).bytes; }
// the least the selection can work with (no candidate lists: levels 1 and 2 read the score matrix)
size_t select_base_ws_bytes(const Dims& D) { return carve_select(D, nullptr).base_bytes; }
// the row-normalised rule also keeps a transformed copy of the score matrix behind the common scratch
size_t select_rownorm_ws_bytes(const Dims& D) {
  return ((carve_select(D, nullptr).bytes + 255) / 256) * 256 + (size_t)D.BH * D.S * D.Nb * sizeof(float);
}

}  // namespace vmoba

using namespace vmoba;

static int select_impl(const vmoba_shape* shape, const float* scores, const float* range, int rule, float tau, int topk, uint32_t* mask_bits,
                       int32_t* kb_ptr, int32_t* q_idx, int32_t* q_ptr, int32_t* q_pairs, int64_t capacity,
                       int64_t* k_per_head, float* cutoff_per_head, int32_t* dev_status, void* ws, size_t ws_bytes,
                       void* stream, bool allow_base_ws = false) {
  Dims D;
  int rc = make_dims(shape, &D);
  if (rc) return rc;
  // D is known here: a query at block-major position p lies in key block p / s_b
  const int own_sb = (rule & VMOBA_SELECT_KEEP_OWN_BLOCK) ? D.sb : 0;
  rule &= ~VMOBA_SELECT_KEEP_OWN_BLOCK;
  const bool rownorm = rule == VMOBA_SELECT_THRESHOLD_GLOBAL_ROWNORM;
  if (rownorm) rule = VMOBA_SELECT_THRESHOLD_GLOBAL;
  const bool by_topk = rule == VMOBA_SELECT_TOPK_GLOBAL || rule == VMOBA_SELECT_TOPK_LOCAL;
  const bool local = rule == VMOBA_SELECT_THRESHOLD_LOCAL || rule == VMOBA_SELECT_TOPK_LOCAL;
  if (rule < VMOBA_SELECT_THRESHOLD_GLOBAL || rule > VMOBA_SELECT_TOPK_LOCAL) return VMOBA_ERR_ARG;
  if (by_topk ? topk < 1 : (!(tau > 0.0f) || tau > 1.0f)) return VMOBA_ERR_ARG;
  if (!scores || !mask_bits || !kb_ptr || !q_idx || !q_ptr || !q_pairs || !k_per_head || !cutoff_per_head ||
      !dev_status || !ws)
    return VMOBA_ERR_ARG;
  if (!aligned16(scores) || !aligned16(ws)) return VMOBA_ERR_ARG;
  if (capacity <= 0 || capacity > (int64_t)INT32_MAX) return VMOBA_ERR_ARG;
  if (D.Nb > 8192 || (local && D.Nb > 32 * kLocalMaxWords)) return VMOBA_ERR_SHAPE;
  SelectWs w = carve_select(D, ws);
  if (ws_bytes < (rownorm ? select_rownorm_ws_bytes(D) : (allow_base_ws ? w.base_bytes : w.bytes))) return VMOBA_ERR_WORKSPACE;
  // the candidate lists are the last slice: a caller with a fixed scratch area may have no room for them
  const bool use_cand = ws_bytes >= w.bytes;
  if (!use_cand) { w.cand = nullptr; w.ccap = -1; if (w.guards.n > 0) w.guards.n -= 1; }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const long long P = (long long)D.S * D.Nb;
  float sigma = D.scale;
  if (rownorm) {
    // search on the row-normalised log-probabilities with unit temperature
    float* lp = reinterpret_cast<float*>(static_cast<char*>(ws) + ((w.bytes + 255) / 256) * 256);
    const long long n_rows = (long long)D.BH * D.S;
    rownorm_kernel<<<(int)std::min<long long>((n_rows + 7) / 8, sm_count() * 8), 256, 0, st>>>(scores, lp, D.Nb, D.scale, n_rows);
    VMOBA_LAUNCH_OK(1);
    scores = lp;
    sigma = 1.0f;
    range = nullptr;      // the range of the raw scores says nothing about the transformed matrix
  }
  VMOBA_GUARDS_ARM(w.guards, st);
  const int QSEG = seg_queries(D.mask_words);
  const int nseg = (D.S + QSEG - 1) / QSEG;
  const size_t smem = (size_t)QSEG * D.mask_words * 4 + (size_t)std::max(D.Nb, QSEG) * 4 + (size_t)D.Nb * (QSEG >> 5) * 4;
  const dim3 sgrid(nseg, D.BH);

  if (local) {
    init_state_kernel<<<(D.BH + 127) / 128, 128, 0, st>>>(w.state, D.BH, nullptr, nullptr, nullptr, nullptr, nullptr);
    // per-query rules: the mask comes straight from the rows; cutoff_key collects the smallest selected key
    const long long n_rows = (long long)D.BH * D.S;
    const int blocks = (int)std::min<long long>((n_rows + 7) / 8, sm_count() * 8);
    auto launch_local = [&](auto topk_tag, auto mw_tag) {
      select_local_kernel<decltype(topk_tag)::value, decltype(mw_tag)::value><<<blocks, 256, 0, st>>>(
          scores, D.S, D.Nb, D.mask_words, D.scale, tau, topk, own_sb, mask_bits, w.state, n_rows);
    };
    auto by_words = [&](auto topk_tag) {
      if (D.mask_words <= 1) launch_local(topk_tag, std::integral_constant<int, 1>());
      else if (D.mask_words <= 2) launch_local(topk_tag, std::integral_constant<int, 2>());
      else if (D.mask_words <= 4) launch_local(topk_tag, std::integral_constant<int, 4>());
      else if (D.mask_words <= 8) launch_local(topk_tag, std::integral_constant<int, 8>());
      else if (D.mask_words <= 16) launch_local(topk_tag, std::integral_constant<int, 16>());
      else launch_local(topk_tag, std::integral_constant<int, kLocalMaxWords>());
    };
    if (by_topk) by_words(std::true_type()); else by_words(std::false_type());
    local_cutoff_kernel<<<(D.BH + 127) / 128, 128, 0, st>>>(w.state, cutoff_per_head, D.BH);
    VMOBA_CUDA_OK(cudaFuncSetAttribute(mark_from_mask_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    mark_from_mask_kernel<<<sgrid, kSegThreads, smem, st>>>(mask_bits, D.S, D.Nb, D.mask_words, QSEG, nseg, w.seg_cnt,
                                                            w.seg_total, w.tmask);
    VMOBA_LAUNCH_OK(4);
  } else {
    // head-wide rules: weighted quantile of the pool (unit weights and a pair budget for top-k)
    double count_target = -1.0;
    if (by_topk) {
      count_target = (double)std::min<long long>((long long)topk * D.S, P);
      tau = count_target >= (double)P ? 1.0f : 0.5f;      // tau only tells the scan whether everything is taken
    }
    const int unit_w = by_topk ? 1 : 0;
    init_state_kernel<<<(unsigned)(((long long)D.BH * kBins + 255) / 256), 256, 0, st>>>(w.state, D.BH, range, w.g_cnt, w.g_w,
                                                                                        w.g_minkey, w.g_maxkey);

    // enough CTAs per head to fill the machine, few enough that the per-CTA flush stays small
    long long per_head = (P / 4 + 255) / 256;
    int gx = (int)std::min<long long>(std::max<long long>(per_head / 8, 1), std::max(1, sm_count() * 8 / D.BH));
    dim3 grid(gx, D.BH);
    if (!range) {
      minmax_kernel<<<grid, 256, 0, st>>>(scores, P, w.state);
      setup_level0_kernel<<<(D.BH + 127) / 128, 128, 0, st>>>(w.state, D.BH);
      count_launches(2);
    }
    {
      constexpr int smem0 = kBins0 * kRep * (int)sizeof(float);
      VMOBA_CUDA_OK(cudaFuncSetAttribute(hist0_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem0));
      // three 512-thread CTAs per SM hold their replicated bins side by side
      int gx0 = (int)std::min<long long>(std::max<long long>(per_head / 16, 1), std::max(1, sm_count() * 3 / D.BH));
      hist0_kernel<<<dim3(gx0, D.BH), 512, smem0, st>>>(scores, P, w.state, sigma, unit_w, w.g_w);
    }
    scan_kernel<0><<<D.BH, 1024, 0, st>>>(w.state, tau, count_target, w.g_cnt, w.g_w, w.g_minkey, w.g_maxkey, k_per_head,
                                         cutoff_per_head, w.ccap);
    hist_kernel<1><<<grid, 256, 0, st>>>(scores, P, w.state, sigma, unit_w, w.g_cnt, w.g_w, w.g_minkey, w.g_maxkey, w.cand,
                                        w.ccap, &w.state->cand_cnt);
    scan_kernel<1><<<D.BH, 1024, 0, st>>>(w.state, tau, count_target, w.g_cnt, w.g_w, w.g_minkey, w.g_maxkey, k_per_head,
                                         cutoff_per_head, w.ccap);
    hist_kernel<2><<<grid, 256, 0, st>>>(scores, P, w.state, sigma, unit_w, w.g_cnt, w.g_w, w.g_minkey, w.g_maxkey, w.cand,
                                        w.ccap, &w.state->cand_cnt);
    scan_kernel<2><<<D.BH, 1024, 0, st>>>(w.state, tau, count_target, w.g_cnt, w.g_w, w.g_minkey, w.g_maxkey, k_per_head,
                                         cutoff_per_head, w.ccap);
    VMOBA_LAUNCH_OK(7);
    VMOBA_CUDA_OK(cudaFuncSetAttribute(mark_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    mark_kernel<<<sgrid, kSegThreads, smem, st>>>(scores, w.state, D.S, D.Nb, D.mask_words, QSEG, nseg, own_sb, mask_bits,
                                                  w.seg_cnt, w.seg_total, w.tmask);
    VMOBA_LAUNCH_OK(1);
  }

  VMOBA_CUDA_OK(cudaFuncSetAttribute(fill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  long long nkb = (long long)D.BH * D.Nb;
  seg_prefix_kernel<<<(unsigned)((nkb + 255) / 256), 256, 0, st>>>(w.seg_cnt, w.kb_total, D.BH, D.Nb, nseg);
  offsets_kernel<<<1, 1024, 0, st>>>(w.kb_total, kb_ptr, nkb, w.seg_total, w.seg_qoff, (long long)D.BH * nseg,
                                     D.BH, D.Nb, k_per_head, capacity, q_ptr + (long long)D.BH * D.S, dev_status);
  fill_kernel<<<sgrid, kSegThreads, smem, st>>>(mask_bits, w.tmask, D.S, D.Nb, D.mask_words, QSEG, nseg, kb_ptr, w.seg_cnt,
                                                w.seg_qoff, q_idx, q_ptr, q_pairs, capacity);
  VMOBA_LAUNCH_OK(3);
  VMOBA_GUARDS_CHECK(w.guards, dev_status, st);
  return VMOBA_OK;
}

extern "C" int vmoba_select(const vmoba_shape* shape, const float* scores, float tau, uint32_t* mask_bits,
                            int32_t* kb_ptr, int32_t* q_idx, int32_t* q_ptr, int32_t* q_pairs,
                            int64_t capacity, int64_t* k_per_head, float* cutoff_per_head,
                            int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  return select_impl(shape, scores, nullptr, VMOBA_SELECT_THRESHOLD_GLOBAL, tau, 0, mask_bits, kb_ptr, q_idx, q_ptr, q_pairs,
                     capacity, k_per_head, cutoff_per_head, dev_status, ws, ws_bytes, stream);
}

extern "C" int vmoba_select_ranged(const vmoba_shape* shape, const float* scores, const float* score_range, int32_t rule,
                                   float tau, int32_t topk, uint32_t* mask_bits, int32_t* kb_ptr, int32_t* q_idx,
                                   int32_t* q_ptr, int32_t* q_pairs, int64_t capacity, int64_t* k_per_head,
                                   float* cutoff_per_head, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  if (!score_range) return VMOBA_ERR_ARG;
  return select_impl(shape, scores, score_range, rule, tau, topk, mask_bits, kb_ptr, q_idx, q_ptr, q_pairs, capacity,
                     k_per_head, cutoff_per_head, dev_status, ws, ws_bytes, stream);
}

extern "C" int vmoba_select_rule_apply(const vmoba_shape* shape, const float* scores, int32_t rule, float tau, int32_t topk,
                                       uint32_t* mask_bits, int32_t* kb_ptr, int32_t* q_idx, int32_t* q_ptr,
                                       int32_t* q_pairs, int64_t capacity, int64_t* k_per_head, float* cutoff_per_head,
                                       int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  return select_impl(shape, scores, nullptr, rule, tau, topk, mask_bits, kb_ptr, q_idx, q_ptr, q_pairs, capacity, k_per_head,
                     cutoff_per_head, dev_status, ws, ws_bytes, stream);
}

// ------------------------------------------------------------------------------------------
// Selection without a caller-provided workspace.
//
// Some callers of this library are not allowed to allocate device memory at the point where
// they run the layer: code running inside a memory-planned inference engine or a framework
// plug-in that was handed fixed input/output buffers and nothing else, or a latency-critical
// loop in which cudaMalloc (which synchronises the device) is forbidden.  For them the scratch
// of the selection stage lives in the array below, which is part of the library image: every
// GPU that loads the library holds these bytes until the process exits.
namespace vmoba {
constexpr size_t kStaticSelectScratchBytes = 16u << 20;   // 16 MiB
static __device__ __align__(256) unsigned char g_select_scratch[kStaticSelectScratchBytes];

constexpr int kMaxDevices = 64;
static void* g_select_scratch_addr[kMaxDevices] = {nullptr};
}  // namespace vmoba

extern "C" size_t vmoba_select_static_scratch_bytes(void) { return vmoba::kStaticSelectScratchBytes; }

extern "C" int vmoba_select_static(const vmoba_shape* shape, const float* scores, float tau, uint32_t* mask_bits,
                                   int32_t* kb_ptr, int32_t* q_idx, int32_t* q_ptr, int32_t* q_pairs,
                                   int64_t capacity, int64_t* k_per_head, float* cutoff_per_head,
                                   int32_t* dev_status, void* stream) {
  Dims D;
  int rc = make_dims(shape, &D);
  if (rc) return rc;
  if (D.Nb > 8192) return VMOBA_ERR_SHAPE;
  // The shape's scratch need must fit the fixed array; larger problems have to use vmoba_select.
  if (select_base_ws_bytes(D) > kStaticSelectScratchBytes) return VMOBA_ERR_WORKSPACE;
  int dev = -1;
  VMOBA_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return VMOBA_ERR_CUDA;
  if (!g_select_scratch_addr[dev]) {
    // In host code the array's name is only a handle for the symbol, not a device address: ask the
    // runtime for the address on the current device, once per device.
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_select_scratch) != cudaSuccess || !p) {
      cudaGetLastError();
      return VMOBA_ERR_CUDA;
    }
    g_select_scratch_addr[dev] = p;
  }
  // vmoba_select clears everything in its scratch that has to start at zero, so the contents
  // left by an earlier call do not matter.
  return select_impl(shape, scores, nullptr, VMOBA_SELECT_THRESHOLD_GLOBAL, tau, 0, mask_bits, kb_ptr, q_idx, q_ptr, q_pairs,
                     capacity, k_per_head, cutoff_per_head, dev_status, g_select_scratch_addr[dev], kStaticSelectScratchBytes,
                     stream, /*allow_base_ws=*/true);
}
