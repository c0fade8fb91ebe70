// Tensor-core attention forward for bf16, head_dim 128 (Step 3 of VMoBA and its dense limit).
//
// One persistent CTA per SM walks the work items.  An item is up to 256 query rows (sparse: a chunk of
// the queries that selected key block j, gathered by index; dense: 256 consecutive rows) against a
// contiguous key range (the block, or the whole sequence), streamed in tiles of 128 keys.
// With 128 query rows per CTA every 128-key tile of K and V (64 KB) feeds only 1024 tensor-pipe
// cycles, and the L2-to-SM path, not the tensor pipe, sets the pace.  Here a CTA owns TWO 128-row
// query tiles (A and B) that share each K/V tile, which halves the bytes per MMA, and the two
// tiles are worked in opposite phase: while the softmax warps of A turn S_A(t) into P_A(t) the
// tensor pipe runs P_B(t-1) V and Q_B K(t)^T, and vice versa.
//
//   warp 0        TMA producer: K and V tiles into two 2-stage rings
//   warp 1        MMA issuer (one thread)
//   warps 4-7     softmax of tile A: thread = one query row, all 128 keys of the tile
//   warps 8-11    softmax of tile B
//   warps 2,3,12,13  loaders: gather the 256 Q rows (and per-row output bookkeeping) of the NEXT item
//
// TMEM: S_A, S_B (128 columns each; the bf16 P of a tile is written over columns 64..127 of its S)
// and the accumulators O_A, O_B (128 columns each).  A softmax thread reads its row in two halves,
// first for the maximum and, after the second half has been turned into P, once more for the first
// half, so that it never holds more than 64 scores.
#include <algorithm>

#include <cuda_fp16.h>

#include "attn_simt.cuh"
#include "sm100.cuh"

namespace vmoba {
namespace tcw {

using namespace sm100;

constexpr int BM = 128;              // rows per query tile
constexpr int IM = 2 * BM;           // query rows per item
constexpr int BN = 128;              // keys per tile
constexpr int DH = 128;              // head dim
constexpr int STAGES = 2;            // K ring depth = V ring depth
constexpr int PANEL = BM * 128;      // bytes of one 64-column panel of a 128-row tile (16 KB)
constexpr int TILE = 2 * PANEL;      // bytes of a [128 x 128] bf16 tile (32 KB)
constexpr int THREADS = 448;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t O_COL = 256;      // S_X at 128 X, P_X at 128 X + 64, O_X at 256 + 128 X
constexpr float RESCALE_LOG2 = 8.0f;

struct Smem {
  uint64_t k_full[STAGES], v_full[STAGES], k_empty[STAGES], v_empty[STAGES];
  uint64_t s_full[2], p_ready[2];    // per query tile: scores written (commit) / P written (128 arrivals)
  uint64_t o_done[2];                // per query tile: P V of a key tile complete (commit)
  uint64_t o_free[2];                // per query tile: epilogue has read the accumulator (128 arrivals)
  uint64_t q_full, q_empty;          // Q tiles of an item gathered (128 arrivals) / no longer needed (commit)
  uint32_t tmem_base;
  int abort_flag;
  int qpos[4][IM];                   // [item % 4][row]: in-head position of the query, -1 for padding rows
  int direct[4][IM];                 // [item % 4][row]: query has a single block -> final result
};
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + 2 * TILE /*Q*/ + 2 * STAGES * TILE + sizeof(Smem) + 32;

struct Params {
  const __nv_bfloat16* q;
  const int* kb_ptr;
  const int* q_idx;
  const int* q_ptr;
  const int* item_ptr;
  const int* item_tab;
  int n_kb, S, Nb, sb, BH;
  float scale_log2;      // softmax scale * log2(e)
  __nv_bfloat16* o;
  __nv_bfloat16* o_resid;
  RowMap o_map;          // where the rows of o go (block-major, or raster order through perm); o_resid is block-major
  float* lse;
  __half* part_o;        // partial rows: fp16 values times part_scale[row]
  float* part_lse;
  float* part_scale;
  long long capacity;
  int part_o_32;         // part_o is 32-byte aligned: rows go out with 32-byte stores
  int32_t* status;
  unsigned long long* prof;   // optional per-section cycle counters (diagnostics), or null
};

struct FwdItem {
  int bh, key_begin, n_keys, list_lo, n_rows, ntiles, nx;   // nx: query tiles in use (1 or 2)
  long long head_off;
};

template <bool DENSE>
__device__ __forceinline__ FwdItem decode_item(const Params& p, int item) {
  FwdItem it;
  if (DENSE) {
    const int tiles = (p.S + IM - 1) / IM;
    it.bh = item / tiles;
    const int t = item - it.bh * tiles;
    it.key_begin = 0; it.n_keys = p.S; it.list_lo = t * IM; it.n_rows = min(IM, p.S - it.list_lo);
  } else {
    const int kbi = checked_index(__ldg(p.item_tab + item), p.n_kb, p.status);
    const int chunk = item - __ldg(p.item_ptr + kbi);
    it.bh = kbi / p.Nb;
    const int j = kbi - it.bh * p.Nb;
    it.key_begin = j * p.sb; it.n_keys = p.sb;
    const long long end = min((long long)__ldg(p.kb_ptr + kbi + 1), p.capacity);
    it.list_lo = __ldg(p.kb_ptr + kbi) + chunk * IM;
    it.n_rows = (int)min((long long)IM, end - it.list_lo);
  }
  it.ntiles = (it.n_keys + BN - 1) / BN;
  it.nx = it.n_rows > BM ? 2 : 1;
  it.head_off = (long long)it.bh * p.S;
  return it;
}

__device__ __forceinline__ constexpr uint32_t koff(int ks) { return (uint32_t)(((ks >> 2) * PANEL + (ks & 3) * 32) >> 4); }
__device__ __forceinline__ constexpr uint32_t mnoff(int ks) { return (uint32_t)((ks * 2048) >> 4); }

// keys at or beyond `valid` (counted inside these 64) get score -inf
__device__ __forceinline__ void mask_tail(uint32_t (&sv)[64], int valid) {
#pragma unroll
  for (int i = 0; i < 64; ++i)
    if (i >= valid) sv[i] = 0xff800000u;
}

__device__ __forceinline__ float max64(const uint32_t (&sv)[64], float mx) {
  float mx0 = mx, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
  for (int i = 0; i < 64; i += 8) {
    mx0 = max3(mx0, __uint_as_float(sv[i]), __uint_as_float(sv[i + 1]));
    mx1 = max3(mx1, __uint_as_float(sv[i + 2]), __uint_as_float(sv[i + 3]));
    mx2 = max3(mx2, __uint_as_float(sv[i + 4]), __uint_as_float(sv[i + 5]));
    mx3 = max3(mx3, __uint_as_float(sv[i + 6]), __uint_as_float(sv[i + 7]));
  }
  return fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
}

// p = 2^(s * scale - m) for 64 scores; bf16 pairs (keys 2i, 2i+1 -> word i); s0/s1 collect the exact
// weights, r0/r1 the bf16-rounded ones (the tensor core multiplies the ROUNDED weights: O is
// normalised by their sum, so that the rounding perturbs the weights but never their total).
__device__ __forceinline__ void exp_pack64(const uint32_t (&sv)[64], float scale, float neg_m, uint32_t (&pk)[32],
                                           float& s0, float& s1, float& r0, float& r1) {
#pragma unroll
  for (int i = 0; i < 32; ++i) {
    float p0, p1;
    fma2(p0, p1, __uint_as_float(sv[2 * i]), __uint_as_float(sv[2 * i + 1]), scale, scale, neg_m, neg_m);
    p0 = ex2(p0);
    p1 = ex2(p1);
    add2(s0, s1, s0, s1, p0, p1);
    pk[i] = pack_bf16(p0, p1);
    add2(r0, r1, r0, r1, __uint_as_float(pk[i] << 16), __uint_as_float(pk[i] & 0xffff0000u));
  }
}

// Partial rows are stored as fp16 times a power of two per row: the smallest one at or above the row's largest
// magnitude (1 for a row of zeros), so that the values use the format's full precision whatever the scale of V.
__device__ __forceinline__ float pow2_at_or_above(float x) {
  const uint32_t u = (__float_as_uint(x) + 0x007fffffu) & 0x7f800000u;
  return u ? __uint_as_float(u) : 1.0f;
}
__device__ __forceinline__ uint32_t pack_half2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// N (8 or 16) consecutive outputs as bf16 (one 16- or 32-byte store) and, if asked for, their rounding
// residuals bf16(v - bf16(v)), computed in registers.
template <int N>
__device__ __forceinline__ void store_resid(__nv_bfloat16* dst, __nv_bfloat16* rdst, const float (&v)[N]) {
  uint32_t h[N / 2], r[N / 2];
#pragma unroll
  for (int k = 0; k < N / 2; ++k) {
    h[k] = pack_bf16(v[2 * k], v[2 * k + 1]);
    r[k] = pack_bf16(v[2 * k] - __uint_as_float(h[k] << 16), v[2 * k + 1] - __uint_as_float(h[k] & 0xffff0000u));
  }
  if constexpr (N == 16) {
    st_global_v8(dst, h[0], h[1], h[2], h[3], h[4], h[5], h[6], h[7]);
    if (rdst) st_global_v8(rdst, r[0], r[1], r[2], r[3], r[4], r[5], r[6], r[7]);
  } else {
    *reinterpret_cast<uint4*>(dst) = make_uint4(h[0], h[1], h[2], h[3]);
    if (rdst) *reinterpret_cast<uint4*>(rdst) = make_uint4(r[0], r[1], r[2], r[3]);
  }
}

// RASTER: the directly written rows of o go through p.o_map (a kernel of its own: with the map's address
// arithmetic compiled into the one kernel, the block-major case ran 6 % slower on the 720p-shaped layers).
template <bool DENSE, bool RASTER = false>
__global__ void __launch_bounds__(THREADS, 1)
attn_fwd_wide_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = base;                      // [2 query tiles][TILE]
  uint8_t* sK = base + 2 * TILE;           // [STAGES][TILE]
  uint8_t* sV = sK + STAGES * TILE;        // [STAGES][TILE]
  Smem* sm = reinterpret_cast<Smem*>(sV + STAGES * TILE);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &sm->abort_flag;
  // diagnostics: cycles one representative thread per role spends in each section
  unsigned long long wp[6] = {0, 0, 0, 0, 0, 0};
  long long t_mark = clock64();
  const long long t_begin = t_mark;
  auto lap = [&](int site) {
    if (p.prof) {
      const long long now = clock64();
      wp[site] += (unsigned long long)(now - t_mark);
      t_mark = now;
    }
  };
  auto tflush = [&](int base_site) {
    if (p.prof) {
      for (int i = 0; i < 6; ++i) atomicAdd(p.prof + base_site + i, wp[i]);
      atomicAdd(p.prof + base_site + 6, (unsigned long long)(clock64() - t_begin));
    }
  };

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(&sm->k_full[s], 1); mbar_init(&sm->v_full[s], 1);
      mbar_init(&sm->k_empty[s], 1); mbar_init(&sm->v_empty[s], 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(&sm->s_full[x], 1); mbar_init(&sm->p_ready[x], 128);
      mbar_init(&sm->o_done[x], 1); mbar_init(&sm->o_free[x], 128);
    }
    mbar_init(&sm->q_full, 128); mbar_init(&sm->q_empty, 1);
    sm->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmK);
    prefetch_tmap(&tmV);
  }
  if (warp == 1) {
    tmem_alloc(&sm->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm->tmem_base;
  const int n_items = DENSE ? p.BH * ((p.S + IM - 1) / IM) : p.item_ptr[p.n_kb];
  constexpr uint32_t IDESC_PV = make_idesc_bf16(BM, DH, false, true);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t fills = 0;
      for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const FwdItem it = decode_item<DENSE>(p, item);
        const int row0 = (int)it.head_off + it.key_begin;
        for (int t = 0; t < it.ntiles; ++t, ++fills) {
          const int s = fills % STAGES;
          const uint32_t par = ((fills / STAGES) - 1) & 1;
          const int y = row0 + t * BN;
          // a K stage is free once both query tiles' Q K^T of the key tile have run, a V stage only
          // after both P V
          if (fills >= STAGES) mbar_wait(&sm->k_empty[s], par, abort_flag, p.status);
          mbar_expect_tx(&sm->k_full[s], TILE);
          tma_load_2d(sK + s * TILE, &tmK, &sm->k_full[s], 0, y);
          tma_load_2d(sK + s * TILE + PANEL, &tmK, &sm->k_full[s], 64, y);
          if (fills >= STAGES) mbar_wait(&sm->v_empty[s], par, abort_flag, p.status);
          mbar_expect_tx(&sm->v_full[s], TILE);
          tma_load_2d(sV + s * TILE, &tmV, &sm->v_full[s], 0, y);
          tma_load_2d(sV + s * TILE + PANEL, &tmV, &sm->v_full[s], 64, y);
        }
      }
      // drain: every issued load must have landed before the CTA may exit (only matters after a timeout)
      if (*abort_flag) {
        const uint32_t first = fills > STAGES ? fills - STAGES : 0;
        for (uint32_t f = first; f < fills; ++f) {
          mbar_wait(&sm->k_full[f % STAGES], (f / STAGES) & 1, abort_flag, p.status);
          mbar_wait(&sm->v_full[f % STAGES], (f / STAGES) & 1, abort_flag, p.status);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: the whole warp walks the loop, one
    // elected lane issues (warp-uniform control flow; see elect_one)
    {
      const bool leader = elect_one();
      const int n_items_u = __reduce_max_sync(0xffffffffu, n_items);
      uint32_t fills = 0;              // key tiles consumed so far (ring position of K and of V)
      uint32_t n = 0;                  // items done so far
      uint32_t tcnt[2] = {0, 0};       // key tiles done per query tile (phase of s_full / p_ready / o_done)
      uint32_t ecnt[2] = {0, 0};       // items done per query tile (phase of o_free)
      const uint64_t dQ[2] = {make_smem_desc(smem_u32(sQ), 16, 1024), make_smem_desc(smem_u32(sQ + TILE), 16, 1024)};
      for (int item = blockIdx.x; item < n_items_u; item += gridDim.x, ++n) {
        FwdItem it = decode_item<DENSE>(p, item);
        it.nx = __reduce_max_sync(0xffffffffu, it.nx);
        lap(5);
        mbar_wait_warp(&sm->q_full, n & 1, abort_flag, p.status);
        lap(0);
        tc_fence_after();
        auto qk = [&](int x, int t, int s) {
          const int n_mma = (min(BN, it.n_keys - t * BN) + 15) & ~15;
          const uint32_t idesc = make_idesc_bf16(BM, n_mma, false, false);
          const uint64_t dK0 = make_smem_desc(smem_u32(sK + s * TILE), 16, 1024);
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks)
            if (leader) mma_ss(tmem + x * 128, dQ[x] + koff(ks), dK0 + koff(ks), idesc, ks > 0 ? 1u : 0u);
          if (leader) mma_commit(&sm->s_full[x]);
        };
        auto pv = [&](int x, int t, uint32_t f) {
          const int s = f % STAGES;
          lap(5);
          mbar_wait_warp(&sm->p_ready[x], tcnt[x] & 1, abort_flag, p.status);
          lap(2);
          mbar_wait_warp(&sm->v_full[s], (f / STAGES) & 1, abort_flag, p.status);
          lap(3);
          // the accumulator was last used by the previous item on this query tile: its epilogue must have read it
          if (t == 0 && ecnt[x] >= 1) mbar_wait_warp(&sm->o_free[x], (ecnt[x] - 1) & 1, abort_flag, p.status);
          lap(4);
          tc_fence_after();
          const int ksteps = (min(BN, it.n_keys - t * BN) + 15) >> 4;
          const uint64_t mV0 = make_smem_desc(smem_u32(sV + s * TILE), PANEL, 1024);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            if (leader && ks < ksteps)   // P of keys 16 ks .. 16 ks + 15 sits in columns 64 + 8 ks .. of the tile's score buffer
              mma_ts(tmem + O_COL + x * 128, tmem + x * 128 + 64 + ks * 8, mV0 + mnoff(ks), IDESC_PV,
                     (t > 0 || ks > 0) ? 1u : 0u);
          if (leader) mma_commit(&sm->o_done[x]);
          tcnt[x] += 1;
        };
        for (int t = 0; t < it.ntiles; ++t) {
          const uint32_t f = fills + t;
          const int s = f % STAGES;
          lap(5);
          mbar_wait_warp(&sm->k_full[s], (f / STAGES) & 1, abort_flag, p.status);
          lap(1);
          tc_fence_after();
          qk(0, t, s);
          if (it.nx == 2) {
            if (t > 0) {
              pv(1, t - 1, f - 1);
              if (leader) mma_commit(&sm->v_empty[(f - 1) % STAGES]);
            }
            qk(1, t, s);
          }
          if (leader) mma_commit(&sm->k_empty[s]);
          if (leader && t == it.ntiles - 1) mma_commit(&sm->q_empty);
          pv(0, t, f);
          if (leader && it.nx == 1) mma_commit(&sm->v_empty[s]);
        }
        if (it.nx == 2) {
          const uint32_t f = fills + it.ntiles - 1;
          pv(1, it.ntiles - 1, f);
          if (leader) mma_commit(&sm->v_empty[f % STAGES]);
        }
        fills += it.ntiles;
        ecnt[0] += 1;
        if (it.nx == 2) ecnt[1] += 1;
      }
      lap(5);
      if (leader) tflush(8);
    }
  } else if (warp < 4 || warp >= 12) {
    // ------------------------------------------------------------------ loaders: Q rows of the next item
    const int lt = (warp < 4 ? warp - 2 : warp - 10) * 32 + lane;   // 0..127
    const int chunk = lt & 15, panel = chunk >> 3, cc = chunk & 7;
    uint32_t n = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const FwdItem it = decode_item<DENSE>(p, item);
      const __nv_bfloat16* qh = p.q + it.head_off * DH;
      for (int x = 0; x < it.nx; ++x) {
        uint4 v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int row = x * BM + (lt >> 4) + 8 * i;
          v[i] = make_uint4(0u, 0u, 0u, 0u);
          if (row < it.n_rows) {
            const int qp = DENSE ? it.list_lo + row : checked_index(__ldg(p.q_idx + it.list_lo + row), p.S, p.status);
            v[i] = __ldg(reinterpret_cast<const uint4*>(qh + (long long)qp * DH) + chunk);
          }
        }
        // both Q tiles are free once the previous item's last Q K^T has run
        if (x == 0 && n >= 1) mbar_wait(&sm->q_empty, (n - 1) & 1, abort_flag, p.status);
        uint8_t* dst = sQ + x * TILE;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int row = (lt >> 4) + 8 * i;
          *reinterpret_cast<uint4*>(dst + panel * PANEL + row * 128 + ((cc ^ (row & 7)) << 4)) = v[i];
        }
      }
      // Four bookkeeping slots: the softmax warps read slot n % 4 in the epilogue of item n, and the
      // loaders can be at most two items ahead of an epilogue.
      for (int x = 0; x < 2; ++x) {
        const int row = x * BM + lt;
        int my_qpos = -1, my_direct = DENSE ? 1 : 0;
        if (row < it.n_rows) {
          my_qpos = DENSE ? it.list_lo + row : checked_index(__ldg(p.q_idx + it.list_lo + row), p.S, p.status);
          if (!DENSE) {
            const long long G_ = it.head_off + my_qpos;
            my_direct = (p.q_ptr[G_ + 1] - p.q_ptr[G_]) == 1;
          }
        }
        sm->qpos[n & 3][row] = my_qpos;
        sm->direct[n & 3][row] = my_direct;
      }
      fence_async_proxy();
      mbar_arrive(&sm->q_full);
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue of one query tile
    const int x = (warp - 4) >> 2;                  // query tile of this warp group
    const int quad = warp & 3;                      // TMEM lane quarter this warp may access
    const int r = quad * 32 + lane;                 // query row inside the tile
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t s_tmem = tmem + lane_addr + x * 128;
    const uint32_t o_tmem = tmem + lane_addr + O_COL + x * 128;
    uint32_t tc = 0, n = 0;                          // key tiles done on this query tile; items seen
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const FwdItem it = decode_item<DENSE>(p, item);
      if (x >= it.nx) continue;
      float m_used = -INFINITY, l = 0.f, l_r = 0.f;   // l: exact sum (for LSE); l_r: sum of the bf16-rounded weights
      for (int t = 0; t < it.ntiles; ++t, ++tc) {
        lap(3);
        mbar_wait(&sm->s_full[x], tc & 1, abort_flag, p.status);
        lap(0);
        tc_fence_after();
        const int valid = min(BN, it.n_keys - t * BN);
        uint32_t sv[64];
        tmem_ld32(s_tmem, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tmem_ld32(s_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        tmem_ld_wait();
        if (valid < 64) mask_tail(sv, valid);
        float mx = max64(sv, -INFINITY);
        tmem_ld32(s_tmem + 64, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tmem_ld32(s_tmem + 96, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        tmem_ld_wait();
        if (valid < 128) mask_tail(sv, valid - 64);
        mx = max64(sv, mx) * p.scale_log2;       // exp2 domain from here on (the scale is positive)
        lap(1);
        // lazy rescale: keep the old reference max unless the new one is more than 2^8 larger
        float factor = 1.0f;
        bool need = false;
        if (t == 0) {
          m_used = mx;
        } else if (mx > m_used + RESCALE_LOG2) {
          factor = ex2(m_used - mx);
          m_used = mx;
          need = true;
        }
        if (t > 0 && __any_sync(0xffffffffu, need)) {
          // O of the previous key tiles must be complete before it is rescaled
          mbar_wait(&sm->o_done[x], (tc - 1) & 1, abort_flag, p.status);
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t ov[32];
            tmem_ld32(o_tmem + c * 32, ov);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * factor);
            tmem_st32(o_tmem + c * 32, ov);
          }
          l *= factor;
          l_r *= factor;
        }
        lap(2);
        float s0 = 0.f, s1 = 0.f, r0 = 0.f, r1 = 0.f;
        uint32_t pk[32];
        const float neg_m = -m_used;
        // keys 64..127 are in registers: their P goes over their own score columns 96..127
        exp_pack64(sv, p.scale_log2, neg_m, pk, s0, s1, r0, r1);
        tmem_st32(s_tmem + 96, pk);
        // keys 0..63 are read again (columns 0..63 are untouched); their P goes to columns 64..95,
        // whose scores have been consumed above
        tmem_ld32(s_tmem, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tmem_ld32(s_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        tmem_ld_wait();
        if (valid < 64) mask_tail(sv, valid);
        exp_pack64(sv, p.scale_log2, neg_m, pk, s0, s1, r0, r1);
        tmem_st32(s_tmem + 64, pk);
        l += s0 + s1;
        l_r += r0 + r1;
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(&sm->p_ready[x]);
      }
      // ---- epilogue: wait for the last P V, normalise, write the row
      lap(3);
      mbar_wait(&sm->o_done[x], (tc - 1) & 1, abort_flag, p.status);
      tc_fence_after();
      const int row = x * BM + r;
      const int qpos = sm->qpos[n & 3][row];
      const bool direct = sm->direct[n & 3][row] != 0;
      const float inv = 1.0f / l_r;
      const float row_lse = (m_used + log2f(l)) * 0.6931471805599453f;
      const bool row_ok = qpos >= 0;
      const long long G_ = it.head_off + (row_ok ? qpos : 0);
      const long long o_row_off = RASTER ? ((row_ok && direct) ? p.o_map.off(G_, DH) : 0) : G_ * DH;
      const long long pos = (long long)it.list_lo + row;
      // a partial row goes out as fp16 times a power of two: find the row's largest magnitude first
      float mul = inv, row_scale = 1.0f;
      if constexpr (!DENSE) {
        const bool partial = row_ok && !direct;
        if (__any_sync(0xffffffffu, partial)) {
          float amax = 0.f;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            uint32_t ov[32];
            tmem_ld32(o_tmem + c * 32, ov);
            tmem_ld_wait();
#pragma unroll
            for (int i = 0; i < 32; ++i) amax = fmaxf(amax, fabsf(__uint_as_float(ov[i])));
          }
          if (partial) {
            row_scale = pow2_at_or_above(amax * inv);
            mul = inv / row_scale;
          }
        }
      }
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t ov[32];
        tmem_ld32(o_tmem + c * 32, ov);
        tmem_ld_wait();
        if (row_ok) {
          const int col = 32 * c;
          if (direct) {
            __nv_bfloat16* dst = p.o + o_row_off + col;
            __nv_bfloat16* rdst = p.o_resid ? p.o_resid + G_ * DH + col : nullptr;
#pragma unroll
            for (int i = 0; i < 32; i += 8) {     // 16-byte stores (32-byte ones were slower here: more values live at once)
              float v8[8];
#pragma unroll
              for (int k = 0; k < 8; ++k) v8[k] = __uint_as_float(ov[i + k]) * inv;
              store_resid<8>(dst + i, rdst ? rdst + i : nullptr, v8);
            }
          } else {
            __half* dst = p.part_o + pos * DH + col;
#pragma unroll
            for (int i = 0; i < 32; i += 16) {
              uint32_t h[8];
#pragma unroll
              for (int k = 0; k < 8; ++k)
                h[k] = pack_half2(__uint_as_float(ov[i + 2 * k]) * mul, __uint_as_float(ov[i + 2 * k + 1]) * mul);
              if (p.part_o_32) {       // one 32-byte store, else two of 16 bytes
                st_global_v8(dst + i, h[0], h[1], h[2], h[3], h[4], h[5], h[6], h[7]);
              } else {
                reinterpret_cast<uint4*>(dst + i)[0] = make_uint4(h[0], h[1], h[2], h[3]);
                reinterpret_cast<uint4*>(dst + i)[1] = make_uint4(h[4], h[5], h[6], h[7]);
              }
            }
          }
        }
      }
      if (row_ok) {
        if (direct) p.lse[G_] = row_lse; else { p.part_lse[pos] = row_lse; p.part_scale[pos] = row_scale; }
      }
      tc_fence_before();
      mbar_arrive(&sm->o_free[x]);
      lap(4);
    }
    if (warp == 4 && lane == 0) tflush(0);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

static int grid_items(long long items) { return (int)std::max<long long>(1, std::min<long long>(items, sm_count())); }

}  // namespace tcw

int tc_sparse_fwd_narrow(const Dims& D, const void* q, const void* k, const void* v, const int* kb_ptr, const int* q_idx,
                         const int* q_ptr, const int* q_pairs, long long cap, void* o, void* o_resid, float* lse,
                         int32_t* status, int* item_ptr, int* item_tab, long long max_items, float* part_o,
                         float* part_lse, float* part_scale, cudaStream_t st, const RowMap& o_map);   // attn_tc_fwd_narrow.cu

// Forward over the work lists (bf16, head_dim 128).  Key blocks of up to thirteen 128-key tiles go to the narrow
// kernel (two CTAs of one query tile per SM), longer ones to the wide kernel of this file.  Returns
// VMOBA_ERR_CUDA if the tensor maps or the launch fail.
int tc_sparse_fwd(const Dims& D, const void* q, const void* k, const void* v, const int* kb_ptr, const int* q_idx,
                       const int* q_ptr, const int* q_pairs, long long cap, void* o, void* o_resid, float* lse,
                       int32_t* status, int* item_ptr, int* item_tab, long long max_items, float* part_o,
                       float* part_lse, float* part_scale, cudaStream_t st, const RowMap& o_map) {
  using namespace tcw;
  // Measured: with blocks of 234 to 1638 keys the narrow kernel is 4 to 14 % faster; from about 1900 keys on the
  // two run level, and the narrow one reads every K / V tile twice as often from the L2, which costs a
  // power-capped step more clock than the forward gains.
  if (D.sb <= 13 * BN)
    return tc_sparse_fwd_narrow(D, q, k, v, kb_ptr, q_idx, q_ptr, q_pairs, cap, o, o_resid, lse, status, item_ptr, item_tab,
                                max_items, part_o, part_lse, part_scale, st, o_map);
  CUtensorMap tmK, tmV;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN))
    return VMOBA_ERR_CUDA;
  const long long n_kb = (long long)D.BH * D.Nb;
  simt::item_ptr_kernel<<<1, 1024, 0, st>>>(kb_ptr, n_kb, IM, cap, item_ptr);
  simt::item_tab_kernel<<<(int)std::min<long long>((n_kb + 255) / 256, sm_count() * 4), 256, 0, st>>>(item_ptr, n_kb, max_items,
                                                                                               item_tab);
  Params p;
  p.q = (const __nv_bfloat16*)q; p.kb_ptr = kb_ptr; p.q_idx = q_idx; p.q_ptr = q_ptr; p.item_ptr = item_ptr;
  p.item_tab = item_tab;
  p.n_kb = (int)n_kb; p.S = D.S; p.Nb = D.Nb; p.sb = D.sb; p.BH = D.BH;
  p.scale_log2 = D.scale * 1.4426950408889634f;
  p.o = (__nv_bfloat16*)o; p.o_resid = (__nv_bfloat16*)o_resid; p.lse = lse;
  p.part_o = reinterpret_cast<__half*>(part_o); p.part_lse = part_lse; p.part_scale = part_scale;
  p.capacity = cap; p.status = status; p.prof = debug_wait_profile();
  p.o_map = o_map;
  p.part_o_32 = (reinterpret_cast<uintptr_t>(part_o) % 32) == 0;
  if (o_map.perm) {
    VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_wide_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)SMEM_BYTES));
    attn_fwd_wide_kernel<false, true><<<grid_items(cap / IM + n_kb), THREADS, SMEM_BYTES, st>>>(tmK, tmV, p);
  } else {
    VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_wide_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)SMEM_BYTES));
    attn_fwd_wide_kernel<false><<<grid_items(cap / IM + n_kb), THREADS, SMEM_BYTES, st>>>(tmK, tmV, p);
  }
  const long long nq = (long long)D.BH * D.S;
  simt::merge_batched_kernel<__nv_bfloat16, __half><<<(int)std::min<long long>((nq + 255) / 256, sm_count() * 8), 256, 0, st>>>(
      q_ptr, q_pairs, nq, p.part_o, part_lse, part_scale, cap, (__nv_bfloat16*)o, (__nv_bfloat16*)o_resid, lse, o_map);
  VMOBA_LAUNCH_OK(4);
  return VMOBA_OK;
}

int tc_dense_fwd(const Dims& D, const void* q, const void* k, const void* v, void* o, void* o_resid, float* lse,
                      int32_t* status, cudaStream_t st) {
  using namespace tcw;
  CUtensorMap tmK, tmV;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN))
    return VMOBA_ERR_CUDA;
  Params p;
  p.q = (const __nv_bfloat16*)q; p.kb_ptr = nullptr; p.q_idx = nullptr; p.q_ptr = nullptr; p.item_ptr = nullptr;
  p.item_tab = nullptr;
  p.n_kb = 0; p.S = D.S; p.Nb = 1; p.sb = D.S; p.BH = D.BH;
  p.scale_log2 = D.scale * 1.4426950408889634f;
  p.o = (__nv_bfloat16*)o; p.o_resid = (__nv_bfloat16*)o_resid; p.lse = lse; p.part_o = nullptr; p.part_lse = nullptr; p.part_scale = nullptr;
  p.capacity = 0; p.part_o_32 = 0; p.o_map = RowMap();
  p.status = status; p.prof = debug_wait_profile();
  VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_wide_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)SMEM_BYTES));
  const long long items = (long long)D.BH * ((D.S + IM - 1) / IM);
  attn_fwd_wide_kernel<true><<<grid_items(items), THREADS, SMEM_BYTES, st>>>(tmK, tmV, p);
  VMOBA_LAUNCH_OK(1);
  return VMOBA_OK;
}

}  // namespace vmoba
