// Tensor-core attention forward for bf16, head_dim 128 (Step 3 of VMoBA and its dense limit).
//
// One persistent CTA per SM walks the work items.  An item is 128 query rows (sparse: a chunk of
// the queries that selected key block j, gathered by index; dense: 128 consecutive rows) against
// a contiguous key range (the block, or the whole sequence), streamed in tiles of 128 keys:
//
//   warp 0       TMA producer: K and V tiles (two 64-column panels each, 128-byte swizzle) into two
//                2-stage rings (a K stage is released by the tile's Q K^T, a V stage by its P V)
//   warp 1       MMA issuer (one thread): S = Q K^T into one of two TMEM score buffers, then
//                O += P V with P read from TMEM; tcgen05.commit signals the other roles
//   warps 2-9    softmax: thread = (query row, 64 of the tile's 128 keys).  The two threads of a row
//                exchange their maxima through shared memory, run the online softmax in the exp2
//                domain, write P (bf16) over their own score columns, rescale O only when the
//                running max moved by more than 2^8, and run the epilogue
//   warps 10-13  loaders: gather the Q rows (and the per-row output bookkeeping) of the NEXT item
//
// Q tiles and the O accumulator are double buffered across items, so gather, MMAs and epilogue of
// neighbouring items overlap; QK^T of tile t+1 is issued before P V of tile t.
// TMEM: 2 x 128 columns of scores (P aliases them) + 2 x 128 columns of O.
#include <algorithm>
#include <cstdlib>

#include "attn_simt.cuh"
#include "sm100.cuh"

namespace vmoba {
namespace tc {

using namespace sm100;

constexpr int BM = 128;              // query rows per item
constexpr int BN = 128;              // keys per tile
constexpr int DH = 128;              // head dim
constexpr int STAGES = 2;            // K/V ring depth
constexpr int PANEL = BM * 128;      // bytes of one 64-column panel of a 128-row tile (16 KB)
constexpr int TILE = 2 * PANEL;      // bytes of a [128 x 128] bf16 tile (32 KB)
constexpr int THREADS = 448;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t S_COL = 0, O_COL = 256;     // S: two 128-column buffers; O: two 128-column accumulators
constexpr float RESCALE_LOG2 = 8.0f;

struct Smem {
  uint64_t k_full[STAGES], v_full[STAGES], k_empty[STAGES], v_empty[STAGES];
  uint64_t s_full[2], p_ready[2];
  uint64_t o_done[2];                // P V of a tile complete (commit), alternating by tile
  uint64_t q_full[2], q_empty[2];    // gathered Q tile of an item (128 loader arrivals / commit)
  uint64_t o_free[2];                // epilogue has read the accumulator (256 arrivals)
  uint32_t tmem_base;
  int abort_flag;
  long long t_issue[STAGES];        // diagnostics: when the K tile of a stage was requested
  float xmax[2][2][128];             // [score buffer][half][row]: row maxima exchanged between the halves
  float xsum[2][2][128];             // [half][l, l_r][row]: row sums exchanged in the epilogue
  int qpos[4][128];                  // [item % 4][row]: in-head position of the query, -1 for padding rows
  int direct[4][128];                // [item % 4][row]: query has a single block -> final result
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
  float* lse;
  float* part_o;
  float* part_lse;
  long long capacity;
  int32_t* status;
  unsigned long long* prof;   // optional per-site cycle counters (diagnostics), or null
};

struct FwdItem {
  int bh, key_begin, n_keys, list_lo, n_rows, ntiles;
  long long head_off;
};

template <bool DENSE>
__device__ __forceinline__ FwdItem decode_item(const Params& p, int item) {
  FwdItem it;
  if (DENSE) {
    const int tiles = (p.S + BM - 1) / BM;
    it.bh = item / tiles;
    const int t = item - it.bh * tiles;
    it.key_begin = 0; it.n_keys = p.S; it.list_lo = t * BM; it.n_rows = min(BM, p.S - it.list_lo);
  } else {
    const int kbi = __ldg(p.item_tab + item);
    const int chunk = item - __ldg(p.item_ptr + kbi);
    it.bh = kbi / p.Nb;
    const int j = kbi - it.bh * p.Nb;
    it.key_begin = j * p.sb; it.n_keys = p.sb;
    const long long end = min((long long)__ldg(p.kb_ptr + kbi + 1), p.capacity);
    it.list_lo = __ldg(p.kb_ptr + kbi) + chunk * BM;
    it.n_rows = (int)min((long long)BM, end - it.list_lo);
  }
  it.ntiles = (it.n_keys + BN - 1) / BN;
  it.head_off = (long long)it.bh * p.S;
  return it;
}

__device__ __forceinline__ constexpr uint32_t koff(int ks) { return (uint32_t)(((ks >> 2) * PANEL + (ks & 3) * 32) >> 4); }
__device__ __forceinline__ constexpr uint32_t mnoff(int ks) { return (uint32_t)((ks * 2048) >> 4); }

// named barrier shared by the two softmax warps of one TMEM lane quarter (64 threads)
__device__ __forceinline__ void pair_sync(int quad) { asm volatile("bar.sync %0, 64;" ::"r"(quad + 1) : "memory"); }

template <bool DENSE>
__global__ void __launch_bounds__(THREADS, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = base;                      // [2][TILE]
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
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sm->k_full[s], 1); mbar_init(&sm->v_full[s], 1); mbar_init(&sm->k_empty[s], 1); mbar_init(&sm->v_empty[s], 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sm->s_full[b], 1); mbar_init(&sm->p_ready[b], 256);
      mbar_init(&sm->o_done[b], 1);
      mbar_init(&sm->q_full[b], 128); mbar_init(&sm->q_empty[b], 1);
      mbar_init(&sm->o_free[b], 256);
    }
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
  const int n_items = DENSE ? p.BH * ((p.S + BM - 1) / BM) : p.item_ptr[p.n_kb];
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
          // a K stage is free once the tile's Q K^T has run, a V stage only after its P V: separate
          // rings, so that the next K tile is already on its way while the softmax of this one runs
          if (fills >= STAGES) mbar_wait(&sm->k_empty[s], ((fills / STAGES) - 1) & 1, abort_flag, p.status);
          const int y = row0 + t * BN;
          if (p.prof) sm->t_issue[s] = clock64();
          mbar_expect_tx(&sm->k_full[s], TILE);
          tma_load_2d(sK + s * TILE, &tmK, &sm->k_full[s], 0, y);
          tma_load_2d(sK + s * TILE + PANEL, &tmK, &sm->k_full[s], 64, y);
          if (fills >= STAGES) mbar_wait(&sm->v_empty[s], ((fills / STAGES) - 1) & 1, abort_flag, p.status);
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
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      unsigned long long lat_sum = 0, lat_cnt = 0;
      uint32_t fills = 0;        // K/V tiles consumed so far (ring position)
      uint32_t tg = 0;           // tiles done so far: score buffer and o_done slot = count & 1
      uint32_t n = 0;            // items done so far: Q slot and O accumulator = count & 1
      for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
        const FwdItem it = decode_item<DENSE>(p, item);
        const int qb = n & 1;
        lap(5);
        mbar_wait(&sm->q_full[qb], (n >> 1) & 1, abort_flag, p.status);
        lap(0);
        tc_fence_after();
        const uint64_t dQ0 = make_smem_desc(smem_u32(sQ + qb * TILE), 16, 1024);
        auto issue_qk = [&](int t) {
          const uint32_t f = fills + t;
          const int s = f % STAGES;
          lap(5);
          mbar_wait(&sm->k_full[s], (f / STAGES) & 1, abort_flag, p.status);
          if (p.prof) {
            const long long now = clock64();
            if (now - t_mark > 100) { lat_sum += (unsigned long long)(now - sm->t_issue[s]); lat_cnt += 1; }
          }
          lap(1);
          tc_fence_after();
          const int n_mma = (min(BN, it.n_keys - t * BN) + 15) & ~15;
          const uint32_t idesc = make_idesc_bf16(BM, n_mma, false, false);
          const uint32_t buf = (tg + t) & 1;
          const uint64_t dK0 = make_smem_desc(smem_u32(sK + s * TILE), 16, 1024);
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks)
            mma_ss(tmem + S_COL + buf * 128, dQ0 + koff(ks), dK0 + koff(ks), idesc, ks > 0 ? 1u : 0u);
          mma_commit(&sm->s_full[buf]);
          mma_commit(&sm->k_empty[s]);
        };
        issue_qk(0);
        for (int t = 0; t < it.ntiles; ++t) {
          if (t + 1 < it.ntiles) issue_qk(t + 1);
          const uint32_t f = fills + t;
          const int s = f % STAGES;
          const uint32_t buf = (tg + t) & 1;
          lap(5);
          mbar_wait(&sm->p_ready[buf], ((tg + t) >> 1) & 1, abort_flag, p.status);
          lap(2);
          mbar_wait(&sm->v_full[s], (f / STAGES) & 1, abort_flag, p.status);
          lap(3);
          // this accumulator was last used two items ago: its epilogue must have read it
          if (t == 0 && n >= 2) mbar_wait(&sm->o_free[qb], ((n >> 1) - 1) & 1, abort_flag, p.status);
          lap(4);
          tc_fence_after();
          const int ksteps = (min(BN, it.n_keys - t * BN) + 15) >> 4;
          const uint32_t p_tmem = tmem + S_COL + buf * 128;
          const uint64_t mV0 = make_smem_desc(smem_u32(sV + s * TILE), PANEL, 1024);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            if (ks < ksteps)   // P of keys 64h + 16kk .. sits in columns 64h + 8kk .. of the score buffer
              mma_ts(tmem + O_COL + qb * 128, p_tmem + (ks >> 2) * 64 + (ks & 3) * 8, mV0 + mnoff(ks), IDESC_PV,
                     (t > 0 || ks > 0) ? 1u : 0u);
          mma_commit(&sm->v_empty[s]);
          mma_commit(&sm->o_done[buf]);
        }
        // Release the Q slot only after the item's last P V: that MMA needed the softmax warps' P, so
        // every waiter of this q_full phase has passed it before the loaders can complete the next one.
        mma_commit(&sm->q_empty[qb]);
        fills += it.ntiles;
        tg += it.ntiles;
      }
      lap(5);
      tflush(8);
      if (p.prof) { atomicAdd(p.prof + 7, lat_sum); atomicAdd(p.prof + 15, lat_cnt); }
    }
  } else if (warp >= 10) {
    // ------------------------------------------------------------------ loaders: Q rows of the next items
    const int lt = threadIdx.x - 320;   // 0..127
    const int chunk = lt & 15, panel = chunk >> 3, cc = chunk & 7;
    uint32_t n = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const FwdItem it = decode_item<DENSE>(p, item);
      const int qb = n & 1;
      const __nv_bfloat16* qh = p.q + it.head_off * DH;
      uint4 v[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int row = (lt >> 4) + 8 * i;
        v[i] = make_uint4(0u, 0u, 0u, 0u);
        if (row < it.n_rows) {
          const int qp = DENSE ? it.list_lo + row : __ldg(p.q_idx + it.list_lo + row);
          v[i] = __ldg(reinterpret_cast<const uint4*>(qh + (long long)qp * DH) + chunk);
        }
      }
      int my_qpos = -1, my_direct = DENSE ? 1 : 0;
      if (lt < it.n_rows) {
        my_qpos = DENSE ? it.list_lo + lt : __ldg(p.q_idx + it.list_lo + lt);
        if (!DENSE) {
          const long long G_ = it.head_off + my_qpos;
          my_direct = (p.q_ptr[G_ + 1] - p.q_ptr[G_]) == 1;
        }
      }
      if (n >= 2) mbar_wait(&sm->q_empty[qb], ((n >> 1) - 1) & 1, abort_flag, p.status);
      uint8_t* dst = sQ + qb * TILE;
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const int row = (lt >> 4) + 8 * i;
        *reinterpret_cast<uint4*>(dst + panel * PANEL + row * 128 + ((cc ^ (row & 7)) << 4)) = v[i];
      }
      // Four slots: q_empty(n - 2) has fired, so the softmax warps finished item n - 2's tiles and copied
      // its bookkeeping (and that of item n - 4, the previous user of this slot) to registers long ago.
      sm->qpos[n & 3][lt] = my_qpos;
      sm->direct[n & 3][lt] = my_direct;
      fence_async_proxy();
      mbar_arrive(&sm->q_full[qb]);
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (8 warps)
    const int quad = warp & 3;                      // TMEM lane quarter this warp may access
    const int half = (warp - 2) >> 2;               // which 64 of the tile's 128 keys / of the 128 output columns
    const int r = quad * 32 + lane;                 // query row of this thread
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint32_t tg = 0, n = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const FwdItem it = decode_item<DENSE>(p, item);
      const int qb = n & 1;
      lap(4);
      mbar_wait(&sm->q_full[qb], (n >> 1) & 1, abort_flag, p.status);     // publishes qpos / direct
      lap(5);
      const int qpos = sm->qpos[n & 3][r];
      const bool direct = sm->direct[n & 3][r] != 0;
      const uint32_t o_tmem = tmem + lane_addr + O_COL + qb * 128 + 64 * half;
      float m_used = -INFINITY, l = 0.f, l_r = 0.f;   // l: exact sum (for LSE); l_r: sum of the bf16-rounded weights
      for (int t = 0; t < it.ntiles; ++t) {
        const uint32_t gt = tg + t;
        const uint32_t buf = gt & 1;
        const uint32_t s_tmem = tmem + lane_addr + S_COL + buf * 128 + 64 * half;
        lap(3);
        mbar_wait(&sm->s_full[buf], (gt >> 1) & 1, abort_flag, p.status);
        lap(0);
        tc_fence_after();
        const int valid = min(BN, it.n_keys - t * BN) - 64 * half;      // valid keys among this thread's 64
        uint32_t sv[2][32];
        tmem_ld32(s_tmem, sv[0]);
        tmem_ld32(s_tmem + 32, sv[1]);
        tmem_ld_wait();
        if (valid < 64) {    // ragged last tile of the key range: keys beyond it get weight zero
#pragma unroll
          for (int c = 0; c < 2; ++c)
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c * 32 + i >= valid) sv[c][i] = 0xff800000u;
        }
        // row maximum of the raw scores (the softmax scale is positive, so it commutes with the max)
        float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
        for (int c = 0; c < 2; ++c)
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            mx0 = max3(mx0, __uint_as_float(sv[c][i]), __uint_as_float(sv[c][i + 1]));
            mx1 = max3(mx1, __uint_as_float(sv[c][i + 2]), __uint_as_float(sv[c][i + 3]));
            mx2 = max3(mx2, __uint_as_float(sv[c][i + 4]), __uint_as_float(sv[c][i + 5]));
            mx3 = max3(mx3, __uint_as_float(sv[c][i + 6]), __uint_as_float(sv[c][i + 7]));
          }
        float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
        // the row's other 64 keys belong to the thread with the same lane in the partner warp
        sm->xmax[buf][half][r] = mx;
        lap(1);
        pair_sync(quad);
        lap(2);
        mx = fmaxf(mx, sm->xmax[buf][half ^ 1][r]) * p.scale_log2;   // exp2 domain from here on
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
          // O of the previous tiles must be complete before it is rescaled
          mbar_wait(&sm->o_done[(gt - 1) & 1], ((gt - 1) >> 1) & 1, abort_flag, p.status);
          tc_fence_after();
#pragma unroll 1
          for (int c = 0; c < 2; ++c) {
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
        // P (bf16 pairs) goes over the first 32 of this thread's 64 score columns: keys 2i, 2i+1 -> column i
        float s0 = 0.f, s1 = 0.f, r0 = 0.f, r1 = 0.f;
        uint32_t pk[32];
        const float neg_m = -m_used;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float p0, p1;
          fma2(p0, p1, __uint_as_float(sv[i >> 4][(2 * i) & 31]), __uint_as_float(sv[i >> 4][((2 * i) & 31) + 1]),
               p.scale_log2, p.scale_log2, neg_m, neg_m);
          p0 = ex2(p0);
          p1 = ex2(p1);
          add2(s0, s1, s0, s1, p0, p1);
          pk[i] = pack_bf16(p0, p1);
          // the tensor core multiplies the ROUNDED weights: normalise O by their sum, so that the
          // rounding of P perturbs the weights but never their total
          add2(r0, r1, r0, r1, __uint_as_float(pk[i] << 16), __uint_as_float(pk[i] & 0xffff0000u));
        }
        tmem_st32(s_tmem, pk);
        l += s0 + s1;
        l_r += r0 + r1;
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(&sm->p_ready[buf]);
      }
      // ---- epilogue: wait for the last P V, combine the two halves' sums, normalise, write 64 columns
      lap(3);
      const uint32_t gl = tg + it.ntiles - 1;
      sm->xsum[half][0][r] = l;
      sm->xsum[half][1][r] = l_r;
      pair_sync(quad);
      l += sm->xsum[half ^ 1][0][r];
      l_r += sm->xsum[half ^ 1][1][r];
      mbar_wait(&sm->o_done[gl & 1], (gl >> 1) & 1, abort_flag, p.status);
      tc_fence_after();
      tg += it.ntiles;
      const float inv = 1.0f / l_r;
      const float row_lse = (m_used + log2f(l)) * 0.6931471805599453f;
      const bool row_ok = qpos >= 0;
      const long long G_ = it.head_off + (row_ok ? qpos : 0);
      const long long pos = (long long)it.list_lo + r;
#pragma unroll 1
      for (int c = 0; c < 2; ++c) {
        uint32_t ov[32];
        tmem_ld32(o_tmem + c * 32, ov);
        tmem_ld_wait();
        if (row_ok) {
          const int col = 64 * half + 32 * c;
          if (direct) {
            __nv_bfloat16* dst = p.o + G_ * DH + col;
            __nv_bfloat16* rdst = p.o_resid ? p.o_resid + G_ * DH + col : nullptr;
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              store4_resid(dst + i, rdst ? rdst + i : nullptr,
                           make_float4(__uint_as_float(ov[i]) * inv, __uint_as_float(ov[i + 1]) * inv,
                                       __uint_as_float(ov[i + 2]) * inv, __uint_as_float(ov[i + 3]) * inv));
          } else {
            float* dst = p.part_o + pos * DH + col;
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<float4*>(dst + i) =
                  make_float4(__uint_as_float(ov[i]) * inv, __uint_as_float(ov[i + 1]) * inv,
                              __uint_as_float(ov[i + 2]) * inv, __uint_as_float(ov[i + 3]) * inv);
          }
        }
      }
      if (row_ok && half == 0) {
        if (direct) p.lse[G_] = row_lse; else p.part_lse[pos] = row_lse;
      }
      tc_fence_before();
      mbar_arrive(&sm->o_free[qb]);
    }
    lap(4);
    if (warp == 2 && lane == 0) tflush(0);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

static int grid_items(long long items) { return (int)std::max<long long>(1, std::min<long long>(items, 148)); }

}  // namespace tc

int tc_sparse_fwd_wide(const Dims& D, const void* q, const void* k, const void* v, const int* kb_ptr, const int* q_idx,
                       const int* q_ptr, const int* q_pairs, long long cap, void* o, void* o_resid, float* lse,
                       int32_t* status, int* item_ptr, int* item_tab, long long max_items, float* part_o,
                       float* part_lse, cudaStream_t st);
int tc_dense_fwd_wide(const Dims& D, const void* q, const void* k, const void* v, void* o, void* o_resid, float* lse,
                      int32_t* status, cudaStream_t st);

// Key ranges of at least this many keys go to the kernel with 256-row items: its per-item set-up is
// longer, and it pays only when an item streams many key tiles.
static int wide_min_keys() {
  static int v = [] { const char* e = getenv("VMOBA_WIDE_MIN_KEYS"); return e ? atoi(e) : 1024; }();
  return v;
}

// Forward over the work lists (bf16, head_dim 128).  Returns VMOBA_ERR_CUDA if the tensor maps or
// the launch fail.
int tc_sparse_fwd(const Dims& D, const void* q, const void* k, const void* v, const int* kb_ptr, const int* q_idx,
                  const int* q_ptr, const int* q_pairs, long long cap, void* o, void* o_resid, float* lse,
                  int32_t* status, int* item_ptr, int* item_tab, long long max_items, float* part_o, float* part_lse,
                  cudaStream_t st) {
  if (D.sb >= wide_min_keys())
    return tc_sparse_fwd_wide(D, q, k, v, kb_ptr, q_idx, q_ptr, q_pairs, cap, o, o_resid, lse, status, item_ptr, item_tab,
                              max_items, part_o, part_lse, st);
  using namespace tc;
  CUtensorMap tmK, tmV;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN))
    return VMOBA_ERR_CUDA;
  const long long n_kb = (long long)D.BH * D.Nb;
  simt::item_ptr_kernel<<<1, 1024, 0, st>>>(kb_ptr, n_kb, BM, cap, item_ptr);
  simt::item_tab_kernel<<<(int)std::min<long long>((n_kb + 255) / 256, 148 * 4), 256, 0, st>>>(item_ptr, n_kb, max_items,
                                                                                               item_tab);
  Params p;
  p.q = (const __nv_bfloat16*)q; p.kb_ptr = kb_ptr; p.q_idx = q_idx; p.q_ptr = q_ptr; p.item_ptr = item_ptr;
  p.item_tab = item_tab;
  p.n_kb = (int)n_kb; p.S = D.S; p.Nb = D.Nb; p.sb = D.sb; p.BH = D.BH;
  p.scale_log2 = D.scale * 1.4426950408889634f;
  p.o = (__nv_bfloat16*)o; p.o_resid = (__nv_bfloat16*)o_resid; p.lse = lse; p.part_o = part_o; p.part_lse = part_lse;
  p.capacity = cap; p.status = status; p.prof = debug_wait_profile();
  VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)SMEM_BYTES));
  attn_fwd_tc_kernel<false><<<grid_items(cap / BM + n_kb), THREADS, SMEM_BYTES, st>>>(tmK, tmV, p);
  const long long nq = (long long)D.BH * D.S;
  simt::merge_kernel<__nv_bfloat16, 128, float><<<(int)std::min<long long>((nq + 7) / 8, 148 * 16), 256, 0, st>>>(
      q_ptr, q_pairs, nq, part_o, part_lse, cap, (__nv_bfloat16*)o, (__nv_bfloat16*)o_resid, lse);
  VMOBA_LAUNCH_OK(4);
  return VMOBA_OK;
}

int tc_dense_fwd(const Dims& D, const void* q, const void* k, const void* v, void* o, void* o_resid, float* lse,
                 int32_t* status, cudaStream_t st) {
  if (D.S >= wide_min_keys()) return tc_dense_fwd_wide(D, q, k, v, o, o_resid, lse, status, st);
  using namespace tc;
  CUtensorMap tmK, tmV;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN))
    return VMOBA_ERR_CUDA;
  Params p;
  p.q = (const __nv_bfloat16*)q; p.kb_ptr = nullptr; p.q_idx = nullptr; p.q_ptr = nullptr; p.item_ptr = nullptr;
  p.item_tab = nullptr;
  p.n_kb = 0; p.S = D.S; p.Nb = 1; p.sb = D.S; p.BH = D.BH;
  p.scale_log2 = D.scale * 1.4426950408889634f;
  p.o = (__nv_bfloat16*)o; p.o_resid = (__nv_bfloat16*)o_resid; p.lse = lse; p.part_o = nullptr; p.part_lse = nullptr;
  p.capacity = 0; p.status = status; p.prof = debug_wait_profile();
  VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)SMEM_BYTES));
  const long long items = (long long)D.BH * ((D.S + BM - 1) / BM);
  attn_fwd_tc_kernel<true><<<grid_items(items), THREADS, SMEM_BYTES, st>>>(tmK, tmV, p);
  VMOBA_LAUNCH_OK(1);
  return VMOBA_OK;
}

}  // namespace vmoba
