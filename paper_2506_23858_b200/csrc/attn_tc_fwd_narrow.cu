// Tensor-core attention forward for short and medium key blocks (bf16, head_dim 128; Step 3 of VMoBA): written for
// key blocks of a few 128-key tiles, where a work item is over after two or three tiles, and used up to thirteen.
//
// The wide kernel (attn_tc_fwd.cu) keeps the tensor pipe busy by running two query tiles of one item in opposite
// phase; that phase needs many key tiles to establish itself.  On a 270-key block both tiles run their softmax at
// the same time, the tensor pipe waits for both, and the item's fixed costs (finding its list, gathering 256 query
// rows into a single buffer, the epilogue's stores) are paid with nothing else in flight.  Here the overlap comes
// from the hardware instead: an item is ONE 128-row query tile, a CTA needs 100 KB of shared memory, 256 TMEM
// columns and 256 threads of 128 registers, and TWO CTAs share an SM.  While one of them gathers, waits for a key tile or
// writes its rows, the other one has the tensor pipe and the exponential unit.
//
//   warp 0        TMA producer: K and V tiles, one stage each (a K tile is reloaded as soon as its Q K^T has run)
//   warp 1        MMA issuer (all lanes walk the loop, one elected lane issues)
//   warps 4-7     softmax (+ epilogue, unless warps 8-11 exist): thread = one query row
//   warps 2,3     loaders: gather the 128 Q rows (and per-row output bookkeeping) of the NEXT item
//   warps 8-11    (key blocks of up to four tiles only) epilogue: read the accumulator, write the rows
//
// Rows of queries with a single block are final and go to o; the others are partial results that the merge pass
// combines: fp16 values times a power of two per row, beside the row's lse.
//
// TMEM: S (128 columns; the bf16 P is written over columns 64..127) and the accumulator O (128 columns).  A softmax
// thread reads its row in two halves, first for the maximum and, after the second half has been turned into P,
// once more for the first half, so that it never holds more than 64 scores; a tail tile of up to 64 keys takes
// one half only.  Items are described by 16-byte records (list, first position, rows) that every role fetches one
// item ahead.
#include <algorithm>

#include <cuda_fp16.h>

#include "attn_simt.cuh"
#include "sm100.cuh"

namespace vmoba {
namespace tcn {

using namespace sm100;

constexpr int BM = 128;              // query rows per item
constexpr int BN = 128;              // keys per tile
constexpr int DH = 128;              // head dim
constexpr int PANEL = BM * 128;      // bytes of one 64-column panel of a 128-row tile (16 KB)
constexpr int TILE = 2 * PANEL;      // bytes of a [128 x 128] bf16 tile (32 KB)
constexpr int THREADS = 256;
constexpr int THREADS_SPLIT = 384;   // with four epilogue warps
constexpr uint32_t TMEM_COLS = 256;
constexpr uint32_t O_COL = 128;      // S at 0, P at 64, O at 128
constexpr float RESCALE_LOG2 = 8.0f;

struct Smem {
  uint64_t k_full, k_empty, v_full, v_empty;
  uint64_t s_full, p_ready;          // scores written (commit) / P written (128 arrivals)
  uint64_t o_done;                   // P V of a key tile complete (commit)
  uint64_t q_full, q_empty;          // Q tile of an item gathered (64 arrivals) / no longer needed (commit)
  uint64_t ep_ready;                 // SPLIT: an item's normalisers are in ep_inv / ep_lse (128 softmax arrivals)
  uint64_t o_free;                   // SPLIT: the epilogue warps have read the accumulator (128 arrivals)
  uint32_t tmem_base;
  int abort_flag;
  float ep_inv[2][BM], ep_lse[2][BM];   // SPLIT, [item % 2][row]: 1 / sum of the rounded weights, natural-log lse
  int qinfo[4][BM];                  // [item % 4][row]: 2 * in-head position + (query has a single block), -1 for padding rows
};
// two CTAs per SM: each may use half of the SM's shared memory
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + 3 * TILE /*Q, K, V*/ + sizeof(Smem) + 32;
static_assert(SMEM_BYTES <= 113 * 1024, "narrow forward: two CTAs must fit one SM");
static_assert(3 * SMEM_BYTES > 228 * 1024, "narrow forward: a third CTA on an SM would wait for TMEM columns forever");

struct Params {
  const __nv_bfloat16* q;
  const int* q_idx;
  const int* q_ptr;
  const int* item_ptr;
  const int4* item_desc;   // per item {list index, first list position, rows, 0}
  int n_kb, S, Nb, sb;
  float scale_log2;        // softmax scale * log2(e)
  __nv_bfloat16* o;
  __nv_bfloat16* o_resid;
  RowMap o_map;            // where the rows of o go (block-major, or raster order through perm); o_resid is block-major
  float* lse;
  __half* part_o;          // partial rows: fp16 values times part_scale[row]
  float* part_lse;
  float* part_scale;
  int part_o_32;           // part_o is 32-byte aligned: rows go out with 32-byte stores
  int32_t* status;
  unsigned long long* prof;   // optional per-section cycle counters (diagnostics), or null
};

struct Item {
  int key_begin, n_keys, list_lo, n_rows, ntiles;
  long long head_off;
};

__device__ __forceinline__ Item item_from_desc(const Params& p, const int4 d) {
  Item it;
  const int kbi = checked_index(d.x, p.n_kb, p.status);
  const int bh = kbi / p.Nb;
  it.key_begin = (kbi - bh * p.Nb) * p.sb;
  it.n_keys = p.sb;
  it.list_lo = d.y;
  it.n_rows = d.z;
  it.ntiles = (it.n_keys + BN - 1) / BN;
  it.head_off = (long long)bh * p.S;
  return it;
}

// item_desc[item] = {index of the (batch, head, key block) list, first list position, rows (<= rows_per_item), 0}
static __global__ void __launch_bounds__(256)
item_desc_kernel(const int* __restrict__ item_ptr, const int* __restrict__ kb_ptr, long long n_kb, long long max_items,
                 long long capacity, int rows_per_item, int4* __restrict__ desc) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_kb; i += (long long)gridDim.x * blockDim.x) {
    const long long t0 = item_ptr[i], t1 = min((long long)item_ptr[i + 1], max_items);
    const long long lo = min((long long)kb_ptr[i], capacity), hi = min((long long)kb_ptr[i + 1], capacity);
    for (long long t = t0; t < t1; ++t) {
      const long long l = lo + (t - t0) * rows_per_item;
      desc[t] = make_int4((int)i, (int)l, (int)min((long long)rows_per_item, hi - l), 0);
    }
  }
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

// p = 2^(s * scale - m) for 64 scores; bf16 pairs (keys 2i, 2i+1 -> word i); s0/s1 collect the exact weights, r0/r1
// the bf16-rounded ones (the tensor core multiplies the ROUNDED weights: O is normalised by their sum, so that the
// rounding perturbs the weights but never their total).
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

// sixteen fp16 values of a partial row: one 32-byte store if the buffer allows it, else two of 16 bytes
__device__ __forceinline__ void store_part16(__half* dst, const uint32_t (&h)[8], int aligned32) {
  if (aligned32) {
    st_global_v8(dst, h[0], h[1], h[2], h[3], h[4], h[5], h[6], h[7]);
  } else {
    reinterpret_cast<uint4*>(dst)[0] = make_uint4(h[0], h[1], h[2], h[3]);
    reinterpret_cast<uint4*>(dst)[1] = make_uint4(h[4], h[5], h[6], h[7]);
  }
}

// eight consecutive outputs as bf16 (one 16-byte store) and, if asked for, their rounding residuals
// bf16(v - bf16(v)), computed in registers
__device__ __forceinline__ void store8_resid(__nv_bfloat16* dst, __nv_bfloat16* rdst, const float (&v)[8]) {
  uint32_t h[4], r[4];
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    h[k] = pack_bf16(v[2 * k], v[2 * k + 1]);
    r[k] = pack_bf16(v[2 * k] - __uint_as_float(h[k] << 16), v[2 * k + 1] - __uint_as_float(h[k] & 0xffff0000u));
  }
  *reinterpret_cast<uint4*>(dst) = make_uint4(h[0], h[1], h[2], h[3]);
  if (rdst) *reinterpret_cast<uint4*>(rdst) = make_uint4(r[0], r[1], r[2], r[3]);
}

// RASTER: the directly written rows of o go through p.o_map.
// SPLIT: four more warps (8-11) take the epilogue: they read the accumulator and write the rows while the softmax
// warps are already on the next item's first tile.  With 384 threads two CTAs leave 80 registers per thread, so the
// warp groups trade registers at the start: the softmax group takes 128, the first group keeps 72, the epilogue
// group 40.  Its loaders then have no room to hold rows in registers: they ask the L2 for an item's rows ahead of
// time and, once the Q tile is free, bring them in as asynchronous 16-byte copies straight into the swizzled tile.
template <bool RASTER, bool SPLIT>
__global__ void __launch_bounds__(SPLIT ? THREADS_SPLIT : THREADS, 2)
attn_fwd_narrow_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = base;
  uint8_t* sK = base + TILE;
  uint8_t* sV = base + 2 * TILE;
  Smem* sm = reinterpret_cast<Smem*>(base + 3 * TILE);
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
    mbar_init(&sm->k_full, 1); mbar_init(&sm->v_full, 1);
    mbar_init(&sm->k_empty, 1); mbar_init(&sm->v_empty, 1);
    mbar_init(&sm->s_full, 1); mbar_init(&sm->p_ready, 128);
    mbar_init(&sm->o_done, 1);
    mbar_init(&sm->q_full, 64); mbar_init(&sm->q_empty, 1);
    mbar_init(&sm->ep_ready, 128); mbar_init(&sm->o_free, 128);
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
  const int n_items = p.item_ptr[p.n_kb];
  constexpr uint32_t IDESC_PV = make_idesc_bf16(BM, DH, false, true);
  // the item of this trip comes from the record fetched during the trip before; the next one is requested here
  int4 next_desc = make_int4(0, 0, 0, 0);
  if ((int)blockIdx.x < n_items) next_desc = __ldg(p.item_desc + blockIdx.x);
  auto get_item = [&](int item) -> Item {
    const int4 d = next_desc;
    const int nxt = item + (int)gridDim.x;
    if (nxt < n_items) next_desc = __ldg(p.item_desc + nxt);
    return item_from_desc(p, d);
  };

  // SPLIT: every role starts by taking or giving back registers (the whole warp group executes the same one)
  if (warp < 4) {
    if constexpr (SPLIT) asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
  }
  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t fills = 0;
      for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        const Item it = get_item(item);
        const int row0 = (int)it.head_off + it.key_begin;
        for (int t = 0; t < it.ntiles; ++t, ++fills) {
          const uint32_t par = (fills - 1) & 1;
          const int y = row0 + t * BN;
          // the K stage is free once the Q K^T of the tile before has run, the V stage after its P V
          if (fills >= 1) mbar_wait(&sm->k_empty, par, abort_flag, p.status);
          mbar_expect_tx(&sm->k_full, TILE);
          tma_load_2d(sK, &tmK, &sm->k_full, 0, y);
          tma_load_2d(sK + PANEL, &tmK, &sm->k_full, 64, y);
          if (fills >= 1) mbar_wait(&sm->v_empty, par, abort_flag, p.status);
          mbar_expect_tx(&sm->v_full, TILE);
          tma_load_2d(sV, &tmV, &sm->v_full, 0, y);
          tma_load_2d(sV + PANEL, &tmV, &sm->v_full, 64, y);
        }
      }
      // drain: every issued load must have landed before the CTA may exit (only matters after a timeout)
      if (*abort_flag && fills >= 1) {
        mbar_wait(&sm->k_full, (fills - 1) & 1, abort_flag, p.status);
        mbar_wait(&sm->v_full, (fills - 1) & 1, abort_flag, p.status);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: the whole warp walks the loop, one
    // elected lane issues (warp-uniform control flow; see elect_one)
    const bool leader = elect_one();
    const int n_items_u = __reduce_max_sync(0xffffffffu, n_items);
    uint32_t fills = 0;              // key tiles consumed so far (phase of the K, V, score and P barriers)
    uint32_t n = 0;                  // items done so far
    const uint64_t dQ = make_smem_desc(smem_u32(sQ), 16, 1024);
    const uint64_t dK0 = make_smem_desc(smem_u32(sK), 16, 1024);
    const uint64_t mV0 = make_smem_desc(smem_u32(sV), PANEL, 1024);
    for (int item = blockIdx.x; item < n_items_u; item += gridDim.x, ++n) {
      const Item it = get_item(item);
      const int ntiles = __reduce_max_sync(0xffffffffu, it.ntiles);
      const int n_keys = __reduce_max_sync(0xffffffffu, it.n_keys);
      lap(5);
      mbar_wait_warp(&sm->q_full, n & 1, abort_flag, p.status);
      lap(0);
      for (int t = 0; t < ntiles; ++t) {
        const uint32_t f = fills + t;
        const int keys = min(BN, n_keys - t * BN);
        lap(5);
        mbar_wait_warp(&sm->k_full, f & 1, abort_flag, p.status);
        lap(1);
        tc_fence_after();
        {
          const uint32_t idesc = make_idesc_bf16(BM, (keys + 15) & ~15, false, false);
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks)
            if (leader) mma_ss(tmem, dQ + koff(ks), dK0 + koff(ks), idesc, ks > 0 ? 1u : 0u);
          if (leader) mma_commit(&sm->s_full);
          if (leader) mma_commit(&sm->k_empty);
          if (leader && t == ntiles - 1) mma_commit(&sm->q_empty);
        }
        lap(5);
        // P of this tile; it also says that the softmax threads have left the epilogue of the item before, i.e.
        // that its accumulator has been read
        mbar_wait_warp(&sm->p_ready, f & 1, abort_flag, p.status);
        lap(2);
        mbar_wait_warp(&sm->v_full, f & 1, abort_flag, p.status);
        lap(3);
        if constexpr (SPLIT) {
          // the accumulator still holds the item before until the epilogue warps have read it
          if (t == 0 && n >= 1) mbar_wait_warp(&sm->o_free, (n - 1) & 1, abort_flag, p.status);
          lap(4);
        }
        tc_fence_after();
        {
          const int ksteps = (keys + 15) >> 4;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks)
            if (leader && ks < ksteps)   // P of keys 16 ks .. 16 ks + 15 sits in columns 64 + 8 ks ..
              mma_ts(tmem + O_COL, tmem + 64 + ks * 8, mV0 + mnoff(ks), IDESC_PV, (t > 0 || ks > 0) ? 1u : 0u);
          if (leader) mma_commit(&sm->o_done);
          if (leader) mma_commit(&sm->v_empty);
        }
      }
      fills += ntiles;
    }
    lap(5);
    if (leader) tflush(8);
  } else if (warp < 4) {
    // ------------------------------------------------------------------ loaders: Q rows of the next item
    const int lt = (warp - 2) * 32 + lane;   // 0..63
    const int chunk = lt & 15, panel = chunk >> 3, cc = chunk & 7;
    uint32_t n = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const Item it = get_item(item);
      const __nv_bfloat16* qh = p.q + it.head_off * DH;
      // Four bookkeeping slots: the softmax warps read slot n % 4 in the epilogue of item n, and the loaders can be
      // at most two items ahead of an epilogue.
      int info[2];
      if constexpr (SPLIT) {
        if ((chunk & 7) == 0) {       // one L2 request per 128-byte line of every row of the item
#pragma unroll 4
          for (int i = 0; i < BM / 4; ++i) {
            const int row = (lt >> 4) + 4 * i;
            if (row < it.n_rows) {
              const int qp = checked_index(__ldg(p.q_idx + it.list_lo + row), p.S, p.status);
              asm volatile("prefetch.global.L2 [%0];" ::"l"(qh + (long long)qp * DH + chunk * 8));
            }
          }
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          info[h] = -1;
          if (h * 64 + lt < it.n_rows) {
            const int qp = checked_index(__ldg(p.q_idx + it.list_lo + h * 64 + lt), p.S, p.status);
            const long long G_ = it.head_off + qp;
            info[h] = 2 * qp + ((p.q_ptr[G_ + 1] - p.q_ptr[G_]) == 1 ? 1 : 0);
          }
        }
        if (n >= 1) mbar_wait(&sm->q_empty, (n - 1) & 1, abort_flag, p.status);
        const uint32_t q_base = smem_u32(sQ) + panel * PANEL;
#pragma unroll 8
        for (int i = 0; i < BM / 4; ++i) {
          const int row = (lt >> 4) + 4 * i;
          const bool ok = row < it.n_rows;
          const int qp = ok ? checked_index(__ldg(p.q_idx + it.list_lo + row), p.S, p.status) : 0;
          // rows beyond the item's are zero-filled (source size 0)
          asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(q_base + row * 128 + ((cc ^ (row & 7)) << 4)),
                       "l"(reinterpret_cast<const uint4*>(qh + (long long)qp * DH) + chunk), "r"(ok ? 16u : 0u)
                       : "memory");
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        asm volatile("cp.async.wait_group 0;" ::: "memory");
      }
      // without epilogue warps the loaders have 128 registers: two rounds of 64 rows that wait in registers
      constexpr int RR = 64;
      constexpr int NI = RR / 4;
      if constexpr (!SPLIT)
      for (int rnd = 0; rnd < BM / RR; ++rnd) {
        uint4 v[NI];
#pragma unroll
        for (int i = 0; i < NI; ++i) {
          const int row = rnd * RR + (lt >> 4) + 4 * i;
          v[i] = make_uint4(0u, 0u, 0u, 0u);
          if (row < it.n_rows) {
            const int qp = checked_index(__ldg(p.q_idx + it.list_lo + row), p.S, p.status);
            v[i] = __ldg(reinterpret_cast<const uint4*>(qh + (long long)qp * DH) + chunk);
          }
        }
        if (rnd == 0) {
          // per-row bookkeeping of rows lt and 64 + lt, fetched while the rows are in flight
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            info[h] = -1;
            if (h * 64 + lt < it.n_rows) {
              const int qp = checked_index(__ldg(p.q_idx + it.list_lo + h * 64 + lt), p.S, p.status);
              const long long G_ = it.head_off + qp;
              info[h] = 2 * qp + ((p.q_ptr[G_ + 1] - p.q_ptr[G_]) == 1 ? 1 : 0);
            }
          }
          // the later rounds' rows are fetched only after this round has been stored: ask the L2 for them now
          // (one request per 128-byte line)
          if ((chunk & 7) == 0) {
#pragma unroll 4
            for (int i = 0; i < (BM - RR) / 4; ++i) {
              const int row = RR + (lt >> 4) + 4 * i;
              if (row < it.n_rows) {
                const int qp = checked_index(__ldg(p.q_idx + it.list_lo + row), p.S, p.status);
                asm volatile("prefetch.global.L2 [%0];" ::"l"(qh + (long long)qp * DH + chunk * 8));
              }
            }
          }
          // the Q tile is free once the previous item's last Q K^T has run
          if (n >= 1) mbar_wait(&sm->q_empty, (n - 1) & 1, abort_flag, p.status);
        }
#pragma unroll
        for (int i = 0; i < NI; ++i) {
          const int row = rnd * RR + (lt >> 4) + 4 * i;
          *reinterpret_cast<uint4*>(sQ + panel * PANEL + row * 128 + ((cc ^ (row & 7)) << 4)) = v[i];
        }
      }
      sm->qinfo[n & 3][lt] = info[0];
      sm->qinfo[n & 3][64 + lt] = info[1];
      fence_async_proxy();
      mbar_arrive(&sm->q_full);
    }
  } else if (SPLIT && warp >= 8) {
    // ------------------------------------------------------------------ epilogue warps (SPLIT): thread = one query row
    if constexpr (SPLIT) asm volatile("setmaxnreg.dec.sync.aligned.u32 40;");
    const int quad = warp & 3;
    const int r = quad * 32 + lane;
    const uint32_t o_tmem = tmem + ((uint32_t)(quad * 32) << 16) + O_COL;
    uint32_t tc = 0, n = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const Item it = get_item(item);
      tc += it.ntiles;
      mbar_wait(&sm->ep_ready, n & 1, abort_flag, p.status);
      mbar_wait(&sm->o_done, (tc - 1) & 1, abort_flag, p.status);
      tc_fence_after();
      const int info = sm->qinfo[n & 3][r];
      const float inv = sm->ep_inv[n & 1][r];
      const float row_lse = sm->ep_lse[n & 1][r];
      const bool row_ok = info >= 0;
      const int qpos = row_ok ? info >> 1 : 0;
      const bool direct = (info & 1) != 0;
      const long long G_ = it.head_off + qpos;
      const long long o_row_off = RASTER ? ((row_ok && direct) ? p.o_map.off(G_, DH) : 0) : G_ * DH;
      const long long pos = (long long)it.list_lo + r;
      const bool partial = row_ok && !direct;
      // a partial row goes out as fp16 times a power of two: find the row's largest magnitude first
      float mul = inv, row_scale = 1.0f;
      if (__any_sync(0xffffffffu, partial)) {
        float amax = 0.f;
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
          uint32_t ov[16];
          tmem_ld16(o_tmem + c * 16, ov);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) amax = fmaxf(amax, fabsf(__uint_as_float(ov[i])));
        }
        if (partial) {
          row_scale = pow2_at_or_above(amax * inv);
          mul = inv / row_scale;
        }
      }
#pragma unroll 1
      for (int c = 0; c < 8; ++c) {
        uint32_t ov[16];
        tmem_ld16(o_tmem + c * 16, ov);
        tmem_ld_wait();
        if (c == 7) {          // the accumulator has been read: the next item's first P V may overwrite it
          tc_fence_before();
          mbar_arrive(&sm->o_free);
        }
        if (row_ok) {
          const int col = 16 * c;
          if (direct) {
            __nv_bfloat16* dst = p.o + o_row_off + col;
            __nv_bfloat16* rdst = p.o_resid ? p.o_resid + G_ * DH + col : nullptr;
#pragma unroll
            for (int i = 0; i < 16; i += 8) {
              float v8[8];
#pragma unroll
              for (int k = 0; k < 8; ++k) v8[k] = __uint_as_float(ov[i + k]) * inv;
              store8_resid(dst + i, rdst ? rdst + i : nullptr, v8);
            }
          } else {
            uint32_t h[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) h[i] = pack_half2(__uint_as_float(ov[2 * i]) * mul, __uint_as_float(ov[2 * i + 1]) * mul);
            store_part16(p.part_o + pos * DH + col, h, p.part_o_32);
          }
        }
      }
      if (row_ok) {
        if (direct) p.lse[G_] = row_lse; else { p.part_lse[pos] = row_lse; p.part_scale[pos] = row_scale; }
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue
    if constexpr (SPLIT) asm volatile("setmaxnreg.inc.sync.aligned.u32 128;");
    const int quad = warp & 3;                      // TMEM lane quarter this warp may access
    const int r = quad * 32 + lane;                 // query row inside the tile
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const uint32_t s_tmem = tmem + lane_addr;
    const uint32_t o_tmem = tmem + lane_addr + O_COL;
    uint32_t tc = 0, n = 0;                          // key tiles done; items seen
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const Item it = get_item(item);
      float m_used = -INFINITY, l = 0.f, l_r = 0.f;   // l: exact sum (for LSE); l_r: sum of the bf16-rounded weights
      for (int t = 0; t < it.ntiles; ++t, ++tc) {
        lap(3);
        mbar_wait(&sm->s_full, tc & 1, abort_flag, p.status);
        lap(0);
        tc_fence_after();
        const int valid = min(BN, it.n_keys - t * BN);
        uint32_t sv[64];
        tmem_ld32(s_tmem, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
        tmem_ld32(s_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
        tmem_ld_wait();
        if (valid < 64) mask_tail(sv, valid);
        float mx = max64(sv, -INFINITY);
        if (valid > 64) {                            // else the MMA wrote the first 64 columns at most
          tmem_ld32(s_tmem + 64, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
          tmem_ld32(s_tmem + 96, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
          tmem_ld_wait();
          if (valid < 128) mask_tail(sv, valid - 64);
          mx = max64(sv, mx);
        }
        mx *= p.scale_log2;                          // exp2 domain from here on (the scale is positive)
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
          mbar_wait(&sm->o_done, (tc - 1) & 1, abort_flag, p.status);
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
        const float neg_m = -m_used;
        uint32_t pk[32];
        if (valid > 64) {
          // keys 64..127 are in registers: their P goes over their own score columns 96..127
          exp_pack64(sv, p.scale_log2, neg_m, pk, s0, s1, r0, r1);
          tmem_st32(s_tmem + 96, pk);
          // keys 0..63 are read again (columns 0..63 are untouched); their P goes to columns 64..95, whose scores
          // have been consumed above
          tmem_ld32(s_tmem, *reinterpret_cast<uint32_t(*)[32]>(&sv[0]));
          tmem_ld32(s_tmem + 32, *reinterpret_cast<uint32_t(*)[32]>(&sv[32]));
          tmem_ld_wait();
        }
        exp_pack64(sv, p.scale_log2, neg_m, pk, s0, s1, r0, r1);    // valid <= 64: the masked scores are still here
        tmem_st32(s_tmem + 64, pk);
        l += s0 + s1;
        l_r += r0 + r1;
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(&sm->p_ready);
      }
      if constexpr (SPLIT) {
        // hand the row's normalisers to the epilogue warps and go on with the next item
        sm->ep_inv[n & 1][r] = 1.0f / l_r;
        sm->ep_lse[n & 1][r] = (m_used + log2f(l)) * 0.6931471805599453f;
        mbar_arrive(&sm->ep_ready);
        lap(4);
        continue;
      }
      // ---- epilogue: wait for the last P V, normalise, write the row
      lap(3);
      mbar_wait(&sm->o_done, (tc - 1) & 1, abort_flag, p.status);
      tc_fence_after();
      const int info = sm->qinfo[n & 3][r];
      const bool row_ok = info >= 0;
      const int qpos = row_ok ? info >> 1 : 0;
      const bool direct = (info & 1) != 0;
      const float inv = 1.0f / l_r;
      const float row_lse = (m_used + log2f(l)) * 0.6931471805599453f;
      const long long G_ = it.head_off + qpos;
      const long long o_row_off = RASTER ? ((row_ok && direct) ? p.o_map.off(G_, DH) : 0) : G_ * DH;
      const long long pos = (long long)it.list_lo + r;
      const bool partial = row_ok && !direct;
      // a partial row goes out as fp16 times a power of two: find the row's largest magnitude first
      float mul = inv, row_scale = 1.0f;
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
            for (int i = 0; i < 32; i += 8) {
              float v8[8];
#pragma unroll
              for (int k = 0; k < 8; ++k) v8[k] = __uint_as_float(ov[i + k]) * inv;
              store8_resid(dst + i, rdst ? rdst + i : nullptr, v8);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 32; i += 16) {
              uint32_t h[8];
#pragma unroll
              for (int k = 0; k < 8; ++k)
                h[k] = pack_half2(__uint_as_float(ov[i + 2 * k]) * mul, __uint_as_float(ov[i + 2 * k + 1]) * mul);
              store_part16(p.part_o + pos * DH + col + i, h, p.part_o_32);
            }
          }
        }
      }
      if (row_ok) {
        if (direct) p.lse[G_] = row_lse; else { p.part_lse[pos] = row_lse; p.part_scale[pos] = row_scale; }
      }
      // No barrier tells the MMA warp that the accumulator has been read: the next thing it waits for from these
      // threads is the P of the next item's first tile, which they write after this point.
      tc_fence_before();
      lap(4);
    }
    if (warp == 4 && lane == 0) tflush(0);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

}  // namespace tcn

// Forward over the work lists with one 128-row query tile per item (bf16, head_dim 128).
// item_tab must hold four ints per item.  Returns VMOBA_ERR_CUDA if the tensor maps or the launch fail.
int tc_sparse_fwd_narrow(const Dims& D, const void* q, const void* k, const void* v, const int* kb_ptr, const int* q_idx,
                         const int* q_ptr, const int* q_pairs, long long cap, void* o, void* o_resid, float* lse,
                         int32_t* status, int* item_ptr, int* item_tab, long long max_items, float* part_o,
                         float* part_lse, float* part_scale, cudaStream_t st, const RowMap& o_map) {
  using namespace tcn;
  CUtensorMap tmK, tmV;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN))
    return VMOBA_ERR_CUDA;
  const long long n_kb = (long long)D.BH * D.Nb;
  simt::item_ptr_kernel<<<1, 1024, 0, st>>>(kb_ptr, n_kb, BM, cap, item_ptr);
  item_desc_kernel<<<(int)std::min<long long>((n_kb + 255) / 256, sm_count() * 4), 256, 0, st>>>(
      item_ptr, kb_ptr, n_kb, max_items, cap, BM, reinterpret_cast<int4*>(item_tab));
  Params p;
  p.q = (const __nv_bfloat16*)q; p.q_idx = q_idx; p.q_ptr = q_ptr; p.item_ptr = item_ptr;
  p.item_desc = reinterpret_cast<const int4*>(item_tab);
  p.n_kb = (int)n_kb; p.S = D.S; p.Nb = D.Nb; p.sb = D.sb;
  p.scale_log2 = D.scale * 1.4426950408889634f;
  p.o = (__nv_bfloat16*)o; p.o_resid = (__nv_bfloat16*)o_resid; p.lse = lse;
  p.part_o = reinterpret_cast<__half*>(part_o); p.part_lse = part_lse; p.part_scale = part_scale;
  p.status = status; p.prof = debug_wait_profile();
  p.part_o_32 = (reinterpret_cast<uintptr_t>(part_o) % 32) == 0;
  p.o_map = o_map;
  const long long items = std::max<long long>(1, std::min<long long>(cap / BM + n_kb, 2LL * sm_count()));
  // Epilogue warps pay when an item is a few tiles long and its epilogue a quarter of it (C4 forward stage 0.42 ->
  // 0.37 ms, C2 0.212 -> 0.190 ms, 3D layer of C5 with 4 heads 0.84 -> 0.81 ms); on key blocks of 1560 and 1638
  // keys the plain variant is 2 % faster.
  const bool split_mode = D.sb <= 4 * BN;
  if (o_map.perm) {
    VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_narrow_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    attn_fwd_narrow_kernel<true, false><<<(int)items, THREADS, SMEM_BYTES, st>>>(tmK, tmV, p);
  } else if (split_mode) {
    VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_narrow_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    attn_fwd_narrow_kernel<false, true><<<(int)items, THREADS_SPLIT, SMEM_BYTES, st>>>(tmK, tmV, p);
  } else {
    VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_narrow_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
    attn_fwd_narrow_kernel<false, false><<<(int)items, THREADS, SMEM_BYTES, st>>>(tmK, tmV, p);
  }
  const long long nq = (long long)D.BH * D.S;
  simt::merge_batched_kernel<__nv_bfloat16, __half><<<(int)std::min<long long>((nq + 255) / 256, sm_count() * 8), 256, 0, st>>>(
      q_ptr, q_pairs, nq, p.part_o, part_lse, part_scale, cap, (__nv_bfloat16*)o, (__nv_bfloat16*)o_resid, lse, o_map);
  VMOBA_LAUNCH_OK(4);
  return VMOBA_OK;
}

}  // namespace vmoba
