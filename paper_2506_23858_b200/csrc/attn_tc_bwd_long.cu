// Backward kernels of the dense path (bf16, head_dim 128): one key range spanning the sequence, so
// each query meets every key tile and dQ is kept query-stationary instead of being reduced through
// memory.  The same math as attn_tc_bwd.cu, in two kernels:
//
//   * every contraction runs as N = 128 MMAs (an N = 64 shared-memory MMA is bound by operand
//     reads at about 60 % of the tensor rate; N = 128 runs at the full rate);
//   * the element-wise step and the second pair of MMAs are pipelined at a granularity of 32
//     columns: as soon as the compute warps have turned 32 columns of S / dP into bf16 P / dS in
//     TMEM, the MMA warp issues the two k-steps that consume them.
//
// dK/dV: item = 128 keys x all queries, in units of 128 queries (eight loader warps copy the Q / dO
//        rows).  TMEM: S^T | dP^T | dV | dK, 128 columns each.  K/V tile single-buffered, Q/dO ring of 2.
// dQ:    item = 128 queries x the key range, in units of 128 keys.
//        TMEM: S | dP | dQ (x2, alternating by item).  Q/dO tile single-buffered, K/V ring of 2.
#include <algorithm>

#include "attn_simt.cuh"
#include "sm100.cuh"

namespace vmoba {
namespace tcl {

using namespace sm100;

constexpr int BM = 128, BN = 128, DH = 128;
constexpr int PANEL = 128 * 128;
constexpr int TILE = 2 * PANEL;
constexpr uint32_t TMEM_COLS = 512;
constexpr int THREADS = 320;     // warp 0 producer, warp 1 MMA, warps 2-9 compute
constexpr int KV_THREADS = 576;  // dK/dV: plus 8 loader warps
constexpr uint32_t IDESC_KK = make_idesc_bf16(128, 128, false, false);
constexpr uint32_t IDESC_TN = make_idesc_bf16(128, 128, false, true);

__device__ __forceinline__ constexpr uint32_t koff(int ks) { return (uint32_t)(((ks >> 2) * PANEL + (ks & 3) * 32) >> 4); }
__device__ __forceinline__ constexpr uint32_t mnoff(int ks) { return (uint32_t)((ks * 2048) >> 4); }
__device__ __forceinline__ uint64_t desc_k0(uint32_t tile_addr) { return make_smem_desc(tile_addr, 16, 1024); }
__device__ __forceinline__ uint64_t desc_mn0(uint32_t tile_addr) { return make_smem_desc(tile_addr, PANEL, 1024); }

// Order in which the four 32-column groups become ready: warps 2-5 do groups 0 then 1, warps 6-9 do
// groups 2 then 3, so the MMA warp consumes 0, 2, 1, 3.
__device__ __forceinline__ constexpr int group_order(int i) { return i == 0 ? 0 : i == 1 ? 2 : i == 2 ? 1 : 3; }

// ==========================================================================================
// dK / dV
// ==========================================================================================
struct KvSmem {
  uint64_t kv_full, kv_empty;
  uint64_t chunk_full[2], chunk_empty[2];
  uint64_t sdp_full;
  uint64_t grp_ready[4];       // 128 arrivals each: the compute threads owning that column group
  uint64_t acc_done, acc_free;
  uint32_t tmem_base;
  int abort_flag;
  alignas(16) float lse2[2][128];
  alignas(16) float Dq[2][128];
};
constexpr size_t KV_SMEM_BYTES = 1024 + 2 * TILE + 2 * 2 * TILE + sizeof(KvSmem) + 32;

struct KvParams {
  const __nv_bfloat16 *q, *d_o;
  const float *lse, *Dv;
  int S, BH;
  float scale, scale_log2;
  __nv_bfloat16 *dk, *dv;
  int32_t* status;
  unsigned long long* prof;    // optional wait-time counters (diagnostics), or null
};

struct KvItem {
  int bh, key0, valid, n_units;
  long long list_lo, list_hi, head_off;
};

// item = (batch * heads + head, key tile); every query of the head meets the tile
__device__ __forceinline__ KvItem kv_decode(const KvParams& p, long long item, int tiles) {
  KvItem it;
  const int tile = (int)(item % tiles);
  it.bh = (int)(item / tiles);
  it.key0 = tile * BN;
  it.valid = min(BN, p.S - tile * BN);
  it.list_lo = 0; it.list_hi = p.S;
  it.n_units = (int)((it.list_hi - it.list_lo + BM - 1) / BM);
  it.head_off = (long long)it.bh * p.S;
  return it;
}

__global__ void __launch_bounds__(KV_THREADS, 1)
dkdv_long_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
                 const __grid_constant__ CUtensorMap tmQrow, const __grid_constant__ CUtensorMap tmOrow, const KvParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sK = base;
  uint8_t* sV = base + TILE;
  uint8_t* sC = base + 2 * TILE;           // [2][Q tile | dO tile]
  KvSmem* sm = reinterpret_cast<KvSmem*>(sC + 4 * TILE);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &sm->abort_flag;
  unsigned long long wp[4] = {0, 0, 0, 0};     // diagnostics: cycles per wait site
  const long long t_begin = clock64();
  auto twait = [&](int site, uint64_t* bar, uint32_t parity) {
    if (p.prof) {
      const long long t0 = clock64();
      mbar_wait(bar, parity, abort_flag, p.status);
      wp[site] += (unsigned long long)(clock64() - t0);
    } else {
      mbar_wait(bar, parity, abort_flag, p.status);
    }
  };
  auto tflush = [&](int base_site, int nsites) {
    if (p.prof) {
      for (int i = 0; i < nsites; ++i) atomicAdd(p.prof + base_site + i, wp[i]);
      atomicAdd(p.prof + base_site + nsites, (unsigned long long)(clock64() - t_begin));
    }
  };

  if (threadIdx.x == 0) {
    mbar_init(&sm->kv_full, 1); mbar_init(&sm->kv_empty, 1);
    for (int b = 0; b < 2; ++b) { mbar_init(&sm->chunk_full[b], 256); mbar_init(&sm->chunk_empty[b], 1); }
    mbar_init(&sm->sdp_full, 1);
    for (int g = 0; g < 4; ++g) mbar_init(&sm->grp_ready[g], 128);
    mbar_init(&sm->acc_done, 1);
    mbar_init(&sm->acc_free, 256);
    sm->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmK); prefetch_tmap(&tmV); prefetch_tmap(&tmQrow); prefetch_tmap(&tmOrow);
  }
  if (warp == 1) {
    tmem_alloc(&sm->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm->tmem_base;
  constexpr uint32_t ST_COL = 0, DPT_COL = 128, DV_COL = 256, DK_COL = 384;

  const int tiles = (p.S + BN - 1) / BN;
  const long long n_items = (long long)p.BH * tiles;

  if (warp == 0) {
    // ------------------------------------------------------------------ producer: the item's K and V tiles
    if (lane == 0) {
      uint32_t n = 0;
      for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const KvItem it = kv_decode(p, item, tiles);
        if (it.n_units == 0) continue;
        if (n >= 1) twait(0, &sm->kv_empty, (n - 1) & 1);
        const int y = (int)it.head_off + it.key0;
        mbar_expect_tx(&sm->kv_full, 2 * TILE);
        tma_load_2d(sK, &tmK, &sm->kv_full, 0, y);
        tma_load_2d(sK + PANEL, &tmK, &sm->kv_full, 64, y);
        tma_load_2d(sV, &tmV, &sm->kv_full, 0, y);
        tma_load_2d(sV + PANEL, &tmV, &sm->kv_full, 64, y);
        ++n;
      }
      if (*abort_flag && n > 0) mbar_wait(&sm->kv_full, (n - 1) & 1, abort_flag, p.status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: the whole warp walks the loop, one
    // elected lane issues (warp-uniform control flow; see elect_one)
    {
      const bool leader = elect_one();
      auto wwait = [&](int site, uint64_t* bar, uint32_t parity) { twait(site, bar, parity); __syncwarp(); };
      uint32_t n = 0, u0 = 0;
      const uint64_t dK0 = desc_k0(smem_u32(sK)), dV0 = desc_k0(smem_u32(sV));
      for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const KvItem it = kv_decode(p, item, tiles);
        if (it.n_units == 0) continue;
        wwait(0, &sm->kv_full, n & 1);
        for (int i = 0; i < it.n_units; ++i) {
          const uint32_t u = u0 + i;
          const int cb = u & 1;
          wwait(1, &sm->chunk_full[cb], (u >> 1) & 1);
          tc_fence_after();
          const uint32_t sQ_addr = smem_u32(sC + cb * 2 * TILE);
          const uint64_t dQ0 = desc_k0(sQ_addr), dO0 = desc_k0(sQ_addr + TILE);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) if (leader) mma_ss(tmem + ST_COL, dK0 + koff(ks), dQ0 + koff(ks), IDESC_KK, ks > 0 ? 1u : 0u);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) if (leader) mma_ss(tmem + DPT_COL, dV0 + koff(ks), dO0 + koff(ks), IDESC_KK, ks > 0 ? 1u : 0u);
          if (leader) mma_commit(&sm->sdp_full);
          // dV / dK still hold the previous item until its epilogue has read them
          if (i == 0 && n > 0) wwait(3, &sm->acc_free, (n - 1) & 1);
          const int rows = (int)min((long long)BM, it.list_hi - it.list_lo - (long long)i * BM);
          const int ksteps = (rows + 15) >> 4;
          const uint64_t mQ0 = desc_mn0(sQ_addr), mO0 = desc_mn0(sQ_addr + TILE);
#pragma unroll
          for (int gi = 0; gi < 4; ++gi) {
            const int g = group_order(gi);
            wwait(2, &sm->grp_ready[g], u & 1);
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
              const int ks = 2 * g + kk;
              if (leader && ks < ksteps) {
                const uint32_t first = (i == 0 && gi == 0 && kk == 0) ? 0u : 1u;
                // P^T / dS^T of queries 32g .. 32g+31 sit in columns 32g .. 32g+15 of their buffer
                mma_ts(tmem + DV_COL, tmem + ST_COL + 32 * g + 8 * kk, mO0 + mnoff(ks), IDESC_TN, first);
                mma_ts(tmem + DK_COL, tmem + DPT_COL + 32 * g + 8 * kk, mQ0 + mnoff(ks), IDESC_TN, first);
              }
            }
          }
          if (leader) mma_commit(&sm->chunk_empty[cb]);
        }
        if (leader) mma_commit(&sm->kv_empty);
        if (leader) mma_commit(&sm->acc_done);
        u0 += it.n_units;
        ++n;
      }
      if (leader) tflush(2, 4);      // [2] kv_full, [3] chunk_full, [4] grp_ready, [5] acc_free, [6] total
    }
  } else if (warp >= 10) {
    // ------------------------------------------------------------------ loaders (8 warps): gather Q / dO units, one ahead
    // 16 threads per 256-byte row, 16 rows per pass, 8 passes per tensor; every load of a unit is
    // issued before the wait for its slot, so the gather latency overlaps the previous unit.
    const int lt = threadIdx.x - 320;    // 0..255
    const int chunk = lt & 15, panel = chunk >> 3, cc = chunk & 7;
    uint32_t u0 = 0;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
      const KvItem it = kv_decode(p, item, tiles);
      const __nv_bfloat16* qh = p.q + it.head_off * DH;
      const __nv_bfloat16* oh = p.d_o + it.head_off * DH;
      for (int i = 0; i < it.n_units; ++i) {
        const uint32_t u = u0 + i;
        const int cb = u & 1;
        const long long lo = it.list_lo + (long long)i * BM;
        const int rows = (int)min((long long)BM, it.list_hi - lo);
        uint4 vq[8], vo[8];
#pragma unroll
        for (int k2 = 0; k2 < 8; ++k2) {
          const int row = (lt >> 4) + 16 * k2;
          vq[k2] = make_uint4(0u, 0u, 0u, 0u);
          vo[k2] = vq[k2];
          if (row < rows) {
            const long long src = lo + row;
            vq[k2] = __ldg(reinterpret_cast<const uint4*>(qh + src * DH) + chunk);
            vo[k2] = __ldg(reinterpret_cast<const uint4*>(oh + src * DH) + chunk);
          }
        }
        float l2 = INFINITY, dd = 0.f;     // padded queries: P = exp2(-inf) = 0
        if (lt < rows) {
          const long long G_ = it.head_off + lo + lt;
          l2 = p.lse[G_] * 1.4426950408889634f;
          dd = p.Dv[G_];
        }
        if (u >= 2) twait(1, &sm->chunk_empty[cb], ((u >> 1) - 1) & 1);
        uint8_t* dst = sC + cb * 2 * TILE;
#pragma unroll
        for (int k2 = 0; k2 < 8; ++k2) {
          const int row = (lt >> 4) + 16 * k2;
          const int off = panel * PANEL + row * 128 + ((cc ^ (row & 7)) << 4);
          *reinterpret_cast<uint4*>(dst + off) = vq[k2];
          *reinterpret_cast<uint4*>(dst + TILE + off) = vo[k2];
        }
        if (lt < BM) { sm->lse2[cb][lt] = l2; sm->Dq[cb][lt] = dd; }
        fence_async_proxy();
        mbar_arrive(&sm->chunk_full[cb]);
      }
      u0 += it.n_units;
    }
    if (lt == 0) tflush(7, 2);      // [7] -, [8] chunk_empty, [9] total
  } else {
    // ------------------------------------------------------------------ compute: thread = (key row, two 32-query groups)
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    const int r = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint32_t n = 0, u0 = 0;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
      const KvItem it = kv_decode(p, item, tiles);
      __nv_bfloat16* dv_row = p.dv + (it.head_off + it.key0 + r) * DH;
      __nv_bfloat16* dk_row = p.dk + (it.head_off + it.key0 + r) * DH;
      if (it.n_units == 0) {
        if (r < it.valid) {
          const uint4 z = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            reinterpret_cast<uint4*>(dk_row)[half * 8 + i] = z;
            reinterpret_cast<uint4*>(dv_row)[half * 8 + i] = z;
          }
        }
        continue;
      }
      for (int i = 0; i < it.n_units; ++i) {
        const uint32_t u = u0 + i;
        const int cb = u & 1;
        twait(0, &sm->chunk_full[cb], (u >> 1) & 1);   // publishes lse2 / Dq of this unit
        twait(1, &sm->sdp_full, u & 1);
        tc_fence_after();
#pragma unroll 1
        for (int gg = 0; gg < 2; ++gg) {
          const int g = 2 * half + gg;
          const float4* lse2 = reinterpret_cast<const float4*>(sm->lse2[cb] + 32 * g);
          const float4* Dq = reinterpret_cast<const float4*>(sm->Dq[cb] + 32 * g);
          const uint32_t st_t = tmem + lane_addr + ST_COL + 32 * g, dp_t = tmem + lane_addr + DPT_COL + 32 * g;
          uint32_t sv[32], dv_[32];
          tmem_ld32(st_t, sv);
          tmem_ld32(dp_t, dv_);
          tmem_ld_wait();
          uint32_t pk[16], dk_[16];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float4 l4 = lse2[e], d4 = Dq[e];
            const float p0 = ex2(fmaf(__uint_as_float(sv[4 * e]), p.scale_log2, -l4.x));
            const float p1 = ex2(fmaf(__uint_as_float(sv[4 * e + 1]), p.scale_log2, -l4.y));
            const float p2 = ex2(fmaf(__uint_as_float(sv[4 * e + 2]), p.scale_log2, -l4.z));
            const float p3 = ex2(fmaf(__uint_as_float(sv[4 * e + 3]), p.scale_log2, -l4.w));
            pk[2 * e] = pack_bf16(p0, p1);
            pk[2 * e + 1] = pack_bf16(p2, p3);
            dk_[2 * e] = pack_bf16(p0 * (__uint_as_float(dv_[4 * e]) - d4.x), p1 * (__uint_as_float(dv_[4 * e + 1]) - d4.y));
            dk_[2 * e + 1] = pack_bf16(p2 * (__uint_as_float(dv_[4 * e + 2]) - d4.z), p3 * (__uint_as_float(dv_[4 * e + 3]) - d4.w));
          }
          tmem_st16(st_t, pk);
          tmem_st16(dp_t, dk_);
          tmem_st_wait();
          tc_fence_before();
          mbar_arrive(&sm->grp_ready[g]);
        }
      }
      // ---- epilogue: each half writes 64 of the 128 dV / dK columns of its key row
      twait(2, &sm->acc_done, n & 1);
      tc_fence_after();
#pragma unroll 1
      for (int cg2 = 0; cg2 < 2; ++cg2) {
        const int cgrp = half * 2 + cg2;
        uint32_t a[32], bb[32];
        tmem_ld32(tmem + lane_addr + DV_COL + cgrp * 32, a);
        tmem_ld32(tmem + lane_addr + DK_COL + cgrp * 32, bb);
        tmem_ld_wait();
        if (r < it.valid) {
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            store4(dv_row + cgrp * 32 + i, make_float4(__uint_as_float(a[i]), __uint_as_float(a[i + 1]),
                                                       __uint_as_float(a[i + 2]), __uint_as_float(a[i + 3])));
            store4(dk_row + cgrp * 32 + i,
                   make_float4(__uint_as_float(bb[i]) * p.scale, __uint_as_float(bb[i + 1]) * p.scale,
                               __uint_as_float(bb[i + 2]) * p.scale, __uint_as_float(bb[i + 3]) * p.scale));
          }
        }
      }
      tc_fence_before();
      mbar_arrive(&sm->acc_free);
      u0 += it.n_units;
      ++n;
    }
    if (threadIdx.x == 64) tflush(10, 3);   // [10] chunk_full, [11] sdp_full, [12] acc_done, [13] total
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}


// ==========================================================================================
// dQ
// ==========================================================================================
struct DqSmem {
  uint64_t kv_full[2], kv_empty[2];
  uint64_t qdo_full, qdo_empty;
  uint64_t sdp_full;
  uint64_t grp_ready[4];
  uint64_t dq_done[2], dq_free[2];
  uint32_t tmem_base;
  int abort_flag;
  float lse2[128];
  float Dr[128];
  int G[128];                  // flat output row of each query (b*heads+head)*S + p, -1 for padding rows
};
constexpr size_t DQ_SMEM_BYTES = 1024 + 2 * TILE + 2 * 2 * TILE + sizeof(DqSmem) + 32;

struct DqParams {
  const float *lse, *Dv;
  int S, BH;
  float scale, scale_log2;
  __nv_bfloat16* dq;
  int32_t* status;
};

struct DqItem {
  int bh, key_begin, n_keys, list_lo, n_rows, n_units;
  long long head_off;
};

// item = (batch * heads + head, tile of 128 consecutive queries) against all keys of the head
__device__ __forceinline__ DqItem dq_decode(const DqParams& p, int item) {
  DqItem it;
  const int tiles = (p.S + BM - 1) / BM;
  it.bh = item / tiles;
  const int t = item - it.bh * tiles;
  it.key_begin = 0; it.n_keys = p.S; it.list_lo = t * BM; it.n_rows = min(BM, p.S - it.list_lo);
  it.n_units = (it.n_keys + BN - 1) / BN;
  it.head_off = (long long)it.bh * p.S;
  return it;
}

__global__ void __launch_bounds__(THREADS, 1)
dq_long_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
               const __grid_constant__ CUtensorMap tmQrow, const __grid_constant__ CUtensorMap tmOrow, const DqParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = base;
  uint8_t* sdO = base + TILE;
  uint8_t* sKV = base + 2 * TILE;          // [2][K tile | V tile]
  DqSmem* sm = reinterpret_cast<DqSmem*>(sKV + 4 * TILE);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &sm->abort_flag;

  if (threadIdx.x == 0) {
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sm->kv_full[b], 1); mbar_init(&sm->kv_empty[b], 1);
      mbar_init(&sm->dq_done[b], 1); mbar_init(&sm->dq_free[b], 256);
    }
    mbar_init(&sm->qdo_full, 1); mbar_init(&sm->qdo_empty, 1);
    mbar_init(&sm->sdp_full, 1);
    for (int g = 0; g < 4; ++g) mbar_init(&sm->grp_ready[g], 128);
    sm->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmK); prefetch_tmap(&tmV); prefetch_tmap(&tmQrow); prefetch_tmap(&tmOrow);
  }
  if (warp == 1) {
    tmem_alloc(&sm->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm->tmem_base;
  constexpr uint32_t S_COL = 0, DP_COL = 128, DQ_COL = 256;
  const int n_items = p.BH * ((p.S + BM - 1) / BM);

  if (warp == 0) {
    // ------------------------------------------------------------------ producer: gathered Q / dO of the item, K/V units
    uint32_t n = 0, f = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const DqItem it = dq_decode(p, item);
      int rc[4], gi[4];
      float l2[4], dd[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int r = 4 * lane + k;
        const bool ok = r < it.n_rows;
        const int qpos = it.list_lo + (ok ? r : 0);
        const long long G_ = it.head_off + qpos;
        rc[k] = (int)G_;
        gi[k] = ok ? (int)G_ : -1;
        l2[k] = ok ? p.lse[G_] * 1.4426950408889634f : INFINITY;
        dd[k] = ok ? p.Dv[G_] : 0.f;
      }
      if (n >= 1) mbar_wait(&sm->qdo_empty, (n - 1) & 1, abort_flag, p.status);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        sm->lse2[4 * lane + k] = l2[k]; sm->Dr[4 * lane + k] = dd[k]; sm->G[4 * lane + k] = gi[k];
      }
      __syncwarp();
      if (lane == 0) mbar_expect_tx(&sm->qdo_full, 2 * TILE);
      __syncwarp();
      tma_gather_tile128(sQ, &tmQrow, &sm->qdo_full, lane, rc);
      tma_gather_tile128(sdO, &tmOrow, &sm->qdo_full, lane, rc);
      if (lane == 0) {
        const int row0 = (int)it.head_off + it.key_begin;
        for (int t = 0; t < it.n_units; ++t, ++f) {
          const int s = f & 1;
          if (f >= 2) mbar_wait(&sm->kv_empty[s], ((f >> 1) - 1) & 1, abort_flag, p.status);
          uint8_t* dst = sKV + s * 2 * TILE;
          const int y = row0 + t * BN;
          mbar_expect_tx(&sm->kv_full[s], 2 * TILE);
          tma_load_2d(dst, &tmK, &sm->kv_full[s], 0, y);
          tma_load_2d(dst + PANEL, &tmK, &sm->kv_full[s], 64, y);
          tma_load_2d(dst + TILE, &tmV, &sm->kv_full[s], 0, y);
          tma_load_2d(dst + TILE + PANEL, &tmV, &sm->kv_full[s], 64, y);
        }
      }
      f = __shfl_sync(0xffffffffu, f, 0);
    }
    if (*abort_flag && lane == 0) {
      if (n > 0) mbar_wait(&sm->qdo_full, (n - 1) & 1, abort_flag, p.status);
      for (uint32_t g = f > 2 ? f - 2 : 0; g < f; ++g) mbar_wait(&sm->kv_full[g & 1], (g >> 1) & 1, abort_flag, p.status);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: the whole warp walks the loop, one
    // elected lane issues (warp-uniform control flow; see elect_one)
    {
      const bool leader = elect_one();
      uint32_t n = 0, f = 0;
      const uint64_t dQ0 = desc_k0(smem_u32(sQ)), dO0 = desc_k0(smem_u32(sdO));
      for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
        const DqItem it = dq_decode(p, item);
        const int acc = n & 1;
        mbar_wait_warp(&sm->qdo_full, n & 1, abort_flag, p.status);
        for (int t = 0; t < it.n_units; ++t, ++f) {
          const int s = f & 1;
          mbar_wait_warp(&sm->kv_full[s], (f >> 1) & 1, abort_flag, p.status);
          tc_fence_after();
          const int n_mma = (min(BN, it.n_keys - t * BN) + 15) & ~15;
          const uint32_t idesc = make_idesc_bf16(BM, n_mma, false, false);
          const uint32_t sK_addr = smem_u32(sKV + s * 2 * TILE);
          const uint64_t dK0 = desc_k0(sK_addr), dV0 = desc_k0(sK_addr + TILE), mK0 = desc_mn0(sK_addr);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) if (leader) mma_ss(tmem + S_COL, dQ0 + koff(ks), dK0 + koff(ks), idesc, ks > 0 ? 1u : 0u);
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) if (leader) mma_ss(tmem + DP_COL, dO0 + koff(ks), dV0 + koff(ks), idesc, ks > 0 ? 1u : 0u);
          if (leader) mma_commit(&sm->sdp_full);
          // this accumulator was last used two items ago: its epilogue must have read it
          if (t == 0 && n >= 2) mbar_wait_warp(&sm->dq_free[acc], ((n >> 1) - 1) & 1, abort_flag, p.status);
          const int ksteps = n_mma >> 4;
#pragma unroll
          for (int gi = 0; gi < 4; ++gi) {
            const int g = group_order(gi);
            mbar_wait_warp(&sm->grp_ready[g], f & 1, abort_flag, p.status);
            tc_fence_after();
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {
              const int ks = 2 * g + kk;
              if (leader && ks < ksteps)
                mma_ts(tmem + DQ_COL + acc * 128, tmem + DP_COL + 32 * g + 8 * kk, mK0 + mnoff(ks), IDESC_TN,
                       (t == 0 && gi == 0 && kk == 0) ? 0u : 1u);
            }
          }
          if (leader) mma_commit(&sm->kv_empty[s]);
        }
        if (leader) mma_commit(&sm->qdo_empty);
        if (leader) mma_commit(&sm->dq_done[acc]);
      }
    }
  } else {
    // ------------------------------------------------------------------ compute: thread = (query row, two 32-key groups)
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;
    const int r = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint32_t n = 0, f = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++n) {
      const DqItem it = dq_decode(p, item);
      const int acc = n & 1;
      mbar_wait(&sm->qdo_full, n & 1, abort_flag, p.status);     // publishes the per-row scalars
      const float lse2 = sm->lse2[r], Dr = sm->Dr[r];
      const int G_ = sm->G[r];
      for (int t = 0; t < it.n_units; ++t, ++f) {
        const int valid_t = min(BN, it.n_keys - t * BN);
        mbar_wait(&sm->sdp_full, f & 1, abort_flag, p.status);
        tc_fence_after();
#pragma unroll 1
        for (int gg = 0; gg < 2; ++gg) {
          const int g = 2 * half + gg;
          const int valid = valid_t - 32 * g;                     // valid keys among this group's 32
          const uint32_t s_t = tmem + lane_addr + S_COL + 32 * g, dp_t = tmem + lane_addr + DP_COL + 32 * g;
          uint32_t sv[32], dv_[32];
          tmem_ld32(s_t, sv);
          tmem_ld32(dp_t, dv_);
          tmem_ld_wait();
          uint32_t ds[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float p0 = ex2(fmaf(__uint_as_float(sv[2 * e]), p.scale_log2, -lse2));
            const float p1 = ex2(fmaf(__uint_as_float(sv[2 * e + 1]), p.scale_log2, -lse2));
            const float x0 = (2 * e < valid) ? p0 * (__uint_as_float(dv_[2 * e]) - Dr) : 0.f;
            const float x1 = (2 * e + 1 < valid) ? p1 * (__uint_as_float(dv_[2 * e + 1]) - Dr) : 0.f;
            ds[e] = pack_bf16(x0, x1);
          }
          tmem_st16(dp_t, ds);
          tmem_st_wait();
          tc_fence_before();
          mbar_arrive(&sm->grp_ready[g]);
        }
      }
      // ---- epilogue: each half writes 64 of the 128 dQ columns of its row
      mbar_wait(&sm->dq_done[acc], (n >> 1) & 1, abort_flag, p.status);
      tc_fence_after();
#pragma unroll 1
      for (int cg2 = 0; cg2 < 2; ++cg2) {
        const int cgrp = half * 2 + cg2;
        uint32_t a[32];
        tmem_ld32(tmem + lane_addr + DQ_COL + acc * 128 + cgrp * 32, a);
        tmem_ld_wait();
        if (G_ >= 0) {      // the item holds every key of the row: the result is final
          __nv_bfloat16* dst = p.dq + (long long)G_ * DH + cgrp * 32;
#pragma unroll
          for (int i = 0; i < 32; i += 4)
            store4(dst + i, make_float4(__uint_as_float(a[i]) * p.scale, __uint_as_float(a[i + 1]) * p.scale,
                                        __uint_as_float(a[i + 2]) * p.scale, __uint_as_float(a[i + 3]) * p.scale));
        }
      }
      tc_fence_before();
      mbar_arrive(&sm->dq_free[acc]);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

static int grid_items(long long items) { return (int)std::max<long long>(1, std::min<long long>(items, sm_count())); }

}  // namespace tcl

// dK, dV of the dense path.  The q / d_o rows are fetched as row gathers, which need one-row tensor maps.
int tc_long_dkdv(const Dims& D, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                 const float* Dv, void* dk, void* dv, int32_t* status, unsigned long long* prof, cudaStream_t st) {
  using namespace tcl;
  CUtensorMap tmK, tmV, tmQ, tmO;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN) ||
      !sm100::make_tmap_bf16_rows(&tmQ, q, rows, DH, 1) || !sm100::make_tmap_bf16_rows(&tmO, d_o, rows, DH, 1))
    return VMOBA_ERR_CUDA;
  KvParams kp;
  kp.q = (const __nv_bfloat16*)q; kp.d_o = (const __nv_bfloat16*)d_o; kp.lse = lse; kp.Dv = Dv; kp.S = D.S; kp.BH = D.BH;
  kp.scale = D.scale; kp.scale_log2 = D.scale * 1.4426950408889634f;
  kp.dk = (__nv_bfloat16*)dk; kp.dv = (__nv_bfloat16*)dv; kp.status = status; kp.prof = prof;
  VMOBA_CUDA_OK(cudaFuncSetAttribute(dkdv_long_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)KV_SMEM_BYTES));
  const long long items = (long long)D.BH * ((D.S + BN - 1) / BN);
  dkdv_long_kernel<<<grid_items(items), KV_THREADS, KV_SMEM_BYTES, st>>>(tmK, tmV, tmQ, tmO, kp);
  VMOBA_LAUNCH_OK(1);
  return VMOBA_OK;
}

// dQ of the dense path.
int tc_long_dq(const Dims& D, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
               const float* Dv, void* dq, int32_t* status, cudaStream_t st) {
  using namespace tcl;
  CUtensorMap tmK, tmV, tmQ, tmO;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN) ||
      !sm100::make_tmap_bf16_rows(&tmQ, q, rows, DH, 1) || !sm100::make_tmap_bf16_rows(&tmO, d_o, rows, DH, 1))
    return VMOBA_ERR_CUDA;
  DqParams qp;
  qp.lse = lse; qp.Dv = Dv; qp.S = D.S; qp.BH = D.BH;
  qp.scale = D.scale; qp.scale_log2 = D.scale * 1.4426950408889634f;
  qp.dq = (__nv_bfloat16*)dq; qp.status = status;
  VMOBA_CUDA_OK(cudaFuncSetAttribute(dq_long_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)DQ_SMEM_BYTES));
  const long long items = (long long)D.BH * ((D.S + BM - 1) / BM);
  dq_long_kernel<<<grid_items(items), THREADS, DQ_SMEM_BYTES, st>>>(tmK, tmV, tmQ, tmO, qp);
  VMOBA_LAUNCH_OK(1);
  return VMOBA_OK;
}

}  // namespace vmoba
