// Tensor-core path of the similarity map S_hat = q b^T (Section 3.3) for bf16 queries, head_dim 128.
//
// The scores must carry fp32 accuracy (the selection cutoff is compared in fp32), but the
// centroids b are fp32.  An fp32 number is exactly the sum of three bf16 numbers (3 x 8 mantissa
// bits), so each centroid row is split b = b1 + b2 + b3 and the product runs as three bf16 MMAs
// into one fp32 TMEM accumulator; q is bf16 already, so every product is exact and only the fp32
// accumulation rounds.
//
// Persistent CTAs walk (head, block range, 128-query tile) items: the three centroid parts of
// the block range stay in shared memory, query tiles stream through a 2-stage TMA ring, the
// accumulator is double buffered in TMEM so that the epilogue (the fp32 stores of the [S, N_b]
// matrix -- the HBM-bound part) overlaps the next tile's MMAs.  The epilogue threads (thread = query
// row) put 32 columns at a time into a swizzled shared-memory slab and one TMA store writes the slab
// as full 128-byte row segments; when rows are not 16-byte multiples (N_b % 4 != 0) each thread
// stores its own row instead.
#include <algorithm>

#include "sm100.cuh"

namespace vmoba {
namespace sct {

using namespace sm100;

constexpr int BM = 128, DH = 128;
constexpr int PANEL = 128 * 128;
constexpr int TILE = 2 * PANEL;
constexpr int NT_MAX = 160;              // centroid rows (key blocks) per pass
constexpr int THREADS = 192;
constexpr uint32_t TMEM_COLS = 512;      // two accumulators of up to 160 columns, at columns 0 and 256

struct Smem {
  uint64_t q_full[2], q_empty[2];
  uint64_t b_full, b_empty;
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
};
// B parts: 3 x (two 64-column panels of NT_MAX rows x 128 bytes)
constexpr int BPANEL = NT_MAX * 128;
constexpr int BPART = 2 * BPANEL;
constexpr int SLAB = BM * 128;            // 128 rows x 32 fp32 columns (16 KB), two of them
constexpr size_t SMEM_BYTES = 1024 + 2 * TILE + 3 * BPART + 2 * SLAB + sizeof(Smem) + 64;

struct Params {
  float* scores;
  int S, Nb, Nb_pad, BH;
  int n_pass, rows_pass;    // block ranges per head, rows per range (multiple of 16, <= NT_MAX)
  int tma_store;            // rows are multiples of 16 bytes: the epilogue writes through tmS
  float* range;             // optional [BH][2]: smallest and largest score of each head (starts at +inf, -inf)
  int32_t* status;
};

// Splits fp32 centroids into three bf16 parts: parts[part][bh][Nb_pad][128]; pad rows are zero.
__global__ void __launch_bounds__(256)
split_centroids_kernel(const float* __restrict__ cent, __nv_bfloat16* __restrict__ parts, int Nb, int Nb_pad, int BH,
                       float* __restrict__ range) {
  const long long n = (long long)BH * Nb_pad * DH;
  if (range) {     // the scores kernel that follows takes minima / maxima into these words
    const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (t < BH) { range[2 * t] = INFINITY; range[2 * t + 1] = -INFINITY; }
  }
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(i % DH);
    const long long row = i / DH;
    const int j = (int)(row % Nb_pad);
    const long long bh = row / Nb_pad;
    float x = 0.f;
    if (j < Nb) x = cent[(bh * Nb + j) * DH + c];
    const __nv_bfloat16 b1 = __float2bfloat16_rn(x);
    const float r1 = x - __bfloat162float(b1);
    const __nv_bfloat16 b2 = __float2bfloat16_rn(r1);
    const float r2 = r1 - __bfloat162float(b2);
    const __nv_bfloat16 b3 = __float2bfloat16_rn(r2);
    parts[i] = b1;
    parts[n + i] = b2;
    parts[2 * n + i] = b3;
  }
}

__global__ void __launch_bounds__(THREADS, 1)
scores_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmB,
                 const __grid_constant__ CUtensorMap tmS, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = base;                    // [2][TILE]
  uint8_t* sB = base + 2 * TILE;         // [3][BPART]
  uint8_t* sOut = sB + 3 * BPART;        // [2][SLAB]; BPART is a multiple of 1024
  Smem* sm = reinterpret_cast<Smem*>(sOut + 2 * SLAB);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &sm->abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sm->q_full[i], 1); mbar_init(&sm->q_empty[i], 1);
      mbar_init(&sm->acc_full[i], 1); mbar_init(&sm->acc_empty[i], 128);
    }
    mbar_init(&sm->b_full, 1);
    mbar_init(&sm->b_empty, 1);
    sm->abort_flag = 0;
    fence_barrier_init();
    prefetch_tmap(&tmQ);
    prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    tmem_alloc(&sm->tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = sm->tmem_base;

  // items: (bh, pass, tile), tile fastest; each CTA takes one contiguous range so that the centroid
  // parts of a (bh, pass) are loaded once per CTA
  const int tiles = (p.S + BM - 1) / BM;
  const long long n_items = (long long)p.BH * p.n_pass * tiles;
  const long long per = (n_items + gridDim.x - 1) / gridDim.x;
  const long long it0_ = (long long)blockIdx.x * per;
  const long long it0 = it0_ < n_items ? it0_ : n_items;
  const long long it1 = it0 + per < n_items ? it0 + per : n_items;
  const long long n_part_rows = (long long)p.BH * p.Nb_pad;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t qn = 0, bn = 0;
      long long cur_group = -1;
      for (long long it = it0; it < it1; ++it, ++qn) {
        const int tile = (int)(it % tiles);
        const long long group = it / tiles;            // bh * n_pass + pass
        const int pass = (int)(group % p.n_pass);
        const long long bh = group / p.n_pass;
        if (group != cur_group) {
          // new centroid range: wait until the MMAs that read the old one are done
          if (bn > 0) mbar_wait(&sm->b_empty, (bn - 1) & 1, abort_flag, p.status);
          const int y0 = (int)(bh * p.Nb_pad + (long long)pass * p.rows_pass);
          mbar_expect_tx(&sm->b_full, 3 * 2 * p.rows_pass * 128);
          for (int part = 0; part < 3; ++part) {
            const int y = (int)(part * n_part_rows) + y0;
            tma_load_2d(sB + part * BPART, &tmB, &sm->b_full, 0, y);
            tma_load_2d(sB + part * BPART + BPANEL, &tmB, &sm->b_full, 64, y);
          }
          cur_group = group;
          ++bn;
        }
        const int s = qn & 1;
        if (qn >= 2) mbar_wait(&sm->q_empty[s], ((qn >> 1) - 1) & 1, abort_flag, p.status);
        const int y = (int)(bh * p.S) + tile * BM;
        mbar_expect_tx(&sm->q_full[s], TILE);
        tma_load_2d(sQ + s * TILE, &tmQ, &sm->q_full[s], 0, y);
        tma_load_2d(sQ + s * TILE + PANEL, &tmQ, &sm->q_full[s], 64, y);
      }
      if (*abort_flag) {
        for (uint32_t f = qn > 2 ? qn - 2 : 0; f < qn; ++f) mbar_wait(&sm->q_full[f & 1], (f >> 1) & 1, abort_flag, p.status);
        if (bn > 0) mbar_wait(&sm->b_full, (bn - 1) & 1, abort_flag, p.status);
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: the whole warp walks the loop, one
    // elected lane issues (warp-uniform control flow; see elect_one)
    {
      const bool leader = elect_one();
      uint32_t qn = 0, bn = 0;
      long long cur_group = -1;
      const uint32_t idesc = make_idesc_bf16(BM, p.rows_pass, false, false);
      for (long long it = it0; it < it1; ++it, ++qn) {
        const long long group = it / tiles;
        if (group != cur_group) {
          // all MMAs on the previous range were issued before this point: release it to the producer
          if (leader && cur_group >= 0) mma_commit(&sm->b_empty);
          mbar_wait_warp(&sm->b_full, bn & 1, abort_flag, p.status);
          cur_group = group;
          ++bn;
        }
        const int s = qn & 1;
        mbar_wait_warp(&sm->q_full[s], (qn >> 1) & 1, abort_flag, p.status);
        if (qn >= 2) mbar_wait_warp(&sm->acc_empty[s], ((qn >> 1) - 1) & 1, abort_flag, p.status);
        tc_fence_after();
        const uint32_t d_tmem = tmem + (s ? 256u : 0u);
        const uint32_t sQ_addr = smem_u32(sQ + s * TILE);
#pragma unroll 1
        for (int part = 0; part < 3; ++part) {
          const uint32_t sB_addr = smem_u32(sB + part * BPART);
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks) {
            const uint64_t a = make_smem_desc(sQ_addr + (ks >> 2) * PANEL + (ks & 3) * 32, 16, 1024);
            const uint64_t b = make_smem_desc(sB_addr + (ks >> 2) * BPANEL + (ks & 3) * 32, 16, 1024);
            if (leader) mma_ss(d_tmem, a, b, idesc, (part > 0 || ks > 0) ? 1u : 0u);
          }
        }
        if (leader) mma_commit(&sm->q_empty[s]);
        if (leader) mma_commit(&sm->acc_full[s]);
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue: thread = query row
    const int quad = warp & 3;
    const int r = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint32_t qn = 0, slabs = 0;
    // smallest / largest score seen by this thread for the current head (the selection's first pass, taken
    // here while the scores are in registers); handed over with one atomic pair per warp when the head changes
    float rmin = INFINITY, rmax = -INFINITY;
    long long range_bh = -1;
    auto flush_range = [&]() {
      if (p.range && range_bh >= 0) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          rmin = fminf(rmin, __shfl_xor_sync(0xffffffffu, rmin, o));
          rmax = fmaxf(rmax, __shfl_xor_sync(0xffffffffu, rmax, o));
        }
        if (lane == 0 && rmin <= rmax) {
          atomic_min_f32(p.range + 2 * range_bh, rmin);
          atomic_max_f32(p.range + 2 * range_bh + 1, rmax);
        }
      }
      rmin = INFINITY; rmax = -INFINITY;
    };
    for (long long it = it0; it < it1; ++it, ++qn) {
      const int tile = (int)(it % tiles);
      const long long group = it / tiles;
      const int pass = (int)(group % p.n_pass);
      const long long bh = group / p.n_pass;
      if (bh != range_bh) { flush_range(); range_bh = bh; }
      const int s = qn & 1;
      mbar_wait(&sm->acc_full[s], (qn >> 1) & 1, abort_flag, p.status);
      tc_fence_after();
      const int row = tile * BM + r;
      const int j0 = pass * p.rows_pass;
      const int ncols = min(p.rows_pass, p.Nb - j0);       // real blocks in this range
      float* out = p.scores + ((long long)bh * p.S + row) * p.Nb + j0;
      const uint32_t a_tmem = tmem + lane_addr + (s ? 256u : 0u);
      if (p.tma_store) {
#pragma unroll 1
        for (int c0 = 0; c0 < p.rows_pass; c0 += 32) {
          if (j0 + c0 >= p.Nb) break;                         // the remaining slabs are padding (uniform)
          uint32_t v[32];
          tmem_ld32(a_tmem + c0, v);
          tmem_ld_wait();
          if (p.range && row < p.S) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (c0 + i < ncols) { rmin = fminf(rmin, __uint_as_float(v[i])); rmax = fmaxf(rmax, __uint_as_float(v[i])); }
          }
          uint8_t* slab = sOut + (slabs & 1) * SLAB;
          // the slab's previous store (two slabs ago) must have read it
          if (threadIdx.x == 64) bulk_wait_group_read<1>();
          asm volatile("bar.sync 1, 128;" ::: "memory");
#pragma unroll
          for (int i = 0; i < 8; ++i)
            *reinterpret_cast<uint4*>(slab + r * 128 + ((i ^ (r & 7)) << 4)) = make_uint4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
          fence_async_proxy();
          asm volatile("bar.sync 1, 128;" ::: "memory");
          if (threadIdx.x == 64) {
            tma_store_3d(&tmS, slab, j0 + c0, tile * BM, (int)bh);   // rows beyond S and columns beyond N_b are clipped
            bulk_commit_group();
          }
          ++slabs;
        }
      } else {
#pragma unroll 1
      for (int c0 = 0; c0 < p.rows_pass; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(a_tmem + c0, v);
        tmem_ld_wait();
        if (row < p.S) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c0 + i < ncols) {
              out[c0 + i] = __uint_as_float(v[i]);
              rmin = fminf(rmin, __uint_as_float(v[i])); rmax = fmaxf(rmax, __uint_as_float(v[i]));
            }
        }
      }
      }
      tc_fence_before();
      mbar_arrive(&sm->acc_empty[s]);
    }
    flush_range();
    if (threadIdx.x == 64) bulk_wait_group<0>();      // shared memory must outlive the last stores' reads
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

}  // namespace sct

size_t scores_tc_ws_bytes(const Dims& D) {
  const size_t Nb_pad = (size_t)(D.Nb + 31) / 32 * 32;
  return 3 * (size_t)D.BH * Nb_pad * sct::DH * sizeof(__nv_bfloat16) + 1024;
}

// scores [BH, S, Nb] fp32 from block-major bf16 q and fp32 centroids (already computed).
int scores_tc(const Dims& D, const void* q_bm, const float* cent, float* scores, float* range, void* ws,
              int32_t* status, cudaStream_t st) {
  using namespace sct;
  // ranges of whole 32-column slabs (the epilogue's store unit)
  const int Nb_pad = (D.Nb + 31) / 32 * 32;
  const int n_pass = (Nb_pad + NT_MAX - 1) / NT_MAX;
  const int rows_pass = ((Nb_pad + n_pass - 1) / n_pass + 31) / 32 * 32;
  __nv_bfloat16* parts = reinterpret_cast<__nv_bfloat16*>((reinterpret_cast<uintptr_t>(ws) + 1023) & ~uintptr_t(1023));
  const long long n = (long long)D.BH * Nb_pad * DH;
  split_centroids_kernel<<<(int)std::min<long long>((n + 255) / 256, sm_count() * 8), 256, 0, st>>>(cent, parts, D.Nb, Nb_pad, D.BH, range);
  CUtensorMap tmQ, tmB, tmS;
  const int tma_store = (D.Nb % 4 == 0) && (reinterpret_cast<uintptr_t>(scores) % 16 == 0);
  if (tma_store) {
    if (!sm100::make_tmap_f32_planes(&tmS, scores, (uint64_t)D.BH, (uint64_t)D.S, (uint64_t)D.Nb, BM)) return VMOBA_ERR_CUDA;
  } else {
    tmS = CUtensorMap{};
  }
  if (!sm100::make_tmap_bf16_rows(&tmQ, q_bm, (uint64_t)D.BH * D.S, DH, BM) ||
      !sm100::make_tmap_bf16_rows(&tmB, parts, (uint64_t)3 * D.BH * Nb_pad, DH, rows_pass))
    return VMOBA_ERR_CUDA;
  Params p;
  p.scores = scores; p.S = D.S; p.Nb = D.Nb; p.Nb_pad = Nb_pad; p.BH = D.BH; p.n_pass = n_pass; p.rows_pass = rows_pass;
  p.tma_store = tma_store;
  p.range = range;
  p.status = status;
  VMOBA_CUDA_OK(cudaFuncSetAttribute(scores_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM_BYTES));
  const long long items = (long long)D.BH * n_pass * ((D.S + BM - 1) / BM);
  scores_tc_kernel<<<(int)std::max<long long>(1, std::min<long long>(items, sm_count())), THREADS, SMEM_BYTES, st>>>(tmQ, tmB, tmS, p);
  VMOBA_LAUNCH_OK(2);
  return VMOBA_OK;
}

}  // namespace vmoba
