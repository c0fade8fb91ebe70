// Tensor-core attention forward for bf16, head_dim 128 (Step 3 of VMoBA and its dense limit).
//
// One persistent CTA per SM walks the work items.  An item is 128 query rows (sparse: a chunk of
// the queries that selected key block j, gathered by index; dense: 128 consecutive rows) against
// a contiguous key range (the block, or the whole sequence), streamed in tiles of 128 keys:
//
//   warp 0      TMA producer: K and V tiles (two 64-column panels each, 128-byte swizzle) into a
//               3-stage ring, completion on mbarriers
//   warp 1      MMA issuer (one thread): S = Q K^T into one of two TMEM score buffers, then
//               O += P V with P read from TMEM; tcgen05.commit signals the other roles
//   warps 2-5   softmax: thread = query row.  Reads S from TMEM, online softmax in the exp2
//               domain, writes P (bf16) over S in TMEM, rescales O in TMEM only when the running
//               max moved by more than 2^8, and runs the epilogue (normalise, write O / partials)
//
// QK^T of tile t+1 is issued before P V of tile t, so the tensor pipe works on the next scores
// while the softmax warps process the current ones.  TMEM: 2 x 128 columns of scores (P aliases the
// first 64 columns of its score buffer) + 128 columns of O.
#include <algorithm>

#include "attn_simt.cuh"
#include "sm100.cuh"

namespace vmoba {
namespace tc {

using namespace sm100;

constexpr int BM = 128;              // query rows per item
constexpr int BN = 128;              // keys per tile
constexpr int DH = 128;              // head dim
constexpr int STAGES = 3;            // K/V ring depth
constexpr int PANEL = BM * 128;      // bytes of one 64-column panel of a 128-row tile (16 KB)
constexpr int TILE = 2 * PANEL;      // bytes of a [128 x 128] bf16 tile (32 KB)
constexpr int THREADS = 192;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t S_COL0 = 0, S_COL1 = 128, O_COL = 256;
constexpr float RESCALE_LOG2 = 8.0f;

struct Smem {
  uint64_t k_full[STAGES], v_full[STAGES], kv_empty[STAGES];
  uint64_t s_full[2], p_ready[2];
  uint64_t o_done[2], q_ready;
  uint32_t tmem_base;
  int abort_flag;
};
constexpr size_t SMEM_BYTES = 1024 /*alignment slack*/ + TILE /*Q*/ + 2 * STAGES * TILE + sizeof(Smem) + 64;

struct Params {
  const __nv_bfloat16* q;
  const int* kb_ptr;
  const int* q_idx;
  const int* q_ptr;
  const int* item_ptr;
  int n_kb, S, Nb, sb, BH;
  float scale_log2;      // softmax scale * log2(e)
  __nv_bfloat16* o;
  __nv_bfloat16* o_resid;
  float* lse;
  float* part_o;
  float* part_lse;
  long long capacity;
  int32_t* status;
};

template <bool DENSE>
__device__ __forceinline__ void decode_item(const Params& p, int item, int& bh, int& key_begin, int& n_keys, int& list_lo,
                                            int& n_rows) {
  if (DENSE) {
    const int tiles = (p.S + BM - 1) / BM;
    bh = item / tiles;
    const int t = item - bh * tiles;
    key_begin = 0;
    n_keys = p.S;
    list_lo = t * BM;
    n_rows = min(BM, p.S - list_lo);
  } else {
    simt::Item it = simt::decode_sparse(item, p.item_ptr, p.n_kb, p.kb_ptr, p.Nb, p.sb, BM, p.capacity);
    bh = it.bh;
    key_begin = it.key_begin;
    n_keys = p.sb;
    list_lo = it.list_lo;
    n_rows = it.list_hi - it.list_lo;
  }
}

template <bool DENSE>
__global__ void __launch_bounds__(THREADS, 1)
attn_fwd_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = base;
  uint8_t* sK = base + TILE;
  uint8_t* sV = sK + STAGES * TILE;
  Smem* sm = reinterpret_cast<Smem*>(sV + STAGES * TILE);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &sm->abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(&sm->k_full[s], 1); mbar_init(&sm->v_full[s], 1); mbar_init(&sm->kv_empty[s], 1); }
    for (int b = 0; b < 2; ++b) { mbar_init(&sm->s_full[b], 1); mbar_init(&sm->p_ready[b], 128); }
    mbar_init(&sm->o_done[0], 1);
    mbar_init(&sm->o_done[1], 1);
    mbar_init(&sm->q_ready, 128);
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
  constexpr uint32_t IDESC_QK_FULL = make_idesc_bf16(BM, BN, false, false);
  constexpr uint32_t IDESC_PV = make_idesc_bf16(BM, DH, false, true);

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t fills = 0;
      for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
        int bh, key_begin, n_keys, list_lo, n_rows;
        decode_item<DENSE>(p, item, bh, key_begin, n_keys, list_lo, n_rows);
        const int row0 = bh * p.S + key_begin;
        const int ntiles = (n_keys + BN - 1) / BN;
        for (int t = 0; t < ntiles; ++t, ++fills) {
          const int s = fills % STAGES;
          if (fills >= STAGES) mbar_wait(&sm->kv_empty[s], ((fills / STAGES) - 1) & 1, abort_flag, p.status);
          const int y = row0 + t * BN;
          mbar_expect_tx(&sm->k_full[s], TILE);
          tma_load_2d(sK + s * TILE, &tmK, &sm->k_full[s], 0, y);
          tma_load_2d(sK + s * TILE + PANEL, &tmK, &sm->k_full[s], 64, y);
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
      uint32_t fills = 0;        // K/V tiles consumed so far (global ring position)
      uint32_t tiles_done = 0;   // score buffers used so far (global): buffer = count & 1
      uint32_t items_done = 0;
      const uint32_t sQ_addr = smem_u32(sQ);
      for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++items_done) {
        int bh, key_begin, n_keys, list_lo, n_rows;
        decode_item<DENSE>(p, item, bh, key_begin, n_keys, list_lo, n_rows);
        const int ntiles = (n_keys + BN - 1) / BN;
        mbar_wait(&sm->q_ready, items_done & 1, abort_flag, p.status);
        tc_fence_after();
        auto issue_qk = [&](int t) {
          const uint32_t f = fills + t;
          const int s = f % STAGES;
          mbar_wait(&sm->k_full[s], (f / STAGES) & 1, abort_flag, p.status);
          tc_fence_after();
          const int valid = min(BN, n_keys - t * BN);
          const int n_mma = (valid + 15) & ~15;
          const uint32_t idesc = (n_mma == BN) ? IDESC_QK_FULL : make_idesc_bf16(BM, n_mma, false, false);
          const uint32_t buf = (tiles_done + t) & 1;
          const uint32_t d_tmem = tmem + (buf ? S_COL1 : S_COL0);
          const uint32_t sK_addr = smem_u32(sK + s * TILE);
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks) {
            const uint32_t off = (ks >> 2) * PANEL + (ks & 3) * 32;
            mma_ss(d_tmem, make_smem_desc(sQ_addr + off, 16, 1024), make_smem_desc(sK_addr + off, 16, 1024), idesc,
                   ks > 0 ? 1u : 0u);
          }
          mma_commit(&sm->s_full[buf]);
        };
        issue_qk(0);
        for (int t = 0; t < ntiles; ++t) {
          if (t + 1 < ntiles) issue_qk(t + 1);
          const uint32_t f = fills + t;
          const int s = f % STAGES;
          const uint32_t buf = (tiles_done + t) & 1;
          mbar_wait(&sm->p_ready[buf], ((tiles_done + t) >> 1) & 1, abort_flag, p.status);
          mbar_wait(&sm->v_full[s], (f / STAGES) & 1, abort_flag, p.status);
          tc_fence_after();
          const int valid = min(BN, n_keys - t * BN);
          const int ksteps = (valid + 15) >> 4;
          const uint32_t p_tmem = tmem + (buf ? S_COL1 : S_COL0);
          const uint32_t sV_addr = smem_u32(sV + s * TILE);
          for (int ks = 0; ks < ksteps; ++ks) {
            mma_ts(tmem + O_COL, p_tmem + ks * 8, make_smem_desc(sV_addr + ks * 2048, PANEL, 1024), IDESC_PV,
                   (t > 0 || ks > 0) ? 1u : 0u);
          }
          mma_commit(&sm->kv_empty[s]);
          mma_commit(&sm->o_done[(tiles_done + t) & 1]);
        }
        fills += ntiles;
        tiles_done += ntiles;
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax + epilogue (128 threads)
    const int quad = warp & 3;                      // TMEM lane quarter this warp may access
    const int r = quad * 32 + lane;                 // query row of this thread
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int st = threadIdx.x - 64;                // 0..127
    uint32_t tiles_done = 0, pv_done = 0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
      int bh, key_begin, n_keys, list_lo, n_rows;
      decode_item<DENSE>(p, item, bh, key_begin, n_keys, list_lo, n_rows);
      const int ntiles = (n_keys + BN - 1) / BN;
      const long long head_off = (long long)bh * p.S;
      // ---- gather Q rows into the swizzled K-major tile: 16 threads per row, 8 rows per pass
      {
        const int chunk = st & 15;                 // 16-byte chunk of the 256-byte row
        const int panel = chunk >> 3, cc = chunk & 7;
        uint4 v[16];                               // all loads in flight before the first store
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int row = (st >> 4) + 8 * i;
          v[i] = make_uint4(0u, 0u, 0u, 0u);
          if (row < n_rows) {
            const int qpos = DENSE ? list_lo + row : p.q_idx[list_lo + row];
            v[i] = __ldg(reinterpret_cast<const uint4*>(p.q + (head_off + qpos) * DH) + chunk);
          }
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const int row = (st >> 4) + 8 * i;
          *reinterpret_cast<uint4*>(sQ + panel * PANEL + row * 128 + ((cc ^ (row & 7)) << 4)) = v[i];
        }
      }
      fence_async_proxy();
      mbar_arrive(&sm->q_ready);

      const bool row_ok = r < n_rows;
      int qpos = 0;
      long long pos = 0;
      if (row_ok) {
        pos = (long long)list_lo + r;
        qpos = DENSE ? list_lo + r : p.q_idx[pos];
      }
      float m_used = -INFINITY, l = 0.f, l_r = 0.f;   // l: exact sum (for LSE); l_r: sum of the bf16-rounded weights
      for (int t = 0; t < ntiles; ++t) {
        const uint32_t buf = (tiles_done + t) & 1;
        const uint32_t s_tmem = tmem + lane_addr + (buf ? S_COL1 : S_COL0);
        mbar_wait(&sm->s_full[buf], ((tiles_done + t) >> 1) & 1, abort_flag, p.status);
        tc_fence_after();
        const int valid = min(BN, n_keys - t * BN);
        uint32_t sv[4][32];
        tmem_ld32(s_tmem + 0, sv[0]);
        tmem_ld32(s_tmem + 32, sv[1]);
        tmem_ld32(s_tmem + 64, sv[2]);
        tmem_ld32(s_tmem + 96, sv[3]);
        tmem_ld_wait();
        float mx = -INFINITY;
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            float x = __uint_as_float(sv[c][i]) * p.scale_log2;
            x = (c * 32 + i < valid) ? x : -INFINITY;
            sv[c][i] = __float_as_uint(x);
            mx = fmaxf(mx, x);
          }
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
          mbar_wait(&sm->o_done[(pv_done + t - 1) & 1], ((pv_done + t - 1) >> 1) & 1, abort_flag, p.status);
          tc_fence_after();
          const uint32_t o_tmem = tmem + lane_addr + O_COL;
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
        float sum = 0.f, sum_r = 0.f;
        // P (bf16 pairs) goes over the first 64 columns of this score buffer: keys 2i, 2i+1 -> column i
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint32_t pk[32];
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const float p0 = ex2(__uint_as_float(sv[2 * h + (i >> 4)][(2 * i) & 31]) - m_used);
            const float p1 = ex2(__uint_as_float(sv[2 * h + (i >> 4)][((2 * i) & 31) + 1]) - m_used);
            sum += p0 + p1;
            pk[i] = pack_bf16(p0, p1);
            // the tensor core multiplies the ROUNDED weights: normalise O by their sum, so that the
            // rounding of P perturbs the weights but never their total
            sum_r += __uint_as_float(pk[i] << 16) + __uint_as_float(pk[i] & 0xffff0000u);
          }
          tmem_st32(s_tmem + h * 32, pk);
        }
        l += sum;
        l_r += sum_r;
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(&sm->p_ready[buf]);
      }
      // ---- epilogue: wait for the last P V, normalise, write
      mbar_wait(&sm->o_done[(pv_done + ntiles - 1) & 1], ((pv_done + ntiles - 1) >> 1) & 1, abort_flag, p.status);
      tc_fence_after();
      pv_done += ntiles;
      tiles_done += ntiles;
      const float inv = 1.0f / l_r;
      const float row_lse = (m_used + log2f(l)) * 0.6931471805599453f;
      const long long G_ = head_off + qpos;
      bool direct = DENSE;
      if (!DENSE && row_ok) direct = (p.q_ptr[G_ + 1] - p.q_ptr[G_]) == 1;
      const uint32_t o_tmem = tmem + lane_addr + O_COL;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        uint32_t ov[32];
        tmem_ld32(o_tmem + c * 32, ov);
        tmem_ld_wait();
        if (row_ok) {
          if (direct) {
            __nv_bfloat16* dst = p.o + G_ * DH + c * 32;
            __nv_bfloat16* rdst = p.o_resid ? p.o_resid + G_ * DH + c * 32 : nullptr;
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              store4_resid(dst + i, rdst ? rdst + i : nullptr,
                           make_float4(__uint_as_float(ov[i]) * inv, __uint_as_float(ov[i + 1]) * inv,
                                       __uint_as_float(ov[i + 2]) * inv, __uint_as_float(ov[i + 3]) * inv));
          } else {
            float* dst = p.part_o + pos * DH + c * 32;
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<float4*>(dst + i) =
                  make_float4(__uint_as_float(ov[i]) * inv, __uint_as_float(ov[i + 1]) * inv,
                              __uint_as_float(ov[i + 2]) * inv, __uint_as_float(ov[i + 3]) * inv);
          }
        }
      }
      if (row_ok) {
        if (direct) p.lse[G_] = row_lse; else p.part_lse[pos] = row_lse;
      }
      // the next item's first P V overwrites O: order our TMEM reads before the q_ready arrival
      tc_fence_before();
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem, TMEM_COLS);
}

static int grid_items(long long items) { return (int)std::max<long long>(1, std::min<long long>(items, 148)); }

}  // namespace tc

// Forward over the work lists (bf16, head_dim 128).  Returns VMOBA_ERR_CUDA if the tensor maps or
// the launch fail.
int tc_sparse_fwd(const Dims& D, const void* q, const void* k, const void* v, const int* kb_ptr, const int* q_idx,
                  const int* q_ptr, const int* q_pairs, long long cap, void* o, void* o_resid, float* lse,
                  int32_t* status, int* item_ptr, float* part_o, float* part_lse, cudaStream_t st) {
  using namespace tc;
  CUtensorMap tmK, tmV;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN))
    return VMOBA_ERR_CUDA;
  const long long n_kb = (long long)D.BH * D.Nb;
  simt::item_ptr_kernel<<<1, 1024, 0, st>>>(kb_ptr, n_kb, BM, cap, item_ptr);
  Params p;
  p.q = (const __nv_bfloat16*)q; p.kb_ptr = kb_ptr; p.q_idx = q_idx; p.q_ptr = q_ptr; p.item_ptr = item_ptr;
  p.n_kb = (int)n_kb; p.S = D.S; p.Nb = D.Nb; p.sb = D.sb; p.BH = D.BH;
  p.scale_log2 = D.scale * 1.4426950408889634f;
  p.o = (__nv_bfloat16*)o; p.o_resid = (__nv_bfloat16*)o_resid; p.lse = lse; p.part_o = part_o; p.part_lse = part_lse;
  p.capacity = cap; p.status = status;
  VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)SMEM_BYTES));
  attn_fwd_tc_kernel<false><<<grid_items(cap / BM + n_kb), THREADS, SMEM_BYTES, st>>>(tmK, tmV, p);
  const long long nq = (long long)D.BH * D.S;
  simt::merge_kernel<__nv_bfloat16, 128, float><<<(int)std::min<long long>((nq + 7) / 8, 148 * 16), 256, 0, st>>>(
      q_ptr, q_pairs, nq, part_o, part_lse, cap, (__nv_bfloat16*)o, (__nv_bfloat16*)o_resid, lse);
  VMOBA_LAUNCH_OK(3);
  return VMOBA_OK;
}

int tc_dense_fwd(const Dims& D, const void* q, const void* k, const void* v, void* o, void* o_resid, float* lse,
                 int32_t* status, cudaStream_t st) {
  using namespace tc;
  CUtensorMap tmK, tmV;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN))
    return VMOBA_ERR_CUDA;
  Params p;
  p.q = (const __nv_bfloat16*)q; p.kb_ptr = nullptr; p.q_idx = nullptr; p.q_ptr = nullptr; p.item_ptr = nullptr;
  p.n_kb = 0; p.S = D.S; p.Nb = 1; p.sb = D.S; p.BH = D.BH;
  p.scale_log2 = D.scale * 1.4426950408889634f;
  p.o = (__nv_bfloat16*)o; p.o_resid = (__nv_bfloat16*)o_resid; p.lse = lse; p.part_o = nullptr; p.part_lse = nullptr;
  p.capacity = 0; p.status = status;
  VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_fwd_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)SMEM_BYTES));
  const long long items = (long long)D.BH * ((D.S + BM - 1) / BM);
  attn_fwd_tc_kernel<true><<<grid_items(items), THREADS, SMEM_BYTES, st>>>(tmK, tmV, p);
  VMOBA_LAUNCH_OK(1);
  return VMOBA_OK;
}

}  // namespace vmoba
