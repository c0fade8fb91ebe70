// Tensor-core attention backward for bf16, head_dim 128: the training backward of Step 3 of
// VMoBA (mask constant).  One persistent kernel (one CTA per SM), key-stationary:
//
//   Item = 128 keys of one key block.  The K and V tiles stay in shared memory; the queries that
//   selected the block stream through in gathered chunks of 64 (Q and dO rows, 4-deep ring).  Per
//   chunk, with keys on the TMEM lanes:
//     S^T = K Q^T,  dP^T = V dO^T                        (two SS MMAs, N = 64)
//     P^T = exp2(c S^T - lse),  dS^T = P^T (dP^T - D)    (threads = key rows)
//     dQ^T = K^T dS^T                                    (SS MMA: K tile read MN-major as A, dS^T from a
//                                                         [keys][queries] bf16 tile in shared memory)
//     dV += P^T dO,  dK += dS^T Q                        (two TS MMAs, A = bf16 P^T / dS^T in TMEM;
//                                                         B = the same dO / Q tiles read MN-major)
//   Every key belongs to exactly one item: dK and dV are written once, no atomics.  dQ^T of a chunk
//   is read out of TMEM by eight writer warps (lane = head-dim index), transposed four queries at a
//   time among groups of four lanes with shuffles, and added into an fp32 accumulator with
//   red.global.add.v4.f32 (per warp instruction: complete 128-byte lines of four query rows).
//
// D = rowsum(dO * O) and lse come in per query; exp runs in the exp2 domain (c = scale * log2 e).
// The dense path uses the kernels with 128-query units in the companion file.
#include <algorithm>

#include "attn_simt.cuh"
#include "sm100.cuh"

namespace vmoba {
namespace tcb {

using namespace sm100;

constexpr int BN = 128, DH = 128;
constexpr int PANEL = 128 * 128;
constexpr int TILE = 2 * PANEL;
constexpr uint32_t TMEM_COLS = 512;
constexpr float LOG2E = 1.4426950408889634f;
// Diagnostics: when a device buffer of 16 counters is registered, the dK/dV kernels add the cycles
// their roles spend in each wait (one representative thread per role and CTA).
static unsigned long long* g_wait_profile = nullptr;
constexpr uint32_t IDESC_TN = make_idesc_bf16(128, 128, false, true);    // A from TMEM, B MN-major

// Asynchronous 16-byte copy global -> shared (bypassing L1); `bytes` = 16, or 0 to write zeros.
__device__ __forceinline__ void cp_async16(uint32_t smem_dst, const void* gsrc, uint32_t bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_dst), "l"(gsrc), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// 16-byte vector reduction into global memory (fp32 add)
__device__ __forceinline__ void red_add_v4(float* addr, float a, float b, float c, float d) {
  asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(addr), "f"(a), "f"(b), "f"(c), "f"(d) : "memory");
}

// Descriptor arithmetic: the start-address field sits in the low 14 bits (in 16-byte units), so a
// byte offset inside the tile is a plain add on the descriptor (the MMA-issuing thread must not
// rebuild descriptors per instruction: it is the serial bottleneck of these kernels).
__device__ __forceinline__ constexpr uint32_t koff(int ks, int panel_bytes) { return (uint32_t)(((ks >> 2) * panel_bytes + (ks & 3) * 32) >> 4); }
__device__ __forceinline__ constexpr uint32_t mnoff(int ks) { return (uint32_t)((ks * 2048) >> 4); }

// K-major operand descriptor for k-step ks (16 of the 128 head-dim columns) of a swizzled tile.
__device__ __forceinline__ uint64_t desc_k(uint32_t tile_addr, int ks) {
  return make_smem_desc(tile_addr + (ks >> 2) * PANEL + (ks & 3) * 32, 16, 1024);
}
// MN-major B operand descriptor: N = the 128 head-dim columns, K = rows 16*ks .. 16*ks+15 of the tile.
__device__ __forceinline__ uint64_t desc_mn(uint32_t tile_addr, int ks) {
  return make_smem_desc(tile_addr + ks * 2048, PANEL, 1024);
}

// ==========================================================================================
// dK / dV / dQ
// ==========================================================================================
// Units of 64 queries flow through a ring of gathered (Q, dO) chunks; S^T / dP^T are double
// buffered in TMEM (64 columns each), so the tensor pipe computes unit u+1 while the compute warps
// turn unit u into P^T / dS^T.  One K / V pair is resident per item; the loader warps run ahead of
// the MMA warp across item boundaries.
constexpr int QC = 64;                       // queries per unit
constexpr int CPANEL = QC * 128;             // bytes of one 64-column panel of a 64-row chunk (8 KB)
constexpr int CTILE = 2 * CPANEL;            // [64 x 128] bf16 (16 KB)
constexpr int NQ = 4;                        // chunk ring depth
struct KvSmem {
  uint64_t kv_full[2], kv_empty[2];          // K+V tiles of an item (TMA / commit); index 0 is in use
  uint64_t chunk_full[NQ], chunk_empty[NQ];  // gathered Q/dO chunk (128 loader arrivals / commit)
  uint64_t sdp_full[2];                      // S^T and dP^T of a unit ready (commit)
  uint64_t pds_ready[2];                     // P^T and dS^T written (128 compute arrivals)
  uint64_t acc_done;                         // all MMAs of the item done (commit)
  uint64_t acc_free;                         // epilogue has read dV / dK (128 compute arrivals)
  uint32_t tmem_base;
  int abort_flag;
  uint64_t dq_full[2];                       // dQ^T of a unit complete (commit)
  uint64_t dq_free[2];                       // dQ^T read out of TMEM (256 writer arrivals)
  alignas(16) float lse2[NQ][QC];
  alignas(16) float Dq[NQ][QC];
};
constexpr int DSTILE = 128 * 128;            // dS^T of a unit in shared memory: [128 keys][64 queries] bf16 (16 KB)
// one K/V pair, the chunk ring, one dS^T tile
// no alignment slack: the kernel checks that its dynamic shared memory starts on a 1024-byte boundary
constexpr size_t KVF_SMEM_BYTES = 2 * TILE + NQ * 2 * CTILE + DSTILE + sizeof(KvSmem) + 32;
static_assert(KVF_SMEM_BYTES <= 232448, "fused backward: shared memory");
// warps: TMA, MMA, 8 compute, 4 loaders, 8 dQ writers
constexpr int KVF_THREADS = 704;
constexpr uint32_t IDESC_K64 = make_idesc_bf16(128, QC, false, false);   // S^T, dP^T: N = 64 queries
constexpr uint32_t IDESC_DQT = make_idesc_bf16(128, QC, true, true);     // dQ^T = K^T dS^T: both operands MN-major

struct KvParams {
  const __nv_bfloat16 *q, *d_o;
  const float *lse, *Dv;
  const int *kb_ptr, *q_idx;
  int S, Nb, sb, BH;
  float scale, scale_log2;
  long long capacity;
  __nv_bfloat16 *dk, *dv;
  int dkv_32;                  // dk and dv are 32-byte aligned: rows go out with 32-byte stores
  RowMap out_map;              // where the dK / dV rows go (block-major, or raster order through perm)
  RowMap do_map;               // where the dO rows come from (likewise)
  float* dq_acc;               // fp32 [queries][head_dim], zeroed rows of all selecting queries
  int32_t* status;
  unsigned long long* prof;    // optional wait-time counters (diagnostics), or null
};

// chunk tile as K-major B operand (N = 64 queries, K = head dim), k-step ks of 8
__device__ __forceinline__ uint64_t cdesc_k(uint32_t tile_addr, int ks) {
  return make_smem_desc(tile_addr + (ks >> 2) * CPANEL + (ks & 3) * 32, 16, 1024);
}
// chunk tile as MN-major B operand (N = head dim, K = 16 queries of k-step ks of 4)
__device__ __forceinline__ uint64_t cdesc_mn(uint32_t tile_addr, int ks) {
  return make_smem_desc(tile_addr + ks * 2048, CPANEL, 1024);
}

struct KvItem {
  int bh, key0, valid, n_units;
  long long list_lo, list_hi, head_off;
};

__device__ __forceinline__ KvItem kv_decode(const KvParams& p, long long item, int tiles) {
  KvItem it;
  const int tile = (int)(item % tiles);
  const long long kbi = item / tiles;
  it.bh = (int)(kbi / p.Nb);
  const int j = (int)(kbi - (long long)it.bh * p.Nb);
  it.key0 = j * p.sb + tile * BN;
  it.valid = min(BN, p.sb - tile * BN);
  it.list_lo = min((long long)p.kb_ptr[kbi], p.capacity);
  it.list_hi = min((long long)p.kb_ptr[kbi + 1], p.capacity);
#ifdef VMOBA_DEBUG
  if (it.list_lo < 0 || it.list_hi < it.list_lo) {      // offsets must be non-negative and ascending
    set_status(p.status, VMOBA_ERR_BOUNDS);
    it.list_lo = it.list_hi = 0;
  }
#endif
  it.n_units = (int)((it.list_hi - it.list_lo + QC - 1) / QC);
  it.head_off = (long long)it.bh * p.S;
  return it;
}

__global__ void __launch_bounds__(KVF_THREADS, 1)
attn_bwd_dkdv_tc_kernel(const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV, const KvParams p) {
  extern __shared__ uint8_t smem_raw[];
  // the swizzled tiles need 1024-byte alignment and there is no room for alignment slack
  if ((smem_u32(smem_raw) & 1023u) != 0) {
    if (threadIdx.x == 0) set_status(p.status, VMOBA_ERR_CUDA);
    return;
  }
  uint8_t* base = smem_raw;
  uint8_t* sK = base;                  // [TILE]
  uint8_t* sV = base + TILE;           // [TILE]
  uint8_t* sC = base + 2 * TILE;       // [NQ][Q chunk | dO chunk]
  uint8_t* sDS = sC + NQ * 2 * CTILE;  // dS^T of the current unit [DSTILE]
  KvSmem* sm = reinterpret_cast<KvSmem*>(sDS + DSTILE);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &sm->abort_flag;
  // diagnostics: cycles spent in each wait site by one representative thread per role
  unsigned long long wp[4] = {0, 0, 0, 0};
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
    for (int b = 0; b < 2; ++b) {
      mbar_init(&sm->kv_full[b], 1); mbar_init(&sm->kv_empty[b], 1);
      mbar_init(&sm->sdp_full[b], 1); mbar_init(&sm->pds_ready[b], 256);
      mbar_init(&sm->dq_full[b], 1); mbar_init(&sm->dq_free[b], 256);
    }
    for (int b = 0; b < NQ; ++b) { mbar_init(&sm->chunk_full[b], 128); mbar_init(&sm->chunk_empty[b], 1); }
    mbar_init(&sm->acc_done, 1);
    mbar_init(&sm->acc_free, 256);
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
  constexpr uint32_t ST_COL = 0, DPT_COL = 128, DV_COL = 256, DK_COL = 384;   // ST/DPT: two 64-column buffers each

  const int tiles = (p.sb + BN - 1) / BN;
  const long long n_items = (long long)p.BH * p.Nb * tiles;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA: K and V tiles, one pair per item
    if (lane == 0) {
      uint32_t n = 0;
      for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        const KvItem it = kv_decode(p, item, tiles);
        if (it.n_units == 0) continue;
        // one K / V pair: the next item's tiles wait for the current item's last MMA
        if (n >= 1) twait(0, &sm->kv_empty[0], (n - 1) & 1);
        const int y = (int)it.head_off + it.key0;
        mbar_expect_tx(&sm->kv_full[0], 2 * TILE);
        tma_load_2d(sK, &tmK, &sm->kv_full[0], 0, y);
        tma_load_2d(sK + PANEL, &tmK, &sm->kv_full[0], 64, y);
        tma_load_2d(sV, &tmV, &sm->kv_full[0], 0, y);
        tma_load_2d(sV + PANEL, &tmV, &sm->kv_full[0], 64, y);
        ++n;
        // The one K / V pair is reloaded only when the item's last MMA has run: ask the L2 for the next item's
        // tiles now, so that the reload finds them there.
        if (item + gridDim.x < n_items) {
          const KvItem nx = kv_decode(p, item + gridDim.x, tiles);
          const int yn = (int)nx.head_off + nx.key0;
          if (nx.n_units > 0) {
            tma_prefetch_2d(&tmK, 0, yn); tma_prefetch_2d(&tmK, 64, yn);
            tma_prefetch_2d(&tmV, 0, yn); tma_prefetch_2d(&tmV, 64, yn);
          }
        }
      }
      if (*abort_flag)
        for (uint32_t f = n > 2 ? n - 2 : 0; f < n; ++f) mbar_wait(&sm->kv_full[0], f & 1, abort_flag, p.status);
      tflush(0, 1);      // [0] kv_empty, [1] total
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer: the whole warp walks the loop, one
    // elected lane issues (warp-uniform control flow; see elect_one)
    {
      const bool leader = elect_one();
      auto wwait = [&](int site, uint64_t* bar, uint32_t parity) { twait(site, bar, parity); __syncwarp(); };
      uint32_t n = 0, u0 = 0;      // items and units done so far
      for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
        KvItem it = kv_decode(p, item, tiles);
        // the list bounds come from memory: a warp reduction marks them as warp-uniform
        const int n_list = __reduce_max_sync(0xffffffffu, (int)(it.list_hi - it.list_lo));
        it.n_units = (n_list + QC - 1) / QC;
        if (it.n_units == 0) continue;
        wwait(0, &sm->kv_full[0], n & 1);
        tc_fence_after();
        const uint64_t dK0 = desc_k(smem_u32(sK), 0), dV0 = desc_k(smem_u32(sV), 0);
        const uint64_t mK0 = desc_mn(smem_u32(sK), 0);     // K^T as MN-major A operand (fused dQ^T)
        auto issue_sdp = [&](int i) {
          const uint32_t u = u0 + i;
          const int cb = u % NQ, tb = u & 1;
          wwait(1, &sm->chunk_full[cb], (u / NQ) & 1);
          tc_fence_after();
          const uint32_t sQ_addr = smem_u32(sC + cb * 2 * CTILE);
          const uint64_t dQ0 = cdesc_k(sQ_addr, 0), dO0 = cdesc_k(sQ_addr + CTILE, 0);
          const uint32_t st = tmem + ST_COL + tb * QC, dp = tmem + DPT_COL + tb * QC;
          // S^T first: its buffer is free (the MMAs that read P^T / dS^T of unit u - 2 were issued before),
          // while the dP^T buffer last held dQ^T of unit u - 2, which the writer warps must have read;
          // that hand-off completes behind the eight S^T MMAs instead of stalling the issue
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks)
            if (leader) mma_ss(st, dK0 + koff(ks, PANEL), dQ0 + koff(ks, CPANEL), IDESC_K64, ks > 0 ? 1u : 0u);
          if (u >= 2) {
            wwait(3, &sm->dq_free[tb], ((u - 2) >> 1) & 1);
            tc_fence_after();
          }
#pragma unroll
          for (int ks = 0; ks < DH / 16; ++ks)
            if (leader) mma_ss(dp, dV0 + koff(ks, PANEL), dO0 + koff(ks, CPANEL), IDESC_K64, ks > 0 ? 1u : 0u);
          if (leader) mma_commit(&sm->sdp_full[tb]);
        };
        issue_sdp(0);
        if (it.n_units > 1) issue_sdp(1);
        for (int i = 0; i < it.n_units; ++i) {
          const uint32_t u = u0 + i;
          const int cb = u % NQ, tb = u & 1;
          wwait(2, &sm->pds_ready[tb], (u >> 1) & 1);
          // dV / dK still hold the previous item until its epilogue has read them
          if (i == 0 && n > 0) wwait(3, &sm->acc_free, (n - 1) & 1);
          tc_fence_after();
          const int rows = min(QC, n_list - i * QC);
          const int ksteps = (rows + 15) >> 4;
          const uint32_t sQ_addr = smem_u32(sC + cb * 2 * CTILE);
          const uint64_t mQ0 = cdesc_mn(sQ_addr, 0), mO0 = cdesc_mn(sQ_addr + CTILE, 0);
          const uint32_t pt = tmem + ST_COL + tb * QC, dst_ = tmem + DPT_COL + tb * QC;
          const uint32_t acc0 = i > 0 ? 1u : 0u;
          {
            // dQ^T [head dim x 64 queries] = K^T dS^T over the tile's keys, into the unit's dP^T columns
            // (already read by the compute warps); issued first so that its read-out overlaps dV / dK
            const uint64_t mS0 = make_smem_desc(smem_u32(sDS), DSTILE, 1024);
            const int kk = (it.valid + 15) >> 4;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
              if (leader && ks < kk) mma_ss(dst_, mK0 + mnoff(ks), mS0 + mnoff(ks), IDESC_DQT, ks > 0 ? 1u : 0u);
            if (leader) mma_commit(&sm->dq_full[tb]);
          }
          // P^T of queries 32h .. 32h+31 sits in columns 32h .. 32h+15 of the S^T buffer, dS^T in columns
          // 32h+16 .. 32h+31 (the dP^T columns are receiving dQ^T)
          const uint32_t ds_t = pt + 16;
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            if (leader && ks < ksteps) {
              mma_ts(tmem + DV_COL, pt + (ks >> 1) * 32 + (ks & 1) * 8, mO0 + mnoff(ks), IDESC_TN, ks > 0 ? 1u : acc0);
              mma_ts(tmem + DK_COL, ds_t + (ks >> 1) * 32 + (ks & 1) * 8, mQ0 + mnoff(ks), IDESC_TN, ks > 0 ? 1u : acc0);
            }
          if (leader) mma_commit(&sm->chunk_empty[cb]);
          if (i + 2 < it.n_units) issue_sdp(i + 2);
        }
        if (leader) mma_commit(&sm->kv_empty[0]);
        if (leader) mma_commit(&sm->acc_done);
        u0 += it.n_units;
        ++n;
      }
      if (leader) tflush(2, 4);      // [2] kv_full, [3] chunk_full, [4] pds_ready, [5] acc_free, [6] total
    }
  } else if (warp >= 10 && warp < 14) {
    // ------------------------------------------------------------------ loaders: gather Q / dO chunks (run ahead)
    // The rows go from global to shared memory as asynchronous 16-byte copies (no registers, no
    // st.shared); a unit is published in the next iteration, once its copies have landed.
    const int lt = threadIdx.x - 320;   // 0..127
    const int chunk = lt & 15, panel = chunk >> 3, cc = chunk & 7;
    auto publish = [&](uint32_t u) {
      fence_async_proxy();
      mbar_arrive(&sm->chunk_full[u % NQ]);
    };
    uint32_t u0 = 0;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
      const KvItem it = kv_decode(p, item, tiles);
      const __nv_bfloat16* qh = p.q + it.head_off * DH + chunk * 8;
      // dO rows: block-major, or in raster order through perm (the batch / head part of the address once per item)
      const bool do_raster = p.do_map.perm != nullptr;
      const int b_ = it.bh / p.do_map.heads, hd_ = it.bh - b_ * p.do_map.heads;
      const __nv_bfloat16* oh = p.d_o + (do_raster ? b_ * p.do_map.sb + hd_ * p.do_map.sh : it.head_off * DH) + chunk * 8;
      for (int i = 0; i < it.n_units; ++i) {
        const uint32_t u = u0 + i;
        const int cb = u % NQ;
        const long long lo = it.list_lo + (long long)i * QC;
        const int rows = (int)min((long long)QC, it.list_hi - lo);
        auto row_of = [&](int r) { return checked_index(__ldg(p.q_idx + lo + r), p.S, p.status); };
        int idx[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int row = (lt >> 4) + 8 * k;
          idx[k] = row < rows ? row_of(row) : -1;       // -1: padding row, zero-filled
        }
        float l2 = INFINITY, dd = 0.f;     // padded queries: P = exp2(-inf) = 0
        if (lt < rows) {
          const long long G_ = it.head_off + row_of(lt);
          l2 = p.lse[G_] * LOG2E;
          dd = p.Dv[G_];
        }
        // the previous unit is published as soon as its copies have landed (this unit's row indices and
        // scalars are already on their way), not behind this unit's wait for a free ring slot
        if (u >= 1) {
          cp_async_wait<0>();
          publish(u - 1);
        }
        if (u >= NQ) twait(0, &sm->chunk_empty[cb], ((u / NQ) - 1) & 1);
        const uint32_t dst = smem_u32(sC + cb * 2 * CTILE);
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          const int row = (lt >> 4) + 8 * k;
          const uint32_t off = panel * CPANEL + row * 128 + ((cc ^ (row & 7)) << 4);
          const int ik = idx[k] < 0 ? 0 : idx[k];
          const long long src = (long long)ik * DH;
          const long long osrc = do_raster ? (long long)__ldg(p.do_map.perm + ik) * p.do_map.st : src;
          const uint32_t bytes = idx[k] < 0 ? 0u : 16u;
          cp_async16(dst + off, qh + src, bytes);
          cp_async16(dst + CTILE + off, oh + osrc, bytes);
        }
        if (lt < QC) { sm->lse2[cb][lt] = l2; sm->Dq[cb][lt] = dd; }
        cp_async_commit();
      }
      u0 += it.n_units;
    }
    cp_async_wait<0>();
    if (u0 >= 1) publish(u0 - 1);
    if (lt == 0) tflush(7, 1);     // [7] chunk_empty, [8] total
  } else if (warp >= 14) {
    // ------------------------------------------------------------------ dQ writers: thread = head-dim index
    // Read dQ^T of a unit out of TMEM (lane = head-dim index, 64 query columns), release the buffer and add
    // it into the fp32 accumulator.  The four lanes 4i .. 4i+3 transpose each group of four queries among
    // themselves with two exchange steps (one shuffle per value), after which lane 4i + j holds head-dim
    // columns 4i .. 4i+3 of query j of the group: one red.global.add.v4.f32 warp instruction then adds four
    // complete 128-byte lines, one in each of four accumulator rows.  (Measured per SM with all SMs busy:
    // reductions that cover whole 128-byte lines reach 23 B/cycle however the lines are spread over rows;
    // 16 bytes per lane in 32 different rows reach 12.5; scalar line-wide reductions reach 23 alone but
    // made this kernel 1.5x slower.  An earlier version transposed through a shared-memory tile: a third
    // of the load/store wavefronts of a unit, on the unit that binds this kernel.)
    // Eight warps: two per TMEM lane quarter, each taking 32 of a unit's 64 query columns.
    const int quad = warp & 3;
    const int qhalf = (warp - 14) >> 2;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int j4 = lane & 3;
    const bool odd1 = (lane & 1) != 0, odd2 = (lane & 2) != 0;
    float* acc_col = p.dq_acc + quad * 32 + (lane & ~3);
    // x[0..3]: this lane's head-dim column for four queries -> head-dim columns 4i .. 4i+3 of query j4
    auto transpose4 = [&](float x0, float x1, float x2, float x3, float4& y) {
      // step 1, partner lane ^ 1: even lanes keep queries 0, 2, odd lanes keep queries 1, 3
      const float r0 = __shfl_xor_sync(0xffffffffu, odd1 ? x0 : x1, 1);
      const float r1 = __shfl_xor_sync(0xffffffffu, odd1 ? x2 : x3, 1);
      // (query 0 or 1: columns c, c ^ 1), (query 2 or 3: likewise), in column order
      const float a0 = odd1 ? r0 : x0, a1 = odd1 ? x1 : r0;
      const float b0 = odd1 ? r1 : x2, b1 = odd1 ? x3 : r1;
      // step 2, partner lane ^ 2: lanes 0, 1 keep the first query of their pair, lanes 2, 3 the second
      const float s0 = __shfl_xor_sync(0xffffffffu, odd2 ? a0 : b0, 2);
      const float s1 = __shfl_xor_sync(0xffffffffu, odd2 ? a1 : b1, 2);
      y = odd2 ? make_float4(s0, s1, b0, b1) : make_float4(a0, a1, s0, s1);
    };
    uint32_t u0 = 0;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
      const KvItem it = kv_decode(p, item, tiles);
      float* acc_head = acc_col + it.head_off * DH;
      for (int i = 0; i < it.n_units; ++i) {
        const uint32_t u = u0 + i;
        const int tb = u & 1;
        // accumulator row of query 32 qhalf + lane of the unit (-1 beyond the list)
        const long long lo = it.list_lo + (long long)i * QC + 32 * qhalf;
        const int row_lane = lo + lane < it.list_hi ? checked_index(__ldg(p.q_idx + lo + lane), p.S, p.status) : -1;
        long long tw0 = p.prof ? clock64() : 0;
        mbar_wait(&sm->dq_full[tb], (u >> 1) & 1, abort_flag, p.status);
        if (p.prof) { const long long t = clock64(); wp[0] += t - tw0; tw0 = t; }
        tc_fence_after();
        uint32_t x[32];
        tmem_ld32(tmem + lane_addr + DPT_COL + tb * QC + 32 * qhalf, x);
        tmem_ld_wait();
        tc_fence_before();
        mbar_arrive(&sm->dq_free[tb]);
        if (p.prof) { const long long t = clock64(); wp[1] += t - tw0; tw0 = t; }
        // The transpositions first, in place, then the eight reductions back to back from eight different
        // register quadruples: a reduction holds its source registers until the load/store unit has taken them
        // (about 200 cycles under this kernel's memory traffic), so a loop that reuses one quadruple sends one
        // reduction per 200 cycles.
        int rw[8];
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          float4 y;
          transpose4(__uint_as_float(x[4 * g]), __uint_as_float(x[4 * g + 1]), __uint_as_float(x[4 * g + 2]),
                     __uint_as_float(x[4 * g + 3]), y);
          x[4 * g] = __float_as_uint(y.x * p.scale); x[4 * g + 1] = __float_as_uint(y.y * p.scale);
          x[4 * g + 2] = __float_as_uint(y.z * p.scale); x[4 * g + 3] = __float_as_uint(y.w * p.scale);
          rw[g] = __shfl_sync(0xffffffffu, row_lane, 4 * g + j4);
        }
#pragma unroll
        for (int g = 0; g < 8; ++g)
          if (rw[g] >= 0)
            red_add_v4(acc_head + (long long)rw[g] * DH, __uint_as_float(x[4 * g]), __uint_as_float(x[4 * g + 1]),
                       __uint_as_float(x[4 * g + 2]), __uint_as_float(x[4 * g + 3]));
        if (p.prof) { const long long t = clock64(); wp[3] += t - tw0; tw0 = t; }
      }
      u0 += it.n_units;
    }
    if (p.prof && warp == 14 && lane == 0) {
      atomicAdd(p.prof + 9, wp[0]); atomicAdd(p.prof + 14, wp[1]); atomicAdd(p.prof + 15, wp[2]); atomicAdd(p.prof + 1, wp[3]);
    }
  } else {
    // ------------------------------------------------------------------ compute: thread = (key row, half of the unit's queries)
    const int quad = warp & 3;
    const int half = (warp - 2) >> 2;                 // warps 2-5: queries 0-31 of a unit, warps 6-9: queries 32-63
    const int r = quad * 32 + lane;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    uint32_t n = 0, u0 = 0;
    for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
      const KvItem it = kv_decode(p, item, tiles);
      const long long row_off = r < it.valid ? p.out_map.off(it.head_off + it.key0 + r, DH) : 0;
      __nv_bfloat16* dv_row = p.dv + row_off;
      __nv_bfloat16* dk_row = p.dk + row_off;
      if (it.n_units == 0) {
        // no query selected this block: its keys get zero gradients
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
        const int cb = u % NQ, tb = u & 1;
        twait(0, &sm->chunk_full[cb], (u / NQ) & 1);   // publishes lse2 / Dq of this unit
        twait(1, &sm->sdp_full[tb], (u >> 1) & 1);
        tc_fence_after();
        // lane l holds the log-sum-exp and D of query 32 half + l: one 128-byte load each per warp, handed
        // round by shuffles (broadcast 16-byte loads from shared memory cost four wavefronts each)
        const float my_lse2 = sm->lse2[cb][32 * half + lane], my_D = sm->Dq[cb][32 * half + lane];
        const uint32_t st_t = tmem + lane_addr + ST_COL + tb * QC + 32 * half;
        const uint32_t dp_t = tmem + lane_addr + DPT_COL + tb * QC + 32 * half;
        // Two passes of 16 queries each (a thread then holds 16 scores and 16 dP values at a time).  P^T goes
        // over the first 16 of this thread's 32 S^T columns and dS^T over the other 16 (the dP^T columns are
        // about to receive dQ^T), so the first pass keeps its dS^T in registers until the second pass has read
        // the remaining scores.  dS^T is written once more, as the row of this key in the [keys][queries]
        // shared-memory tile that dQ^T reads; rows beyond the key range hold other blocks' keys and must not
        // contribute.
        uint8_t* dsrow = sDS + r * 128;
        const bool live = r < it.valid;
        uint32_t dk_first[8];
#pragma unroll
        for (int pass = 0; pass < 2; ++pass) {
          uint32_t sv[16], dv_[16];
          tmem_ld16(st_t + 16 * pass, sv);
          tmem_ld16(dp_t + 16 * pass, dv_);
          tmem_ld_wait();
          if (pass == 1) tmem_st8(st_t + 16, dk_first);
          uint32_t pk[8], dk_[8];
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int l0 = 16 * pass + 4 * e;
            float4 l4, d4;
            l4.x = __shfl_sync(0xffffffffu, my_lse2, l0);     l4.y = __shfl_sync(0xffffffffu, my_lse2, l0 + 1);
            l4.z = __shfl_sync(0xffffffffu, my_lse2, l0 + 2); l4.w = __shfl_sync(0xffffffffu, my_lse2, l0 + 3);
            d4.x = __shfl_sync(0xffffffffu, my_D, l0);        d4.y = __shfl_sync(0xffffffffu, my_D, l0 + 1);
            d4.z = __shfl_sync(0xffffffffu, my_D, l0 + 2);    d4.w = __shfl_sync(0xffffffffu, my_D, l0 + 3);
            const float p0 = ex2(fmaf(__uint_as_float(sv[4 * e]), p.scale_log2, -l4.x));
            const float p1 = ex2(fmaf(__uint_as_float(sv[4 * e + 1]), p.scale_log2, -l4.y));
            const float p2 = ex2(fmaf(__uint_as_float(sv[4 * e + 2]), p.scale_log2, -l4.z));
            const float p3 = ex2(fmaf(__uint_as_float(sv[4 * e + 3]), p.scale_log2, -l4.w));
            pk[2 * e] = pack_bf16(p0, p1);
            pk[2 * e + 1] = pack_bf16(p2, p3);
            dk_[2 * e] = pack_bf16(p0 * (__uint_as_float(dv_[4 * e]) - d4.x), p1 * (__uint_as_float(dv_[4 * e + 1]) - d4.y));
            dk_[2 * e + 1] = pack_bf16(p2 * (__uint_as_float(dv_[4 * e + 2]) - d4.z), p3 * (__uint_as_float(dv_[4 * e + 3]) - d4.w));
          }
          tmem_st8(st_t + 8 * pass, pk);
          if (pass == 0) {
#pragma unroll
            for (int k = 0; k < 8; ++k) dk_first[k] = dk_[k];
            // one shared-memory tile: the previous unit's dQ^T must have finished reading it
            if (u >= 1) mbar_wait(&sm->dq_full[(u - 1) & 1], ((u - 1) >> 1) & 1, abort_flag, p.status);
          } else {
            tmem_st8(st_t + 24, dk_);
          }
#pragma unroll
          for (int j = 0; j < 2; ++j)
            *reinterpret_cast<uint4*>(dsrow + (((4 * half + 2 * pass + j) ^ (r & 7)) << 4)) =
                live ? make_uint4(dk_[4 * j], dk_[4 * j + 1], dk_[4 * j + 2], dk_[4 * j + 3]) : make_uint4(0u, 0u, 0u, 0u);
        }
        fence_async_proxy();
        tmem_st_wait();
        tc_fence_before();
        mbar_arrive(&sm->pds_ready[tb]);
      }
      // ---- epilogue: each half writes 64 of the 128 dV / dK columns of its key row
      twait(2, &sm->acc_done, n & 1);
      tc_fence_after();
#pragma unroll 1
      for (int pass = 0; pass < 4; ++pass) {      // dV columns, then dK columns, 32 at a time
        const int cgrp = half * 2 + (pass & 1);
        const bool is_dk = pass >= 2;
        uint32_t a[32];
        tmem_ld32(tmem + lane_addr + (is_dk ? DK_COL : DV_COL) + cgrp * 32, a);
        tmem_ld_wait();
        if (r < it.valid) {
          const float mul = is_dk ? p.scale : 1.0f;
          __nv_bfloat16* row = (is_dk ? dk_row : dv_row) + cgrp * 32;
#pragma unroll
          for (int i = 0; i < 32; i += 16) {      // sixteen bf16 = one 32-byte store (two 16-byte stores if unaligned)
            uint32_t hv[8];
#pragma unroll
            for (int k = 0; k < 8; ++k)
              hv[k] = pack_bf16(__uint_as_float(a[i + 2 * k]) * mul, __uint_as_float(a[i + 2 * k + 1]) * mul);
            if (p.dkv_32) {
              st_global_v8(row + i, hv[0], hv[1], hv[2], hv[3], hv[4], hv[5], hv[6], hv[7]);
            } else {
              *reinterpret_cast<uint4*>(row + i) = make_uint4(hv[0], hv[1], hv[2], hv[3]);
              *reinterpret_cast<uint4*>(row + i + 8) = make_uint4(hv[4], hv[5], hv[6], hv[7]);
            }
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

static int grid_items(long long items) { return (int)std::max<long long>(1, std::min<long long>(items, sm_count())); }

}  // namespace tcb

// attn_tc_bwd_long.cu
int tc_long_dkdv(const Dims& D, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                 const float* Dv, void* dk, void* dv, int32_t* status, unsigned long long* prof, cudaStream_t st);
int tc_long_dq(const Dims& D, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
               const float* Dv, void* dq, int32_t* status, cudaStream_t st);
// Backward over the work lists (bf16, head_dim 128).  Dv holds rowsum(dO * O) per query; dq_acc is
// an fp32 accumulator whose rows of selecting queries are zero; the caller converts it to bf16.
int tc_sparse_bwd(const Dims& D, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                  const float* Dv, const int* kb_ptr, const int* q_idx, long long cap, float* dq_acc, void* dk, void* dv,
                  int32_t* status, cudaStream_t st, const RowMap& out_map, const RowMap& do_map) {
  using namespace tcb;
  CUtensorMap tmK, tmV;
  const uint64_t rows = (uint64_t)D.BH * D.S;
  if (!sm100::make_tmap_bf16_rows(&tmK, k, rows, DH, BN) || !sm100::make_tmap_bf16_rows(&tmV, v, rows, DH, BN))
    return VMOBA_ERR_CUDA;
  const long long n_kb = (long long)D.BH * D.Nb;
  KvParams kp;
  kp.q = (const __nv_bfloat16*)q; kp.d_o = (const __nv_bfloat16*)d_o; kp.lse = lse; kp.Dv = Dv;
  kp.kb_ptr = kb_ptr; kp.q_idx = q_idx; kp.S = D.S; kp.Nb = D.Nb; kp.sb = D.sb; kp.BH = D.BH;
  kp.scale = D.scale; kp.scale_log2 = D.scale * LOG2E; kp.capacity = cap;
  kp.dk = (__nv_bfloat16*)dk; kp.dv = (__nv_bfloat16*)dv; kp.status = status; kp.prof = tcb::g_wait_profile;
  kp.dq_acc = dq_acc;
  kp.out_map = out_map;
  kp.do_map = do_map;
  kp.dkv_32 = (reinterpret_cast<uintptr_t>(dk) % 32) == 0 && (reinterpret_cast<uintptr_t>(dv) % 32) == 0 &&
              (!out_map.perm || (out_map.sb % 16 == 0 && out_map.st % 16 == 0 && out_map.sh % 16 == 0));
  const long long kv_items = n_kb * ((D.sb + BN - 1) / BN);
  VMOBA_CUDA_OK(cudaFuncSetAttribute(attn_bwd_dkdv_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)KVF_SMEM_BYTES));
  attn_bwd_dkdv_tc_kernel<<<grid_items(kv_items), KVF_THREADS, KVF_SMEM_BYTES, st>>>(tmK, tmV, kp);
  VMOBA_LAUNCH_OK(1);
  return VMOBA_OK;
}

// Dense backward: the kernels with 128-query units (one key range spanning the sequence).
int tc_dense_bwd(const Dims& D, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                 const float* Dv, void* dq, void* dk, void* dv, int32_t* status, cudaStream_t st) {
  int rc = tc_long_dkdv(D, q, k, v, d_o, lse, Dv, dk, dv, status, tcb::g_wait_profile, st);
  if (rc) return rc;
  return tc_long_dq(D, q, k, v, d_o, lse, Dv, dq, status, st);
}

}  // namespace vmoba

// Registers (or clears, with null) a device buffer of 16 uint64 counters for the dK/dV kernel's
// wait-time diagnostics.  Not part of the method; see the kernel for the counter layout.
namespace vmoba {
unsigned long long* debug_wait_profile() { return tcb::g_wait_profile; }
}  // namespace vmoba

extern "C" void vmoba_debug_wait_profile(void* dev_counters16) {
  vmoba::tcb::g_wait_profile = static_cast<unsigned long long*>(dev_counters16);
}
