// fp32 CUDA-core attention kernels: Step 3 of VMoBA (attention of each query over the keys
// of its selected blocks), its backward, and the dense tau = 1 limit.  These serve the fp32
// dtype (any supported head_dim) and bf16 shapes without a tensor-core kernel; all arithmetic
// is fp32.
//
// Work decomposition follows the key-block CSR: a work item is (batch, head, key block j,
// a chunk of <= 64 queries that selected j).  A query that selected several blocks gets one
// partial (o, lse) per block, merged afterwards; queries with a single block are written
// directly, queries with none are zero-filled by the merge kernel.
#pragma once

#include <cuda_fp16.h>

#include "common.cuh"

namespace vmoba {
namespace simt {

constexpr int kRows = 64;      // rows (queries, or keys in the dK/dV kernel) per CTA
constexpr int kTile = 32;      // rows of the streamed operand per shared-memory tile
constexpr int kThreads = 256;  // 4 threads per row, each owning head_dim/4 channels

// chunk-count prefix over the (batch, head, key block) lists: item_ptr[i] = number of work
// items before list i when every list is cut into chunks of `rows` queries.
static __global__ void __launch_bounds__(1024)
item_ptr_kernel(const int* __restrict__ kb_ptr, long long n_kb, int rows, long long capacity,
                int* __restrict__ item_ptr) {
  __shared__ long long total;
  block_exclusive_scan(
      [&](long long i) {
        long long lo = min((long long)kb_ptr[i], capacity), hi = min((long long)kb_ptr[i + 1], capacity);
        return (hi - lo + rows - 1) / rows;
      },
      item_ptr, n_kb, &total);
}

// item_tab[item] = index of the (batch, head, key block) list the item belongs to.
static __global__ void __launch_bounds__(256)
item_tab_kernel(const int* __restrict__ item_ptr, long long n_kb, long long max_items, int* __restrict__ item_tab) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n_kb; i += (long long)gridDim.x * blockDim.x) {
    const long long lo = item_ptr[i], hi = min((long long)item_ptr[i + 1], max_items);
    for (long long t = lo; t < hi; ++t) item_tab[t] = (int)i;
  }
}

struct Item {
  int bh;          // batch * heads + head
  int key_begin;   // key range inside the head (block-major positions)
  int key_end;
  int list_lo;     // sparse: range of CSR positions handled by this item
  int list_hi;
};

// Sparse item decode: binary search of the chunk prefix.
__device__ __forceinline__ Item decode_sparse(int item, const int* __restrict__ item_ptr, int n_kb,
                                              const int* __restrict__ kb_ptr, int Nb, int sb, int rows,
                                              long long capacity) {
  int lo = 0, hi = n_kb;   // find the last i with item_ptr[i] <= item
  while (hi - lo > 1) {
    int mid = (lo + hi) >> 1;
    if (item_ptr[mid] <= item) lo = mid; else hi = mid;
  }
  Item it;
  it.bh = lo / Nb;
  int j = lo - it.bh * Nb;
  it.key_begin = j * sb;
  it.key_end = it.key_begin + sb;
  int chunk = item - item_ptr[lo];
  long long end = min((long long)kb_ptr[lo + 1], capacity);
  it.list_lo = kb_ptr[lo] + chunk * rows;
  it.list_hi = (int)min((long long)it.list_lo + rows, end);
  return it;
}

// Cooperative load of `kTile` rows x DH channels (converted to fp32) into shared memory;
// rows beyond `n_valid` are zero-filled.  row_of(i) gives the in-head position of tile row i.
template <typename T, int DH, typename RowOf>
__device__ __forceinline__ void load_tile(float* __restrict__ dst, const T* __restrict__ head_base, int n_valid,
                                          RowOf row_of) {
  constexpr int V = DH / 4;
  for (int i = threadIdx.x; i < kTile * V; i += kThreads) {
    int r = i / V, c4 = i % V;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (r < n_valid) x = load4(head_base + (long long)row_of(r) * DH + c4 * 4);
    *reinterpret_cast<float4*>(dst + r * DH + c4 * 4) = x;
  }
}

__device__ __forceinline__ float quad_sum(float x) {
  x += __shfl_xor_sync(0xffffffffu, x, 1);
  x += __shfl_xor_sync(0xffffffffu, x, 2);
  return x;
}

// ------------------------------------------------------------------------------ forward
template <typename T, int DH, bool DENSE>
__global__ void __launch_bounds__(kThreads)
attn_fwd_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                const int* __restrict__ kb_ptr, const int* __restrict__ q_idx, const int* __restrict__ q_ptr,
                const int* __restrict__ item_ptr, int n_kb, int S, int Nb, int sb, int BH, float scale,
                T* __restrict__ o, T* __restrict__ o_resid, float* __restrict__ lse, float* __restrict__ part_o,
                float* __restrict__ part_lse, long long capacity) {
  constexpr int DP = DH / 4;   // channels per thread
  constexpr int G = DP / 4;    // float4 groups per thread
  __shared__ __align__(16) float Ks[kTile * DH];
  __shared__ __align__(16) float Vs[kTile * DH];
  const int r = threadIdx.x >> 2, part = threadIdx.x & 3;
  const int tiles_per_head = (S + kRows - 1) / kRows;
  const int n_items = DENSE ? BH * tiles_per_head : item_ptr[n_kb];
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    Item it;
    int qpos = -1;
    long long pos = -1;
    if (DENSE) {
      it.bh = item / tiles_per_head;
      int row = (item - it.bh * tiles_per_head) * kRows + r;
      it.key_begin = 0; it.key_end = S;
      if (row < S) qpos = row;
    } else {
      it = decode_sparse(item, item_ptr, n_kb, kb_ptr, Nb, sb, kRows, capacity);
      if (it.list_lo + r < it.list_hi) { pos = it.list_lo + r; qpos = q_idx[pos]; }
    }
    const long long head_off = (long long)it.bh * S;
    const T* kh = k + head_off * DH;
    const T* vh = v + head_off * DH;
    float qr[DP], acc[DP];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
      if (qpos >= 0) x = load4(q + (head_off + qpos) * DH + (part + 4 * g) * 4);
      qr[4 * g] = x.x; qr[4 * g + 1] = x.y; qr[4 * g + 2] = x.z; qr[4 * g + 3] = x.w;
      acc[4 * g] = acc[4 * g + 1] = acc[4 * g + 2] = acc[4 * g + 3] = 0.f;
    }
    float m = -INFINITY, l = 0.f;
    for (int t0 = it.key_begin; t0 < it.key_end; t0 += kTile) {
      const int nv = min(kTile, it.key_end - t0);
      __syncthreads();
      load_tile<T, DH>(Ks, kh, nv, [&](int i) { return t0 + i; });
      load_tile<T, DH>(Vs, vh, nv, [&](int i) { return t0 + i; });
      __syncthreads();
#pragma unroll 1
      for (int kk = 0; kk < kTile; kk += 16) {
        if (kk >= nv) break;
        float s[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float a = 0.f;
#pragma unroll
          for (int g = 0; g < G; ++g) {
            float4 kv = *reinterpret_cast<const float4*>(Ks + (kk + i) * DH + (part + 4 * g) * 4);
            a = fmaf(qr[4 * g], kv.x, a); a = fmaf(qr[4 * g + 1], kv.y, a);
            a = fmaf(qr[4 * g + 2], kv.z, a); a = fmaf(qr[4 * g + 3], kv.w, a);
          }
          a = quad_sum(a);
          s[i] = (kk + i < nv) ? a * scale : -INFINITY;
        }
        float mx = s[0];
#pragma unroll
        for (int i = 1; i < 16; ++i) mx = fmaxf(mx, s[i]);
        const float m_new = fmaxf(m, mx);
        const float corr = (m == -INFINITY) ? 0.f : expf(m - m_new);
        l *= corr;
#pragma unroll
        for (int c = 0; c < DP; ++c) acc[c] *= corr;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float p = (s[i] == -INFINITY) ? 0.f : expf(s[i] - m_new);
          l += p;
#pragma unroll
          for (int g = 0; g < G; ++g) {
            float4 vv = *reinterpret_cast<const float4*>(Vs + (kk + i) * DH + (part + 4 * g) * 4);
            acc[4 * g] = fmaf(p, vv.x, acc[4 * g]); acc[4 * g + 1] = fmaf(p, vv.y, acc[4 * g + 1]);
            acc[4 * g + 2] = fmaf(p, vv.z, acc[4 * g + 2]); acc[4 * g + 3] = fmaf(p, vv.w, acc[4 * g + 3]);
          }
        }
        m = m_new;
      }
    }
    if (qpos >= 0) {
      const float inv = 1.0f / l;
      const float row_lse = m + logf(l);
      const long long G_ = head_off + qpos;
      bool direct = DENSE;
      if (!DENSE) direct = (q_ptr[G_ + 1] - q_ptr[G_]) == 1;
      if (direct) {
#pragma unroll
        for (int g = 0; g < G; ++g)
          store4_resid(o + G_ * DH + (part + 4 * g) * 4, o_resid ? o_resid + G_ * DH + (part + 4 * g) * 4 : nullptr,
                       make_float4(acc[4 * g] * inv, acc[4 * g + 1] * inv, acc[4 * g + 2] * inv, acc[4 * g + 3] * inv));
        if (part == 0) lse[G_] = row_lse;
      } else {
#pragma unroll
        for (int g = 0; g < G; ++g)
          store4(part_o + pos * DH + (part + 4 * g) * 4,
                 make_float4(acc[4 * g] * inv, acc[4 * g + 1] * inv, acc[4 * g + 2] * inv, acc[4 * g + 3] * inv));
        if (part == 0) part_lse[pos] = row_lse;
      }
    }
  }
}

// Merge of the per-block partials of each query (one warp per query).  Queries with a single
// pair were written by the attention kernel; queries with none get o = 0, lse = -inf.
template <typename T, int DH, typename PT>
__global__ void __launch_bounds__(256)
merge_kernel(const int* __restrict__ q_ptr, const int* __restrict__ q_pairs, long long n_queries,
             const PT* __restrict__ part_o, const float* __restrict__ part_lse, long long capacity,
             T* __restrict__ o, T* __restrict__ o_resid, float* __restrict__ lse, const RowMap o_map = RowMap()) {
  constexpr int C = DH / 32;   // channels per lane
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long g = warp; g < n_queries; g += nwarps) {
    const long long lo = q_ptr[g], hi = min((long long)q_ptr[g + 1], capacity);
    const long long n = hi - lo;
    if (n == 1 && q_ptr[g + 1] - lo == 1) continue;
    float acc[C];
#pragma unroll
    for (int c = 0; c < C; ++c) acc[c] = 0.f;
    float out_lse = -INFINITY;
    if (n > 0) {
      // lane i of each group of 32 pairs fetches the position and lse of pair i once; the row
      // weights then travel by shuffle.  A truncated list (capacity exceeded) may hold unwritten
      // entries: keep every index in range.
      float mx = -INFINITY;
      for (long long i0 = lo; i0 < hi; i0 += 32) {
        const long long i = i0 + lane;
        const float l = i < hi ? part_lse[min(max(q_pairs[i], 0), (int)(capacity - 1))] : -INFINITY;
        mx = fmaxf(mx, l);
      }
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
      float tot = 0.f;
      for (long long i0 = lo; i0 < hi; i0 += 32) {
        const long long i = i0 + lane;
        int my_pos = 0;
        float my_w = 0.f;
        if (i < hi) {
          my_pos = min(max(q_pairs[i], 0), (int)(capacity - 1));
          my_w = expf(part_lse[my_pos] - mx);
        }
        tot += my_w;
        const int m = (int)min((long long)32, hi - i0);
#pragma unroll 4
        for (int k = 0; k < m; ++k) {
          const long long pos = __shfl_sync(0xffffffffu, my_pos, k);
          const float wgt = __shfl_sync(0xffffffffu, my_w, k);
          if constexpr (C == 4 && sizeof(PT) == 4) {
            const float4 v = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(part_o) + pos * DH + lane * 4);
            acc[0] = fmaf(wgt, v.x, acc[0]); acc[1] = fmaf(wgt, v.y, acc[1]);
            acc[2] = fmaf(wgt, v.z, acc[2]); acc[3] = fmaf(wgt, v.w, acc[3]);
          } else {
#pragma unroll
            for (int c = 0; c < C; ++c) acc[c] = fmaf(wgt, to_f32<PT>(part_o[pos * DH + lane * C + c]), acc[c]);
          }
        }
      }
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, s);
      const float inv = 1.0f / tot;
#pragma unroll
      for (int c = 0; c < C; ++c) acc[c] *= inv;
      out_lse = mx + logf(tot);
    }
    // o goes to the caller's layout (block-major, or raster order through perm); the residual stays block-major
    T* o_row = o + o_map.off(g, DH);
    if constexpr (C == 4) {
      store4_resid(o_row + lane * 4, o_resid ? o_resid + g * DH + lane * 4 : nullptr,
                   make_float4(acc[0], acc[1], acc[2], acc[3]));
    } else {
#pragma unroll
      for (int c = 0; c < C; ++c) {
        const T hi_ = from_f32<T>(acc[c]);
        o_row[lane * C + c] = hi_;
        if (o_resid) o_resid[g * DH + lane * C + c] = from_f32<T>(acc[c] - to_f32<T>(hi_));
      }
    }
    if (lane == 0) lse[g] = out_lse;
  }
}

// The same merge for head_dim 128 and fp32 partials, 32 consecutive queries per warp and trip.  With one
// query per warp the four dependent loads of a query (list bounds, pair positions, partial lse, rows) are
// paid one after the other for every query; here lane l reads the bounds, the first kInLane pair positions
// and their lse of query g0 + l, works out the weights on its own, and the warp then walks the queries that
// need a row written, fetching all rows of a query at once.  Queries with more pairs than a lane keeps take
// the warp-wide loop of merge_kernel.
//
// PT = __half: a partial row is stored as fp16 values times a power of two (part_scale, one per row; the row's
// largest magnitude rounded up), which halves the bytes the forward writes and this pass reads; a value is then off
// by at most 2^-11 of its row's largest one.  The scale is folded into the row's merge weight.
constexpr int kInLane = 8;
template <typename PT>
__device__ __forceinline__ float4 load_part4(const PT* p);
template <>
__device__ __forceinline__ float4 load_part4<float>(const float* p) { return *reinterpret_cast<const float4*>(p); }
template <>
__device__ __forceinline__ float4 load_part4<__half>(const __half* p) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&u.x));
  const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&u.y));
  return make_float4(a.x, a.y, b.x, b.y);
}
template <typename T, typename PT>
__global__ void __launch_bounds__(256)
merge_batched_kernel(const int* __restrict__ q_ptr, const int* __restrict__ q_pairs, long long n_queries,
                     const PT* __restrict__ part_o, const float* __restrict__ part_lse,
                     const float* __restrict__ part_scale, long long capacity,
                     T* __restrict__ o, T* __restrict__ o_resid, float* __restrict__ lse, const RowMap o_map = RowMap()) {
  constexpr int DH = 128;
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
  const int last = (int)(capacity - 1);
  for (long long g0 = warp * 32; g0 < n_queries; g0 += nwarps * 32) {
    const long long g = g0 + lane;
    int lo = 0, n = 1, n_raw = 1;        // lanes beyond the last query behave like a directly written row
    if (g < n_queries) {
      lo = q_ptr[g];
      const int hi_raw = q_ptr[g + 1];
      n_raw = hi_raw - lo;
      n = (int)(min((long long)hi_raw, capacity) - lo);
      if (n < 0) n = 0;
    }
    const bool direct = n == 1 && n_raw == 1;
    int pos[kInLane];
    float w[kInLane], sc[kInLane];
    float out_lse = -INFINITY;
    if (!direct && n > 0 && n <= kInLane) {
      float mx = -INFINITY;
#pragma unroll
      for (int k = 0; k < kInLane; ++k) {
        pos[k] = 0; w[k] = -INFINITY;
        if (k < n) pos[k] = min(max(q_pairs[lo + k], 0), last);
      }
#pragma unroll
      for (int k = 0; k < kInLane; ++k) {
        sc[k] = 1.0f;
        if (k < n) {
          w[k] = part_lse[pos[k]];
          if (part_scale) sc[k] = part_scale[pos[k]];
          mx = fmaxf(mx, w[k]);
        }
      }
      float tot = 0.f;
#pragma unroll
      for (int k = 0; k < kInLane; ++k) {
        w[k] = k < n ? expf(w[k] - mx) : 0.f;
        tot += w[k];
      }
      const float inv = 1.0f / tot;
#pragma unroll
      for (int k = 0; k < kInLane; ++k) w[k] *= inv * sc[k];
      out_lse = mx + logf(tot);
    } else {
#pragma unroll
      for (int k = 0; k < kInLane; ++k) { pos[k] = 0; w[k] = 0.f; }
    }
    uint32_t todo = __ballot_sync(0xffffffffu, !direct);
    while (todo) {
      const int b = __ffs(todo) - 1;
      todo &= todo - 1;
      const long long gq = g0 + b;
      const int nb = __shfl_sync(0xffffffffu, n, b);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float row_lse = __shfl_sync(0xffffffffu, out_lse, b);
      if (nb <= kInLane) {
        float4 v[kInLane];
        float wk[kInLane];
#pragma unroll
        for (int k = 0; k < kInLane; ++k) {
          const int pk = __shfl_sync(0xffffffffu, pos[k], b);
          wk[k] = __shfl_sync(0xffffffffu, w[k], b);
          v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (k < nb) v[k] = load_part4<PT>(part_o + (long long)pk * DH + lane * 4);
        }
#pragma unroll
        for (int k = 0; k < kInLane; ++k) {
          acc.x = fmaf(wk[k], v[k].x, acc.x); acc.y = fmaf(wk[k], v[k].y, acc.y);
          acc.z = fmaf(wk[k], v[k].z, acc.z); acc.w = fmaf(wk[k], v[k].w, acc.w);
        }
      } else {
        // many pairs: lane i of each group of 32 pairs fetches position and lse of pair i, the weights travel by shuffle
        const long long qlo = __shfl_sync(0xffffffffu, lo, b), qhi = qlo + nb;
        float mx = -INFINITY;
        for (long long i0 = qlo; i0 < qhi; i0 += 32) {
          const long long i = i0 + lane;
          mx = fmaxf(mx, i < qhi ? part_lse[min(max(q_pairs[i], 0), last)] : -INFINITY);
        }
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, s));
        float tot = 0.f;
        for (long long i0 = qlo; i0 < qhi; i0 += 32) {
          const long long i = i0 + lane;
          int my_pos = 0;
          float my_w = 0.f, my_ws = 0.f;
          if (i < qhi) {
            my_pos = min(max(q_pairs[i], 0), last);
            my_w = expf(part_lse[my_pos] - mx);
            my_ws = part_scale ? my_w * part_scale[my_pos] : my_w;
          }
          tot += my_w;
          const int m = (int)min((long long)32, qhi - i0);
#pragma unroll 4
          for (int k = 0; k < m; ++k) {
            const long long pk = __shfl_sync(0xffffffffu, my_pos, k);
            const float wgt = __shfl_sync(0xffffffffu, my_ws, k);
            const float4 v = load_part4<PT>(part_o + pk * DH + lane * 4);
            acc.x = fmaf(wgt, v.x, acc.x); acc.y = fmaf(wgt, v.y, acc.y);
            acc.z = fmaf(wgt, v.z, acc.z); acc.w = fmaf(wgt, v.w, acc.w);
          }
        }
#pragma unroll
        for (int s = 16; s > 0; s >>= 1) tot += __shfl_xor_sync(0xffffffffu, tot, s);
        const float inv = 1.0f / tot;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        row_lse = mx + logf(tot);
      }
      T* o_row = o + o_map.off(gq, DH);
      store4_resid(o_row + lane * 4, o_resid ? o_resid + gq * DH + lane * 4 : nullptr, acc);
      if (lane == 0) lse[gq] = row_lse;
    }
  }
}

// ------------------------------------------------------------------------------ backward
// D = rowsum(dO * O), one warp per query; o and dO block-major or in raster order through their maps, the
// rounding residual of o always block-major.  If zero_acc is given, the fp32 dQ accumulator rows of the queries
// with at least one selected block are cleared in the same pass (the only rows the backward kernel adds into).
template <typename T, int DH>
__global__ void __launch_bounds__(256)
rowdot_kernel(const T* __restrict__ o, const T* __restrict__ o_resid, const T* __restrict__ d_o, long long n_queries,
              float* __restrict__ Dv, const RowMap do_map = RowMap(), const RowMap o_map = RowMap(),
              float* __restrict__ zero_acc = nullptr, const int* __restrict__ q_ptr = nullptr) {
  constexpr int C = DH / 32;
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
  if constexpr (C == 4 && sizeof(T) == 2) {
    // Four rows per warp and trip, in phases (row offsets, loads, sums, stores), so that the twelve 8-byte
    // loads of a lane are in flight together.
    constexpr int R = 4;
    for (long long g0 = warp * R; g0 < n_queries; g0 += nwarps * R) {
      uint2 ov[R], rv[R], dv[R];
      bool zero[R], used[R];
      // with the lists at hand, a query without a selected block is skipped: nothing reads its D
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const long long g = min(g0 + r, n_queries - 1);
        used[r] = !q_ptr || __ldg(q_ptr + g + 1) - __ldg(q_ptr + g) >= 1;
        zero[r] = zero_acc && q_ptr && g0 + r < n_queries && used[r];
      }
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const long long g = min(g0 + r, n_queries - 1);
        ov[r] = dv[r] = rv[r] = make_uint2(0u, 0u);
        if (used[r]) {
          ov[r] = *reinterpret_cast<const uint2*>(o + o_map.off(g, DH) + lane * 4);
          dv[r] = *reinterpret_cast<const uint2*>(d_o + do_map.off(g, DH) + lane * 4);
          if (o_resid) rv[r] = *reinterpret_cast<const uint2*>(o_resid + g * DH + lane * 4);
        }
      }
      float a[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        auto lo = [](uint32_t u) { return __uint_as_float(u << 16); };
        auto hi = [](uint32_t u) { return __uint_as_float(u & 0xffff0000u); };
        a[r] = (lo(ov[r].x) + lo(rv[r].x)) * lo(dv[r].x);
        a[r] = fmaf(hi(ov[r].x) + hi(rv[r].x), hi(dv[r].x), a[r]);
        a[r] = fmaf(lo(ov[r].y) + lo(rv[r].y), lo(dv[r].y), a[r]);
        a[r] = fmaf(hi(ov[r].y) + hi(rv[r].y), hi(dv[r].y), a[r]);
      }
#pragma unroll
      for (int s = 16; s > 0; s >>= 1)
#pragma unroll
        for (int r = 0; r < R; ++r) a[r] += __shfl_xor_sync(0xffffffffu, a[r], s);
#pragma unroll
      for (int r = 0; r < R; ++r) {
        if (g0 + r >= n_queries) break;
        if (lane == 0) Dv[g0 + r] = a[r];
        if (zero[r]) reinterpret_cast<float4*>(zero_acc + (g0 + r) * DH)[lane] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    return;
  }
  for (long long g = warp; g < n_queries; g += nwarps) {
    float a = 0.f;
    const T* do_row = d_o + do_map.off(g, DH);
    const T* o_row = o + o_map.off(g, DH);
    if (zero_acc && __ldg(q_ptr + g + 1) - __ldg(q_ptr + g) >= 1) {
      float4* row = reinterpret_cast<float4*>(zero_acc + g * DH);
      for (int c = lane; c < DH / 4; c += 32) row[c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int c = 0; c < C; ++c) {
      float ov = to_f32<T>(o_row[lane * C + c]);
      if (o_resid) ov += to_f32<T>(o_resid[g * DH + lane * C + c]);
      a = fmaf(ov, to_f32<T>(do_row[lane * C + c]), a);
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) a += __shfl_xor_sync(0xffffffffu, a, s);
    if (lane == 0) Dv[g] = a;
  }
}

// dK, dV: key-stationary.  A CTA owns 64 keys of one key block (or of the whole sequence when
// DENSE) and streams the queries that selected the block; no atomics, deterministic.
template <typename T, int DH, bool DENSE>
__global__ void __launch_bounds__(kThreads)
attn_bwd_dkdv_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                     const T* __restrict__ d_o, const float* __restrict__ lse, const float* __restrict__ Dv,
                     const int* __restrict__ kb_ptr, const int* __restrict__ q_idx, int S, int Nb, int sb, int BH,
                     float scale, long long capacity, T* __restrict__ dk, T* __restrict__ dv) {
  constexpr int DP = DH / 4, G = DP / 4;
  __shared__ __align__(16) float Qs[kTile * DH];
  __shared__ __align__(16) float dOs[kTile * DH];
  __shared__ float s_lse[kTile], s_D[kTile];
  const int r = threadIdx.x >> 2, part = threadIdx.x & 3;
  const int span = DENSE ? S : sb;
  const int tiles = (span + kRows - 1) / kRows;
  const long long n_items = (long long)BH * (DENSE ? 1 : Nb) * tiles;
  for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int tile = (int)(item % tiles);
    const long long kbi = item / tiles;          // DENSE: bh ; sparse: bh * Nb + j
    const int bh = DENSE ? (int)kbi : (int)(kbi / Nb);
    const int j = DENSE ? 0 : (int)(kbi - (long long)bh * Nb);
    const int key_in_span = tile * kRows + r;
    const bool key_ok = key_in_span < span;
    const int kpos = j * sb + key_in_span;
    const long long head_off = (long long)bh * S;
    long long list_lo = 0, list_hi = S;
    if (!DENSE) { list_lo = min((long long)kb_ptr[kbi], capacity); list_hi = min((long long)kb_ptr[kbi + 1], capacity); }
    float kr[DP], vr[DP], dkr[DP], dvr[DP];
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
      if (key_ok) {
        x = load4(k + (head_off + kpos) * DH + (part + 4 * g) * 4);
        y = load4(v + (head_off + kpos) * DH + (part + 4 * g) * 4);
      }
      kr[4 * g] = x.x; kr[4 * g + 1] = x.y; kr[4 * g + 2] = x.z; kr[4 * g + 3] = x.w;
      vr[4 * g] = y.x; vr[4 * g + 1] = y.y; vr[4 * g + 2] = y.z; vr[4 * g + 3] = y.w;
#pragma unroll
      for (int c = 0; c < 4; ++c) dkr[4 * g + c] = dvr[4 * g + c] = 0.f;
    }
    for (long long t0 = list_lo; t0 < list_hi; t0 += kTile) {
      const int nv = (int)min((long long)kTile, list_hi - t0);
      __syncthreads();
      auto row_of = [&](int i) { return DENSE ? (int)(t0 + i) : q_idx[t0 + i]; };
      load_tile<T, DH>(Qs, q + head_off * DH, nv, row_of);
      load_tile<T, DH>(dOs, d_o + head_off * DH, nv, row_of);
      if (threadIdx.x < kTile) {
        float a = INFINITY, b = 0.f;
        if (threadIdx.x < nv) {
          long long g_ = head_off + row_of(threadIdx.x);
          a = lse[g_]; b = Dv[g_];
        }
        s_lse[threadIdx.x] = a; s_D[threadIdx.x] = b;
      }
      __syncthreads();
#pragma unroll 2
      for (int i = 0; i < kTile; ++i) {
        if (i >= nv) break;
        float s = 0.f, dp = 0.f;
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float4 qv = *reinterpret_cast<const float4*>(Qs + i * DH + (part + 4 * g) * 4);
          float4 gv = *reinterpret_cast<const float4*>(dOs + i * DH + (part + 4 * g) * 4);
          s = fmaf(qv.x, kr[4 * g], s); s = fmaf(qv.y, kr[4 * g + 1], s);
          s = fmaf(qv.z, kr[4 * g + 2], s); s = fmaf(qv.w, kr[4 * g + 3], s);
          dp = fmaf(gv.x, vr[4 * g], dp); dp = fmaf(gv.y, vr[4 * g + 1], dp);
          dp = fmaf(gv.z, vr[4 * g + 2], dp); dp = fmaf(gv.w, vr[4 * g + 3], dp);
        }
        s = quad_sum(s); dp = quad_sum(dp);
        const float p = expf(s * scale - s_lse[i]);      // lse = +inf for padded rows -> p = 0
        const float ds = p * (dp - s_D[i]);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float4 qv = *reinterpret_cast<const float4*>(Qs + i * DH + (part + 4 * g) * 4);
          float4 gv = *reinterpret_cast<const float4*>(dOs + i * DH + (part + 4 * g) * 4);
          dkr[4 * g] = fmaf(ds, qv.x, dkr[4 * g]); dkr[4 * g + 1] = fmaf(ds, qv.y, dkr[4 * g + 1]);
          dkr[4 * g + 2] = fmaf(ds, qv.z, dkr[4 * g + 2]); dkr[4 * g + 3] = fmaf(ds, qv.w, dkr[4 * g + 3]);
          dvr[4 * g] = fmaf(p, gv.x, dvr[4 * g]); dvr[4 * g + 1] = fmaf(p, gv.y, dvr[4 * g + 1]);
          dvr[4 * g + 2] = fmaf(p, gv.z, dvr[4 * g + 2]); dvr[4 * g + 3] = fmaf(p, gv.w, dvr[4 * g + 3]);
        }
      }
    }
    if (key_ok) {
#pragma unroll
      for (int g = 0; g < G; ++g) {
        store4(dk + (head_off + kpos) * DH + (part + 4 * g) * 4,
               make_float4(dkr[4 * g] * scale, dkr[4 * g + 1] * scale, dkr[4 * g + 2] * scale, dkr[4 * g + 3] * scale));
        store4(dv + (head_off + kpos) * DH + (part + 4 * g) * 4,
               make_float4(dvr[4 * g], dvr[4 * g + 1], dvr[4 * g + 2], dvr[4 * g + 3]));
      }
    }
  }
}

// dQ: query-stationary over the same work items as the forward.  Sparse: the per-block
// contributions of a query are added into an fp32 accumulator (atomics); dense: written directly.
template <typename T, int DH, bool DENSE>
__global__ void __launch_bounds__(kThreads)
attn_bwd_dq_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                   const T* __restrict__ d_o, const float* __restrict__ lse, const float* __restrict__ Dv,
                   const int* __restrict__ kb_ptr, const int* __restrict__ q_idx, const int* __restrict__ item_ptr,
                   int n_kb, int S, int Nb, int sb, int BH, float scale, long long capacity,
                   float* __restrict__ dq_acc, T* __restrict__ dq) {
  constexpr int DP = DH / 4, G = DP / 4;
  __shared__ __align__(16) float Ks[kTile * DH];
  __shared__ __align__(16) float Vs[kTile * DH];
  const int r = threadIdx.x >> 2, part = threadIdx.x & 3;
  const int tiles_per_head = (S + kRows - 1) / kRows;
  const int n_items = DENSE ? BH * tiles_per_head : item_ptr[n_kb];
  for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
    Item it;
    int qpos = -1;
    if (DENSE) {
      it.bh = item / tiles_per_head;
      int row = (item - it.bh * tiles_per_head) * kRows + r;
      it.key_begin = 0; it.key_end = S;
      if (row < S) qpos = row;
    } else {
      it = decode_sparse(item, item_ptr, n_kb, kb_ptr, Nb, sb, kRows, capacity);
      if (it.list_lo + r < it.list_hi) qpos = q_idx[it.list_lo + r];
    }
    const long long head_off = (long long)it.bh * S;
    const T* kh = k + head_off * DH;
    const T* vh = v + head_off * DH;
    float qr[DP], gr[DP], acc[DP];
    float row_lse = INFINITY, row_D = 0.f;
    if (qpos >= 0) { row_lse = lse[head_off + qpos]; row_D = Dv[head_off + qpos]; }
#pragma unroll
    for (int g = 0; g < G; ++g) {
      float4 x = make_float4(0.f, 0.f, 0.f, 0.f), y = x;
      if (qpos >= 0) {
        x = load4(q + (head_off + qpos) * DH + (part + 4 * g) * 4);
        y = load4(d_o + (head_off + qpos) * DH + (part + 4 * g) * 4);
      }
      qr[4 * g] = x.x; qr[4 * g + 1] = x.y; qr[4 * g + 2] = x.z; qr[4 * g + 3] = x.w;
      gr[4 * g] = y.x; gr[4 * g + 1] = y.y; gr[4 * g + 2] = y.z; gr[4 * g + 3] = y.w;
      acc[4 * g] = acc[4 * g + 1] = acc[4 * g + 2] = acc[4 * g + 3] = 0.f;
    }
    for (int t0 = it.key_begin; t0 < it.key_end; t0 += kTile) {
      const int nv = min(kTile, it.key_end - t0);
      __syncthreads();
      load_tile<T, DH>(Ks, kh, nv, [&](int i) { return t0 + i; });
      load_tile<T, DH>(Vs, vh, nv, [&](int i) { return t0 + i; });
      __syncthreads();
#pragma unroll 2
      for (int i = 0; i < kTile; ++i) {
        if (i >= nv) break;
        float s = 0.f, dp = 0.f;
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float4 kv = *reinterpret_cast<const float4*>(Ks + i * DH + (part + 4 * g) * 4);
          float4 vv = *reinterpret_cast<const float4*>(Vs + i * DH + (part + 4 * g) * 4);
          s = fmaf(qr[4 * g], kv.x, s); s = fmaf(qr[4 * g + 1], kv.y, s);
          s = fmaf(qr[4 * g + 2], kv.z, s); s = fmaf(qr[4 * g + 3], kv.w, s);
          dp = fmaf(gr[4 * g], vv.x, dp); dp = fmaf(gr[4 * g + 1], vv.y, dp);
          dp = fmaf(gr[4 * g + 2], vv.z, dp); dp = fmaf(gr[4 * g + 3], vv.w, dp);
        }
        s = quad_sum(s); dp = quad_sum(dp);
        const float p = expf(s * scale - row_lse);
        const float ds = p * (dp - row_D);
#pragma unroll
        for (int g = 0; g < G; ++g) {
          float4 kv = *reinterpret_cast<const float4*>(Ks + i * DH + (part + 4 * g) * 4);
          acc[4 * g] = fmaf(ds, kv.x, acc[4 * g]); acc[4 * g + 1] = fmaf(ds, kv.y, acc[4 * g + 1]);
          acc[4 * g + 2] = fmaf(ds, kv.z, acc[4 * g + 2]); acc[4 * g + 3] = fmaf(ds, kv.w, acc[4 * g + 3]);
        }
      }
    }
    if (qpos >= 0) {
      const long long G_ = head_off + qpos;
#pragma unroll
      for (int g = 0; g < G; ++g) {
        if (DENSE) {
          store4(dq + G_ * DH + (part + 4 * g) * 4,
                 make_float4(acc[4 * g] * scale, acc[4 * g + 1] * scale, acc[4 * g + 2] * scale, acc[4 * g + 3] * scale));
        } else {
#pragma unroll
          for (int c = 0; c < 4; ++c) atomicAdd(dq_acc + G_ * DH + (part + 4 * g) * 4 + c, acc[4 * g + c] * scale);
        }
      }
    }
  }
}

// fp32 accumulator rows -> output dtype, one warp per query.  With `sparse_rows` set only queries with
// two or more selected blocks own an accumulator row: queries with exactly one block were written
// directly by the attention kernel (skipped here) and queries with none get zeros without a read.
template <typename T, int DH>
__global__ void __launch_bounds__(256)
cast_rows_kernel(const float* __restrict__ src, T* __restrict__ dst, const int* __restrict__ q_ptr, long long n_queries,
                 int sparse_rows, int min_nb, const RowMap map = RowMap()) {
  constexpr int C = DH / 32;
  const int lane = threadIdx.x & 31;
  const long long warp = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * (blockDim.x >> 5);
  if constexpr (C == 4) {
    // Four rows per warp and trip, in phases (list bounds, row offsets, loads, stores), so that the
    // loads of the four rows are in flight together.
    constexpr int R = 4;
    for (long long g0 = warp * R; g0 < n_queries; g0 += nwarps * R) {
      int nb[R];
      long long off[R];
      float4 v[R];
#pragma unroll
      for (int r = 0; r < R; ++r) {
        const long long g = g0 + r;
        nb[r] = g >= n_queries ? 1 : (sparse_rows ? __ldg(q_ptr + g + 1) - __ldg(q_ptr + g) : 2);
        if (g >= n_queries || (nb[r] > 0 && nb[r] < min_nb)) nb[r] = -1;   // no row, or written by the attention kernel
      }
#pragma unroll
      for (int r = 0; r < R; ++r) off[r] = nb[r] >= 0 ? map.off(g0 + r, DH) : 0;
#pragma unroll
      for (int r = 0; r < R; ++r)
        v[r] = nb[r] > 0 ? *reinterpret_cast<const float4*>(src + (g0 + r) * DH + lane * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int r = 0; r < R; ++r)
        if (nb[r] >= 0) store4(dst + off[r] + lane * 4, v[r]);
    }
  } else {
    for (long long g = warp; g < n_queries; g += nwarps) {
      const int nb = sparse_rows ? q_ptr[g + 1] - q_ptr[g] : 2;
      if (nb > 0 && nb < min_nb) continue;   // written directly by the attention kernel
      T* out = dst + map.off(g, DH);
#pragma unroll
      for (int c = 0; c < C; ++c) out[lane * C + c] = from_f32<T>(nb == 0 ? 0.f : src[g * DH + lane * C + c]);
    }
  }
}

// fp32 accumulator -> output dtype.
template <typename T>
__global__ void __launch_bounds__(256)
cast_kernel(const float* __restrict__ src, T* __restrict__ dst, long long n4) {
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x)
    store4(dst + 4 * i, *reinterpret_cast<const float4*>(src + 4 * i));
}

}  // namespace simt
}  // namespace vmoba
