// Step 1 of VMoBA (Eq. 1): reorder tokens of the T x H x W latent into 1D / 2D / 3D blocks,
// and the inverse reordering.  A pure permutation of head_dim-wide rows, bound by HBM
// bandwidth: every row is read once and written once with 16-byte vector accesses.
#include "common.cuh"

namespace vmoba {

struct PermGeom {
  int H, W, bT, bH, bW, nH, nW, sb;
};

// Eq. 1: raster index of the token at block-major position p.
__device__ __forceinline__ int perm_of(const PermGeom& g, int p) {
  int j = p / g.sb, r = p - j * g.sb;
  int jw = j % g.nW, jt_h = j / g.nW;
  int jh = jt_h % g.nH, jt = jt_h / g.nH;
  int rw = r % g.bW, rt_h = r / g.bW;
  int rh = rt_h % g.bH, rt = rt_h / g.bH;
  int t = jt * g.bT + rt, h = jh * g.bH + rh, w = jw * g.bW + rw;
  return (t * g.H + h) * g.W + w;
}

__global__ void perm_table_kernel(PermGeom g, int S, int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm) {
  int p = blockIdx.x * blockDim.x + threadIdx.x;
  if (p >= S) return;
  int r = perm_of(g, p);
  if (perm) perm[p] = r;
  if (inv_perm) inv_perm[r] = p;
}

// Rows are enumerated as ((b * S + p) * heads + head): consecutive rows share a token, so the
// raster side is touched in runs of heads * head_dim contiguous elements.  A warp takes 32 rows
// at a time: lane l derives the two byte offsets of row l once, then the warp streams the
// rows' 16-byte vectors with the offsets broadcast by shuffle.
template <int VEC_PER_ROW>   // 16-byte vectors per row: head_dim * elem_size / 16
__global__ void __launch_bounds__(256)
partition_kernel(PermGeom g, int S, int heads, long long n_rows, int inverse,
                 const uint4* __restrict__ src, uint4* __restrict__ dst,
                 long long rs_b, long long rs_s, long long rs_h /* raster strides in 16-byte vectors */) {
  constexpr int ROWS_PER_PASS = 32 / VEC_PER_ROW > 0 ? 32 / VEC_PER_ROW : 1;
  constexpr int PASSES = 32 / ROWS_PER_PASS;        // passes to cover 32 rows
  constexpr int VITER = VEC_PER_ROW > 32 ? VEC_PER_ROW / 32 : 1;
  const int lane = threadIdx.x & 31;
  const long long warp_id = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long n_warps = (long long)gridDim.x * (blockDim.x >> 5);
  for (long long base = warp_id * 32; base < n_rows; base += n_warps * 32) {
    long long row = base + lane;
    long long off_r = 0, off_bm = 0;
    if (row < n_rows) {
      int head = (int)(row % heads);
      long long bp = row / heads;
      int p = (int)(bp % S);
      int b = (int)(bp / S);
      int r = perm_of(g, p);
      off_r = b * rs_b + (long long)r * rs_s + head * rs_h;
      off_bm = (((long long)b * heads + head) * S + p) * VEC_PER_ROW;
    }
    long long off_src = inverse ? off_bm : off_r;
    long long off_dst = inverse ? off_r : off_bm;
#pragma unroll 4
    for (int pass = 0; pass < PASSES; ++pass) {
      int sub = (VEC_PER_ROW >= 32) ? 0 : lane / VEC_PER_ROW;
      int vec = (VEC_PER_ROW >= 32) ? lane : lane % VEC_PER_ROW;
      int src_lane = pass * ROWS_PER_PASS + sub;
      long long so = __shfl_sync(0xffffffffu, off_src, src_lane);
      long long dof = __shfl_sync(0xffffffffu, off_dst, src_lane);
      bool ok = base + src_lane < n_rows;
#pragma unroll
      for (int it = 0; it < VITER; ++it) {
        if (ok) {
          uint4 v = __ldg(src + so + vec + it * 32);
          dst[dof + vec + it * 32] = v;
        }
      }
    }
  }
}

template <int V>
static int launch_partition(const Dims& D, const PermGeom& g, int inverse, const void* src, void* dst,
                            const int64_t* rs, cudaStream_t st) {
  long long n_rows = (long long)D.BH * D.S;
  long long warps = (n_rows + 31) / 32;
  long long blocks = (warps + 7) / 8;
  long long cap = (long long)sm_count() * 8 * 4;
  if (blocks > cap) blocks = cap;
  long long per_vec = 16 / D.es;
  partition_kernel<V><<<(unsigned)blocks, 256, 0, st>>>(
      g, D.S, D.heads, n_rows, inverse, static_cast<const uint4*>(src), static_cast<uint4*>(dst),
      rs[0] / per_vec, rs[1] / per_vec, rs[2] / per_vec);
  VMOBA_LAUNCH_OK(1);
  return VMOBA_OK;
}

}  // namespace vmoba

using namespace vmoba;

extern "C" int vmoba_partition(const vmoba_shape* shape, int inverse, const void* src, void* dst,
                               const int64_t raster_strides_bsh[3], int32_t* perm_or_null,
                               int32_t* inv_perm_or_null, void* stream) {
  Dims D;
  int rc = make_dims(shape, &D);
  if (rc) return rc;
  if (!src || !dst || !raster_strides_bsh || !aligned16(src) || !aligned16(dst)) return VMOBA_ERR_ARG;
  if (inverse != 0 && inverse != 1) return VMOBA_ERR_ARG;
  int per_vec = 16 / D.es;
  for (int i = 0; i < 3; ++i)
    if (raster_strides_bsh[i] < 0 || raster_strides_bsh[i] % per_vec) return VMOBA_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  PermGeom g{D.H, D.W, D.bT, D.bH, D.bW, D.nH, D.nW, D.sb};
  if (perm_or_null || inv_perm_or_null) {
    perm_table_kernel<<<(D.S + 255) / 256, 256, 0, st>>>(g, D.S, perm_or_null, inv_perm_or_null);
    VMOBA_LAUNCH_OK(1);
  }
  int V = D.d * D.es / 16;
  switch (V) {
    case 8: return launch_partition<8>(D, g, inverse, src, dst, raster_strides_bsh, st);
    case 16: return launch_partition<16>(D, g, inverse, src, dst, raster_strides_bsh, st);
    case 32: return launch_partition<32>(D, g, inverse, src, dst, raster_strides_bsh, st);
    default: return VMOBA_ERR_NOT_IMPLEMENTED;
  }
}
