// Step 1b + Step 2a of VMoBA: mean key-block centroids (Eq. 2) and the query x centroid
// similarity map S_hat = q b^T (Section 3.3), both in fp32.
//
// Both kernels are bound by HBM traffic: K is read once for the centroids, Q once for the
// scores, and the [S, N_b] fp32 score matrix is written once.  The contraction itself
// (2 * S * N_b * d flops) is small next to that and runs on the fp32 FMA pipe so that the
// scores carry fp32 accuracy (the selection cutoff is compared in fp32).
#include <algorithm>

#include "common.cuh"

namespace vmoba {

// scores_tc.cu: tensor-core scores for bf16 / head_dim 128
size_t scores_tc_ws_bytes(const Dims& D);
int scores_tc(const Dims& D, const void* q_bm, const float* cent, float* scores, float* range, void* ws,
              int32_t* status, cudaStream_t st);

size_t scores_ws_bytes(const Dims& D) {
  return (D.dtype == VMOBA_BF16 && D.d == 128) ? scores_tc_ws_bytes(D) : 256;
}

// One CTA per (batch, head, block): 256 threads = (256 / V) row lanes x V float4-column lanes.
template <typename T, int DH>
__global__ void __launch_bounds__(256)
centroid_kernel(const T* __restrict__ k_bm, float* __restrict__ cent, int sb) {
  constexpr int V = DH / 4;            // float4 columns per row
  constexpr int RL = 256 / V;          // row lanes
  __shared__ float4 red[RL][V];
  const long long blk = blockIdx.x;    // (b*heads + head) * Nb + j : blocks are contiguous in block-major order
  const T* base = k_bm + blk * (long long)sb * DH;
  const int col = threadIdx.x % V, rl = threadIdx.x / V;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int r = rl; r < sb; r += RL) {
    float4 x = load4(base + (long long)r * DH + col * 4);
    acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
  }
  red[rl][col] = acc;
  __syncthreads();
  if (rl == 0) {
    float4 s = red[0][col];
    for (int i = 1; i < RL; ++i) {
      float4 x = red[i][col];
      s.x += x.x; s.y += x.y; s.z += x.z; s.w += x.w;
    }
    float inv = 1.0f / (float)sb;
    s.x *= inv; s.y *= inv; s.z *= inv; s.w *= inv;
    store4(cent + blk * DH + col * 4, s);
  }
}

// fp32 tile GEMM: a CTA computes 64 queries x 64 blocks with the whole head_dim in shared
// memory (operands stored transposed so that each thread reads its 4x4 micro-tile as float4).
template <typename T, int DH>
__global__ void __launch_bounds__(256)
scores_kernel(const T* __restrict__ q_bm, const float* __restrict__ cent, float* __restrict__ scores,
              int S, int Nb) {
  extern __shared__ float smem[];
  constexpr int LD = 64 + 4;
  float* qT = smem;                 // [DH][LD]
  float* bT = smem + DH * LD;       // [DH][LD]
  const int bh = blockIdx.z;
  const int q0 = blockIdx.x * 64;
  const int tid = threadIdx.x;
  const T* qh = q_bm + ((long long)bh * S + q0) * DH;
  // Load the query tile once: thread t reads float4 #(t % (DH/4)) of row (t / (DH/4)) + k * rows_per_pass.
  constexpr int V = DH / 4;
  for (int i = tid; i < 64 * V; i += 256) {
    int r = i / V, c4 = i % V;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (q0 + r < S) x = load4(qh + (long long)r * DH + c4 * 4);
    qT[(c4 * 4 + 0) * LD + r] = x.x;
    qT[(c4 * 4 + 1) * LD + r] = x.y;
    qT[(c4 * 4 + 2) * LD + r] = x.z;
    qT[(c4 * 4 + 3) * LD + r] = x.w;
  }
  const int ty = tid / 16, tx = tid % 16;
  const float* ch = cent + (long long)bh * Nb * DH;
  float* out = scores + ((long long)bh * S + q0) * Nb;
  for (int j0 = 0; j0 < Nb; j0 += 64) {
    __syncthreads();
    for (int i = tid; i < 64 * V; i += 256) {
      int r = i / V, c4 = i % V;
      float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
      if (j0 + r < Nb) x = *reinterpret_cast<const float4*>(ch + (long long)(j0 + r) * DH + c4 * 4);
      bT[(c4 * 4 + 0) * LD + r] = x.x;
      bT[(c4 * 4 + 1) * LD + r] = x.y;
      bT[(c4 * 4 + 2) * LD + r] = x.z;
      bT[(c4 * 4 + 3) * LD + r] = x.w;
    }
    __syncthreads();
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
#pragma unroll 8
    for (int c = 0; c < DH; ++c) {
      float4 a = *reinterpret_cast<const float4*>(qT + c * LD + ty * 4);
      float4 b = *reinterpret_cast<const float4*>(bT + c * LD + tx * 4);
      float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      int r = ty * 4 + i;
      if (q0 + r >= S) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        int col = j0 + tx * 4 + j;
        if (col < Nb) out[(long long)r * Nb + col] = acc[i][j];
      }
    }
  }
}

// Smallest and largest score of each head (the paths whose scores kernel does not take them on the way).
__global__ void range_init_kernel(float* __restrict__ range, int BH) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < BH) { range[2 * i] = INFINITY; range[2 * i + 1] = -INFINITY; }
}
__global__ void __launch_bounds__(256)
range_kernel(const float* __restrict__ scores, long long P, float* __restrict__ range) {
  const int bh = blockIdx.y;
  const float* base = scores + (long long)bh * P;
  float lo = INFINITY, hi = -INFINITY;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < P; i += (long long)gridDim.x * blockDim.x) {
    const float s = base[i];
    lo = fminf(lo, s); hi = fmaxf(hi, s);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
    hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
  }
  if ((threadIdx.x & 31) == 0 && lo <= hi) { atomic_min_f32(range + 2 * bh, lo); atomic_max_f32(range + 2 * bh + 1, hi); }
}

template <typename T, int DH>
static int run_scores(const Dims& D, const void* q, const void* k, float* cent, float* scores, float* range, void* ws,
                      int32_t* status, cudaStream_t st) {
  centroid_kernel<T, DH><<<D.BH * D.Nb, 256, 0, st>>>(static_cast<const T*>(k), cent, D.sb);
  VMOBA_LAUNCH_OK(1);
  if (D.dtype == VMOBA_BF16 && DH == 128) return scores_tc(D, q, cent, scores, range, ws, status, st);
  size_t smem = 2 * DH * (64 + 4) * sizeof(float);
  VMOBA_CUDA_OK(cudaFuncSetAttribute(scores_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
  dim3 grid((D.S + 63) / 64, 1, D.BH);
  scores_kernel<T, DH><<<grid, 256, smem, st>>>(static_cast<const T*>(q), cent, scores, D.S, D.Nb);
  VMOBA_LAUNCH_OK(1);
  if (range) {
    const long long P = (long long)D.S * D.Nb;
    range_init_kernel<<<(D.BH + 127) / 128, 128, 0, st>>>(range, D.BH);
    const int gx = (int)std::min<long long>(std::max<long long>(P / 2048, 1), std::max(1, sm_count() * 8 / D.BH));
    range_kernel<<<dim3(gx, D.BH), 256, 0, st>>>(scores, P, range);
    VMOBA_LAUNCH_OK(2);
  }
  return VMOBA_OK;
}

}  // namespace vmoba

using namespace vmoba;

static int block_scores_impl(const vmoba_shape* shape, const void* q_bm, const void* k_bm, float* centroids,
                             float* scores, float* range, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  Dims D;
  int rc = make_dims(shape, &D);
  if (rc) return rc;
  if (!q_bm || !k_bm || !centroids || !scores || !dev_status || !ws) return VMOBA_ERR_ARG;
  if (!aligned16(q_bm) || !aligned16(k_bm) || !aligned16(centroids) || !aligned16(scores) || !aligned16(ws))
    return VMOBA_ERR_ARG;
  if (ws_bytes < scores_ws_bytes(D)) return VMOBA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (D.dtype == VMOBA_BF16) {
    if (D.d == 128) return run_scores<__nv_bfloat16, 128>(D, q_bm, k_bm, centroids, scores, range, ws, dev_status, st);
    return run_scores<__nv_bfloat16, 64>(D, q_bm, k_bm, centroids, scores, range, ws, dev_status, st);
  }
  if (D.d == 128) return run_scores<float, 128>(D, q_bm, k_bm, centroids, scores, range, ws, dev_status, st);
  return run_scores<float, 64>(D, q_bm, k_bm, centroids, scores, range, ws, dev_status, st);
}

extern "C" int vmoba_block_scores(const vmoba_shape* shape, const void* q_bm, const void* k_bm,
                                  float* centroids, float* scores, int32_t* dev_status, void* ws,
                                  size_t ws_bytes, void* stream) {
  return block_scores_impl(shape, q_bm, k_bm, centroids, scores, nullptr, dev_status, ws, ws_bytes, stream);
}

extern "C" int vmoba_block_scores_range(const vmoba_shape* shape, const void* q_bm, const void* k_bm,
                                        float* centroids, float* scores, float* score_range, int32_t* dev_status,
                                        void* ws, size_t ws_bytes, void* stream) {
  if (!score_range) return VMOBA_ERR_ARG;
  return block_scores_impl(shape, q_bm, k_bm, centroids, scores, score_range, dev_status, ws, ws_bytes, stream);
}
