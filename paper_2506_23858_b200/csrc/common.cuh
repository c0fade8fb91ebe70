// Shared host/device helpers of the VMoBA library: derived dimensions, argument checks,
// dtype load/store, error plumbing.  Not part of the public ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "../../include/vmoba.h"

namespace vmoba {

struct Dims {
  int B, heads, d;
  int T, H, W, bT, bH, bW;
  int nT, nH, nW;
  int Nb;        // key blocks per head
  int sb;        // tokens per block
  int S;         // tokens per head
  int BH;        // B * heads
  int dtype;
  int es;        // element size in bytes
  int mask_words;  // ceil(Nb / 32)
  float scale;
};

// Where row (batch, head, block-major position p) of an output tensor lives.  perm == nullptr: block-major,
// row G = (batch * heads + head) * S + p at G * head_dim.  Otherwise raster order [B, S, heads, head_dim]
// through element strides: batch * sb + perm[p] * st + head * sh (the inverse of Eq. 1 folded into the
// kernel that writes the rows).
struct RowMap {
  const int* perm = nullptr;
  long long sb = 0, st = 0, sh = 0;
  int heads = 1, S = 1;
#ifdef __CUDACC__
  __device__ __forceinline__ long long off(long long G, int dh) const {
    if (!perm) return G * dh;
    long long b, hd;
    int p;
    if ((unsigned long long)G <= 0x7fffffffull) {   // the usual case: 32-bit quotients
      const unsigned g = (unsigned)G, bh = g / (unsigned)S, b32 = bh / (unsigned)heads;
      p = (int)(g - bh * (unsigned)S);
      b = b32;
      hd = bh - b32 * (unsigned)heads;
    } else {
      const long long bh = G / S;
      p = (int)(G - bh * S);
      b = bh / heads;
      hd = bh - b * heads;
    }
    return b * sb + (long long)__ldg(perm + p) * st + hd * sh;
  }
#endif
};

// Validates a shape and fills the derived sizes (Eq. 1 needs the grid divisible by the block).
inline int make_dims(const vmoba_shape* s, Dims* o) {
  if (!s) return VMOBA_ERR_ARG;
  if (s->dtype != VMOBA_F32 && s->dtype != VMOBA_BF16) return VMOBA_ERR_ARG;
  if (s->B <= 0 || s->heads <= 0 || s->T <= 0 || s->H <= 0 || s->W <= 0 || s->bT <= 0 ||
      s->bH <= 0 || s->bW <= 0)
    return VMOBA_ERR_SHAPE;
  if (s->head_dim != 64 && s->head_dim != 128) return VMOBA_ERR_SHAPE;
  if (s->T % s->bT || s->H % s->bH || s->W % s->bW) return VMOBA_ERR_SHAPE;
  if (!(s->softmax_scale >= 0.0f) || s->softmax_scale > 1e30f) return VMOBA_ERR_ARG;
  long long S = (long long)s->T * s->H * s->W;
  long long total = S * s->B * s->heads;
  if (S > (1ll << 24) || total > (1ll << 30)) return VMOBA_ERR_SHAPE;
  o->B = s->B; o->heads = s->heads; o->d = s->head_dim;
  o->T = s->T; o->H = s->H; o->W = s->W; o->bT = s->bT; o->bH = s->bH; o->bW = s->bW;
  o->nT = s->T / s->bT; o->nH = s->H / s->bH; o->nW = s->W / s->bW;
  o->Nb = o->nT * o->nH * o->nW;
  o->sb = s->bT * s->bH * s->bW;
  o->S = (int)S;
  o->BH = s->B * s->heads;
  o->dtype = s->dtype;
  o->es = s->dtype == VMOBA_BF16 ? 2 : 4;
  o->mask_words = (o->Nb + 31) / 32;
  o->scale = s->softmax_scale > 0.0f ? s->softmax_scale : 1.0f / sqrtf((float)s->head_dim);
  if ((long long)o->BH * o->Nb > (1ll << 24)) return VMOBA_ERR_SHAPE;
  return VMOBA_OK;
}

// Number of SMs of the current device, read once per device and thread (grids of the persistent kernels are
// one CTA per SM; the streaming kernels size theirs as a multiple of it).
inline int sm_count() {
  thread_local int cached_dev = -1, cached_n = 0;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return 1;
  if (dev != cached_dev) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 1;
    cached_dev = dev; cached_n = n;
  }
  return cached_n;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// The debug build (-DVMOBA_DEBUG, lib/libvmoba_debug.so) stands in for a memory checker: every index read from a
// work list is range-checked before it is used (a violation records VMOBA_ERR_BOUNDS in the status word and the
// access goes to element 0 instead: no trap, the kernel carries on), and every slice of a workspace is followed by
// a 256-byte guard zone that is filled with a pattern before the stage's kernels run and verified after them.
#ifdef VMOBA_DEBUG
constexpr size_t kGuardBytes = 256;
#else
constexpr size_t kGuardBytes = 0;
#endif
constexpr uint32_t kGuardWord = 0xC0FFEE5Au;
struct Guards {
  char* base = nullptr;
  size_t off[16] = {};
  int n = 0;
};

// Carves 256-byte aligned slices out of a caller-provided workspace.
struct Carver {
  char* base;
  size_t off = 0;
  Guards guards;
  explicit Carver(void* p) : base(static_cast<char*>(p)) { guards.base = base; }
  template <typename T>
  T* take(size_t n) {
    off = align_up(off, 256);
    T* r = reinterpret_cast<T*>(base ? base + off : nullptr);
    off += n * sizeof(T);
    if (kGuardBytes) {
      off = align_up(off, 256);
      if (guards.n < 16) guards.off[guards.n++] = off;
      off += kGuardBytes;
    }
    return r;
  }
  size_t total() const { return align_up(off, 256); }
};

#define VMOBA_CUDA_OK(expr)                      \
  do {                                           \
    cudaError_t e__ = (expr);                    \
    if (e__ != cudaSuccess) return VMOBA_ERR_CUDA; \
  } while (0)

// Number of kernels this library has launched since it was loaded (reported by
// vmoba_kernel_launches(); benchmarks use it to show that the CUDA path did the work).
inline std::atomic<unsigned long long> g_kernel_launches{0};
inline void count_launches(int n) { g_kernel_launches.fetch_add((unsigned long long)n, std::memory_order_relaxed); }

// Checks the launches issued since the last check; n = how many kernels those were.
#define VMOBA_LAUNCH_OK(n)                                  \
  do {                                                      \
    if (cudaPeekAtLastError() != cudaSuccess) {             \
      cudaGetLastError();                                   \
      return VMOBA_ERR_CUDA;                                \
    }                                                       \
    ::vmoba::count_launches(n);                             \
  } while (0)

// ---------------------------------------------------------------- device helpers
__device__ __forceinline__ void set_status(int32_t* st, int code) {
  if (st) atomicCAS(st, 0, code);
}

// An index read from a work list, about to address one of n elements.
__device__ __forceinline__ int checked_index(int v, int n, int32_t* st) {
#ifdef VMOBA_DEBUG
  if ((unsigned)v >= (unsigned)n) {
    set_status(st, VMOBA_ERR_BOUNDS);
    return 0;
  }
#endif
  return v;
}

#ifdef VMOBA_DEBUG
static __global__ void guard_arm_kernel(Guards g) {
  reinterpret_cast<uint32_t*>(g.base + g.off[blockIdx.x])[threadIdx.x] = kGuardWord;
}
static __global__ void guard_check_kernel(Guards g, int32_t* status) {
  if (reinterpret_cast<const uint32_t*>(g.base + g.off[blockIdx.x])[threadIdx.x] != kGuardWord)
    set_status(status, VMOBA_ERR_BOUNDS);
}
#define VMOBA_GUARDS_ARM(g, st) \
  do { if ((g).n && (g).base) guard_arm_kernel<<<(g).n, (int)(kGuardBytes / 4), 0, st>>>(g); } while (0)
#define VMOBA_GUARDS_CHECK(g, status, st) \
  do { if ((g).n && (g).base) guard_check_kernel<<<(g).n, (int)(kGuardBytes / 4), 0, st>>>(g, status); } while (0)
#else
#define VMOBA_GUARDS_ARM(g, st) do { } while (0)
#define VMOBA_GUARDS_CHECK(g, status, st) do { } while (0)
#endif

template <typename T>
__device__ __forceinline__ float to_f32(T x);
template <>
__device__ __forceinline__ float to_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Load 4 consecutive elements as floats (p must be 4-element aligned).
__device__ __forceinline__ float4 load4(const float* p) { return *reinterpret_cast<const float4*>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  float4 r;
  r.x = __uint_as_float(u.x << 16);
  r.y = __uint_as_float(u.x & 0xffff0000u);
  r.z = __uint_as_float(u.y << 16);
  r.w = __uint_as_float(u.y & 0xffff0000u);
  return r;
}
__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

// Store 4 values and, for bf16 with a residual buffer, the rounding residual bf16(v - bf16(v)).
__device__ __forceinline__ void store4_resid(float* p, float* /*resid*/, float4 v) { store4(p, v); }
__device__ __forceinline__ void store4_resid(__nv_bfloat16* p, __nv_bfloat16* resid, float4 v) {
  // the rounded values are rebuilt from the packed words in registers (no read-back of the row just stored)
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
  if (resid)
    store4(resid, make_float4(v.x - __uint_as_float(u.x << 16), v.y - __uint_as_float(u.x & 0xffff0000u),
                              v.z - __uint_as_float(u.y << 16), v.w - __uint_as_float(u.y & 0xffff0000u)));
}

// Atomic minimum / maximum of fp32 values in global memory (the integer order of the bit patterns agrees with
// the float order for non-negative values and is reversed for negative ones).  The word starts at +inf / -inf.
__device__ __forceinline__ void atomic_min_f32(float* addr, float v) {
  if (!(v < 0.f)) atomicMin(reinterpret_cast<int*>(addr), __float_as_int(v));
  else atomicMax(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}
__device__ __forceinline__ void atomic_max_f32(float* addr, float v) {
  if (!(v < 0.f)) atomicMax(reinterpret_cast<int*>(addr), __float_as_int(v));
  else atomicMin(reinterpret_cast<unsigned int*>(addr), __float_as_uint(v));
}

// Order-preserving map from fp32 to uint32 (larger float <-> larger key).
__device__ __forceinline__ uint32_t float_key(float f) {
  uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(uint32_t k) {
  uint32_t u = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
  return __uint_as_float(u);
}

// Single-CTA exclusive scan of in(0..n-1) (64-bit running total, outputs clamped to int32);
// out[n] receives the total.  Must be called by every thread of the CTA.
template <typename In>
__device__ void block_exclusive_scan(In in, int* __restrict__ out, long long n, long long* total_out) {
  __shared__ long long s_warp[32];
  __shared__ long long s_carry;
  const int t = threadIdx.x, lane = t & 31, warp = t >> 5;
  __syncthreads();
  if (t == 0) s_carry = 0;
  __syncthreads();
  for (long long base = 0; base < n; base += blockDim.x) {
    long long i = base + t;
    long long v = i < n ? (long long)in(i) : 0;
    long long inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      long long x = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += x;
    }
    if (lane == 31) s_warp[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      long long x = lane < (int)(blockDim.x >> 5) ? s_warp[lane] : 0;
      long long xi = x;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        long long y = __shfl_up_sync(0xffffffffu, xi, o);
        if (lane >= o) xi += y;
      }
      s_warp[lane] = xi - x;
    }
    __syncthreads();
    long long excl = s_carry + s_warp[warp] + inc - v;
    if (i < n) out[i] = (int)min(excl, (long long)INT32_MAX);
    __syncthreads();
    if (t == (int)blockDim.x - 1) s_carry = excl + v;
    __syncthreads();
  }
  if (t == 0) {
    out[n] = (int)min(s_carry, (long long)INT32_MAX);
    *total_out = s_carry;
  }
  __syncthreads();
}

// Device counters set through vmoba_debug_wait_profile (null when diagnostics are off).
unsigned long long* debug_wait_profile();

}  // namespace vmoba
