// Entry points of Step 3 of VMoBA (attention over the selected blocks), its training
// backward and the dense tau = 1 path: argument checks, workspace carving and kernel dispatch.
#include <algorithm>

#include "attn_simt.cuh"
#include "common.cuh"

namespace vmoba {

size_t select_ws_bytes(const Dims& D);   // select.cu
size_t select_rownorm_ws_bytes(const Dims& D);
size_t scores_ws_bytes(const Dims& D);   // scores.cu

// attn_tc_fwd.cu: tensor-core forward kernel (bf16, head_dim 128)
int tc_sparse_fwd(const Dims& D, const void* q, const void* k, const void* v, const int* kb_ptr, const int* q_idx,
                  const int* q_ptr, const int* q_pairs, long long cap, void* o, void* o_resid, float* lse,
                  int32_t* status, int* item_ptr, int* item_tab, long long max_items, float* part_o, float* part_lse,
                  float* part_scale, cudaStream_t st, const RowMap& o_map);
int tc_dense_fwd(const Dims& D, const void* q, const void* k, const void* v, void* o, void* o_resid, float* lse,
                 int32_t* status, cudaStream_t st);

// attn_tc_bwd.cu: tensor-core backward kernels (bf16, head_dim 128)
int tc_sparse_bwd(const Dims& D, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                  const float* Dv, const int* kb_ptr, const int* q_idx, long long cap, float* dq_acc, void* dk, void* dv,
                  int32_t* status, cudaStream_t st, const RowMap& out_map, const RowMap& do_map);
int tc_dense_bwd(const Dims& D, const void* q, const void* k, const void* v, const void* d_o, const float* lse,
                 const float* Dv, void* dq, void* dk, void* dv, int32_t* status, cudaStream_t st);

static bool use_tensor_cores(const Dims& D) { return D.dtype == VMOBA_BF16 && D.d == 128; }

static long long max_items_128(const Dims& D, long long cap) { return cap / 128 + (long long)D.BH * D.Nb + 1; }

struct FwdWs { int* item_ptr; int* item_tab; float* part_o; float* part_lse; float* part_scale; size_t bytes; Guards guards; };
static FwdWs carve_fwd(const Dims& D, long long cap, void* ws) {
  Carver c(ws);
  FwdWs w;
  w.item_ptr = c.take<int>((size_t)D.BH * D.Nb + 1);
  w.item_tab = c.take<int>(4 * (size_t)max_items_128(D, cap));   // one int per item, or a 16-byte descriptor
  w.part_lse = c.take<float>((size_t)cap);
  w.part_scale = c.take<float>((size_t)cap);     // per partial row: the power of two its fp16 values are scaled by
  // fp32 rows on the CUDA-core path, fp16 rows (scaled per row) on the tensor-core path
  w.part_o = c.take<float>((size_t)cap * D.d / (use_tensor_cores(D) ? 2 : 1));
  w.bytes = c.total();
  w.guards = c.guards;
  return w;
}

struct BwdWs { int* item_ptr; int* item_tab; float* Dv; float* dq_acc; void* o_resid; size_t bytes; Guards guards; };
static BwdWs carve_bwd(const Dims& D, bool dense, void* ws, long long cap = 0) {
  Carver c(ws);
  BwdWs w;
  w.item_ptr = c.take<int>((size_t)D.BH * D.Nb + 1);
  w.item_tab = dense ? nullptr : c.take<int>((size_t)max_items_128(D, cap));
  w.Dv = c.take<float>((size_t)D.BH * D.S);
  w.dq_acc = dense ? nullptr : c.take<float>((size_t)D.BH * D.S * D.d);
  w.o_resid = (dense && D.dtype == VMOBA_BF16) ? c.take<__nv_bfloat16>((size_t)D.BH * D.S * D.d) : nullptr;
  w.bytes = c.total();
  w.guards = c.guards;
  return w;
}

static int grid_for(long long items, int per_sm) {
  long long g = std::min<long long>(items, (long long)sm_count() * per_sm);
  return (int)std::max<long long>(g, 1);
}

template <typename T, int DH>
static int simt_sparse_fwd(const Dims& D, const void* q, const void* k, const void* v, const int* kb_ptr,
                           const int* q_idx, const int* q_ptr, const int* q_pairs, long long cap, void* o,
                           void* o_resid, float* lse, int32_t* status, void* ws, cudaStream_t st) {
  FwdWs w = carve_fwd(D, cap, ws);
  VMOBA_GUARDS_ARM(w.guards, st);
  const long long n_kb = (long long)D.BH * D.Nb;
  simt::item_ptr_kernel<<<1, 1024, 0, st>>>(kb_ptr, n_kb, simt::kRows, cap, w.item_ptr);
  long long max_items = cap / simt::kRows + n_kb;
  simt::attn_fwd_kernel<T, DH, false><<<grid_for(max_items, 8), simt::kThreads, 0, st>>>(
      (const T*)q, (const T*)k, (const T*)v, kb_ptr, q_idx, q_ptr, w.item_ptr, (int)n_kb, D.S, D.Nb, D.sb, D.BH,
      D.scale, (T*)o, (T*)o_resid, lse, w.part_o, w.part_lse, cap);
  long long nq = (long long)D.BH * D.S;
  simt::merge_kernel<T, DH, float><<<grid_for((nq + 7) / 8, 16), 256, 0, st>>>(
      q_ptr, q_pairs, nq, w.part_o, w.part_lse, cap, (T*)o, (T*)o_resid, lse);
  VMOBA_LAUNCH_OK(3);
  VMOBA_GUARDS_CHECK(w.guards, status, st);
  return VMOBA_OK;
}

template <typename T, int DH>
static int simt_sparse_bwd(const Dims& D, const void* q, const void* k, const void* v, const void* o,
                           const void* o_resid, const float* lse, const void* d_o, const int* kb_ptr, const int* q_idx,
                           const int* q_ptr, long long cap, void* dq, void* dk, void* dv, int32_t* status, void* ws,
                           cudaStream_t st, const RowMap& out_map, const RowMap& do_map, const RowMap& o_map) {
  // raster-order o / dO / gradients (perm set) are handled by the tensor-core kernels only
  if ((out_map.perm || do_map.perm || o_map.perm) && !use_tensor_cores(D)) return VMOBA_ERR_NOT_IMPLEMENTED;
  BwdWs w = carve_bwd(D, false, ws, cap);
  VMOBA_GUARDS_ARM(w.guards, st);
  const long long n_kb = (long long)D.BH * D.Nb;
  const long long nq = (long long)D.BH * D.S;
  if (use_tensor_cores(D)) {
    // the backward kernel adds every dQ contribution into the fp32 accumulator: the row-dot pass also clears the
    // rows of all selecting queries; they are converted afterwards (rows of queries without a block become zero)
    const int min_nb = 1;
    simt::rowdot_kernel<T, DH><<<grid_for((nq + 7) / 8, 16), 256, 0, st>>>(
        (const T*)o, (const T*)o_resid, (const T*)d_o, nq, w.Dv, do_map, o_map, w.dq_acc, q_ptr);
    count_launches(1);
    int rc = tc_sparse_bwd(D, q, k, v, d_o, lse, w.Dv, kb_ptr, q_idx, cap, w.dq_acc, dk, dv, status, st, out_map, do_map);
    if (rc) return rc;
    simt::cast_rows_kernel<T, DH><<<grid_for((nq + 7) / 8, 16), 256, 0, st>>>(w.dq_acc, (T*)dq, q_ptr, nq, 1, min_nb, out_map);
    VMOBA_LAUNCH_OK(1);
    VMOBA_GUARDS_CHECK(w.guards, status, st);
    return VMOBA_OK;
  }
  simt::rowdot_kernel<T, DH><<<grid_for((nq + 7) / 8, 16), 256, 0, st>>>((const T*)o, (const T*)o_resid,
                                                                        (const T*)d_o, nq, w.Dv, do_map);
  count_launches(1);
  VMOBA_CUDA_OK(cudaMemsetAsync(w.dq_acc, 0, (size_t)nq * DH * sizeof(float), st));
  simt::item_ptr_kernel<<<1, 1024, 0, st>>>(kb_ptr, n_kb, simt::kRows, cap, w.item_ptr);
  long long tiles = (D.sb + simt::kRows - 1) / simt::kRows;
  simt::attn_bwd_dkdv_kernel<T, DH, false><<<grid_for(n_kb * tiles, 4), simt::kThreads, 0, st>>>(
      (const T*)q, (const T*)k, (const T*)v, (const T*)d_o, lse, w.Dv, kb_ptr, q_idx, D.S, D.Nb, D.sb, D.BH,
      D.scale, cap, (T*)dk, (T*)dv);
  simt::attn_bwd_dq_kernel<T, DH, false><<<grid_for(nq / simt::kRows * D.Nb + n_kb, 4), simt::kThreads, 0, st>>>(
      (const T*)q, (const T*)k, (const T*)v, (const T*)d_o, lse, w.Dv, kb_ptr, q_idx, w.item_ptr, (int)n_kb, D.S,
      D.Nb, D.sb, D.BH, D.scale, cap, w.dq_acc, (T*)dq);
  simt::cast_kernel<T><<<grid_for((nq * DH / 4 + 255) / 256, 16), 256, 0, st>>>(w.dq_acc, (T*)dq, nq * DH / 4);
  VMOBA_LAUNCH_OK(4);
  VMOBA_GUARDS_CHECK(w.guards, status, st);
  return VMOBA_OK;
}

template <typename T, int DH>
static int simt_dense(const Dims& D, const void* q, const void* k, const void* v, void* o, float* lse,
                      const void* d_o, void* dq, void* dk, void* dv, void* ws, int32_t* status, cudaStream_t st) {
  const long long nq = (long long)D.BH * D.S;
  const long long tiles = (D.S + simt::kRows - 1) / simt::kRows;
  BwdWs w = carve_bwd(D, true, d_o ? ws : nullptr);
  if (use_tensor_cores(D)) {
    int rc = tc_dense_fwd(D, q, k, v, o, d_o ? w.o_resid : nullptr, lse, status, st);
    if (rc) return rc;
  } else {
    simt::attn_fwd_kernel<T, DH, true><<<grid_for(D.BH * tiles, 8), simt::kThreads, 0, st>>>(
        (const T*)q, (const T*)k, (const T*)v, nullptr, nullptr, nullptr, nullptr, 0, D.S, 1, D.S, D.BH, D.scale,
        (T*)o, d_o ? (T*)w.o_resid : nullptr, lse, nullptr, nullptr, 0);
    count_launches(1);
  }
  if (d_o) {
    simt::rowdot_kernel<T, DH><<<grid_for((nq + 7) / 8, 16), 256, 0, st>>>((const T*)o, (const T*)w.o_resid,
                                                                          (const T*)d_o, nq, w.Dv);
    if (use_tensor_cores(D)) {
      VMOBA_LAUNCH_OK(1);
      return tc_dense_bwd(D, q, k, v, d_o, lse, w.Dv, dq, dk, dv, status, st);
    }
    simt::attn_bwd_dkdv_kernel<T, DH, true><<<grid_for(D.BH * tiles, 4), simt::kThreads, 0, st>>>(
        (const T*)q, (const T*)k, (const T*)v, (const T*)d_o, lse, w.Dv, nullptr, nullptr, D.S, 1, D.S, D.BH,
        D.scale, 0, (T*)dk, (T*)dv);
    simt::attn_bwd_dq_kernel<T, DH, true><<<grid_for(D.BH * tiles, 4), simt::kThreads, 0, st>>>(
        (const T*)q, (const T*)k, (const T*)v, (const T*)d_o, lse, w.Dv, nullptr, nullptr, nullptr, 0, D.S, 1, D.S,
        D.BH, D.scale, 0, nullptr, (T*)dq);
  }
  VMOBA_LAUNCH_OK(d_o ? 3 : 0);
  return VMOBA_OK;
}

#define VMOBA_DISPATCH(FN, ...)                                                        \
  do {                                                                                 \
    if (D.dtype == VMOBA_BF16) {                                                       \
      if (D.d == 128) return FN<__nv_bfloat16, 128>(__VA_ARGS__);                      \
      return FN<__nv_bfloat16, 64>(__VA_ARGS__);                                       \
    }                                                                                  \
    if (D.d == 128) return FN<float, 128>(__VA_ARGS__);                                \
    return FN<float, 64>(__VA_ARGS__);                                                 \
  } while (0)

}  // namespace vmoba

using namespace vmoba;

extern "C" const char* vmoba_status_string(int status) {
  switch (status) {
    case VMOBA_OK: return "ok";
    case VMOBA_ERR_ARG: return "invalid argument";
    case VMOBA_ERR_SHAPE: return "invalid shape";
    case VMOBA_ERR_WORKSPACE: return "workspace too small";
    case VMOBA_ERR_CAPACITY: return "work-list capacity exceeded";
    case VMOBA_ERR_TIMEOUT: return "device-side wait timed out";
    case VMOBA_ERR_CUDA: return "CUDA error";
    case VMOBA_ERR_NOT_IMPLEMENTED: return "not implemented";
    case VMOBA_ERR_BOUNDS: return "index out of range or workspace guard overwritten (debug build)";
    default: return "unknown status";
  }
}

extern "C" uint64_t vmoba_kernel_launches(void) { return g_kernel_launches.load(std::memory_order_relaxed); }

extern "C" size_t vmoba_workspace_bytes(const vmoba_shape* shape, int stage, int64_t capacity) {
  Dims D;
  if (make_dims(shape, &D)) return 0;
  if (capacity < 0) return 0;
  switch (stage) {
    case VMOBA_STAGE_SCORES: return scores_ws_bytes(D);
    case VMOBA_STAGE_SELECT: return select_ws_bytes(D);
    case VMOBA_STAGE_SELECT_ROWNORM: return select_rownorm_ws_bytes(D);
    case VMOBA_STAGE_ATTN_FWD: return carve_fwd(D, capacity, nullptr).bytes;
    case VMOBA_STAGE_ATTN_BWD: return carve_bwd(D, false, nullptr, capacity).bytes;
    case VMOBA_STAGE_FULL_FWD: return 256;
    case VMOBA_STAGE_FULL_BWD: return carve_bwd(D, true, nullptr).bytes;
    default: return 0;
  }
}

extern "C" int vmoba_attn_fwd(const vmoba_shape* shape, const void* q_bm, const void* k_bm, const void* v_bm,
                              const int32_t* kb_ptr, const int32_t* q_idx, const int32_t* q_ptr,
                              const int32_t* q_pairs, int64_t capacity, void* o_bm, void* o_resid_or_null,
                              float* lse, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  Dims D;
  int rc = make_dims(shape, &D);
  if (rc) return rc;
  if (!q_bm || !k_bm || !v_bm || !kb_ptr || !q_idx || !q_ptr || !q_pairs || !o_bm || !lse || !dev_status || !ws)
    return VMOBA_ERR_ARG;
  if (!aligned16(q_bm) || !aligned16(k_bm) || !aligned16(v_bm) || !aligned16(o_bm) || !aligned16(ws) ||
      !aligned16(o_resid_or_null))
    return VMOBA_ERR_ARG;
  if (capacity <= 0 || capacity > (int64_t)INT32_MAX) return VMOBA_ERR_ARG;
  if (ws_bytes < carve_fwd(D, capacity, nullptr).bytes) return VMOBA_ERR_WORKSPACE;
  if (D.dtype != VMOBA_BF16) o_resid_or_null = nullptr;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (use_tensor_cores(D)) {
    FwdWs w = carve_fwd(D, capacity, ws);
    VMOBA_GUARDS_ARM(w.guards, st);
    rc = tc_sparse_fwd(D, q_bm, k_bm, v_bm, kb_ptr, q_idx, q_ptr, q_pairs, capacity, o_bm, o_resid_or_null, lse,
                       dev_status, w.item_ptr, w.item_tab, max_items_128(D, capacity), w.part_o, w.part_lse, w.part_scale, st,
                       RowMap());
    VMOBA_GUARDS_CHECK(w.guards, dev_status, st);
    return rc;
  }
  VMOBA_DISPATCH(simt_sparse_fwd, D, q_bm, k_bm, v_bm, kb_ptr, q_idx, q_ptr, q_pairs, capacity, o_bm, o_resid_or_null,
                 lse, dev_status, ws, st);
}

extern "C" int vmoba_attn_bwd(const vmoba_shape* shape, const void* q_bm, const void* k_bm, const void* v_bm,
                              const void* o_bm, const void* o_resid_or_null, const float* lse, const void* do_bm,
                              const int32_t* kb_ptr,
                              const int32_t* q_idx, const int32_t* q_ptr, int64_t capacity, void* dq_bm, void* dk_bm,
                              void* dv_bm, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  Dims D;
  int rc = make_dims(shape, &D);
  if (rc) return rc;
  if (!q_bm || !k_bm || !v_bm || !o_bm || !lse || !do_bm || !kb_ptr || !q_idx || !q_ptr || !dq_bm || !dk_bm ||
      !dv_bm || !dev_status || !ws)
    return VMOBA_ERR_ARG;
  if (!aligned16(q_bm) || !aligned16(k_bm) || !aligned16(v_bm) || !aligned16(o_bm) || !aligned16(do_bm) ||
      !aligned16(dq_bm) || !aligned16(dk_bm) || !aligned16(dv_bm) || !aligned16(ws))
    return VMOBA_ERR_ARG;
  if (capacity <= 0 || capacity > (int64_t)INT32_MAX) return VMOBA_ERR_ARG;
  if (ws_bytes < carve_bwd(D, false, nullptr, capacity).bytes) return VMOBA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (D.dtype != VMOBA_BF16) o_resid_or_null = nullptr;
  if (!aligned16(o_resid_or_null)) return VMOBA_ERR_ARG;
  VMOBA_DISPATCH(simt_sparse_bwd, D, q_bm, k_bm, v_bm, o_bm, o_resid_or_null, lse, do_bm, kb_ptr, q_idx, q_ptr,
                 capacity, dq_bm, dk_bm, dv_bm, dev_status, ws, st, RowMap(), RowMap(), RowMap());
}

extern "C" int vmoba_attn_fwd_raster(const vmoba_shape* shape, const void* q_bm, const void* k_bm, const void* v_bm,
                                     const int32_t* kb_ptr, const int32_t* q_idx, const int32_t* q_ptr,
                                     const int32_t* q_pairs, int64_t capacity, void* o, const int64_t o_strides_bsh[3],
                                     const int32_t* perm, void* o_resid_bm_or_null, float* lse, int32_t* dev_status,
                                     void* ws, size_t ws_bytes, void* stream) {
  Dims D;
  int rc = make_dims(shape, &D);
  if (rc) return rc;
  if (!q_bm || !k_bm || !v_bm || !kb_ptr || !q_idx || !q_ptr || !q_pairs || !o || !o_strides_bsh || !perm || !lse ||
      !dev_status || !ws)
    return VMOBA_ERR_ARG;
  if (!aligned16(q_bm) || !aligned16(k_bm) || !aligned16(v_bm) || !aligned16(o) || !aligned16(ws) ||
      !aligned16(o_resid_bm_or_null))
    return VMOBA_ERR_ARG;
  for (int i = 0; i < 3; ++i)
    if (o_strides_bsh[i] < 0 || o_strides_bsh[i] % (16 / D.es)) return VMOBA_ERR_ARG;     // rows stay 16-byte aligned
  if (capacity <= 0 || capacity > (int64_t)INT32_MAX) return VMOBA_ERR_ARG;
  if (ws_bytes < carve_fwd(D, capacity, nullptr).bytes) return VMOBA_ERR_WORKSPACE;
  if (!use_tensor_cores(D)) return VMOBA_ERR_NOT_IMPLEMENTED;
  RowMap o_map;
  o_map.perm = perm; o_map.heads = D.heads; o_map.S = D.S;
  o_map.sb = o_strides_bsh[0]; o_map.st = o_strides_bsh[1]; o_map.sh = o_strides_bsh[2];
  FwdWs w = carve_fwd(D, capacity, ws);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  VMOBA_GUARDS_ARM(w.guards, st);
  rc = tc_sparse_fwd(D, q_bm, k_bm, v_bm, kb_ptr, q_idx, q_ptr, q_pairs, capacity, o, o_resid_bm_or_null, lse,
                     dev_status, w.item_ptr, w.item_tab, max_items_128(D, capacity), w.part_o, w.part_lse, w.part_scale, st,
                     o_map);
  VMOBA_GUARDS_CHECK(w.guards, dev_status, st);
  return rc;
}

extern "C" int vmoba_attn_bwd_raster(const vmoba_shape* shape, const void* q_bm, const void* k_bm, const void* v_bm,
                                     const void* o_bm, const int64_t o_strides_bsh[3], const void* o_resid_or_null,
                                     const float* lse, const void* d_o, const int64_t do_strides_bsh[3],
                                     const int32_t* kb_ptr,
                                     const int32_t* q_idx, const int32_t* q_ptr, int64_t capacity, void* dq, void* dk,
                                     void* dv, const int64_t grad_strides_bsh[3], const int32_t* perm,
                                     int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  Dims D;
  int rc = make_dims(shape, &D);
  if (rc) return rc;
  if (!q_bm || !k_bm || !v_bm || !o_bm || !lse || !d_o || !kb_ptr || !q_idx || !q_ptr || !dq || !dk || !dv ||
      !grad_strides_bsh || !perm || !dev_status || !ws)
    return VMOBA_ERR_ARG;
  if (!aligned16(q_bm) || !aligned16(k_bm) || !aligned16(v_bm) || !aligned16(o_bm) || !aligned16(d_o) ||
      !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(ws))
    return VMOBA_ERR_ARG;
  // rows must stay 16-byte aligned
  const int per16 = 16 / D.es;
  for (int i = 0; i < 3; ++i) {
    if (grad_strides_bsh[i] < 0 || grad_strides_bsh[i] % per16) return VMOBA_ERR_ARG;
    if (do_strides_bsh && (do_strides_bsh[i] < 0 || do_strides_bsh[i] % per16)) return VMOBA_ERR_ARG;
    if (o_strides_bsh && (o_strides_bsh[i] < 0 || o_strides_bsh[i] % per16)) return VMOBA_ERR_ARG;
  }
  if (capacity <= 0 || capacity > (int64_t)INT32_MAX) return VMOBA_ERR_ARG;
  if (ws_bytes < carve_bwd(D, false, nullptr, capacity).bytes) return VMOBA_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (D.dtype != VMOBA_BF16) o_resid_or_null = nullptr;
  if (!aligned16(o_resid_or_null)) return VMOBA_ERR_ARG;
  RowMap out_map, do_map, o_map;
  out_map.perm = perm;
  out_map.heads = do_map.heads = o_map.heads = D.heads;
  out_map.S = do_map.S = o_map.S = D.S;
  if (o_strides_bsh) {      // else o is block-major
    o_map.perm = perm;
    o_map.sb = o_strides_bsh[0]; o_map.st = o_strides_bsh[1]; o_map.sh = o_strides_bsh[2];
  }
  out_map.sb = grad_strides_bsh[0]; out_map.st = grad_strides_bsh[1]; out_map.sh = grad_strides_bsh[2];
  if (do_strides_bsh) {     // else d_o is block-major
    do_map.perm = perm;
    do_map.sb = do_strides_bsh[0]; do_map.st = do_strides_bsh[1]; do_map.sh = do_strides_bsh[2];
  }
  VMOBA_DISPATCH(simt_sparse_bwd, D, q_bm, k_bm, v_bm, o_bm, o_resid_or_null, lse, d_o, kb_ptr, q_idx, q_ptr,
                 capacity, dq, dk, dv, dev_status, ws, st, out_map, do_map, o_map);
}

extern "C" int vmoba_full_attn(const vmoba_shape* shape, const void* q, const void* k, const void* v, void* o,
                               float* lse, const void* do_or_null, void* dq, void* dk, void* dv,
                               int32_t* dev_status, void* ws, size_t ws_bytes, void* stream) {
  Dims D;
  int rc = make_dims(shape, &D);
  if (rc) return rc;
  if (!q || !k || !v || !o || !lse || !dev_status) return VMOBA_ERR_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return VMOBA_ERR_ARG;
  if (do_or_null) {
    if (!dq || !dk || !dv || !ws) return VMOBA_ERR_ARG;
    if (!aligned16(do_or_null) || !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(ws))
      return VMOBA_ERR_ARG;
    if (ws_bytes < carve_bwd(D, true, nullptr).bytes) return VMOBA_ERR_WORKSPACE;
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  VMOBA_DISPATCH(simt_dense, D, q, k, v, o, lse, do_or_null, dq, dk, dv, ws, dev_status, st);
}
