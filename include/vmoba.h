/*
 * vmoba.h -- C ABI of the VMoBA block-sparse attention layer for NVIDIA B200 (sm_100a).
 *
 * VMoBA (Mixture-of-Block Attention for video diffusion models, arXiv 2506.23858)
 * replaces the dense self-attention of a video DiT layer by three steps (Section 3.1):
 *   Step 1  partition the keys of the T x H x W latent grid into 1D / 2D / 3D blocks and
 *           mean-pool each block into a centroid                     (Eq. 1, Eq. 2)
 *   Step 2  score every query token against every centroid and keep, per head, the
 *           globally best (query, key-block) pairs until their normalised similarity
 *           mass reaches a threshold tau                             (Eq. 3, Eq. 4)
 *   Step 3  softmax attention of each query over the keys of its selected blocks only.
 *
 * Conventions shared by every entry point
 *   - All data pointers are DEVICE pointers, 16-byte aligned, owned by the caller.  The
 *     library allocates no device memory and keeps no state between calls; scratch memory
 *     is passed in as `ws` and must hold vmoba_workspace_bytes() bytes.  Two entry points are
 *     exceptions and say so: vmoba_select_static keeps a 16 MiB device array inside the library
 *     image and a per-device cache of its address, and vmoba_debug_wait_profile keeps the pointer
 *     it was given until it is cleared.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work on it and
 *     return; they never synchronise.
 *   - The return value reports errors the host can see (bad arguments, shapes, workspace
 *     size, a failed launch).  Errors that depend on device data (work-list capacity
 *     exceeded, a bounded device-side wait that expired) are written to the int32 word
 *     `dev_status` (first error wins; the caller zeroes it and reads it after
 *     synchronising).  After any error the outputs are unspecified but every access stayed
 *     inside the buffers described here.
 *   - Token order at the boundary is raster (t, h, w), w fastest, S = T*H*W.  "Block-major"
 *     means position p = block * s_b + slot, blocks ordered (nT, nH, nW) with nW fastest and
 *     slots (sT, sH, sW) with sW fastest (Eq. 1).  Block-major tensors are [B, heads, S, head_dim],
 *     contiguous.  G = (b * heads + head) * S + p is the flat query index used by the lists.
 *   - The partition type is implied by the block shape: (bT, H, W) is the 1D temporal
 *     partition, (T, bH, bW) the 2D spatial one, anything else 3D; one index formula covers
 *     all three.  A layer l of the recurrent schedule uses l mod 3 -> 1D, 2D, 3D.
 *   - dtype VMOBA_BF16 runs QK^T and PV on the tensor cores (head_dim 128); VMOBA_F32 is the
 *     fp32 CUDA-core path (head_dim 64 or 128).  Scores, LSE and all selection arithmetic are
 *     fp32 (fp64 for the cumulative mass) for both.
 */
#ifndef VMOBA_H_
#define VMOBA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  VMOBA_OK = 0,
  VMOBA_ERR_ARG = 1,            /* null or misaligned pointer, tau not in (0, 1], bad enum          */
  VMOBA_ERR_SHAPE = 2,          /* non-positive size, grid not divisible by the block, head_dim     */
  VMOBA_ERR_WORKSPACE = 3,      /* ws_bytes smaller than vmoba_workspace_bytes()                    */
  VMOBA_ERR_CAPACITY = 4,       /* (dev_status) more selected pairs than the lists can hold         */
  VMOBA_ERR_TIMEOUT = 5,        /* (dev_status) a bounded device-side wait expired                  */
  VMOBA_ERR_CUDA = 6,           /* a CUDA runtime / driver call failed                              */
  VMOBA_ERR_NOT_IMPLEMENTED = 7,/* combination of dtype / head_dim without a kernel                 */
  VMOBA_ERR_BOUNDS = 8          /* (dev_status, debug build only) an index read from a work list was out of
                                   range, or a guard zone between two slices of the workspace was overwritten */
} vmoba_status;

typedef enum { VMOBA_F32 = 0, VMOBA_BF16 = 1 } vmoba_dtype;

typedef enum {
  VMOBA_STAGE_SCORES = 0,
  VMOBA_STAGE_SELECT = 1,
  VMOBA_STAGE_ATTN_FWD = 2,
  VMOBA_STAGE_ATTN_BWD = 3,
  VMOBA_STAGE_FULL_FWD = 4,
  VMOBA_STAGE_FULL_BWD = 5,
  VMOBA_STAGE_SELECT_ROWNORM = 6   /* vmoba_select_rule_apply with VMOBA_SELECT_THRESHOLD_GLOBAL_ROWNORM */
} vmoba_stage;

typedef struct {
  int32_t B, heads, head_dim; /* head_dim: 64 or 128                                            */
  int32_t T, H, W;            /* latent grid, S = T*H*W                                         */
  int32_t bT, bH, bW;         /* block shape in tokens; must divide T, H, W                     */
  int32_t dtype;              /* vmoba_dtype of q, k, v, o and the gradients                    */
  float softmax_scale;        /* attention scale and selection temperature; 0 => head_dim^-1/2 */
} vmoba_shape;

const char* vmoba_status_string(int status);

/* Number of CUDA kernels this library has launched in this process since it was loaded
 * (bookkeeping for benchmarks; the paper has no counterpart). */
uint64_t vmoba_kernel_launches(void);

/* Bytes of scratch `ws` a stage needs.  `capacity` is the number of (query, key-block) pairs
 * the work lists can hold (the q_idx_capacity given to vmoba_select); stages that do not
 * depend on it ignore it.  Returns 0 for an invalid shape or stage. */
size_t vmoba_workspace_bytes(const vmoba_shape* shape, int stage, int64_t capacity);

/*
 * Step 1, Eq. 1: reorder tokens into blocks (inverse = 0) or back (inverse = 1).
 *   raster : [B, S, heads, head_dim] addressed by element strides raster_strides_bsh =
 *            {batch, token, head}; head_dim is contiguous; strides must keep rows 16-byte aligned.
 *   bm     : block-major [B, heads, S, head_dim], contiguous.
 * inverse = 0 reads raster and writes bm; inverse = 1 reads bm and writes raster.
 * perm_or_null / inv_perm_or_null: optional int32 [S] outputs, perm[p] = raster index of the
 * token at block-major position p, inv_perm its inverse.
 */
int vmoba_partition(const vmoba_shape* shape, int inverse, const void* src, void* dst,
                    const int64_t raster_strides_bsh[3], int32_t* perm_or_null,
                    int32_t* inv_perm_or_null, void* stream);

/*
 * Step 1 + Step 2a, Eq. 2 and the similarity map of Section 3.3:
 *   centroids [B, heads, N_b, head_dim] fp32 = mean of each key block,
 *   scores    [B, heads, S, N_b]       fp32 = q . centroid, unscaled.
 * q_bm, k_bm are block-major.
 */
int vmoba_block_scores(const vmoba_shape* shape, const void* q_bm, const void* k_bm,
                       float* centroids, float* scores, int32_t* dev_status, void* ws, size_t ws_bytes,
                       void* stream);

/*
 * vmoba_block_scores that also hands over what the selection's first pass would look for: score_range
 * [B*heads][2] fp32 receives the smallest and the largest score of each head's pool, taken in the epilogue of
 * the scores kernel while the values are still in registers (Eq. 4's normalisation is relative to the pool's
 * largest score, and the cutoff search starts from the pool's range).  Give it to vmoba_select_ranged.
 */
int vmoba_block_scores_range(const vmoba_shape* shape, const void* q_bm, const void* k_bm, float* centroids,
                             float* scores, float* score_range, int32_t* dev_status, void* ws, size_t ws_bytes,
                             void* stream);

/*
 * Step 2b, Eq. 3 + Eq. 4: global threshold selection per (batch, head).
 * The head's S*N_b scores are normalised with a softmax at temperature softmax_scale over the
 * whole pool; pairs are taken in descending score order until the cumulative mass is >= tau
 * (tau >= 1 selects everything).  Every pair whose score is >= the score of the last pair
 * taken is selected (exact ties at the cutoff are all kept).
 * Outputs
 *   mask_bits        uint32 [B*heads*S, ceil(N_b/32)]  bit j of a row = block j selected by that query
 *   kb_ptr           int32  [B*heads*N_b + 1]          CSR offsets by (batch, head, key block) into q_idx
 *   q_idx            int32  [capacity]                 per key block: the in-head positions p (ascending) of
 *                                                      the queries that selected it
 *   q_ptr            int32  [B*heads*S + 1]            CSR offsets by flat query G into q_pairs
 *   q_pairs          int32  [capacity]                 per query: positions in q_idx of its pairs, by ascending block
 *   k_per_head       int64  [B*heads]                  number of selected pairs
 *   cutoff_per_head  float  [B*heads]                  score of the last pair taken
 * dev_status gets VMOBA_ERR_CAPACITY if the total exceeds `capacity` (lists are then truncated).
 */
int vmoba_select(const vmoba_shape* shape, const float* scores, float tau, uint32_t* mask_bits,
                 int32_t* kb_ptr, int32_t* q_idx, int32_t* q_ptr, int32_t* q_pairs,
                 int64_t capacity, int64_t* k_per_head, float* cutoff_per_head,
                 int32_t* dev_status, void* ws, size_t ws_bytes, void* stream);

/*
 * The block-choice variants of Table 3b ("Block choice design ablation") and of the training-free
 * setting of Table 4 / Appendix A ("Local + TopK"): the same outputs as vmoba_select, chosen by
 *   VMOBA_SELECT_THRESHOLD_GLOBAL  the method's own rule; identical to vmoba_select(tau)
 *   VMOBA_SELECT_TOPK_GLOBAL       head-wide pool of Eq. 3, fixed budget: the K = min(topk * S, S * N_b)
 *                                  best pairs of the head (every pair tied with the K-th is kept)
 *   VMOBA_SELECT_THRESHOLD_LOCAL   Eq. 4 applied to each query on its own: softmax of its N_b scores at
 *                                  temperature softmax_scale, blocks in descending order until the
 *                                  cumulative mass is >= tau; ties in block order; never an empty row
 *   VMOBA_SELECT_TOPK_LOCAL        each query keeps its min(topk, N_b) best blocks (the MoBA rule);
 *                                  ties in block order; exactly that many per query
 * tau in (0, 1] is read by the threshold modes, topk >= 1 by the top-k modes.  The local modes need
 * N_b <= 1024 (VMOBA_ERR_SHAPE otherwise).  cutoff_per_head receives the score of the last pair taken
 * (global modes) or the smallest score selected in the head (local modes).  Workspace:
 * vmoba_workspace_bytes(shape, VMOBA_STAGE_SELECT, 0), as for vmoba_select.
 */
typedef enum {
  VMOBA_SELECT_THRESHOLD_GLOBAL = 0,
  VMOBA_SELECT_TOPK_GLOBAL = 1,
  VMOBA_SELECT_THRESHOLD_LOCAL = 2,
  VMOBA_SELECT_TOPK_LOCAL = 3,
  /* the method's own rule under the other reading of "normalized similarity scores" (Eq. 4): each
   * query's scores are normalised by a softmax over its own N_b blocks, then pooled over the head
   * (divided by S) and taken in descending order of that probability until the sum reaches tau.
   * cutoff_per_head receives softmax_scale * score - logsumexp(row) of the last pair taken.  Needs
   * the larger workspace vmoba_workspace_bytes(shape, VMOBA_STAGE_SELECT_ROWNORM, 0). */
  VMOBA_SELECT_THRESHOLD_GLOBAL_ROWNORM = 4,
  /* may be OR-ed into any rule: every query also keeps the key block it lies in (the convention of
   * MoBA, which always attends the current block), so that the head-wide rules leave no query
   * without a block.  The paper's own rule does not do this; it is an option, off by default. */
  VMOBA_SELECT_KEEP_OWN_BLOCK = 0x100
} vmoba_select_rule;

int vmoba_select_rule_apply(const vmoba_shape* shape, const float* scores, int32_t rule, float tau, int32_t topk,
                            uint32_t* mask_bits, int32_t* kb_ptr, int32_t* q_idx, int32_t* q_ptr,
                            int32_t* q_pairs, int64_t capacity, int64_t* k_per_head, float* cutoff_per_head,
                            int32_t* dev_status, void* ws, size_t ws_bytes, void* stream);

/*
 * vmoba_select_rule_apply for a caller that already knows each head's score range (score_range [B*heads][2] =
 * minimum, maximum, exactly as vmoba_block_scores_range wrote them for these scores): the head-wide rules then
 * skip their own pass over the score matrix that looks for it (one traversal fewer).  The results are
 * those of vmoba_select_rule_apply bit for bit.  A range that does not bound the scores gives an unspecified
 * selection (every access still stays inside the buffers).  The per-query rules and the row-normalised rule
 * ignore the range.
 */
int vmoba_select_ranged(const vmoba_shape* shape, const float* scores, const float* score_range, int32_t rule, float tau,
                        int32_t topk, uint32_t* mask_bits, int32_t* kb_ptr, int32_t* q_idx, int32_t* q_ptr,
                        int32_t* q_pairs, int64_t capacity, int64_t* k_per_head, float* cutoff_per_head,
                        int32_t* dev_status, void* ws, size_t ws_bytes, void* stream);

/*
 * vmoba_select for callers that cannot hand over scratch memory.  (The paper has no counterpart:
 * this is a packaging variant of the selection stage, not a step of the method.)
 *
 * Who needs it: code that runs where allocating device memory is not possible or not allowed --
 * a plug-in inside a memory-planned inference engine that only receives its input and output
 * buffers, or a serving loop in which cudaMalloc (it synchronises the whole device) is banned.
 * Same arguments and results as vmoba_select minus `ws`: the scratch is a fixed
 * vmoba_select_static_scratch_bytes() = 16 MiB array inside the library image, which every GPU
 * that loads the library keeps resident until the process exits.
 *   - Shapes whose vmoba_workspace_bytes(shape, VMOBA_STAGE_SELECT, 0) fits that size run exactly
 *     as vmoba_select does.  The last slice of that workspace is an optional side list (the larger of
 *     4096 and S * N_b / 32 floats per (batch, head)) that saves the cutoff search one pass over the
 *     scores; a shape that fits only without it still runs, one pass slower, with the same results.
 *     Shapes that do not fit even so are rejected with VMOBA_ERR_WORKSPACE; use vmoba_select with
 *     your own buffer for those.
 *   - The call allocates nothing (no cudaMalloc / cudaFree, no allocating library routine).
 *   - The first call on each device looks up the array's device address (one
 *     cudaGetSymbolAddress, with that device current); make that first call outside of any stream
 *     capture.  Later calls on the device reuse the address.  The address cache is filled without a
 *     lock: two host threads that make the first call on one device at the same time both look the
 *     address up and store the same value.
 *   - The current device must be the device of `stream` and of every buffer: the address that is
 *     used is the current device's copy of the array.
 *   - All calls on one device share the one array.  Every call re-initialises what it needs, so
 *     stale contents are harmless, but two calls whose kernels can overlap on the GPU (different
 *     streams, no ordering between them) race on it: serialise them.
 */
size_t vmoba_select_static_scratch_bytes(void);
int vmoba_select_static(const vmoba_shape* shape, const float* scores, float tau, uint32_t* mask_bits,
                        int32_t* kb_ptr, int32_t* q_idx, int32_t* q_ptr, int32_t* q_pairs,
                        int64_t capacity, int64_t* k_per_head, float* cutoff_per_head,
                        int32_t* dev_status, void* stream);

/*
 * Step 3: attention of every query over the keys of its selected blocks.
 *   o_bm [B, heads, S, head_dim] (dtype), lse [B*heads*S] fp32 natural-log sum-exp of the scaled logits.
 * A query with no selected block gets o = 0 and lse = -inf.
 * o_resid_or_null (bf16 only, same shape as o_bm): if given, receives the rounding residual
 * bf16(o_exact - o_bm).  The backward needs rowsum(dO * O) to better than bf16 accuracy of O
 * (taken from the rounded output alone, dQ loses about 6e-3 relative accuracy); training
 * callers keep this tensor with o_bm and lse for vmoba_attn_bwd.
 * `capacity` is the one given to vmoba_select (bounds the per-pair partial results in ws: for bf16 with
 * head_dim 128 a row of fp16 values with a power-of-two scale per row, else an fp32 row).
 */
int vmoba_attn_fwd(const vmoba_shape* shape, const void* q_bm, const void* k_bm, const void* v_bm,
                   const int32_t* kb_ptr, const int32_t* q_idx, const int32_t* q_ptr,
                   const int32_t* q_pairs, int64_t capacity, void* o_bm, void* o_resid_or_null,
                   float* lse, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream);

/*
 * The same forward with the inverse of Eq. 1 folded into the kernels that write o: o is written in RASTER order,
 * [B, S, heads, head_dim] addressed by element strides o_strides_bsh = {batch, token, head} (head_dim contiguous,
 * every stride a multiple of 16 bytes), the row of block-major position p being token perm[p] (perm: device int32
 * [S], as produced by vmoba_partition).  Saves the inverse partition pass of o.  The rounding residual, if asked
 * for, stays block-major (it only feeds vmoba_attn_bwd*), as does lse.  bf16 with head_dim 128 only
 * (VMOBA_ERR_NOT_IMPLEMENTED otherwise); everything else as for vmoba_attn_fwd.
 */
int vmoba_attn_fwd_raster(const vmoba_shape* shape, const void* q_bm, const void* k_bm, const void* v_bm,
                          const int32_t* kb_ptr, const int32_t* q_idx, const int32_t* q_ptr, const int32_t* q_pairs,
                          int64_t capacity, void* o, const int64_t o_strides_bsh[3], const int32_t* perm,
                          void* o_resid_bm_or_null, float* lse, int32_t* dev_status, void* ws, size_t ws_bytes,
                          void* stream);

/*
 * Training backward of Step 3 with the selection held constant (TopkMask has zero gradient):
 * dq, dk, dv [B, heads, S, head_dim] (dtype) from do_bm, the forward's o_bm (+ o_resid) and lse.
 * Queries without a selected block get dq = 0.  The paper states no gradient formula; this is
 * the softmax-attention gradient restricted to the selected pairs.  `capacity` is the one given
 * to vmoba_select (list positions at or beyond it are never read).
 */
int vmoba_attn_bwd(const vmoba_shape* shape, const void* q_bm, const void* k_bm, const void* v_bm,
                   const void* o_bm, const void* o_resid_or_null, const float* lse, const void* do_bm,
                   const int32_t* kb_ptr,
                   const int32_t* q_idx, const int32_t* q_ptr, int64_t capacity, void* dq_bm, void* dk_bm,
                   void* dv_bm, int32_t* dev_status, void* ws, size_t ws_bytes, void* stream);

/*
 * The same backward with Eq. 1 and its inverse folded into the kernels that read o and dO and write the gradients:
 * o and d_o are read and dq, dk, dv are written in RASTER order, [B, S, heads, head_dim] addressed by element
 * strides {batch, token, head} (o_strides_bsh for o, do_strides_bsh for d_o, grad_strides_bsh for the three
 * gradients; head_dim contiguous, every stride a multiple of 16 bytes), the row of block-major position p being
 * token perm[p] (perm: device int32 [S], as produced by vmoba_partition).  o_strides_bsh and do_strides_bsh may
 * each be NULL: that tensor is then block-major like the other inputs (o_resid always is).  Saves the three inverse partition passes of a training step and, with a raster d_o, the
 * partition pass of dO (its gathered reads from raster order cost more than that pass when the head count is
 * large: see the design notes).  The other inputs, the workspace and the errors are those of vmoba_attn_bwd; bf16
 * with head_dim 128 only (VMOBA_ERR_NOT_IMPLEMENTED otherwise).
 */
int vmoba_attn_bwd_raster(const vmoba_shape* shape, const void* q_bm, const void* k_bm, const void* v_bm,
                          const void* o, const int64_t o_strides_bsh[3], const void* o_resid_or_null, const float* lse,
                          const void* d_o, const int64_t do_strides_bsh[3], const int32_t* kb_ptr, const int32_t* q_idx,
                          const int32_t* q_ptr, int64_t capacity, void* dq, void* dk, void* dv,
                          const int64_t grad_strides_bsh[3], const int32_t* perm, int32_t* dev_status, void* ws,
                          size_t ws_bytes, void* stream);

/*
 * Dense softmax attention over all S keys: the tau = 1 limit of the layer and the speed-up
 * denominator (the "Full Attention" baseline of Section 4.1).  Tensors are [B, heads, S, head_dim]
 * in any one token order.  If do_or_null is given, also computes dq, dk, dv.
 */
int vmoba_full_attn(const vmoba_shape* shape, const void* q, const void* k, const void* v, void* o,
                    float* lse, const void* do_or_null, void* dq, void* dk, void* dv,
                    int32_t* dev_status, void* ws, size_t ws_bytes, void* stream);

/*
 * Diagnostics; not part of the method.  Registers a device buffer of 16 uint64 counters (NULL: clears the
 * registration) into which the tensor-core attention kernels launched afterwards ADD, per CTA, the clock
 * cycles that one representative thread of each warp role spent in each section of its loop; divide by the
 * grid size (one CTA per SM) for cycles per CTA.  The caller zeroes the buffer before a launch, reads it after
 * synchronising, and keeps it alive until it is cleared here.  Process-wide, not thread-safe; kernels run a
 * little slower while a buffer is registered, and their results do not change.
 *   forward kernel:  [0] softmax thread waiting for scores, [1] score read + row maximum, [2] accumulator
 *     rescale, [3] exponentials + P written, [4] epilogue (wait for the last P V, normalise, write), [6] its
 *     total; MMA warp: [8] wait for Q, [9] for K, [10] for P, [11] for V, [12] for a free accumulator,
 *     [13] issuing, [14] its total.
 *   backward kernel: [0] TMA warp waiting for free K / V buffers; [1] the TMA warp's total plus the writer
 *     warp's staging and reductions (one slot); MMA warp: [2] wait for K / V, [3] for a gathered chunk, [4] for
 *     P^T / dS^T, [5] for free accumulators or the dQ^T buffer, [6] its total; loaders: [7] wait for a free
 *     chunk, [8] total; compute warps: [10] wait for a chunk, [11] for S^T / dP^T, [12] for the dK / dV hand-off,
 *     [13] total; writer warp: [9] wait for dQ^T, [14] reading it from TMEM, [15] waiting at the staging barrier.
 */
void vmoba_debug_wait_profile(void* dev_counters16);

/*
 * Diagnostics; not part of the method.  Exercises the failure path of the kernels' bounded device-side waits
 * without starving a real kernel: one CTA waits on a barrier that nothing arrives at, with a limit of `polls`
 * polls (1 .. 65536; the attention kernels use 2^22).  The wait gives up, dev_status receives
 * VMOBA_ERR_TIMEOUT (if it was 0), the CTA's later waits give up after a few polls and the kernel ends by itself.
 * out2_or_null (device int32 [2]) receives the number of waits that gave up (128: two per thread) and a 1 written
 * by the kernel's last instruction.
 */
int vmoba_debug_wait_timeout(int32_t* dev_status, uint32_t polls, int32_t* out2_or_null, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* VMOBA_H_ */
