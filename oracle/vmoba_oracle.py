"""CPU oracle for the VMoBA block-sparse attention layer (arXiv 2506.23858).

TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the smoke check and
the benchmark's CPU-baseline leg may import this module.  It shares nothing with
the CUDA path and never imports it.

Everything here is plain numpy, written to be checked against the paper by eye:
fp32 values in (inputs, centroids and scores are *stored* in fp32, as the layer
stores them), fp64 arithmetic inside, one head at a time, one query at a time
where the definition is per query.  numpy's matmul / sort / cumsum serve as
steps; there is no tiling, fusion or reordering.

Notation follows the paper: a latent grid of T x H x W tokens (s = T*H*W), key
blocks of (s^T, s^H, s^W) tokens, N_b blocks of s_b tokens, centroids B,
similarity S_hat = q b^T, threshold tau, mask M.

Every function below is pinned by tests that do not re-use its own formula
(closed forms, invariants, brute force, finite differences, textbook special
cases); none is "parity unpinned".

Readings of the paper where it is silent (each is the documented choice of this
build, listed with its alternatives in the design notes):
  * "normalized similarity" (Section 3.4, the sentence before Eq. 4) = softmax of
    sigma * S_hat over the whole head's pool of s*N_b pairs, sigma = the
    attention's softmax scale;
  * the comparison in Eq. 4 is ">= tau"; tau >= 1, or a cumulative sum that never
    reaches tau in floating point, selects every pair;
  * ties in the descending order are broken by ascending flat index q*N_b + j;
  * a query that selected no block outputs 0 with LSE = -inf and receives and
    contributes zero gradient;
  * no gradient flows through centroids, scores or the mask (TopkMask is
    piecewise constant).
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------------------
# Step 1a: block partition (Eq. 1)
# --------------------------------------------------------------------------------------
def partition_perm(T, H, W, bT, bH, bW):
    """Eq. 1: the rearrange (nT sT)(nH sH)(nW sW) -> (nT nH nW)(sT sH sW).

    The three partition types are one formula: 1D is (bT, H, W), 2D is (T, bH, bW),
    3D is (bT, bH, bW).  Returns (perm, inv_perm), int32 arrays of length s:
    perm[p] is the raster index (t*H + h)*W + w of the token that sits at
    block-major position p = block*s_b + slot; inv_perm is its inverse.
    Block order is (nT, nH, nW) with nW fastest, slot order (sT, sH, sW) with sW
    fastest (Section 3.2: the first 3D block's width/height/time neighbours are
    the 2nd, 3rd and 5th blocks of a 2x2 spatial grid).
    """
    if min(T, H, W, bT, bH, bW) <= 0 or T % bT or H % bH or W % bW:
        raise ValueError("grid must be positive and divisible by the block shape")
    nT, nH, nW = T // bT, H // bH, W // bW
    s_b = bT * bH * bW
    s = T * H * W
    perm = np.empty(s, dtype=np.int32)
    for t in range(T):
        for h in range(H):
            for w in range(W):
                block = ((t // bT) * nH + (h // bH)) * nW + (w // bW)
                slot = ((t % bT) * bH + (h % bH)) * bW + (w % bW)
                perm[block * s_b + slot] = (t * H + h) * W + w
    inv_perm = np.empty(s, dtype=np.int32)
    inv_perm[perm] = np.arange(s, dtype=np.int32)
    return perm, inv_perm


def partition_apply(x, perm):
    """K' = rearrange(K): x is [s, d] in raster order; returns block-major [s, d]."""
    return x[perm]


def partition_invert(x_bm, perm):
    """Inverse rearrange: block-major [s, d] back to raster order."""
    out = np.empty_like(x_bm)
    out[perm] = x_bm
    return out


def layer_partition(layer, T, H, W, block_1d, block_2d, block_3d):
    """Layer-wise recurrent schedule (Eq. 1's case split): layer l uses l mod 3 -> 1D, 2D, 3D.

    block_1d = s^T; block_2d = (s^H, s^W); block_3d = (s^T, s^H, s^W).
    Returns the (bT, bH, bW) block shape of that layer (0-based layer index).
    """
    m = layer % 3
    if m == 0:
        return (block_1d, H, W)
    if m == 1:
        return (T, block_2d[0], block_2d[1])
    return tuple(block_3d)


# --------------------------------------------------------------------------------------
# Step 1b: mean key blocks (Eq. 2)
# --------------------------------------------------------------------------------------
def centroids(k_bm, n_blocks):
    """Eq. 2: B = mean(K') over the s_b tokens of each block.  k_bm: [s, d] block-major fp32.

    Sum in fp64, result stored in fp32: [N_b, d].
    """
    s, d = k_bm.shape
    s_b = s // n_blocks
    assert s_b * n_blocks == s
    kb = k_bm.astype(np.float64).reshape(n_blocks, s_b, d)
    return (kb.sum(axis=1) / s_b).astype(np.float32)


# --------------------------------------------------------------------------------------
# Step 2: similarity map, global + threshold selection (Eq. 3, Eq. 4)
# --------------------------------------------------------------------------------------
def block_scores(q, cent):
    """S_hat = q b^T (Section 3.3): q [s, d] fp32, cent [N_b, d] fp32 -> [s, N_b] fp32 (fp64 sums), unscaled."""
    return (q.astype(np.float64) @ cent.astype(np.float64).T).astype(np.float32)


def select(scores, tau, sigma):
    """Eq. 3 + Eq. 4 for one head.

    scores: S_hat [s, N_b] fp32.  The pool is all P = s*N_b pairs of the head.
      1. normalise: w = exp(sigma*S_hat - max), p = w / sum(w)   (fp64)
      2. sort pairs by S_hat descending (ties: ascending flat index)
      3. c_m = cumulative sum of the sorted p;  k = min{m : c_m >= tau}
         (tau >= 1 or never reached -> k = P)
      4. M = 1 on the first k pairs of that order (TopkMask).
    Returns (mask [s, N_b] bool, k, cutoff) where cutoff is the fp32 score of the k-th pair.
    """
    if not (tau > 0.0):
        raise ValueError("tau must be in (0, 1]")
    s, n_b = scores.shape
    flat = scores.reshape(-1)
    P = flat.size
    order = np.argsort(-flat.astype(np.float64), kind="stable")   # descending, ties by flat index
    if tau >= 1.0:
        k = P
    else:
        x = sigma * flat.astype(np.float64)
        w = np.exp(x - x.max())
        p = w / w.sum()
        c = np.cumsum(p[order])
        hit = np.nonzero(c >= tau)[0]
        k = int(hit[0]) + 1 if hit.size else P
    mask = np.zeros(P, dtype=bool)
    mask[order[:k]] = True
    cutoff = np.float32(flat[order[k - 1]])
    return mask.reshape(s, n_b), k, cutoff


def select_topk_per_query(scores, k):
    """Per-query ("local") top-k selection, the MoBA-style rule the paper uses for its
    training-free runs (Appendix A, Table 4): each query keeps its k best blocks
    (ties: lower block index first)."""
    s, n_b = scores.shape
    k = min(k, n_b)
    order = np.argsort(-scores.astype(np.float64), axis=1, kind="stable")
    mask = np.zeros((s, n_b), dtype=bool)
    np.put_along_axis(mask, order[:, :k], True, axis=1)
    return mask


def select_threshold_per_query(scores, tau, sigma):
    """"threshold + local" of the block-choice ablation (Table 3b): the cumulative-similarity rule of
    Eq. 4 applied to each query on its own instead of to the head-wide pool.

    For query i: p_ij = softmax_j(sigma * S_hat_ij) over its N_b blocks (fp64), blocks ordered by
    S_hat descending (ties: lower block index first), k_i = min{m : sum of the first m p >= tau}
    (tau >= 1 or never reached -> N_b); the first k_i blocks are kept.  Every query keeps at least
    one block.  Returns (mask [s, N_b] bool, k [s] int).
    """
    if not (tau > 0.0):
        raise ValueError("tau must be in (0, 1]")
    s, n_b = scores.shape
    mask = np.zeros((s, n_b), dtype=bool)
    ks = np.zeros(s, dtype=np.int64)
    for i in range(s):
        row = scores[i].astype(np.float64)
        order = np.argsort(-row, kind="stable")
        if tau >= 1.0:
            k = n_b
        else:
            x = sigma * row
            w = np.exp(x - x.max())
            p = w / w.sum()
            c = np.cumsum(p[order])
            hit = np.nonzero(c >= tau)[0]
            k = int(hit[0]) + 1 if hit.size else n_b
        mask[i, order[:k]] = True
        ks[i] = k
    return mask, ks


def select_rownorm(scores, tau, sigma):
    """Eq. 3 + Eq. 4 under the other reading of "normalized similarity scores": each query's scores
    are normalised on their own, p_ij = softmax_j(sigma * S_hat_ij) / s (fp64; the head's pool then
    sums to one), the pool is ordered by p descending (ties: ascending flat index) and pairs are
    taken until the cumulative p reaches tau (tau >= 1 or never reached: all).  Unlike the pool-wide
    softmax this is not a single raw-score cutoff per head: a query with a flat row needs a higher
    raw score than a query with a peaked one.
    Returns (mask [s, N_b] bool, k, cutoff) with cutoff = ln(s * p) of the last pair taken, i.e.
    sigma * S_hat minus the row's log-sum-exp.
    """
    if not (tau > 0.0):
        raise ValueError("tau must be in (0, 1]")
    s, n_b = scores.shape
    x = sigma * scores.astype(np.float64)
    m = x.max(axis=1, keepdims=True)
    lse = m + np.log(np.exp(x - m).sum(axis=1, keepdims=True))
    logp = (x - lse).reshape(-1)                      # ln(s * p)
    P = logp.size
    order = np.argsort(-logp, kind="stable")
    if tau >= 1.0:
        k = P
    else:
        c = np.cumsum(np.exp(logp[order]) / s)
        hit = np.nonzero(c >= tau)[0]
        k = int(hit[0]) + 1 if hit.size else P
    mask = np.zeros(P, dtype=bool)
    mask[order[:k]] = True
    return mask.reshape(s, n_b), k, float(logp[order[k - 1]])


def select_topk_global(scores, k):
    """"topk + global" of the block-choice ablation (Table 3b): the head-wide pool of Eq. 3 with a
    fixed budget instead of the threshold of Eq. 4.  The budget is the one "topk + local" spends,
    K = k * s pairs per head (capped at the pool size); the K best pairs of the head are kept
    (ties: ascending flat index).  Returns (mask [s, N_b] bool, K, cutoff = fp32 score of the K-th pair).
    """
    if k < 1:
        raise ValueError("k must be positive")
    s, n_b = scores.shape
    flat = scores.reshape(-1)
    K = min(k * s, flat.size)
    order = np.argsort(-flat.astype(np.float64), kind="stable")
    mask = np.zeros(flat.size, dtype=bool)
    mask[order[:K]] = True
    return mask.reshape(s, n_b), K, np.float32(flat[order[K - 1]])


# --------------------------------------------------------------------------------------
# Step 3: attention over the selected blocks (Section 3.1, Step 3) and its gradient
# --------------------------------------------------------------------------------------
def _row_keys(mask_row, s_b):
    """Block-major key positions of the blocks a query selected."""
    blocks = np.nonzero(mask_row)[0]
    if blocks.size == 0:
        return np.empty(0, dtype=np.int64)
    return (blocks[:, None] * s_b + np.arange(s_b)[None, :]).reshape(-1)


def sparse_attn_fwd(q, k, v, mask, scale, rows=None):
    """Each query attends only to the keys/values of its selected blocks.

    q, k, v: [s, d] block-major fp32 (one head); mask [s, N_b] bool (query-major);
    rows: optional list of query positions to evaluate (rows are independent).
    For query i with key set K_i: z_t = scale * q_i.k_t, m = max z, l = sum exp(z - m),
    o_i = sum exp(z_t - m) v_t / l, LSE_i = m + ln l.  Empty K_i: o_i = 0, LSE_i = -inf.
    Returns (o [n_rows, d] fp64, lse [n_rows] fp64).
    """
    s, d = q.shape
    n_b = mask.shape[1]
    s_b = s // n_b
    rows = np.arange(s) if rows is None else np.asarray(rows)
    k64 = k.astype(np.float64)
    v64 = v.astype(np.float64)
    o = np.zeros((rows.size, d), dtype=np.float64)
    lse = np.full(rows.size, -np.inf, dtype=np.float64)
    for n, i in enumerate(rows):
        keys = _row_keys(mask[i], s_b)
        if keys.size == 0:
            continue
        z = scale * (k64[keys] @ q[i].astype(np.float64))
        m = z.max()
        w = np.exp(z - m)
        l = w.sum()
        o[n] = (w @ v64[keys]) / l
        lse[n] = m + np.log(l)
    return o, lse


def sparse_attn_bwd(q, k, v, mask, scale, do, rows=None):
    """Gradient of sparse_attn_fwd with the mask held constant.

    For query i over its key set: P_t = exp(z_t - LSE_i); dV_t += P_t dO_i;
    dP_t = dO_i.v_t; D_i = dO_i.o_i; dS_t = P_t (dP_t - D_i);
    dQ_i = scale * sum_t dS_t k_t;  dK_t += scale * dS_t q_i.
    rows: optional subset of queries (dQ rows are exact for those queries; dK/dV
    then hold only those queries' contributions).
    Returns (dq [n_rows, d], dk [s, d], dv [s, d]) in fp64.
    """
    s, d = q.shape
    n_b = mask.shape[1]
    s_b = s // n_b
    rows = np.arange(s) if rows is None else np.asarray(rows)
    q64, k64, v64, do64 = (a.astype(np.float64) for a in (q, k, v, do))
    dq = np.zeros((rows.size, d), dtype=np.float64)
    dk = np.zeros((s, d), dtype=np.float64)
    dv = np.zeros((s, d), dtype=np.float64)
    for n, i in enumerate(rows):
        keys = _row_keys(mask[i], s_b)
        if keys.size == 0:
            continue
        z = scale * (k64[keys] @ q64[i])
        m = z.max()
        w = np.exp(z - m)
        p = w / w.sum()
        o = p @ v64[keys]
        dp = v64[keys] @ do64[i]
        D = do64[i] @ o
        ds = p * (dp - D)
        dq[n] = scale * (ds @ k64[keys])
        dk[keys] += scale * ds[:, None] * q64[i][None, :]
        dv[keys] += p[:, None] * do64[i][None, :]
    return dq, dk, dv


def sparse_attn_bwd_key_block(q, k, v, mask, scale, do, block):
    """Exact dK, dV rows of one key block: only the queries that selected `block`
    contribute to it, so the full gradient of that block needs just those queries.
    Returns (dk [s_b, d], dv [s_b, d]) fp64."""
    s, d = q.shape
    n_b = mask.shape[1]
    s_b = s // n_b
    rows = np.nonzero(mask[:, block])[0]
    _, dk, dv = sparse_attn_bwd(q, k, v, mask, scale, do, rows=rows)
    sl = slice(block * s_b, (block + 1) * s_b)
    return dk[sl], dv[sl]


def dense_attn_fwd(q, k, v, scale, rows=None):
    """Plain softmax attention (the tau = 1 limit), one row at a time, three-pass softmax."""
    s, d = q.shape
    rows = np.arange(s) if rows is None else np.asarray(rows)
    k64 = k.astype(np.float64)
    v64 = v.astype(np.float64)
    o = np.empty((rows.size, d), dtype=np.float64)
    lse = np.empty(rows.size, dtype=np.float64)
    for n, i in enumerate(rows):
        z = scale * (k64 @ q[i].astype(np.float64))
        m = z.max()
        w = np.exp(z - m)
        l = w.sum()
        o[n] = (w @ v64) / l
        lse[n] = m + np.log(l)
    return o, lse


def dense_attn_bwd(q, k, v, scale, do):
    """Textbook softmax-attention gradient in matrix form (all rows, fp64)."""
    q64, k64, v64, do64 = (a.astype(np.float64) for a in (q, k, v, do))
    z = scale * (q64 @ k64.T)
    z -= z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    o = p @ v64
    dv = p.T @ do64
    dp = do64 @ v64.T
    D = (do64 * o).sum(axis=1, keepdims=True)
    ds = p * (dp - D)
    dq = scale * (ds @ k64)
    dk = scale * (ds.T @ q64)
    return dq, dk, dv


# --------------------------------------------------------------------------------------
# The whole layer for one head, raster order in, raster order out
# --------------------------------------------------------------------------------------
def vmoba_head_forward(q, k, v, grid, block, tau, scale, sigma=None):
    """One head of one VMoBA layer: q, k, v [s, d] fp32 in raster order.

    Returns a dict with perm, centroids, scores, mask, k, cutoff, o (raster order,
    fp64) and lse (raster order)."""
    T, H, W = grid
    sigma = scale if sigma is None else sigma
    perm, inv_perm = partition_perm(T, H, W, *block)
    n_b = (T // block[0]) * (H // block[1]) * (W // block[2])
    q_bm, k_bm, v_bm = q[perm], k[perm], v[perm]
    cent = centroids(k_bm, n_b)
    sc = block_scores(q_bm, cent)
    mask, kk, cutoff = select(sc, tau, sigma)
    o_bm, lse_bm = sparse_attn_fwd(q_bm, k_bm, v_bm, mask, scale)
    return dict(perm=perm, inv_perm=inv_perm, centroids=cent, scores=sc, mask=mask, k=kk,
                cutoff=cutoff, o_bm=o_bm, lse_bm=lse_bm,
                o=partition_invert(o_bm, perm), lse=partition_invert(lse_bm[:, None], perm)[:, 0])


def flops_model(s, d, s_b, k_avg):
    """Section 3.1's estimate, O(s d (s / s_b + k_avg s_b)), with its constants made
    explicit (2 flops per multiply-add; QK^T and PV in the attention term):
    selection 2*s*(s/s_b)*d, attention 4*s*k_avg*s_b*d."""
    return 2.0 * s * (s / s_b) * d + 4.0 * s * k_avg * s_b * d
