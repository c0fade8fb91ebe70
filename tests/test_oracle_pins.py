"""Pins for the CPU oracle: every oracle function is checked against something other
than its own formula -- the paper's printed block counts, a hand-computed selection
example, closed forms, invariants, brute force on tiny inputs, library routines
(scipy softmax/logsumexp, torch autograd) and finite differences."""
import math
import os

import numpy as np
import pytest
import scipy.special

from oracle import vmoba_oracle as orc
from paper_2506_23858_b200 import inputs as gen


# ---------------------------------------------------------------- partition (Eq. 1)
GRIDS = [
    (4, 8, 8, 1, 8, 8), (4, 8, 8, 4, 2, 4), (4, 8, 8, 2, 4, 2),
    (6, 12, 26, 3, 6, 13), (21, 30, 52, 3, 6, 13), (21, 30, 52, 21, 6, 13), (21, 30, 52, 1, 30, 52),
]


@pytest.mark.parametrize("g", GRIDS)
def test_partition_inverse_restores_order(g):
    perm, inv = orc.partition_perm(*g)
    s = g[0] * g[1] * g[2]
    assert np.array_equal(np.sort(perm), np.arange(s))
    assert np.array_equal(inv[perm], np.arange(s))
    assert np.array_equal(perm[inv], np.arange(s))
    x = np.arange(s * 3, dtype=np.float32).reshape(s, 3)
    assert np.array_equal(orc.partition_invert(orc.partition_apply(x, perm), perm), x)


@pytest.mark.parametrize("g", GRIDS)
def test_partition_matches_reshape_transpose(g):
    """Independent statement of the rearrange: numpy reshape + transpose."""
    T, H, W, bT, bH, bW = g
    ref = (np.arange(T * H * W).reshape(T // bT, bT, H // bH, bH, W // bW, bW)
           .transpose(0, 2, 4, 1, 3, 5).reshape(-1))
    perm, _ = orc.partition_perm(*g)
    assert np.array_equal(perm, ref)


@pytest.mark.parametrize("g", GRIDS)
def test_partition_blocks_are_boxes(g):
    """Brute force: decode (t,h,w) of every token of every block; it must lie in that block's box at its slot."""
    T, H, W, bT, bH, bW = g
    perm, _ = orc.partition_perm(*g)
    nH, nW = H // bH, W // bW
    s_b = bT * bH * bW
    for p in range(0, T * H * W, 7):     # stride keeps the big grids quick; small grids are still covered densely
        r = int(perm[p]); t, h, w = r // (H * W), (r // W) % H, r % W
        j, slot = divmod(p, s_b)
        jt, jh, jw = j // (nH * nW), (j // nW) % nH, j % nW
        assert (t // bT, h // bH, w // bW) == (jt, jh, jw)
        assert slot == ((t % bT) * bH + (h % bH)) * bW + (w % bW)


def test_partition_identity_when_one_temporal_block_is_everything():
    perm, inv = orc.partition_perm(5, 4, 6, 5, 4, 6)
    assert np.array_equal(perm, np.arange(120))
    # 1D partition keeps raster order too (frames are contiguous in raster order)
    perm, _ = orc.partition_perm(6, 4, 6, 2, 4, 6)
    assert np.array_equal(perm, np.arange(144))


def test_partition_3d_neighbour_block_ids():
    """Section 3.2: with a 2x2 spatial grid of 3D blocks, the first block's width, height and
    time neighbours are the 2nd, 3rd and 5th blocks (0-based 1, 2, 4)."""
    T, H, W, bT, bH, bW = 4, 4, 4, 2, 2, 2
    _, inv = orc.partition_perm(T, H, W, bT, bH, bW)
    s_b = bT * bH * bW
    blk = lambda t, h, w: inv[(t * H + h) * W + w] // s_b
    assert blk(0, 0, 0) == 0
    assert blk(0, 0, bW) == 1
    assert blk(0, bH, 0) == 2
    assert blk(bT, 0, 0) == 4


def test_partition_block_counts_of_table4(golden_dir):
    rows = [l.split() for l in open(os.path.join(golden_dir, "table4_block_counts.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 11
    for r in rows:
        T, H, W, bT, bH, bW, n = map(int, r)
        perm, _ = orc.partition_perm(T, H, W, bT, bH, bW)
        s_b = bT * bH * bW
        assert perm.size // s_b == n


def test_partition_rejects_indivisible_grid():
    with pytest.raises(ValueError):
        orc.partition_perm(21, 30, 52, 4, 6, 13)


def test_layer_schedule_cycles_1d_2d_3d():
    sched = [orc.layer_partition(l, 21, 30, 52, 1, (6, 13), (3, 6, 13)) for l in range(6)]
    assert sched[:3] == [(1, 30, 52), (21, 6, 13), (3, 6, 13)]
    assert sched[3:] == sched[:3]


# ---------------------------------------------------------------- centroids (Eq. 2)
def test_centroids_constant_keys():
    k = np.tile(np.array([[0.25, -3.0, 7.5]], dtype=np.float32), (24, 1))
    assert np.array_equal(orc.centroids(k, 4), np.tile(k[:1], (4, 1)))


def test_centroids_mean_of_means_and_unit_blocks():
    rng = np.random.default_rng(3)
    k = rng.standard_normal((60, 5)).astype(np.float32)
    c = orc.centroids(k, 6)
    assert np.allclose(c.astype(np.float64).sum(0) * 10, k.astype(np.float64).sum(0), atol=1e-5)
    assert np.array_equal(orc.centroids(k, 60), k)          # s_b = 1: B = K'
    # explicit loop for one block
    j = 4
    acc = np.zeros(5)
    for t in range(j * 10, (j + 1) * 10):
        acc += k[t].astype(np.float64)
    assert np.allclose(c[j], acc / 10, atol=1e-7)


# ---------------------------------------------------------------- scores
def test_scores_loop_and_linearity():
    rng = np.random.default_rng(4)
    q = rng.standard_normal((7, 6)).astype(np.float32)
    b = rng.standard_normal((3, 6)).astype(np.float32)
    s = orc.block_scores(q, b)
    assert s.shape == (7, 3) and s.dtype == np.float32
    for i in range(7):
        for j in range(3):
            acc = 0.0
            for c in range(6):
                acc += float(q[i, c]) * float(b[j, c])
            assert abs(s[i, j] - acc) < 1e-6
    s2 = orc.block_scores((2 * q).astype(np.float32), b)
    assert np.allclose(s2, 2 * s, atol=1e-6)
    # a transposed operand would give the wrong shape or values here
    assert not np.allclose(s[:3, :3], s[:3, :3].T)


# ---------------------------------------------------------------- selection (Eq. 3, Eq. 4)
def test_select_hand_computed_example(golden_dir):
    sc = np.log(np.array([[8, 1], [4, 2], [1, 1], [2, 2]], dtype=np.float64)).astype(np.float32)
    n = 0
    for line in open(os.path.join(golden_dir, "select_hand_case.txt")):
        if not line.strip() or line.startswith("#"):
            continue
        parts = line.split()
        tau, k, idx = float(parts[0]), int(parts[1]), list(map(int, parts[2:]))
        mask, kk, cutoff = orc.select(sc, tau, 1.0)
        assert kk == k, (tau, kk, k)
        assert sorted(np.nonzero(mask.reshape(-1))[0].tolist()) == idx
        n += 1
    assert n == 9


@pytest.mark.parametrize("tau", [0.1, 0.25, 0.333, 0.5, 0.99])
def test_select_all_equal_scores_closed_form(tau):
    sc = np.full((16, 5), 1.75, dtype=np.float32)
    mask, k, cutoff = orc.select(sc, tau, 0.3)
    P = 80
    # masses are m/P; the first m with m/P >= tau (fp64 cumsum of 1/80 may sit an ulp off at exact multiples)
    assert k in (math.ceil(tau * P - 1e-9), math.ceil(tau * P + 1e-9))
    assert np.array_equal(np.nonzero(mask.reshape(-1))[0], np.arange(k))   # ties -> lowest flat indices
    assert cutoff == np.float32(1.75)


def test_select_one_dominant_pair():
    sc = np.zeros((10, 4), dtype=np.float32)
    sc[6, 2] = 500.0
    for tau in (0.01, 0.5, 0.999):
        mask, k, cutoff = orc.select(sc, tau, 0.1)       # gap 50 in the exponent: the rest has mass ~ 39*e^-50
        assert k == 1 and mask[6, 2] and mask.sum() == 1 and cutoff == np.float32(500.0)


def test_select_two_level_closed_form():
    """n_hi pairs at value a, the rest at 0: mass of the top n <= n_hi is n e^{sa} / (n_hi e^{sa} + P - n_hi)."""
    s_, n_b, n_hi, sigma = 12, 6, 9, 0.5
    a = math.log(5.0) / sigma                     # e^{sigma a} = 5
    rng = np.random.default_rng(0)
    sc = np.zeros(s_ * n_b, dtype=np.float32)
    hi = rng.choice(s_ * n_b, n_hi, replace=False)
    sc[hi] = a
    P = s_ * n_b
    Z = n_hi * 5.0 + (P - n_hi)
    for tau in (0.05, 0.2, 0.4, 0.6, 0.9):
        if tau <= n_hi * 5.0 / Z:
            k_ref = math.ceil(tau * Z / 5.0 - 1e-9)
        else:
            k_ref = n_hi + math.ceil(tau * Z - n_hi * 5.0 - 1e-6)
        mask, k, _ = orc.select(sc.reshape(s_, n_b), tau, sigma)
        assert k == k_ref, (tau, k, k_ref)
        if k <= n_hi:
            assert set(np.nonzero(mask.reshape(-1))[0]) <= set(hi.tolist())
        else:
            assert set(hi.tolist()) <= set(np.nonzero(mask.reshape(-1))[0])


def _brute_force_select(sc, tau, sigma):
    """O(P^2) rank counting, no sort: pair a precedes b if larger score, or equal score and lower index."""
    flat = sc.reshape(-1).astype(np.float64)
    P = flat.size
    x = sigma * flat
    w = np.exp(x - x.max())
    Z = math.fsum(w)
    rank = np.empty(P, dtype=np.int64)
    for a in range(P):
        rank[a] = int(np.sum(flat > flat[a]) + np.sum((flat == flat[a])[:a]))
    mass_upto = np.empty(P)
    for a in range(P):
        mass_upto[a] = math.fsum(w[rank <= rank[a]]) / Z
    k = P
    for r in range(P):
        a = int(np.nonzero(rank == r)[0][0])
        if mass_upto[a] >= tau:
            k = r + 1
            break
    return (rank < k).reshape(sc.shape), k


def test_select_brute_force_on_tiny_config():
    w = gen.C1
    data = gen.make_inputs(w, with_do=False)
    scale = w.head_dim ** -0.5
    for head in range(w.heads):
        perm, _ = orc.partition_perm(w.T, w.H, w.W, *w.block)
        q = data["q"][0, :, head][perm]
        k = data["k"][0, :, head][perm]
        sc = orc.block_scores(q, orc.centroids(k, w.n_blocks))
        mask, kk, cutoff = orc.select(sc, w.tau, scale)
        bmask, bk = _brute_force_select(sc, w.tau, scale)
        assert kk == bk
        assert np.array_equal(mask, bmask)
        assert np.isclose(cutoff, np.sort(sc.reshape(-1))[::-1][kk - 1])


def test_select_invariants():
    rng = np.random.default_rng(11)
    sc = (3.0 * rng.standard_normal((300, 7))).astype(np.float32)
    sigma = 0.4
    P = sc.size
    x = sigma * sc.reshape(-1).astype(np.float64)
    p = np.exp(x - x.max()); p /= p.sum()
    prev = None
    for tau in (0.05, 0.1, 0.25, 0.5, 0.75, 0.9):
        mask, k, cutoff = orc.select(sc, tau, sigma)
        assert mask.sum() == k
        mass = p[mask.reshape(-1)].sum()
        assert mass >= tau - 1e-12                                   # Eq. 4: reaches tau ...
        smallest = p[mask.reshape(-1)].min()
        assert mass - smallest < tau + 1e-12                         # ... and is minimal
        assert k <= math.ceil(tau * P)                               # density never exceeds tau
        assert (sc[mask] >= cutoff).all() and (sc[~mask] <= cutoff).all()
        if prev is not None:
            assert not (prev & ~mask).any()                          # nested in tau
        prev = mask
        # adding a constant to every score changes nothing (softmax shift invariance);
        # 4.0 and these scores are exactly representable sums in fp32 only approximately, so compare masks off-ties
        mask_shift, k_shift, _ = orc.select((sc.astype(np.float64) + 4.0).astype(np.float32), tau, sigma)
        assert abs(k_shift - k) <= 2
        # permuting the queries permutes the mask rows
        pr = rng.permutation(sc.shape[0])
        mask_p, k_p, _ = orc.select(sc[pr], tau, sigma)
        assert k_p == k and np.array_equal(mask_p, mask[pr])
    full, k, _ = orc.select(sc, 1.0, sigma)
    assert k == P and full.all()


def test_select_rejects_bad_tau():
    with pytest.raises(ValueError):
        orc.select(np.zeros((2, 2), np.float32), 0.0, 1.0)
    with pytest.raises(ValueError):
        orc.select(np.zeros((2, 2), np.float32), float("nan"), 1.0)


def test_select_topk_per_query():
    sc = np.array([[1, 5, 3, 3], [0, 0, 0, 0], [9, 8, 7, 6]], dtype=np.float32)
    m = orc.select_topk_per_query(sc, 2)
    assert m.tolist() == [[False, True, True, False], [True, True, False, False], [True, True, False, False]]
    assert orc.select_topk_per_query(sc, 9).all()


def test_select_threshold_per_query_hand_case():
    # one row, sigma = 1: weights e^0, e^-1, e^-2, e^-3 -> probabilities 0.6439, 0.2369, 0.0871, 0.0321
    sc = np.array([[3.0, 2.0, 0.0, 1.0]], dtype=np.float32)
    for tau, want in [(0.5, [1, 0, 0, 0]), (0.6439, [1, 0, 0, 0]), (0.65, [1, 1, 0, 0]), (0.88, [1, 1, 0, 0]),
                      (0.89, [1, 1, 0, 1]), (0.97, [1, 1, 1, 1]), (1.0, [1, 1, 1, 1])]:
        m, k = orc.select_threshold_per_query(sc, tau, 1.0)
        assert m[0].astype(int).tolist() == want, tau
        assert k[0] == sum(want)


def test_select_threshold_per_query_is_the_global_rule_on_one_row():
    # with a single query the head-wide pool IS the row: both rules must agree
    rng = np.random.default_rng(5)
    for _ in range(20):
        sc = rng.normal(size=(1, 37)).astype(np.float32) * 3
        tau = float(rng.uniform(0.05, 0.95))
        m_row, k_row = orc.select_threshold_per_query(sc, tau, 0.7)
        m_pool, k_pool, _ = orc.select(sc, tau, 0.7)
        assert (m_row == m_pool).all() and k_row[0] == k_pool


def test_select_threshold_per_query_rows_are_independent_and_never_empty():
    rng = np.random.default_rng(6)
    sc = rng.normal(size=(9, 12)).astype(np.float32)
    m, k = orc.select_threshold_per_query(sc, 0.3, 2.0)
    assert (m.sum(1) == k).all() and (k >= 1).all()
    for i in range(9):
        mi, _ = orc.select_threshold_per_query(sc[i:i + 1], 0.3, 2.0)
        assert (mi[0] == m[i]).all()
    # ties: equal scores are taken in block order
    m, k = orc.select_threshold_per_query(np.zeros((1, 4), np.float32), 0.5, 1.0)
    assert m[0].tolist() == [True, True, False, False]
    with pytest.raises(ValueError):
        orc.select_threshold_per_query(sc, 0.0, 1.0)


def test_select_rownorm():
    # two queries, sigma = 1.  Row 0 is peaked: softmax (0.9526, 0.0474); row 1 is flat: (0.5, 0.5).
    # Pool probabilities (divided by s = 2): 0.4763, 0.0237, 0.25, 0.25 -> order (0,0), (1,0), (1,1), (0,1)
    sc = np.array([[3.0, 0.0], [7.0, 7.0]], dtype=np.float32)
    for tau, want, k_want in [(0.4, [[1, 0], [0, 0]], 1), (0.5, [[1, 0], [1, 0]], 2), (0.73, [[1, 0], [1, 1]], 3),
                              (0.98, [[1, 1], [1, 1]], 4), (1.0, [[1, 1], [1, 1]], 4)]:
        m, k, cut = orc.select_rownorm(sc, tau, 1.0)
        assert m.astype(int).tolist() == want and k == k_want, tau
    # the raw scores of row 1 (7.0) exceed every score of row 0, yet row 0's peak is taken first:
    # the pool-wide softmax of Eq. 4's other reading would take both 7.0s first
    assert orc.select(sc, 0.4, 1.0)[0].astype(int).tolist() == [[0, 0], [1, 0]]
    # one query: both readings coincide (the row is the pool)
    rng = np.random.default_rng(8)
    row = rng.normal(size=(1, 31)).astype(np.float32) * 2
    for tau in (0.1, 0.5, 0.9):
        assert (orc.select_rownorm(row, tau, 0.6)[0] == orc.select(row, tau, 0.6)[0]).all()
    # rows shifted by constants are normalised away: the mask does not change
    sc = rng.normal(size=(12, 9)).astype(np.float32)
    shift = rng.normal(size=(12, 1)).astype(np.float32) * 8
    a, ka, _ = orc.select_rownorm(sc.astype(np.float64), 0.3, 1.0)
    b, kb, _ = orc.select_rownorm(sc.astype(np.float64) + shift.astype(np.float64), 0.3, 1.0)
    assert (a == b).all() and ka == kb
    # brute force: the kept set is exactly the top-k of p and its mass is the first to reach tau
    x = sc.astype(np.float64)
    p = np.exp(x) / np.exp(x).sum(axis=1, keepdims=True) / 12
    assert p[a].min() >= p[~a].max() and p[a].sum() >= 0.3 and p[a].sum() - p[a].min() < 0.3
    with pytest.raises(ValueError):
        orc.select_rownorm(sc, 0.0, 1.0)


def test_select_topk_global():
    sc = np.array([[1, 5, 3, 3], [0, 0, 0, 0], [9, 8, 7, 6]], dtype=np.float32)
    m, K, cut = orc.select_topk_global(sc, 2)          # budget 6 of 12: 9 8 7 6 5 and the first 3
    assert K == 6 and cut == 3.0
    assert m.astype(int).tolist() == [[0, 1, 1, 0], [0, 0, 0, 0], [1, 1, 1, 1]]
    # one query: the pool is the row, so the rule is the per-query one
    rng = np.random.default_rng(7)
    row = rng.normal(size=(1, 23)).astype(np.float32)
    assert (orc.select_topk_global(row, 5)[0] == orc.select_topk_per_query(row, 5)).all()
    # the budget is capped by the pool
    assert orc.select_topk_global(sc, 99)[0].all()
    # brute force: exactly the K largest values
    sc = rng.normal(size=(6, 7)).astype(np.float32)
    m, K, cut = orc.select_topk_global(sc, 3)
    assert m.sum() == K == 18 and sc[m].min() >= sc[~m].max() and cut == sc[m].min()
    with pytest.raises(ValueError):
        orc.select_topk_global(sc, 0)


# ---------------------------------------------------------------- attention forward
def _rand_head(s, d, seed):
    rng = np.random.default_rng(seed)
    return [rng.standard_normal((s, d)).astype(np.float32) for _ in range(4)]


def test_dense_forward_matches_scipy_softmax():
    q, k, v, _ = _rand_head(40, 8, 5)
    scale = 0.31
    o, lse = orc.dense_attn_fwd(q, k, v, scale)
    z = scale * (q.astype(np.float64) @ k.astype(np.float64).T)
    assert np.allclose(o, scipy.special.softmax(z, axis=1) @ v.astype(np.float64), atol=1e-12)
    assert np.allclose(lse, scipy.special.logsumexp(z, axis=1), atol=1e-12)


def test_dense_forward_online_softmax_coding_agrees():
    """Second, independent coding: one key at a time with a running max."""
    q, k, v, _ = _rand_head(12, 4, 6)
    scale = 0.5
    o, lse = orc.dense_attn_fwd(q, k, v, scale)
    for i in range(12):
        m, l, acc = -math.inf, 0.0, np.zeros(4)
        for t in range(12):
            z = scale * float(np.dot(q[i].astype(np.float64), k[t].astype(np.float64)))
            m_new = max(m, z)
            c = math.exp(m - m_new) if m > -math.inf else 0.0
            l = l * c + math.exp(z - m_new)
            acc = acc * c + math.exp(z - m_new) * v[t].astype(np.float64)
            m = m_new
        assert np.allclose(o[i], acc / l, atol=1e-12)
        assert abs(lse[i] - (m + math.log(l))) < 1e-12


def test_sparse_forward_full_mask_equals_dense():
    q, k, v, _ = _rand_head(48, 8, 7)
    mask = np.ones((48, 6), dtype=bool)
    o, lse = orc.sparse_attn_fwd(q, k, v, mask, 0.35)
    od, lsed = orc.dense_attn_fwd(q, k, v, 0.35)
    assert np.allclose(o, od, atol=1e-12) and np.allclose(lse, lsed, atol=1e-12)


def test_sparse_forward_constant_values_and_empty_rows():
    q, k, v, _ = _rand_head(30, 4, 8)
    v[:] = np.array([1.5, -2.0, 0.25, 8.0], dtype=np.float32)
    rng = np.random.default_rng(1)
    mask = rng.random((30, 5)) < 0.4
    mask[3] = False
    o, lse = orc.sparse_attn_fwd(q, k, v, mask, 0.5)
    for i in range(30):
        if mask[i].any():
            assert np.allclose(o[i], v[0], atol=1e-12)
        else:
            assert np.all(o[i] == 0) and lse[i] == -np.inf


def test_sparse_forward_single_block_and_lse_merge():
    """One selected block = dense attention on that block (scipy); several blocks = LSE-weighted merge."""
    s, d, n_b = 36, 6, 4
    s_b = s // n_b
    q, k, v, _ = _rand_head(s, d, 9)
    scale = 0.4
    rng = np.random.default_rng(2)
    mask = rng.random((s, n_b)) < 0.5
    o, lse = orc.sparse_attn_fwd(q, k, v, mask, scale)
    for i in range(s):
        parts = []
        for j in np.nonzero(mask[i])[0]:
            z = scale * (k[j * s_b:(j + 1) * s_b].astype(np.float64) @ q[i].astype(np.float64))
            parts.append((scipy.special.softmax(z) @ v[j * s_b:(j + 1) * s_b].astype(np.float64),
                          scipy.special.logsumexp(z)))
        if not parts:
            assert lse[i] == -np.inf
            continue
        tot = scipy.special.logsumexp([p[1] for p in parts])
        merged = sum(math.exp(p[1] - tot) * p[0] for p in parts)
        assert np.allclose(o[i], merged, atol=1e-12) and abs(lse[i] - tot) < 1e-12


def test_sparse_forward_row_subset():
    q, k, v, _ = _rand_head(40, 4, 10)
    mask = np.random.default_rng(3).random((40, 5)) < 0.5
    o, lse = orc.sparse_attn_fwd(q, k, v, mask, 0.5)
    rows = [0, 7, 39]
    o2, lse2 = orc.sparse_attn_fwd(q, k, v, mask, 0.5, rows=rows)
    assert np.array_equal(o2, o[rows]) and np.array_equal(lse2, lse[rows])


# ---------------------------------------------------------------- attention backward
def _torch_masked_attention_grads(q, k, v, mask, scale, do):
    import torch
    s_b = q.shape[0] // mask.shape[1]
    tq, tk, tv = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (q, k, v))
    tok_mask = torch.tensor(np.repeat(mask, s_b, axis=1))
    z = scale * tq @ tk.T
    z = z.masked_fill(~tok_mask, float("-inf"))
    nonempty = tok_mask.any(dim=1, keepdim=True)
    z = torch.where(nonempty, z, torch.zeros_like(z))            # avoid NaN rows; zeroed below
    p = torch.softmax(z, dim=1) * nonempty
    o = p @ tv
    o.backward(torch.tensor(do, dtype=torch.float64))
    return o.detach().numpy(), tq.grad.numpy(), tk.grad.numpy(), tv.grad.numpy()


def test_sparse_backward_matches_autograd():
    s, d, n_b = 32, 6, 4
    q, k, v, do = _rand_head(s, d, 12)
    mask = np.random.default_rng(5).random((s, n_b)) < 0.45
    mask[5] = False
    o_t, dq_t, dk_t, dv_t = _torch_masked_attention_grads(q, k, v, mask, 0.4, do)
    o, _ = orc.sparse_attn_fwd(q, k, v, mask, 0.4)
    dq, dk, dv = orc.sparse_attn_bwd(q, k, v, mask, 0.4, do)
    assert np.allclose(o, o_t, atol=1e-12)
    assert np.allclose(dq, dq_t, atol=1e-11) and np.allclose(dk, dk_t, atol=1e-11) and np.allclose(dv, dv_t, atol=1e-11)
    assert np.all(dq[5] == 0)


def test_sparse_backward_finite_differences():
    s, d, n_b = 12, 3, 3
    q, k, v, do = (a.astype(np.float64) for a in _rand_head(s, d, 13))
    mask = np.random.default_rng(6).random((s, n_b)) < 0.6
    scale = 0.7
    loss = lambda q_, k_, v_: float((orc.sparse_attn_fwd(q_, k_, v_, mask, scale)[0] * do).sum())
    dq, dk, dv = orc.sparse_attn_bwd(q, k, v, mask, scale, do)
    eps = 1e-6
    for name, arr, grad in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for (i, c) in [(0, 0), (3, 1), (7, 2), (11, 0)]:
            hi = arr.copy(); hi[i, c] += eps
            lo = arr.copy(); lo[i, c] -= eps
            args_hi = {"q": (hi, k, v), "k": (q, hi, v), "v": (q, k, hi)}[name]
            args_lo = {"q": (lo, k, v), "k": (q, lo, v), "v": (q, k, lo)}[name]
            fd = (loss(*args_hi) - loss(*args_lo)) / (2 * eps)
            assert abs(fd - grad[i, c]) < 1e-7, (name, i, c, fd, grad[i, c])


def test_sparse_backward_key_shift_invariance_and_dense_limit():
    s, d, n_b = 24, 4, 4
    q, k, v, do = _rand_head(s, d, 14)
    mask = np.random.default_rng(7).random((s, n_b)) < 0.5
    # shifting every key by the same vector leaves each row's softmax unchanged: each query's dK contribution sums to 0
    for i in (0, 5, 17):
        _, dk, _ = orc.sparse_attn_bwd(q, k, v, mask, 0.5, do, rows=[i])
        assert np.allclose(dk.sum(0), 0, atol=1e-12)
    full = np.ones((s, n_b), dtype=bool)
    dq, dk, dv = orc.sparse_attn_bwd(q, k, v, full, 0.5, do)
    dq2, dk2, dv2 = orc.dense_attn_bwd(q, k, v, 0.5, do)
    assert np.allclose(dq, dq2, atol=1e-12) and np.allclose(dk, dk2, atol=1e-12) and np.allclose(dv, dv2, atol=1e-12)


def test_sparse_backward_key_block_slice():
    s, d, n_b = 30, 4, 5
    q, k, v, do = _rand_head(s, d, 15)
    mask = np.random.default_rng(8).random((s, n_b)) < 0.5
    _, dk, dv = orc.sparse_attn_bwd(q, k, v, mask, 0.5, do)
    for j in range(n_b):
        dkj, dvj = orc.sparse_attn_bwd_key_block(q, k, v, mask, 0.5, do, j)
        assert np.allclose(dkj, dk[j * 6:(j + 1) * 6], atol=1e-13) and np.allclose(dvj, dv[j * 6:(j + 1) * 6], atol=1e-13)


def test_dense_backward_matches_autograd():
    s, d = 20, 5
    q, k, v, do = _rand_head(s, d, 16)
    _, dq_t, dk_t, dv_t = _torch_masked_attention_grads(q, k, v, np.ones((s, 1), bool), 0.45, do)
    dq, dk, dv = orc.dense_attn_bwd(q, k, v, 0.45, do)
    assert np.allclose(dq, dq_t, atol=1e-11) and np.allclose(dk, dk_t, atol=1e-11) and np.allclose(dv, dv_t, atol=1e-11)


# ---------------------------------------------------------------- whole layer
def test_layer_threshold_one_equals_dense_attention():
    """tau = 1 selects every pair, so the layer must reproduce plain softmax attention in raster order."""
    w = gen.C1
    data = gen.make_inputs(w, with_do=False)
    scale = w.head_dim ** -0.5
    for block in ((1, 8, 8), (4, 2, 4), (2, 4, 2)):
        q, k, v = (data[n][0, :, 1] for n in "qkv")
        out = orc.vmoba_head_forward(q, k, v, (w.T, w.H, w.W), block, 1.0, scale)
        od, lsed = orc.dense_attn_fwd(q, k, v, scale)
        assert out["mask"].all()
        assert np.allclose(out["o"], od, atol=1e-10) and np.allclose(out["lse"], lsed, atol=1e-10)


def test_layer_tiny_config_density_and_empty_rows():
    w = gen.C1
    data = gen.make_inputs(w, with_do=False)
    scale = w.head_dim ** -0.5
    for head in range(w.heads):
        q, k, v = (data[n][0, :, head] for n in "qkv")
        out = orc.vmoba_head_forward(q, k, v, (w.T, w.H, w.W), w.block, w.tau, scale)
        dens = out["mask"].mean()
        assert 0.0 < dens <= w.tau
        assert out["k"] == out["mask"].sum()
        empty = ~out["mask"].any(axis=1)
        assert np.all(out["o_bm"][empty] == 0)


def test_flops_model():
    # dense limit: k_avg = s / s_b blocks per query gives 4 s^2 d + the selection term
    s, d, s_b = 32760, 128, 234
    assert math.isclose(orc.flops_model(s, d, s_b, s / s_b), 4.0 * s * s * d + 2.0 * s * (s / s_b) * d)


# ---------------------------------------------------------------- input generator
def test_generator_bf16_rounding_is_rne_and_seeded():
    import torch
    x = np.random.default_rng(0).standard_normal(4096).astype(np.float32)
    bits = gen.f32_to_bf16_bits(x)
    ref = torch.tensor(x).to(torch.bfloat16)
    assert np.array_equal(bits, ref.view(torch.int16).numpy().view(np.uint16))
    assert np.array_equal(gen.bf16_bits_to_f32(bits), ref.float().numpy())
    w = gen.C2.with_(T=6, H=12, W=26, heads=3)
    a = gen.make_inputs(w)
    b = gen.make_inputs(w, heads=[2])
    assert np.array_equal(a["q_bits"][:, :, 2], b["q_bits"][:, :, 0])
    assert a["q"].shape == (1, 6 * 12 * 26, 3, 128)
    # the smooth field gives q.k locality: a query's own-block centroid scores above the average block
    perm, _ = orc.partition_perm(w.T, w.H, w.W, *w.block)
    q = a["q"][0, :, 0][perm]; k = a["k"][0, :, 0][perm]
    sc = orc.block_scores(q, orc.centroids(k, w.n_blocks))
    own = sc[np.arange(w.S), np.arange(w.S) // w.block_tokens]
    assert own.mean() > sc.mean() + 1.0
