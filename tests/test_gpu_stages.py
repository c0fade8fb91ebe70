"""Stage-isolated parity: each CUDA stage is fed the ORACLE's output of the previous stage and
compared element by element with the oracle's output of that stage.  All calls go through the
C-ABI library."""
import numpy as np
import pytest
import torch

from oracle import vmoba_oracle as orc
from paper_2506_23858_b200 import binding as vb
from paper_2506_23858_b200 import inputs as gen
from paper_2506_23858_b200.layer import VmobaLayer, lists_from_mask
from tests import _util as U

pytestmark = pytest.mark.gpu

# Mid-size cases: 1872 tokens (29.25 tiles of 64, 14.6 tiles of 128), several block geometries
# (1 to 15 mask words), both dtypes, both head dims, batch 2.
MID = gen.Workload("mid", 1, 2, 128, 6, 12, 26, (3, 6, 13), 0.25, "bf16", "smooth", 5)
CASES = [
    gen.C1,
    gen.C1.with_(name="c1_3d", block=(2, 4, 2)),
    gen.C1.with_(name="c1_d128", head_dim=128, block=(4, 2, 4)),
    MID,
    MID.with_(name="mid_1d", block=(1, 12, 26)),
    MID.with_(name="mid_2d", block=(6, 6, 13), B=2),
    MID.with_(name="mid_48blk", block=(1, 3, 13)),
    MID.with_(name="mid_468blk", block=(1, 2, 2), tau=0.1),
    MID.with_(name="mid_f32", dtype="f32", head_dim=64, block=(2, 6, 13)),
    MID.with_(name="mid_bf16_d64", head_dim=64, block=(3, 4, 13)),
]
IDS = [c.name for c in CASES]


def _oracle_front(w, data):
    """Oracle partition, centroids, scores, selection for every (b, head)."""
    perm, inv = orc.partition_perm(w.T, w.H, w.W, *w.block)
    scale = w.head_dim ** -0.5
    out = dict(perm=perm, inv=inv, scale=scale, heads=[])
    for b in range(w.B):
        for h in range(w.heads):
            q, k, v = (data[n][b, :, h][perm] for n in "qkv")
            cent = orc.centroids(k, w.n_blocks)
            sc = orc.block_scores(q, cent)
            mask, kk, cutoff = orc.select(sc, w.tau, scale)
            out["heads"].append(dict(q=q, k=k, v=v, cent=cent, scores=sc, mask=mask, k_sel=kk, cutoff=cutoff))
    return out


_cache = {}


def _prep(w):
    if w.name not in _cache:
        data = gen.make_inputs(w)
        _cache[w.name] = (data, _oracle_front(w, data))
    return _cache[w.name]


@pytest.mark.parametrize("w", CASES, ids=IDS)
def test_partition_bit_exact_and_inverse(w):
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    L = VmobaLayer(shape, capacity=1024)
    x = U.to_device(w, data, "q")
    perm = torch.empty(w.S, dtype=torch.int32, device="cuda")
    inv = torch.empty(w.S, dtype=torch.int32, device="cuda")
    L.partition(x, L.q_bm, perm=perm, inv_perm=inv)
    assert np.array_equal(perm.cpu().numpy(), ora["perm"])
    assert np.array_equal(inv.cpu().numpy(), ora["inv"])
    got = L.q_bm.view(torch.int16 if w.dtype == "bf16" else torch.int32).cpu().numpy()
    src = x.view(torch.int16 if w.dtype == "bf16" else torch.int32).cpu().numpy()
    ref = np.ascontiguousarray(src[:, ora["perm"]].transpose(0, 2, 1, 3))
    assert np.array_equal(got, ref)
    back = torch.zeros_like(x)
    L.partition(back, L.q_bm, inverse=True)
    assert torch.equal(back.view(torch.int16 if w.dtype == "bf16" else torch.int32),
                       x.view(torch.int16 if w.dtype == "bf16" else torch.int32))


def test_partition_strided_raster_view():
    """q, k, v often live interleaved in one [B, S, 3, heads, d] projection output."""
    w = MID
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    L = VmobaLayer(shape, capacity=1024)
    qkv = torch.stack([U.to_device(w, data, n) for n in "qkv"], dim=2)      # [B, S, 3, heads, d]
    kview = qkv[:, :, 1]
    L.partition(kview, L.k_bm)
    ref = np.ascontiguousarray(data["k"][:, ora["perm"]].transpose(0, 2, 1, 3))
    assert np.array_equal(U.to_numpy_f32(L.k_bm), ref)


@pytest.mark.parametrize("w", CASES, ids=IDS)
def test_centroids_and_scores(w):
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    L = VmobaLayer(shape, capacity=1024)
    L.q_bm.copy_(U.bm_to_device(w, U.block_major(w, data, "q", ora["perm"])))
    L.k_bm.copy_(U.bm_to_device(w, U.block_major(w, data, "k", ora["perm"])))
    L.block_scores()
    cent = L.centroids.cpu().numpy().reshape(w.B * w.heads, w.n_blocks, w.head_dim)
    sc = L.scores.cpu().numpy().reshape(w.B * w.heads, w.S, w.n_blocks)
    for i, hd in enumerate(ora["heads"]):
        assert U.max_abs(cent[i], hd["cent"]) <= 2e-6
        U.assert_scores_close(sc[i], hd["scores"])


def _check_lists(L, w, mask):
    """kb_ptr/q_idx/q_ptr/q_pairs must be exactly the CSR forms of `mask` [BH, S, Nb]."""
    BH, S, Nb = mask.shape
    kb_ptr = L.kb_ptr.cpu().numpy(); q_idx = L.q_idx.cpu().numpy()
    q_ptr = L.q_ptr.cpu().numpy(); q_pairs = L.q_pairs.cpu().numpy()
    counts = mask.sum(axis=1).reshape(-1)
    assert np.array_equal(np.diff(kb_ptr), counts) and kb_ptr[0] == 0
    assert np.array_equal(np.diff(q_ptr), mask.sum(axis=2).reshape(-1)) and q_ptr[0] == 0
    n = int(mask.sum())
    assert kb_ptr[-1] == n and q_ptr[-1] == n
    for bh in range(BH):
        for j in range(Nb):
            lo, hi = kb_ptr[bh * Nb + j], kb_ptr[bh * Nb + j + 1]
            assert np.array_equal(q_idx[lo:hi], np.nonzero(mask[bh, :, j])[0])
    # q_pairs: for query G its pairs in ascending block order point back at (block j list, entry == q)
    block_of_pos = np.repeat(np.arange(BH * Nb), counts)
    for G in np.random.default_rng(0).choice(BH * S, size=min(BH * S, 600), replace=False):
        bh, qq = divmod(int(G), S)
        pp = q_pairs[q_ptr[G]:q_ptr[G + 1]]
        assert np.array_equal(block_of_pos[pp] - bh * Nb, np.nonzero(mask[bh, qq])[0])
        assert np.all(q_idx[pp] == qq)


@pytest.mark.parametrize("w", CASES, ids=IDS)
def test_select_matches_oracle_outside_the_cutoff_band(w):
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    cap = w.B * w.heads * w.S * w.n_blocks
    L = VmobaLayer(shape, capacity=cap)
    sc = np.stack([hd["scores"] for hd in ora["heads"]]).reshape(w.B, w.heads, w.S, w.n_blocks)
    L.scores.copy_(torch.from_numpy(sc))
    for tau in (w.tau, 0.6, 1.0):
        L.dev_status.zero_()
        L.select(tau)
        L.check_status()
        got = U.unpack_mask(L.mask_bits, w.B * w.heads, w.S, w.n_blocks)
        kph = L.k_per_head.cpu().numpy(); cut = L.cutoff.cpu().numpy()
        for i, hd in enumerate(ora["heads"]):
            m_ref, k_ref, c_ref = orc.select(hd["scores"], tau, ora["scale"])
            decided = np.abs(hd["scores"] - c_ref) > U.SCORE_BAND
            assert np.array_equal(got[i][decided], m_ref[decided]), (tau, i)
            assert kph[i] == got[i].sum()
            # same scores in, so the GPU may only differ by exact ties and fp64 summation order
            assert abs(float(cut[i]) - float(c_ref)) <= U.SCORE_BAND
            assert abs(int(kph[i]) - k_ref) <= max(8, int(1e-4 * k_ref)), (tau, i, kph[i], k_ref)
            assert np.all(hd["scores"][got[i]] >= cut[i]) and np.all(hd["scores"][~got[i]] < cut[i])
        _check_lists(L, w, got)
    assert got.all()          # tau = 1 selects every pair


def test_select_when_the_crossing_bin_does_not_fit_the_side_list():
    """Level 1 of the cutoff search copies the pairs of the level-0 crossing bin to a short list that level 2 reads
    instead of the matrix.  Here nearly all pairs fall into that one bin (a tight cluster between two far outliers),
    far more than the list holds, so level 2 has to go back to the matrix: same answer as the oracle."""
    w = gen.Workload("sel_cluster", 1, 1, 64, 8, 32, 32, (1, 8, 32), 0.25, "bf16", "smooth", 3)
    rng = np.random.default_rng(11)
    sc = (rng.standard_normal((w.S, w.n_blocks)) * 1e-3).astype(np.float32)
    sc[0, 0], sc[1, 1] = 12.0, -12.0           # stretch the range: one level-0 bin is 0.047 wide
    sc[5, 3], sc[7, 9] = 0.5, 0.25
    L = VmobaLayer(vb.shape_of(w), capacity=w.S * w.n_blocks)
    L.scores.copy_(torch.from_numpy(sc.reshape(1, 1, w.S, w.n_blocks)))
    scale = w.head_dim ** -0.5
    for tau in (0.25, 0.6):
        L.dev_status.zero_()
        L.select(tau)
        L.check_status()
        got = U.unpack_mask(L.mask_bits, 1, w.S, w.n_blocks)[0]
        m_ref, k_ref, c_ref = orc.select(sc, tau, scale)
        cut = float(L.cutoff.cpu().numpy()[0])
        decided = np.abs(sc - c_ref) > 1e-5       # the cluster is 1e-3 wide: compare much closer than the usual band
        assert np.array_equal(got[decided], m_ref[decided]), tau
        assert abs(cut - float(c_ref)) <= 1e-5
        assert abs(int(L.k_per_head.cpu().numpy()[0]) - k_ref) <= 64
        assert np.all(sc[got] >= cut) and np.all(sc[~got] < cut)


def test_select_reports_capacity_overflow():
    w = MID
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    L = VmobaLayer(shape, capacity=256)
    sc = np.stack([hd["scores"] for hd in ora["heads"]]).reshape(w.B, w.heads, w.S, w.n_blocks)
    L.scores.copy_(torch.from_numpy(sc))
    L.select(0.25)
    torch.cuda.synchronize()
    assert int(L.dev_status.item()) == vb.ERR_CAPACITY
    # the truncated lists must still be usable without leaving the buffers
    L.q_bm.normal_(); L.k_bm.normal_(); L.v_bm.normal_()
    L.attn_fwd()
    torch.cuda.synchronize()


def _oracle_attention(w, ora, data, masks, with_bwd):
    res = []
    for i, hd in enumerate(ora["heads"]):
        o, lse = orc.sparse_attn_fwd(hd["q"], hd["k"], hd["v"], masks[i], ora["scale"])
        r = dict(o=o, lse=lse)
        if with_bwd:
            b, h = divmod(i, w.heads)
            do = data["do"][b, :, h][ora["perm"]]
            r["dq"], r["dk"], r["dv"] = orc.sparse_attn_bwd(hd["q"], hd["k"], hd["v"], masks[i], ora["scale"], do)
        res.append(r)
    return res


@pytest.mark.parametrize("w", CASES, ids=IDS)
def test_sparse_attention_forward_backward(w):
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    masks = np.stack([hd["mask"] for hd in ora["heads"]])
    kb_ptr, q_idx, q_ptr, q_pairs, n = lists_from_mask(masks)
    L = VmobaLayer(shape, capacity=max(n, 1), with_backward=True)
    for name, buf in (("q", L.q_bm), ("k", L.k_bm), ("v", L.v_bm), ("do", L.do_bm)):
        buf.copy_(U.bm_to_device(w, U.block_major(w, data, name, ora["perm"])))
    L.kb_ptr.copy_(kb_ptr); L.q_idx.copy_(q_idx); L.q_ptr.copy_(q_ptr); L.q_pairs.copy_(q_pairs)
    L.o_bm.fill_(7.0); L.lse.fill_(7.0)
    L.attn_fwd()
    L.attn_bwd()
    L.check_status()
    ref = _oracle_attention(w, ora, data, masks, True)
    BH = w.B * w.heads
    o = U.to_numpy_f32(L.o_bm).reshape(BH, w.S, w.head_dim)
    lse = L.lse.cpu().numpy().reshape(BH, w.S)
    dq, dk, dv = (U.to_numpy_f32(t).reshape(BH, w.S, w.head_dim) for t in (L.dq_bm, L.dk_bm, L.dv_bm))
    for i, r in enumerate(ref):
        empty = ~masks[i].any(axis=1)
        assert np.all(o[i][empty] == 0) and np.all(np.isneginf(lse[i][empty])) and np.all(dq[i][empty] == 0)
        U.assert_close(o[i], r["o"], w.dtype, f"o head {i}")
        assert U.max_abs(lse[i][~empty], r["lse"][~empty]) <= (2e-2 if w.dtype == "bf16" else 1e-4)
        U.assert_close(dq[i], r["dq"], w.dtype, f"dq head {i}")
        U.assert_close(dk[i], r["dk"], w.dtype, f"dk head {i}")
        U.assert_close(dv[i], r["dv"], w.dtype, f"dv head {i}")


@pytest.mark.parametrize("block", [(1, 4, 16), (1, 5, 13), (1, 8, 16), (1, 10, 13), (2, 12, 8)],
                         ids=["64keys", "65keys", "128keys", "130keys", "192keys"])
def test_sparse_attention_item_and_tile_edges(block):
    """Hand-built lists whose lengths sit on the work-item edges of the tensor-core kernels (0, 1, 63, 64, 65, 127,
    128, 129, 255, 256, 257 and 300 queries per key block) against key blocks whose tail tile is full, one key
    long, or absent: forward and backward against the oracle, empty queries zero-filled."""
    grid = {(1, 4, 16): (6, 8, 16), (1, 5, 13): (6, 10, 13), (1, 8, 16): (6, 8, 16), (1, 10, 13): (6, 10, 13),
            (2, 12, 8): (12, 12, 8)}[block]
    w = gen.Workload("edges", 1, 1, 128, *grid, block, 0.25, "bf16", "smooth", 9)
    data = gen.make_inputs(w)
    perm, _ = orc.partition_perm(w.T, w.H, w.W, *w.block)
    q, k, v, do = (data[n][0, :, 0][perm] for n in ("q", "k", "v", "do"))
    rng = np.random.default_rng(3)
    counts = [0, 1, 63, 64, 65, 127, 128, 129, 255, 256, 257, 300] if w.n_blocks >= 12 else [0, 1, 127, 128, 129, 300]
    mask = np.zeros((1, w.S, w.n_blocks), dtype=bool)
    for j in range(w.n_blocks):
        c = min(counts[j % len(counts)], w.S)
        mask[0, rng.choice(w.S, size=c, replace=False), j] = True
    kb_ptr, q_idx, q_ptr, q_pairs, n = lists_from_mask(mask)
    L = VmobaLayer(vb.shape_of(w), capacity=max(n, 1), with_backward=True)
    for name, buf in (("q", L.q_bm), ("k", L.k_bm), ("v", L.v_bm), ("do", L.do_bm)):
        buf.copy_(U.bm_to_device(w, U.block_major(w, data, name, perm)))
    L.kb_ptr.copy_(kb_ptr); L.q_idx.copy_(q_idx); L.q_ptr.copy_(q_ptr); L.q_pairs.copy_(q_pairs)
    L.o_bm.fill_(7.0); L.lse.fill_(7.0)
    L.attn_fwd()
    L.attn_bwd()
    L.check_status()
    scale = w.head_dim ** -0.5
    o_ref, lse_ref = orc.sparse_attn_fwd(q, k, v, mask[0], scale)
    dq_ref, dk_ref, dv_ref = orc.sparse_attn_bwd(q, k, v, mask[0], scale, do)
    o = U.to_numpy_f32(L.o_bm).reshape(w.S, w.head_dim)
    lse = L.lse.cpu().numpy().reshape(w.S)
    dq, dk, dv = (U.to_numpy_f32(t).reshape(w.S, w.head_dim) for t in (L.dq_bm, L.dk_bm, L.dv_bm))
    empty = ~mask[0].any(axis=1)
    assert empty.any() and (~empty).any()
    assert np.all(o[empty] == 0) and np.all(np.isneginf(lse[empty])) and np.all(dq[empty] == 0)
    U.assert_close(o, o_ref, w.dtype, "o")
    assert U.max_abs(lse[~empty], lse_ref[~empty]) <= 2e-2
    U.assert_close(dq, dq_ref, w.dtype, "dq")
    U.assert_close(dk, dk_ref, w.dtype, "dk")
    U.assert_close(dv, dv_ref, w.dtype, "dv")


@pytest.mark.parametrize("block", [(3, 6, 13), (6, 12, 13), (6, 12, 26)], ids=["234keys", "936keys", "1872keys"])
def test_attention_with_no_selected_pair(block):
    """Empty work lists (no query selected any block): every kernel variant of the forward and the backward must
    return with o = 0, lse = -inf and zero gradients."""
    w = MID.with_(name="mid_empty_%d_%d_%d" % block, block=block)
    shape = vb.shape_of(w)
    masks = np.zeros((w.B * w.heads, w.S, w.n_blocks), dtype=bool)
    kb_ptr, q_idx, q_ptr, q_pairs, n = lists_from_mask(masks)
    assert n == 0
    L = VmobaLayer(shape, capacity=1, with_backward=True)
    for buf in (L.q_bm, L.k_bm, L.v_bm, L.do_bm):
        buf.normal_()
    L.kb_ptr.copy_(kb_ptr); L.q_idx.copy_(q_idx); L.q_ptr.copy_(q_ptr); L.q_pairs.copy_(q_pairs)
    L.o_bm.fill_(7.0); L.lse.fill_(7.0)
    for g in (L.dq_bm, L.dk_bm, L.dv_bm):
        g.fill_(7.0)
    L.attn_fwd()
    L.attn_bwd()
    L.check_status()
    assert torch.all(L.o_bm == 0) and torch.all(torch.isneginf(L.lse))
    assert torch.all(L.dq_bm == 0) and torch.all(L.dk_bm == 0) and torch.all(L.dv_bm == 0)


@pytest.mark.parametrize("block", [(3, 6, 13), (1, 12, 26), (6, 12, 13)], ids=["234keys", "312keys", "936keys"])
def test_partial_rows_follow_the_scale_of_v(block):
    """The forward keeps one partial result per (query, block) pair as fp16 values times a power of two chosen per
    row.  Multiplying v by a power of two (exact in bf16) must therefore multiply o by the same factor bit for bit,
    far beyond the range of fp16 itself (v reaches about 5 * 2^20 here) and far below it."""
    w = MID.with_(name="mid_vscale_%d_%d_%d" % block, block=block, tau=0.5)
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    # a random half of all pairs: most queries hold several blocks, so their rows go through the merge
    masks = np.random.default_rng(17).random((w.B * w.heads, w.S, w.n_blocks)) < 0.5
    assert (masks.sum(axis=2) >= 2).any()
    kb_ptr, q_idx, q_ptr, q_pairs, n = lists_from_mask(masks)
    L = VmobaLayer(shape, capacity=max(n, 1))
    for name, buf in (("q", L.q_bm), ("k", L.k_bm), ("v", L.v_bm)):
        buf.copy_(U.bm_to_device(w, U.block_major(w, data, name, ora["perm"])))
    L.kb_ptr.copy_(kb_ptr); L.q_idx.copy_(q_idx); L.q_ptr.copy_(q_ptr); L.q_pairs.copy_(q_pairs)
    v0 = L.v_bm.clone()
    L.attn_fwd(); L.check_status()
    o0, lse0 = L.o_bm.clone(), L.lse.clone()
    for factor in (2.0 ** 20, 2.0 ** -20):
        L.v_bm.copy_(v0 * factor)
        assert torch.equal(L.v_bm.float(), v0.float() * factor)
        L.attn_fwd(); L.check_status()
        assert torch.equal(L.o_bm.float(), o0.float() * factor), factor
        assert torch.equal(L.lse, lse0)


@pytest.mark.parametrize("w", [CASES[0], CASES[3], CASES[8]], ids=[IDS[0], IDS[3], IDS[8]])
def test_sparse_attention_full_mask_equals_dense_oracle(w):
    """tau = 1: the sparse path over every pair must reproduce dense softmax attention."""
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    BH = w.B * w.heads
    masks = np.ones((BH, w.S, w.n_blocks), dtype=bool)
    kb_ptr, q_idx, q_ptr, q_pairs, n = lists_from_mask(masks)
    L = VmobaLayer(shape, capacity=n)
    for name, buf in (("q", L.q_bm), ("k", L.k_bm), ("v", L.v_bm)):
        buf.copy_(U.bm_to_device(w, U.block_major(w, data, name, ora["perm"])))
    L.kb_ptr.copy_(kb_ptr); L.q_idx.copy_(q_idx); L.q_ptr.copy_(q_ptr); L.q_pairs.copy_(q_pairs)
    L.attn_fwd()
    L.check_status()
    o = U.to_numpy_f32(L.o_bm).reshape(BH, w.S, w.head_dim)
    for i, hd in enumerate(ora["heads"]):
        od, _ = orc.dense_attn_fwd(hd["q"], hd["k"], hd["v"], ora["scale"])
        U.assert_close(o[i], od, w.dtype, f"head {i}")


@pytest.mark.parametrize("w", [CASES[0], CASES[3], CASES[8], CASES[9]], ids=[IDS[0], IDS[3], IDS[8], IDS[9]])
def test_dense_attention_forward_backward(w):
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    BH = w.B * w.heads
    dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
    mk = lambda name: U.bm_to_device(w, U.block_major(w, data, name, ora["perm"]))
    q, k, v, do = mk("q"), mk("k"), mk("v"), mk("do")
    o = torch.empty_like(q); dq = torch.empty_like(q); dk = torch.empty_like(q); dv = torch.empty_like(q)
    lse = torch.empty(BH * w.S, dtype=torch.float32, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ws = torch.empty(vb.workspace_bytes(shape, vb.STAGE_FULL_BWD), dtype=torch.uint8, device="cuda")
    vb.vmoba_full_attn(shape, q, k, v, o, lse, do, dq, dk, dv, status, ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    on = U.to_numpy_f32(o).reshape(BH, w.S, -1)
    g = [U.to_numpy_f32(t).reshape(BH, w.S, -1) for t in (dq, dk, dv)]
    for i, hd in enumerate(ora["heads"]):
        b, h = divmod(i, w.heads)
        od, lsed = orc.dense_attn_fwd(hd["q"], hd["k"], hd["v"], ora["scale"])
        U.assert_close(on[i], od, w.dtype, "o")
        assert U.max_abs(lse.cpu().numpy().reshape(BH, w.S)[i], lsed) <= (2e-2 if w.dtype == "bf16" else 1e-4)
        ref = orc.dense_attn_bwd(hd["q"], hd["k"], hd["v"], ora["scale"], data["do"][b, :, h][ora["perm"]])
        for name, got, want in zip(("dq", "dk", "dv"), g, ref):
            U.assert_close(got[i], want, w.dtype, name)


@pytest.mark.parametrize("w", [CASES[0], CASES[3], CASES[4], CASES[6], CASES[7], CASES[8]],
                         ids=[IDS[0], IDS[3], IDS[4], IDS[6], IDS[7], IDS[8]])
def test_score_range_from_the_scores_kernel_and_ranged_selection(w):
    """vmoba_block_scores_range must report exactly the smallest and largest score of every head, and
    vmoba_select_ranged, which skips its own search for them, must return what vmoba_select returns, bit for bit."""
    data, ora = _prep(w)
    shape = vb.shape_of(w)
    cap = w.B * w.heads * w.S * w.n_blocks
    L = VmobaLayer(shape, capacity=cap)
    L.q_bm.copy_(U.bm_to_device(w, U.block_major(w, data, "q", ora["perm"])))
    L.k_bm.copy_(U.bm_to_device(w, U.block_major(w, data, "k", ora["perm"])))
    L.score_range.fill_(float("nan"))
    L.block_scores(with_range=True)
    torch.cuda.synchronize()
    sc = L.scores.view(w.B * w.heads, -1)
    assert torch.equal(L.score_range[:, 0], sc.amin(dim=1)) and torch.equal(L.score_range[:, 1], sc.amax(dim=1))
    plain = L.scores.clone()
    L.block_scores(with_range=False)
    assert torch.equal(L.scores, plain)                       # the scores themselves do not depend on the entry point
    names = ("mask_bits", "kb_ptr", "q_ptr", "k_per_head", "cutoff")
    for tau in (w.tau, 0.6):
        L.select(tau, use_range=False)
        torch.cuda.synchronize()
        n = L.n_selected()
        ref = {k: getattr(L, k).clone() for k in names}
        ref["q_idx"], ref["q_pairs"] = L.q_idx[:n].clone(), L.q_pairs[:n].clone()
        for k in names:
            getattr(L, k).fill_(0)
        L.q_idx.fill_(-1); L.q_pairs.fill_(-1)
        L.select(tau, use_range=True)
        torch.cuda.synchronize()
        L.check_status()
        for k in names:
            assert torch.equal(getattr(L, k), ref[k]), (tau, k)
        assert torch.equal(L.q_idx[:n], ref["q_idx"]) and torch.equal(L.q_pairs[:n], ref["q_pairs"])
