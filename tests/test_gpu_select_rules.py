"""Parity of vmoba_select_rule_apply with the oracle: the four block-choice rules of Table 3b
(threshold / top-k, head-wide / per query), stage-isolated (oracle scores in), then end to end with
the attention forward on the paper's training-free setting (Local + TopK, Table 4)."""
import numpy as np
import pytest
import torch

from oracle import vmoba_oracle as orc
from paper_2506_23858_b200 import binding as vb
from paper_2506_23858_b200 import inputs as gen
from paper_2506_23858_b200.layer import VmobaLayer
from tests import _util as U
from tests.test_gpu_stages import CASES, IDS, MID, _check_lists, _prep

pytestmark = pytest.mark.gpu

# a relative margin below which fp32 exp / summation order may move a row's cumulative mass across tau
MASS_MARGIN = 1e-5


def _layer_with_scores(w, ora):
    shape = vb.shape_of(w)
    L = VmobaLayer(shape, capacity=w.B * w.heads * w.S * w.n_blocks)
    sc = np.stack([hd["scores"] for hd in ora["heads"]]).reshape(w.B, w.heads, w.S, w.n_blocks)
    L.scores.copy_(torch.from_numpy(sc))
    return L


def _run(L, w, rule, tau=0.25, topk=1):
    L.dev_status.zero_()
    L.select_rule(rule, tau=tau, topk=topk)
    L.check_status()
    return U.unpack_mask(L.mask_bits, w.B * w.heads, w.S, w.n_blocks)


@pytest.mark.parametrize("w", CASES, ids=IDS)
def test_topk_local_is_exact(w):
    data, ora = _prep(w)
    L = _layer_with_scores(w, ora)
    for k in (1, 3, w.n_blocks, w.n_blocks + 5):
        got = _run(L, w, vb.SELECT_TOPK_LOCAL, topk=k)
        cut = L.cutoff.cpu().numpy()
        for i, hd in enumerate(ora["heads"]):
            ref = orc.select_topk_per_query(hd["scores"], k)
            assert np.array_equal(got[i], ref), (k, i)
            assert float(cut[i]) == float(hd["scores"][ref].min())
        assert (got.sum(axis=2) == min(k, w.n_blocks)).all()          # never an empty row, exactly k
        assert np.array_equal(L.k_per_head.cpu().numpy(), got.sum(axis=(1, 2)))
        _check_lists(L, w, got)


def test_topk_local_breaks_ties_in_block_order():
    # scores quantised to a handful of values: most rows have ties at their cutoff
    w = MID.with_(name="ties", block=(1, 3, 13))
    rng = np.random.default_rng(11)
    sc = rng.integers(-2, 3, size=(w.B * w.heads, w.S, w.n_blocks)).astype(np.float32)
    L = VmobaLayer(vb.shape_of(w), capacity=w.B * w.heads * w.S * w.n_blocks)
    L.scores.copy_(torch.from_numpy(sc.reshape(w.B, w.heads, w.S, w.n_blocks)))
    for k in (2, 7):
        got = _run(L, w, vb.SELECT_TOPK_LOCAL, topk=k)
        for i in range(sc.shape[0]):
            assert np.array_equal(got[i], orc.select_topk_per_query(sc[i], k))
    # the threshold rule on all-equal rows: the first ceil(tau * N_b) blocks
    L.scores.zero_()
    got = _run(L, w, vb.SELECT_THRESHOLD_LOCAL, tau=0.25)
    want = orc.select_threshold_per_query(np.zeros((4, w.n_blocks), np.float32), 0.25, 1.0)[0]
    assert np.array_equal(got[0, :4], want)


@pytest.mark.parametrize("w", CASES, ids=IDS)
def test_threshold_local_matches_oracle(w):
    data, ora = _prep(w)
    L = _layer_with_scores(w, ora)
    for tau in (0.25, 0.7, 1.0):
        got = _run(L, w, vb.SELECT_THRESHOLD_LOCAL, tau=tau)
        n_exempt = 0
        for i, hd in enumerate(ora["heads"]):
            ref, k_ref = orc.select_threshold_per_query(hd["scores"], tau, ora["scale"])
            # rows whose cumulative mass passes tau by less than the margin may take one block more or less
            x = ora["scale"] * hd["scores"].astype(np.float64)
            p = np.exp(x - x.max(axis=1, keepdims=True))
            p /= p.sum(axis=1, keepdims=True)
            c = np.cumsum(-np.sort(-p, axis=1), axis=1)
            at = np.take_along_axis(c, (k_ref - 1)[:, None], axis=1)[:, 0]
            before = np.where(k_ref > 1, np.take_along_axis(c, np.maximum(k_ref - 2, 0)[:, None], axis=1)[:, 0], 0.0)
            close = (np.abs(at - tau) < MASS_MARGIN) | (np.abs(before - tau) < MASS_MARGIN)
            if tau >= 1.0:
                close[:] = False
            n_exempt += int(close.sum())
            assert np.array_equal(got[i][~close], ref[~close]), (tau, i)
            assert (np.abs(got[i][close].sum(axis=1) - k_ref[close]) <= 1).all()
        assert n_exempt <= max(2, got.shape[0] * got.shape[1] // 1000)
        assert (got.sum(axis=2) >= 1).all()
        _check_lists(L, w, got)
    assert got.all()          # tau = 1 keeps every block of every query


@pytest.mark.parametrize("w", CASES, ids=IDS)
def test_topk_global_matches_oracle(w):
    data, ora = _prep(w)
    L = _layer_with_scores(w, ora)
    for k in (1, 2, w.n_blocks):
        got = _run(L, w, vb.SELECT_TOPK_GLOBAL, topk=k)
        kph = L.k_per_head.cpu().numpy(); cut = L.cutoff.cpu().numpy()
        for i, hd in enumerate(ora["heads"]):
            ref, K, c_ref = orc.select_topk_global(hd["scores"], k)
            # counting is exact: the cutoff is THE K-th largest score; pairs tied with it are all kept
            assert float(cut[i]) == float(c_ref), (k, i)
            untied = hd["scores"] != c_ref
            assert np.array_equal(got[i][untied], ref[untied])
            assert got[i][~untied].all()
            assert K <= kph[i] == got[i].sum()
        _check_lists(L, w, got)
    assert got.all()          # k = N_b: the budget is the whole pool


def test_threshold_global_rule_is_vmoba_select():
    w = MID
    data, ora = _prep(w)
    L = _layer_with_scores(w, ora)
    a = _run(L, w, vb.SELECT_THRESHOLD_GLOBAL, tau=0.25).copy()
    q_idx = L.q_idx.clone()
    L.select(0.25)
    L.check_status()
    assert np.array_equal(a, U.unpack_mask(L.mask_bits, w.B * w.heads, w.S, w.n_blocks))
    assert torch.equal(q_idx, L.q_idx)


def test_rule_argument_checks():
    w = MID
    L = VmobaLayer(vb.shape_of(w), capacity=1024)
    for rule, tau, topk in ((7, 0.25, 1), (vb.SELECT_TOPK_LOCAL, 0.25, 0), (vb.SELECT_THRESHOLD_LOCAL, 0.0, 1),
                            (vb.SELECT_THRESHOLD_LOCAL, 1.5, 1), (vb.SELECT_TOPK_GLOBAL, 0.25, -3)):
        with pytest.raises(vb.VmobaError):
            L.select_rule(rule, tau=tau, topk=topk)


def test_local_topk_feeds_the_attention_forward():
    """The paper's training-free setting (Table 4, Local + TopK): per-query top-k lists through the
    same attention kernel; every query has exactly k blocks, so no row is empty."""
    w = MID.with_(name="mid_topk", block=(3, 6, 13))
    data, ora = _prep(w)
    L = VmobaLayer(vb.shape_of(w), capacity=w.B * w.heads * w.S * 4)
    for name, buf in (("q", L.q_bm), ("k", L.k_bm), ("v", L.v_bm)):
        buf.copy_(U.bm_to_device(w, U.block_major(w, data, name, ora["perm"])))
    L.block_scores()
    L.select_rule(vb.SELECT_TOPK_LOCAL, topk=2)
    L.attn_fwd()
    L.check_status()
    got_mask = U.unpack_mask(L.mask_bits, w.B * w.heads, w.S, w.n_blocks)
    o = L.o_bm.float().cpu().numpy().reshape(w.B * w.heads, w.S, w.head_dim)
    for i, hd in enumerate(ora["heads"]):
        # attention parity on the GPU's own mask (its scores differ from the oracle's in the last bits)
        ref_o, _ = orc.sparse_attn_fwd(hd["q"], hd["k"], hd["v"], got_mask[i], ora["scale"])
        U.assert_close(o[i], ref_o, "bf16", f"o head {i}")
        m_ref = orc.select_topk_per_query(hd["scores"], 2)
        # rows whose 2nd and 3rd best scores are farther apart than the score tolerance must agree
        srt = -np.sort(-hd["scores"], axis=1)
        clear = (srt[:, 1] - srt[:, 2]) > U.SCORE_BAND
        assert np.array_equal(got_mask[i][clear], m_ref[clear])


def test_local_rules_at_full_size_on_sampled_rows():
    """C3's three partitions at 32,760 tokens with the per-query budgets of the paper's training-free
    runs (k = 2 / 6 / 18 for the 1D / 2D / 3D layers, Table 4), and the per-query threshold rule: the
    GPU's own scores go through the oracle's rule on 4,096 sampled rows per layer."""
    rng = np.random.default_rng(3)
    for name, k in (("1d", 2), ("2d", 6), ("3d", 18)):
        w = gen.C2.with_(name=f"c3_{name}_local", block=gen.C3_BLOCKS[name], heads=4)
        data = gen.make_inputs(w)
        perm, _ = orc.partition_perm(w.T, w.H, w.W, *w.block)
        L = VmobaLayer(vb.shape_of(w), capacity=w.B * w.heads * w.S * min(w.n_blocks, 48))
        for nme, buf in (("q", L.q_bm), ("k", L.k_bm)):
            buf.copy_(U.bm_to_device(w, U.block_major(w, data, nme, perm)))
        L.block_scores()
        rows = np.sort(rng.choice(w.B * w.heads * w.S, size=4096, replace=False))
        sc = L.scores.reshape(-1, w.n_blocks)[torch.from_numpy(rows).cuda()].cpu().numpy()
        L.select_rule(vb.SELECT_TOPK_LOCAL, topk=k)
        L.check_status()
        words = L.mask_bits.reshape(-1, L.mask_bits.shape[-1])[torch.from_numpy(rows).cuda()].cpu().numpy()
        got = ((words[:, np.arange(w.n_blocks) >> 5] >> (np.arange(w.n_blocks) & 31)) & 1).astype(bool)
        assert np.array_equal(got, orc.select_topk_per_query(sc, k)), name
        assert int(L.n_selected()) == w.B * w.heads * w.S * min(k, w.n_blocks)
        L.select_rule(vb.SELECT_THRESHOLD_LOCAL, tau=0.5)
        L.check_status()
        words = L.mask_bits.reshape(-1, L.mask_bits.shape[-1])[torch.from_numpy(rows).cuda()].cpu().numpy()
        got = ((words[:, np.arange(w.n_blocks) >> 5] >> (np.arange(w.n_blocks) & 31)) & 1).astype(bool)
        ref, k_ref = orc.select_threshold_per_query(sc, 0.5, w.head_dim ** -0.5)
        differ = (got != ref).any(axis=1)
        assert differ.sum() <= 4 and (np.abs(got.sum(axis=1) - k_ref) <= 1).all(), (name, int(differ.sum()))


def test_keep_own_block_option():
    """VMOBA_SELECT_KEEP_OWN_BLOCK: the mask is the rule's mask OR the block each query lies in."""
    w = MID
    data, ora = _prep(w)
    L = _layer_with_scores(w, ora)
    own = np.zeros((w.S, w.n_blocks), dtype=bool)
    own[np.arange(w.S), np.arange(w.S) // w.block_tokens] = True
    for rule, kw, ref_of in (
            (vb.SELECT_THRESHOLD_GLOBAL, dict(tau=0.25), lambda sc: orc.select(sc, 0.25, ora["scale"])[0]),
            (vb.SELECT_TOPK_LOCAL, dict(topk=2), lambda sc: orc.select_topk_per_query(sc, 2)),
            (vb.SELECT_THRESHOLD_LOCAL, dict(tau=0.25), lambda sc: orc.select_threshold_per_query(sc, 0.25, ora["scale"])[0])):
        base = _run(L, w, rule, **kw).copy()
        got = _run(L, w, rule | vb.SELECT_KEEP_OWN_BLOCK, **kw)
        for i, hd in enumerate(ora["heads"]):
            assert np.array_equal(got[i], base[i] | own), (rule, i)
        assert (got.sum(axis=2) >= 1).all()
        _check_lists(L, w, got)
    # end to end: no query is left without keys, so no output row is zero and every lse is finite
    for name, buf in (("q", L.q_bm), ("k", L.k_bm), ("v", L.v_bm)):
        buf.copy_(U.bm_to_device(w, U.block_major(w, data, name, ora["perm"])))
    L.select_rule(vb.SELECT_THRESHOLD_GLOBAL | vb.SELECT_KEEP_OWN_BLOCK, tau=0.25)
    L.attn_fwd()
    L.check_status()
    assert torch.isfinite(L.lse).all()


@pytest.mark.parametrize("w", CASES, ids=IDS)
def test_rownorm_threshold_matches_oracle(w):
    """Eq. 4 with per-query softmax normalisation: equal to the oracle on every pair whose row-normalised
    log-probability is farther than the score band from the oracle's cutoff."""
    data, ora = _prep(w)
    L = _layer_with_scores(w, ora)
    for tau in (0.25, 0.6, 1.0):
        got = _run(L, w, vb.SELECT_THRESHOLD_GLOBAL_ROWNORM, tau=tau)
        kph = L.k_per_head.cpu().numpy(); cut = L.cutoff.cpu().numpy()
        for i, hd in enumerate(ora["heads"]):
            m_ref, k_ref, c_ref = orc.select_rownorm(hd["scores"], tau, ora["scale"])
            x = ora["scale"] * hd["scores"].astype(np.float64)
            mx = x.max(axis=1, keepdims=True)
            logp = x - (mx + np.log(np.exp(x - mx).sum(axis=1, keepdims=True)))
            decided = np.abs(logp - c_ref) > U.SCORE_BAND
            assert np.array_equal(got[i][decided], m_ref[decided]), (tau, i)
            assert kph[i] == got[i].sum()
            if tau < 1.0:
                assert abs(float(cut[i]) - c_ref) <= U.SCORE_BAND
            assert abs(int(kph[i]) - k_ref) <= max(8, int(2e-3 * k_ref)), (tau, i, kph[i], k_ref)
        _check_lists(L, w, got)
    assert got.all()
    # too small a workspace is refused on the host
    with pytest.raises(vb.VmobaError):
        vb.vmoba_select_rule_apply(L.shape, L.scores, vb.SELECT_THRESHOLD_GLOBAL_ROWNORM, 0.25, 1, L.mask_bits, L.kb_ptr,
                                   L.q_idx, L.q_ptr, L.q_pairs, L.capacity, L.k_per_head, L.cutoff, L.dev_status,
                                   L.ws[:vb.workspace_bytes(L.shape, vb.STAGE_SELECT, 0)])
