"""End-to-end parity of the whole layer (raster order in, raster order out) against the oracle,
on the tiny config in full and on the benchmark configurations at full size with sampled
heads / rows / key blocks (rows of attention are independent, so sampled rows are exact).

Mask parity rule: the GPU mask must equal the oracle's on every pair whose oracle fp32 score
is farther than 1e-3 from the oracle's cutoff.  Output rows that own a pair inside that band
are left out of the O / dQ comparison; dK / dV are compared against the oracle re-run on the
GPU's (validated) mask."""
import numpy as np
import pytest
import torch

from oracle import vmoba_oracle as orc
from paper_2506_23858_b200 import binding as vb
from paper_2506_23858_b200 import inputs as gen
from paper_2506_23858_b200.layer import VmobaLayer, default_capacity
from tests import _util as U

pytestmark = pytest.mark.gpu


def _run_layer(w, data, with_bwd, capacity=None):
    shape = vb.shape_of(w)
    cap = capacity or default_capacity(shape, w.tau)
    L = VmobaLayer(shape, capacity=cap, with_backward=with_bwd)
    q, k, v = (U.to_device(w, data, n) for n in "qkv")
    o = torch.empty_like(q)
    L.forward(q, k, v, w.tau, o)
    out = dict(L=L, o=o)
    if with_bwd:
        do = U.to_device(w, data, "do")
        out["dq"], out["dk"], out["dv"] = torch.empty_like(q), torch.empty_like(q), torch.empty_like(q)
        L.backward(do, out["dq"], out["dk"], out["dv"])
    torch.cuda.synchronize()
    L.check_status()
    return out


def _check_head(w, data, res, b, h, rng, n_rows, n_blocks, with_bwd):
    """Oracle for one (batch, head); compares mask (band rule), O/LSE/dQ on sampled clean rows and
    dK/dV on sampled key blocks."""
    L = res["L"]
    scale = w.head_dim ** -0.5
    perm, inv = orc.partition_perm(w.T, w.H, w.W, *w.block)
    q, k, v = (data[n][b, :, h][perm] for n in "qkv")
    cent = orc.centroids(k, w.n_blocks)
    sc = orc.block_scores(q, cent)
    m_ref, k_ref, c_ref = orc.select(sc, w.tau, scale)
    bh = b * w.heads + h
    S, Nb = w.S, w.n_blocks
    words = L.mask_bits[bh * S:(bh + 1) * S].cpu().numpy().view(np.uint32)
    m_gpu = (((words[:, :, None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(S, -1)[:, :Nb]).astype(bool)
    sc_gpu = L.scores.view(-1, S, Nb)[bh].cpu().numpy()
    U.assert_scores_close(sc_gpu, sc)
    decided = np.abs(sc - c_ref) > U.SCORE_BAND
    assert np.array_equal(m_gpu[decided], m_ref[decided]), f"mask mismatch outside the band, head {bh}"
    assert int(L.k_per_head[bh].item()) == int(m_gpu.sum())
    clean = decided.all(axis=1)
    assert clean.mean() > 0.5
    rows = rng.choice(np.nonzero(clean)[0], size=min(n_rows, int(clean.sum())), replace=False)
    # make sure both empty and non-empty rows are sampled when they exist
    o_ref, lse_ref = orc.sparse_attn_fwd(q, k, v, m_ref, scale, rows=rows)
    raster_rows = torch.from_numpy(perm[rows].astype(np.int64)).cuda()
    o_gpu = U.to_numpy_f32(res["o"][b, raster_rows, h])
    U.assert_close(o_gpu, o_ref, w.dtype, f"o head {bh}")
    lse_gpu = L.lse[bh * S:(bh + 1) * S].cpu().numpy()[rows]
    ne = np.isfinite(lse_ref)
    assert np.all(np.isneginf(lse_gpu[~ne])) and np.all(o_gpu[~ne] == 0)
    assert U.max_abs(lse_gpu[ne], lse_ref[ne]) <= (2e-2 if w.dtype == "bf16" else 1e-4)
    if with_bwd:
        do = data["do"][b, :, h][perm]
        dq_ref, _, _ = orc.sparse_attn_bwd(q, k, v, m_ref, scale, do, rows=rows)
        U.assert_close(U.to_numpy_f32(res["dq"][b, raster_rows, h]), dq_ref, w.dtype, f"dq head {bh}")
        # properties that hold at any size: softmax rows sum to 1, so sum_t dV_t = sum of dO over the
        # non-empty queries; shifting all keys by one vector changes nothing, so sum_t dK_t = 0.
        all_tok = torch.from_numpy(perm.astype(np.int64)).cuda()
        dv_all = res["dv"][b, :, h].float()
        dk_all = res["dk"][b, :, h].float()
        nonempty = m_gpu.any(axis=1)
        want = do[nonempty].astype(np.float64).sum(axis=0)
        eps = 2.0 ** -9 if w.dtype == "bf16" else 1e-6
        tol_v = 6.0 * np.sqrt(S) * eps * float(dv_all.pow(2).mean().sqrt()) + 1e-3 * np.abs(want).max() + 1e-4
        assert U.max_abs(dv_all.double().sum(dim=0).cpu().numpy(), want) <= tol_v
        # D = dO.o is taken from the stored (rounded) output, as in any FlashAttention-style backward, so
        # each query leaves a residual of order eps * sqrt(d) in sum_t dS_qt; these add up over the queries.
        tol_k = (6.0 * np.sqrt(S) * eps * float(dk_all.pow(2).mean().sqrt()) + 1e-4
                 + 3.0 * scale * np.sqrt(S) * eps * np.sqrt(w.head_dim))
        assert float(dk_all.double().sum(dim=0).abs().max()) <= tol_k
        # exact dK / dV rows of sampled key blocks, where the oracle can afford the block's queries
        for j in rng.choice(Nb, size=min(n_blocks, Nb), replace=False):
            n_q = int(m_gpu[:, j].sum())
            keys_per_q = float(m_gpu[m_gpu[:, j]].sum(axis=1).mean()) * w.block_tokens if n_q else 0.0
            if n_q * keys_per_q > 6e7:
                continue
            dk_ref, dv_ref = orc.sparse_attn_bwd_key_block(q, k, v, m_gpu, scale, do, int(j))
            tok = torch.from_numpy(perm[j * w.block_tokens:(j + 1) * w.block_tokens].astype(np.int64)).cuda()
            U.assert_close(U.to_numpy_f32(res["dk"][b, tok, h]), dk_ref, w.dtype, f"dk head {bh} block {j}")
            U.assert_close(U.to_numpy_f32(res["dv"][b, tok, h]), dv_ref, w.dtype, f"dv head {bh} block {j}")
    return float(m_gpu.mean())


def test_tiny_config_forward_full_comparison():
    """Config 1: fp32, 256 tokens, 1D partition, tau 0.25, every row of both heads."""
    w = gen.C1
    data = gen.make_inputs(w)
    res = _run_layer(w, data, with_bwd=True)
    rng = np.random.default_rng(0)
    for h in range(w.heads):
        dens = _check_head(w, data, res, 0, h, rng, n_rows=w.S, n_blocks=w.n_blocks, with_bwd=True)
        assert 0 < dens <= w.tau + 1e-3


MID = gen.Workload("mid", 2, 3, 128, 6, 12, 26, (3, 6, 13), 0.25, "bf16", "smooth", 9)


@pytest.mark.parametrize("block", [(1, 12, 26), (6, 6, 13), (3, 6, 13), (1, 3, 13)], ids=["1d", "2d", "3d", "48blk"])
def test_mid_size_layer_forward_backward(block):
    w = MID.with_(block=block)
    data = gen.make_inputs(w)
    res = _run_layer(w, data, with_bwd=True)
    rng = np.random.default_rng(1)
    for b in range(w.B):
        for h in range(w.heads):
            _check_head(w, data, res, b, h, rng, n_rows=400, n_blocks=3, with_bwd=True)


@pytest.mark.parametrize("block", [(1, 12, 26), (3, 6, 13)], ids=["1d", "3d"])
def test_mid_size_layer_unstructured_inputs(block):
    """Inputs without any locality component: the selection pattern is unstructured and a large share of the
    queries own several pairs (about 1.4 per query with 6 blocks, 11 with 48), so most output rows go through the
    partial rows and the merge instead of being written directly by the forward kernel."""
    w = MID.with_(block=block, recipe="white", heads=2, B=1)
    data = gen.make_inputs(w)
    res = _run_layer(w, data, with_bwd=True, capacity=w.S * w.n_blocks)
    L = res["L"]
    q_ptr = L.q_ptr.cpu().numpy().astype(np.int64)
    per_query = np.diff(q_ptr.reshape(-1))[: w.S]
    assert (per_query >= 2).mean() > 0.3, "the recipe is meant to give a large share of the queries several pairs"
    rng = np.random.default_rng(3)
    for h in range(w.heads):
        _check_head(w, data, res, 0, h, rng, n_rows=400, n_blocks=3, with_bwd=True)


@pytest.mark.parametrize("grid,block", [((6, 9, 20), (3, 9, 10)), ((4, 43, 3), (1, 43, 3)), ((2, 16, 32), (1, 16, 16))],
                         ids=["270keys_tail14", "129keys_tail1", "256keys_no_tail"])
def test_key_block_tails_forward_backward(grid, block):
    """Key blocks whose last 128-key tile holds 14 keys (the 720p 3D blocks), one key, or is full."""
    w = gen.Workload("tails", 1, 2, 128, grid[0], grid[1], grid[2], block, 0.25, "bf16", "smooth", 11)
    data = gen.make_inputs(w)
    res = _run_layer(w, data, with_bwd=True)
    rng = np.random.default_rng(2)
    for h in range(w.heads):
        _check_head(w, data, res, 0, h, rng, n_rows=min(400, w.S), n_blocks=min(3, w.n_blocks), with_bwd=True)


@pytest.mark.parametrize("block", [(1, 12, 26), (3, 6, 13)], ids=["1d", "3d"])
def test_wide_logit_range_forward_backward(block):
    """Queries four times larger (exact in bf16): logits spread over tens of units, so the running maximum
    of a row moves by more than the lazy-rescale threshold between key tiles and the accumulator is rescaled."""
    w = MID.with_(block=block, B=1, heads=2)
    data = gen.make_inputs(w)
    data["q"] = data["q"] * 4.0
    data["q_bits"] = gen.f32_to_bf16_bits(data["q"])
    assert np.array_equal(gen.bf16_bits_to_f32(data["q_bits"]), data["q"])
    res = _run_layer(w, data, with_bwd=True)
    rng = np.random.default_rng(3)
    for h in range(w.heads):
        _check_head(w, data, res, 0, h, rng, n_rows=400, n_blocks=3, with_bwd=True)


@pytest.mark.parametrize("block", [(1, 12, 26), (3, 6, 13)], ids=["1d", "3d"])
def test_backward_writing_raster_order_equals_inverse_partition(block):
    """vmoba_attn_bwd_raster folds Eq. 1 into the reads of dO and its inverse into the gradient writes: dK and dV
    must equal partition + vmoba_attn_bwd + inverse partition bit for bit, dQ up to the order of its fp32 sum."""
    w = MID.with_(block=block)
    data = gen.make_inputs(w)
    shape = vb.shape_of(w)
    L = VmobaLayer(shape, capacity=default_capacity(shape, w.tau), with_backward=True)
    q, k, v, do = (U.to_device(w, data, n) for n in ("q", "k", "v", "do"))
    o = torch.empty_like(q)
    L.forward(q, k, v, w.tau, o)
    got = [torch.full_like(q, float("nan")) for _ in range(3)]
    ref = [torch.empty_like(q) for _ in range(3)]
    L.backward(do, *got, fold_inverse=True, fold_do=True)
    L.backward(do, *ref, fold_inverse=False)
    torch.cuda.synchronize()
    L.check_status()
    assert torch.equal(got[1], ref[1]) and torch.equal(got[2], ref[2])
    assert not torch.isnan(got[0].float()).any()
    diff = (got[0].float() - ref[0].float()).abs().max().item()
    assert diff <= 2.0 ** -6 * max(1.0, ref[0].float().abs().max().item())
    # a strided destination: the gradients of a fused [B, S, heads, 3, d] buffer
    fused = torch.full((w.B, w.S, w.heads, 3, w.head_dim), float("nan"), dtype=q.dtype, device=q.device)
    L.backward(do, fused[:, :, :, 0], fused[:, :, :, 1], fused[:, :, :, 2], fold_inverse=True)     # dO block-major
    torch.cuda.synchronize()
    L.check_status()
    assert torch.equal(fused[:, :, :, 1], ref[1]) and torch.equal(fused[:, :, :, 2], ref[2])


@pytest.mark.parametrize("block", [(1, 12, 26), (3, 6, 13)], ids=["1d", "3d"])
def test_forward_writing_raster_order_equals_inverse_partition(block):
    """vmoba_attn_fwd_raster folds the inverse of Eq. 1 into the forward's row writes (directly written rows and merged
    rows): o must equal vmoba_attn_fwd + inverse partition bit for bit, lse and the rounding residual must not change,
    and the backward reading that raster-order o must give the gradients of the block-major route (dK, dV bit for
    bit, dQ up to the order of its fp32 sum)."""
    w = MID.with_(block=block)
    data = gen.make_inputs(w)
    shape = vb.shape_of(w)
    L = VmobaLayer(shape, capacity=default_capacity(shape, w.tau), with_backward=True)
    q, k, v, do = (U.to_device(w, data, n) for n in ("q", "k", "v", "do"))
    o_ref = torch.empty_like(q)
    L.forward(q, k, v, w.tau, o_ref, fold_o=False)
    g_ref = [torch.empty_like(q) for _ in range(3)]
    L.backward(do, *g_ref)
    torch.cuda.synchronize()
    lse_ref, resid_ref = L.lse.clone(), L.o_resid.clone()
    # a strided destination: o as one slice of a [B, S, heads, 2, d] buffer
    buf = torch.full((w.B, w.S, w.heads, 2, w.head_dim), float("nan"), dtype=q.dtype, device=q.device)
    o_got = buf[:, :, :, 1]
    L.forward(q, k, v, w.tau, o_got, fold_o=True)
    g_got = [torch.empty_like(q) for _ in range(3)]
    L.backward(do, *g_got)
    torch.cuda.synchronize()
    L.check_status()
    assert torch.equal(o_got, o_ref)
    assert torch.isnan(buf[:, :, :, 0].float()).all()
    assert torch.equal(L.lse, lse_ref) and torch.equal(L.o_resid, resid_ref)
    assert torch.equal(g_got[1], g_ref[1]) and torch.equal(g_got[2], g_ref[2])
    diff = (g_got[0].float() - g_ref[0].float()).abs().max().item()
    assert diff <= 2.0 ** -6 * max(1.0, g_ref[0].float().abs().max().item())
    # and the block-major backward after a raster forward (o_bm rebuilt from the raster tensor)
    g_bm = [torch.empty_like(q) for _ in range(3)]
    L.backward(do, *g_bm, fold_inverse=False)
    torch.cuda.synchronize()
    assert torch.equal(g_bm[1], g_ref[1]) and torch.equal(g_bm[2], g_ref[2])


def test_repeated_runs_reproduce():
    """Everything but dQ is written once, by one owner: repeated runs must agree bit for bit (a race between the
    roles of a kernel shows up here first).  dQ is an fp32 sum of per-key-tile parts whose order is not fixed."""
    w = MID.with_(block=(1, 12, 26))
    data = gen.make_inputs(w)
    runs = [_run_layer(w, data, with_bwd=True) for _ in range(3)]
    for r in runs[1:]:
        for name in ("o", "dk", "dv"):
            assert torch.equal(r[name], runs[0][name]), name
        assert torch.equal(r["L"].lse, runs[0]["L"].lse)
        diff = (r["dq"].float() - runs[0]["dq"].float()).abs().max().item()
        assert diff <= 2.0 ** -6 * max(1.0, runs[0]["dq"].float().abs().max().item())


def test_section_timers_leave_results_unchanged():
    """The diagnostic counters (cycles per warp role and loop section) fill in when a buffer is registered and the
    outputs stay bit-identical (dQ up to its summation order)."""
    w = MID.with_(block=(1, 12, 26))
    data = gen.make_inputs(w)
    plain = _run_layer(w, data, with_bwd=True)
    counters = torch.zeros(16, dtype=torch.int64, device="cuda")
    vb.vmoba_debug_wait_profile(counters)
    try:
        timed = _run_layer(w, data, with_bwd=True)
        torch.cuda.synchronize()
    finally:
        vb.vmoba_debug_wait_profile(None)
    c = counters.cpu().numpy()
    assert c[6] > 0 and c[13] > 0 and c[8] > 0      # totals of three roles
    assert np.all(c >= 0)
    for name in ("o", "dk", "dv"):
        assert torch.equal(timed[name], plain[name]), name
    diff = (timed["dq"].float() - plain["dq"].float()).abs().max().item()
    assert diff <= 2.0 ** -6 * max(1.0, plain["dq"].float().abs().max().item())
    after = _run_layer(w, data, with_bwd=True)        # cleared: the buffer is no longer written
    torch.cuda.synchronize()
    assert np.array_equal(counters.cpu().numpy(), c)
    assert torch.equal(after["o"], plain["o"])


def test_mid_size_threshold_one_equals_dense_path():
    """tau = 1.0 through the sparse pipeline must equal the library's dense path and the oracle's dense attention."""
    w = MID.with_(tau=1.0, B=1, heads=2)
    data = gen.make_inputs(w)
    res = _run_layer(w, data, with_bwd=False, capacity=w.B * w.heads * w.S * w.n_blocks)
    shape = vb.shape_of(w)
    q, k, v = (U.to_device(w, data, n).permute(0, 2, 1, 3).contiguous() for n in "qkv")     # [B, heads, S, d] raster order
    o = torch.empty_like(q)
    lse = torch.empty(w.B * w.heads * w.S, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    vb.vmoba_full_attn(shape, q, k, v, o, lse, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    sparse = U.to_numpy_f32(res["o"].permute(0, 2, 1, 3))
    dense = U.to_numpy_f32(o)
    # two independently rounded bf16 results may sit one bf16 ulp apart (1.6e-2 at most below |o| = 4)
    U.assert_close(sparse, dense, w.dtype, "o sparse route at tau = 1 vs dense path")
    for h in range(w.heads):
        od, _ = orc.dense_attn_fwd(data["q"][0, :, h], data["k"][0, :, h], data["v"][0, :, h], w.head_dim ** -0.5,
                                   rows=np.arange(0, w.S, 7))
        U.assert_close(dense[0, h][::7], od, w.dtype, "dense path vs oracle")


# ---- the benchmark configurations at full size, sampled -----------------------------------
def _full_size(w, with_bwd, heads_checked, n_rows=96, n_blocks=2, capacity=None):
    data = gen.make_inputs(w, with_do=with_bwd)
    res = _run_layer(w, data, with_bwd, capacity=capacity)
    rng = np.random.default_rng(2)
    dens = []
    for (b, h) in heads_checked:
        dens.append(_check_head(w, data, res, b, h, rng, n_rows, n_blocks, with_bwd))
    return res, dens


def test_config2_wan_layer_3d_forward():
    res, dens = _full_size(gen.C2, False, [(0, 0), (0, 7)])
    assert all(0 < d <= 0.25 for d in dens)


@pytest.mark.parametrize("name", ["1d", "2d"])
def test_config3_partitions_forward(name):
    w = gen.C2.with_(name="c3_" + name, block=gen.C3_BLOCKS[name])
    _full_size(w, False, [(0, 3)])


@pytest.mark.parametrize("tau", [0.1, 0.5])
def test_config3_threshold_sweep_3d(tau):
    w = gen.C2.with_(name=f"c3_tau{tau}", tau=tau, heads=4)
    res, dens = _full_size(w, False, [(0, 1)])
    assert dens[0] <= tau


def test_config4_training_step():
    res, dens = _full_size(gen.C4, True, [(1, 5)])


@pytest.mark.parametrize("name", ["1d", "2d", "3d"])
def test_config5_720p_shape_forward_backward(name):
    """Config 5's grid and block shapes with 4 of its 40 heads (per-head work is independent;
    the input generator is the bottleneck of this test, not the GPU)."""
    w = gen.C5.with_(name="c5_" + name, block=gen.C5_BLOCKS[name], heads=4)
    shape = vb.shape_of(w)
    cap = int(0.3 * default_capacity(shape, w.tau)) if name == "3d" else None
    _full_size(w, True, [(0, 2)], n_rows=48, n_blocks=1, capacity=cap)


def _measured_capacity(w, data):
    """Work-list capacity from a scores + selection pass of its own (the way bench.py sizes its lists)."""
    shape = vb.shape_of(w)
    probe = VmobaLayer(shape, capacity=1)
    q, k = (U.to_device(w, data, n) for n in "qk")
    probe.partition(q, probe.q_bm); probe.partition(k, probe.k_bm)
    probe.block_scores(); probe.select(w.tau)
    torch.cuda.synchronize()
    n = probe.n_selected()
    del probe, q, k
    torch.cuda.empty_cache()
    return int(n * 1.05) + 4096


@pytest.mark.parametrize("name", ["2d", "3d"])
def test_config5_all_40_heads_one_layer(name):
    """Config 5 exactly as bench.py times it (B=1, 40 heads, 75,600 tokens, lists sized from a selection pass),
    the 2D layer and the 3D layer (17 million pairs, the longest lists), forward and backward; sampled rows and
    key blocks of the first and the last head against the oracle."""
    w = gen.C5.with_(name="c5_full_" + name, block=gen.C5_BLOCKS[name])
    data = gen.make_inputs(w, with_do=True)
    res = _run_layer(w, data, True, capacity=_measured_capacity(w, data))
    rng = np.random.default_rng(2)
    for (b, h) in [(0, 0), (0, 39)]:
        _check_head(w, data, res, b, h, rng, 32, 1, True)


@pytest.mark.parametrize("grid", ["t55k", "t56k"])
@pytest.mark.parametrize("name", ["1d", "2d", "3d"])
def test_paper_training_grids_forward_backward(grid, name):
    """The paper's two fine-tuning grids with its own block sizes (Table 4): latent 24 x 36 x 64 with 8 / 48 / 72
    blocks of 6912 / 1152 / 768 keys, latent 36 x 30 x 52 with 12 / 24 / 36 blocks of 4680 / 2340 / 1560 keys;
    tau = 0.25, forward and backward, four heads, one of them against the oracle on sampled rows and a key block."""
    base, blocks = (gen.T55, gen.T55_BLOCKS) if grid == "t55k" else (gen.T56, gen.T56_BLOCKS)
    w = base.with_(name=f"{grid}_{name}", block=blocks[name], heads=4)
    _full_size(w, True, [(0, 3)], n_rows=48, n_blocks=1)


def test_bounded_wait_runs_out_cleanly_and_the_library_keeps_working():
    """The device-side failure detector: a wait on a barrier that nothing arrives at gives up after its poll limit,
    the status word receives VMOBA_ERR_TIMEOUT, the CTA's later waits drain at once and the kernel ends by itself
    (no trap, no hang); the context stays usable: a forward + backward right afterwards still matches the oracle."""
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = torch.zeros(2, dtype=torch.int32, device="cuda")
    vb.vmoba_debug_wait_timeout(st, 300, out)
    torch.cuda.synchronize()
    assert int(st.item()) == vb.ERR_TIMEOUT
    assert out.tolist() == [128, 1]            # both waits of all 64 threads gave up; the kernel ran to its end
    with pytest.raises(vb.VmobaError):
        vb.vmoba_debug_wait_timeout(st, 0, out)        # host-side argument check
    w = MID.with_(block=(3, 6, 13), B=1, heads=2)
    data = gen.make_inputs(w)
    res = _run_layer(w, data, with_bwd=True)
    rng = np.random.default_rng(4)
    for h in range(w.heads):
        _check_head(w, data, res, 0, h, rng, n_rows=200, n_blocks=2, with_bwd=True)
