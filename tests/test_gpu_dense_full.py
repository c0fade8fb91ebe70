"""The dense path (vmoba_full_attn: the tau = 1 limit of the layer and the speed-up denominator, Section 4.1's
"Full Attention") and the tau = 1 route through the sparse pipeline at the benchmark sequence lengths.

Rows of attention are independent, so o, lse and dq of sampled query rows are exact against the oracle at any
size; dk and dv need every query, so they are compared element by element on a case the oracle can afford in
full (8,190 tokens: 64 query units per key tile) and through column sums that hold at any size
(sum_t dV_t = sum_q dO_q because softmax rows sum to one; sum_t dK_t = 0 because a shift of all keys changes
nothing)."""
import numpy as np
import pytest
import torch

from oracle import vmoba_oracle as orc
from paper_2506_23858_b200 import binding as vb
from paper_2506_23858_b200 import inputs as gen
from paper_2506_23858_b200.layer import VmobaLayer
from tests import _util as U

pytestmark = pytest.mark.gpu


def _dense_run(w, data, with_bwd):
    """vmoba_full_attn on [B, heads, S, d] raster-order tensors; returns torch results."""
    shape = vb.shape_of(w)
    q, k, v = (U.to_device(w, data, n).permute(0, 2, 1, 3).contiguous() for n in "qkv")
    o = torch.empty_like(q)
    lse = torch.empty(w.B * w.heads * w.S, dtype=torch.float32, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = dict(o=o, lse=lse)
    if with_bwd:
        do = U.to_device(w, data, "do").permute(0, 2, 1, 3).contiguous()
        out["dq"], out["dk"], out["dv"] = (torch.empty_like(q) for _ in range(3))
        ws = torch.empty(vb.workspace_bytes(shape, vb.STAGE_FULL_BWD), dtype=torch.uint8, device="cuda")
        vb.vmoba_full_attn(shape, q, k, v, o, lse, do, out["dq"], out["dk"], out["dv"], st, ws)
    else:
        vb.vmoba_full_attn(shape, q, k, v, o, lse, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    return out


def _check_rows(w, data, res, h, rows, with_bwd):
    """o, lse (and dq) of sampled rows of head h against the oracle's dense attention."""
    scale = w.head_dim ** -0.5
    q, k, v = (data[n][0, :, h] for n in "qkv")
    o_ref, lse_ref = orc.dense_attn_fwd(q, k, v, scale, rows=rows)
    ridx = torch.from_numpy(rows.astype(np.int64)).cuda()
    U.assert_close(U.to_numpy_f32(res["o"][0, h, ridx]), o_ref, w.dtype, f"o dense head {h}")
    lse = res["lse"].view(w.B, w.heads, w.S)[0, h, ridx].cpu().numpy()
    assert U.max_abs(lse, lse_ref) <= 2e-2
    if with_bwd:
        everything = np.ones((w.S, 1), dtype=bool)             # one block holding every key: the full mask
        dq_ref, _, _ = orc.sparse_attn_bwd(q, k, v, everything, scale, data["do"][0, :, h], rows=rows)
        U.assert_close(U.to_numpy_f32(res["dq"][0, h, ridx]), dq_ref, w.dtype, f"dq dense head {h}")


def _check_column_sums(w, data, res, h):
    S = w.S
    do = data["do"][0, :, h].astype(np.float64)
    dv = res["dv"][0, h].double()
    dk = res["dk"][0, h].double()
    eps = 2.0 ** -9
    want = do.sum(axis=0)
    tol_v = 6.0 * np.sqrt(S) * eps * float(dv.pow(2).mean().sqrt()) + 1e-3 * np.abs(want).max() + 1e-4
    assert U.max_abs(dv.sum(dim=0).cpu().numpy(), want) <= tol_v
    scale = w.head_dim ** -0.5
    tol_k = 6.0 * np.sqrt(S) * eps * float(dk.pow(2).mean().sqrt()) + 1e-4 + 3.0 * scale * np.sqrt(S) * eps * np.sqrt(w.head_dim)
    assert float(dk.sum(dim=0).abs().max()) <= tol_k


def test_dense_path_8190_tokens_every_gradient_element():
    """Grid 21 x 30 x 13: the dense backward walks 64 query units per key tile (the mid-size cases walk 15);
    o, dq, dk, dv of both heads element by element against the oracle's matrix-form gradient."""
    w = gen.Workload("dense_8k", 1, 2, 128, 21, 30, 13, (21, 30, 13), 1.0, "bf16", "smooth", 21)
    data = gen.make_inputs(w)
    res = _dense_run(w, data, True)
    scale = w.head_dim ** -0.5
    for h in range(w.heads):
        q, k, v, do = (data[n][0, :, h] for n in ("q", "k", "v", "do"))
        o_ref, lse_ref = orc.dense_attn_fwd(q, k, v, scale, rows=np.arange(0, w.S, 5))
        U.assert_close(U.to_numpy_f32(res["o"][0, h, ::5]), o_ref, w.dtype, f"o dense head {h}")
        dq_ref, dk_ref, dv_ref = orc.dense_attn_bwd(q, k, v, scale, do)
        for name, ref in (("dq", dq_ref), ("dk", dk_ref), ("dv", dv_ref)):
            U.assert_close(U.to_numpy_f32(res[name][0, h]), ref, w.dtype, f"{name} dense head {h}")


@pytest.mark.parametrize("base,heads", [(gen.C2, 2), (gen.C5, 1)], ids=["32760_tokens", "75600_tokens"])
def test_dense_path_at_benchmark_lengths(base, heads):
    """vmoba_full_attn forward + backward at the sequence lengths of configs 2-4 and of config 5."""
    w = base.with_(name="dense_full", heads=heads, tau=1.0)
    data = gen.make_inputs(w)
    res = _dense_run(w, data, True)
    rng = np.random.default_rng(5)
    for h in range(w.heads):
        _check_rows(w, data, res, h, rng.choice(w.S, size=24, replace=False), True)
        _check_column_sums(w, data, res, h)


@pytest.mark.parametrize("name", ["1d", "2d", "3d"])
def test_config3_threshold_one_equals_dense_at_full_size(name):
    """Config 3's tau = 1.0 at 32,760 tokens: the sparse pipeline with every pair selected (one head per
    partition type) against the oracle's dense attention on sampled rows, and against the library's dense path."""
    w = gen.C2.with_(name="c3_tau1_" + name, block=gen.C3_BLOCKS[name], heads=1, tau=1.0)
    data = gen.make_inputs(w, with_do=False)
    shape = vb.shape_of(w)
    L = VmobaLayer(shape, capacity=w.S * w.n_blocks)
    q, k, v = (U.to_device(w, data, n) for n in "qkv")
    o = torch.empty_like(q)
    L.forward(q, k, v, 1.0, o)
    torch.cuda.synchronize()
    L.check_status()
    assert L.n_selected() == w.S * w.n_blocks
    rows = np.random.default_rng(6).choice(w.S, size=24, replace=False)
    scale = w.head_dim ** -0.5
    o_ref, lse_ref = orc.dense_attn_fwd(data["q"][0, :, 0], data["k"][0, :, 0], data["v"][0, :, 0], scale, rows=rows)
    ridx = torch.from_numpy(rows.astype(np.int64)).cuda()
    U.assert_close(U.to_numpy_f32(o[0, ridx, 0]), o_ref, w.dtype, "o sparse route at tau = 1")
    perm, inv = orc.partition_perm(w.T, w.H, w.W, *w.block)
    lse = L.lse.cpu().numpy()[inv[rows]]
    assert U.max_abs(lse, lse_ref) <= 2e-2
    dense = _dense_run(w, data, False)
    U.assert_close(U.to_numpy_f32(o[0, :, 0]), U.to_numpy_f32(dense["o"][0, 0]), w.dtype, "o sparse route vs dense path")


def test_sampler_switch_runs_dense_then_sparse():
    """The host-side rule of Section 4.1 (first quarter of the steps dense): step 0 of 4 must give dense attention,
    the later steps the sparse layer's output."""
    from paper_2506_23858_b200.layer import SteppedAttention, default_capacity
    w = gen.Workload("mid", 1, 2, 128, 6, 12, 26, (3, 6, 13), 0.25, "bf16", "smooth", 5)
    data = gen.make_inputs(w, with_do=False)
    shape = vb.shape_of(w)
    L = VmobaLayer(shape, capacity=default_capacity(shape, w.tau))
    sw = SteppedAttention(L, w.tau, n_steps=4)
    q, k, v = (U.to_device(w, data, n) for n in "qkv")
    outs, paths = [], []
    for step in range(4):
        o = torch.empty_like(q)
        paths.append(sw.forward(step, q, k, v, o))
        outs.append(o)
    torch.cuda.synchronize()
    L.check_status()
    assert paths == ["dense", "sparse", "sparse", "sparse"]
    scale = w.head_dim ** -0.5
    for h in range(w.heads):
        od, _ = orc.dense_attn_fwd(data["q"][0, :, h], data["k"][0, :, h], data["v"][0, :, h], scale)
        U.assert_close(U.to_numpy_f32(outs[0][0, :, h]), od, w.dtype, "o dense step")
    ref = torch.empty_like(q)
    L.forward(q, k, v, w.tau, ref)
    torch.cuda.synchronize()
    assert torch.equal(outs[1], ref) and torch.equal(outs[3], ref)
    assert not torch.equal(outs[0], ref)
