"""vmoba_select_static -- the selection stage for callers that cannot allocate device memory
(plug-ins in memory-planned engines, serving loops where cudaMalloc is banned) -- must give the
same lists as vmoba_select.  Called twice in a row, because both calls share the library's one
built-in scratch array and the second sees whatever the first left behind.

This file is collected last on purpose: a run that stops at the first failure has then already
run every other test."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2506_23858_b200 import binding as vb
from paper_2506_23858_b200 import inputs as gen

SCORE_BAND = 1e-3     # the same cutoff band the other selection tests use


def _select_buffers(shape, capacity):
    BH, S, Nb = shape.B * shape.heads, shape.S, shape.n_blocks
    dev = "cuda"
    return dict(
        mask_bits=torch.zeros((BH * S, shape.mask_words), dtype=torch.int32, device=dev),
        kb_ptr=torch.zeros(BH * Nb + 1, dtype=torch.int32, device=dev),
        q_idx=torch.zeros(capacity, dtype=torch.int32, device=dev),
        q_ptr=torch.zeros(BH * S + 1, dtype=torch.int32, device=dev),
        q_pairs=torch.zeros(capacity, dtype=torch.int32, device=dev),
        k_per_head=torch.zeros(BH, dtype=torch.int64, device=dev),
        cutoff=torch.zeros(BH, dtype=torch.float32, device=dev),
        status=torch.zeros(1, dtype=torch.int32, device=dev),
    )


def _compare(a, b, scores, shape):
    """Same inputs, same algorithm: the two entry points may differ only where fp summation order
    moves the cutoff, i.e. on pairs inside the cutoff band."""
    BH, S, Nb = shape.B * shape.heads, shape.S, shape.n_blocks
    ca, cb = a["cutoff"].cpu().numpy(), b["cutoff"].cpu().numpy()
    assert np.all(np.abs(ca - cb) <= SCORE_BAND)
    wa = a["mask_bits"].cpu().numpy().view(np.uint32).reshape(BH, S, -1)
    wb = b["mask_bits"].cpu().numpy().view(np.uint32).reshape(BH, S, -1)
    ma = ((wa[..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(BH, S, -1)[..., :Nb].astype(bool)
    mb = ((wb[..., None] >> np.arange(32, dtype=np.uint32)) & 1).reshape(BH, S, -1)[..., :Nb].astype(bool)
    sc = scores.cpu().numpy().reshape(BH, S, Nb)
    decided = np.abs(sc - cb[:, None, None]) > SCORE_BAND
    assert np.array_equal(ma[decided], mb[decided])
    if np.array_equal(ma, mb):          # the usual case: bit-identical selection => identical lists
        for name in ("kb_ptr", "q_ptr", "k_per_head"):
            assert torch.equal(a[name], b[name]), name
        n = int(a["kb_ptr"][-1].item())
        assert torch.equal(a["q_idx"][:n], b["q_idx"][:n]) and torch.equal(a["q_pairs"][:n], b["q_pairs"][:n])
    assert int(a["status"].item()) == 0 and int(b["status"].item()) == 0


@pytest.mark.gpu
def test_select_static_matches_select_twice_in_a_row():
    torch.manual_seed(0)
    cases = [
        (vb.make_shape(1, 2, 64, (4, 8, 8), (1, 8, 8), "f32"), 0.25),
        (vb.make_shape(2, 3, 128, (6, 12, 26), (1, 3, 13), "bf16"), 0.4),
    ]
    for shape, tau in cases:
        assert vb.workspace_bytes(shape, vb.STAGE_SELECT) <= vb.select_static_scratch_bytes()
        BH, S, Nb = shape.B * shape.heads, shape.S, shape.n_blocks
        capacity = BH * S * Nb
        ws = torch.empty(vb.workspace_bytes(shape, vb.STAGE_SELECT), dtype=torch.uint8, device="cuda")
        for call in range(2):
            scores = (3.0 * torch.randn(BH * S * Nb, device="cuda")).contiguous()
            ref, got = _select_buffers(shape, capacity), _select_buffers(shape, capacity)
            vb.vmoba_select(shape, scores, tau, ref["mask_bits"], ref["kb_ptr"], ref["q_idx"], ref["q_ptr"],
                            ref["q_pairs"], capacity, ref["k_per_head"], ref["cutoff"], ref["status"], ws)
            vb.vmoba_select_static(shape, scores, tau, got["mask_bits"], got["kb_ptr"], got["q_idx"], got["q_ptr"],
                                   got["q_pairs"], capacity, got["k_per_head"], got["cutoff"], got["status"])
            torch.cuda.synchronize()
            assert int(got["k_per_head"].sum().item()) > 0
            _compare(got, ref, scores, shape)


def test_select_static_rejects_shapes_beyond_its_scratch():
    big = vb.make_shape(4, 40, 128, (21, 45, 80), (3, 9, 10), "bf16")
    assert vb.workspace_bytes(big, vb.STAGE_SELECT) > vb.select_static_scratch_bytes()
    fake = ctypes.c_void_p(0x1000)          # never dereferenced: the size check comes first
    rc = vb.lib().vmoba_select_static(ctypes.byref(big), fake, ctypes.c_float(0.25), fake, fake, fake, fake, fake,
                                      1 << 20, fake, fake, fake, None)
    assert rc == vb.ERR_WORKSPACE
