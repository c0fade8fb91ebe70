"""The C-ABI library loads without a GPU and exports every symbol include/vmoba.h declares;
host-side argument checks return the documented codes (no kernel is launched here)."""
import ctypes
import os
import re

from paper_2506_23858_b200 import binding as vb
from paper_2506_23858_b200 import build as vbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "vmoba.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(vmoba_[a-z_]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    vbuild.ensure_built()
    L = ctypes.CDLL(vb.lib_path())
    declared = _declared_symbols()
    assert set(vb.EXPORTS) <= set(declared)
    assert len(declared) >= 8
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings_and_workspace_sizes():
    assert vb.status_string(vb.OK) == "ok"
    assert "capacity" in vb.status_string(vb.ERR_CAPACITY)
    s = vb.make_shape(1, 12, 128, (21, 30, 52), (3, 6, 13), "bf16")
    assert (s.S, s.n_blocks, s.block_tokens, s.mask_words) == (32760, 140, 234, 5)
    for stage in range(6):
        assert vb.workspace_bytes(s, stage, 1 << 20) > 0
    assert vb.workspace_bytes(s, 99, 0) == 0
    assert vb.workspace_bytes(s, vb.STAGE_ATTN_FWD, 2 << 20) > vb.workspace_bytes(s, vb.STAGE_ATTN_FWD, 1 << 20)
    bad = vb.make_shape(1, 12, 128, (21, 30, 52), (4, 6, 13), "bf16")     # 21 % 4 != 0
    assert vb.workspace_bytes(bad, vb.STAGE_SELECT, 0) == 0


def test_host_side_argument_checks():
    L = vb.lib()
    good = vb.make_shape(1, 2, 64, (4, 8, 8), (1, 8, 8), "f32")
    strides = (ctypes.c_int64 * 3)(4 * 8 * 8 * 2 * 64, 2 * 64, 64)
    null = ctypes.c_void_p(None)
    fake = ctypes.c_void_p(0x1000)                     # aligned, never dereferenced: checks fail first
    assert L.vmoba_partition(ctypes.byref(good), 0, null, fake, strides, null, null, null) == vb.ERR_ARG
    assert L.vmoba_partition(ctypes.byref(good), 0, ctypes.c_void_p(0x1004), fake, strides, null, null, null) == vb.ERR_ARG
    assert L.vmoba_partition(ctypes.byref(good), 2, fake, fake, strides, null, null, null) == vb.ERR_ARG
    for bad, code in (
        (vb.make_shape(1, 2, 64, (4, 8, 8), (3, 8, 8), "f32"), vb.ERR_SHAPE),     # grid not divisible
        (vb.make_shape(1, 2, 96, (4, 8, 8), (1, 8, 8), "f32"), vb.ERR_SHAPE),     # head_dim
        (vb.make_shape(0, 2, 64, (4, 8, 8), (1, 8, 8), "f32"), vb.ERR_SHAPE),
        (vb.make_shape(1, 2, 64, (4, 8, 8), (1, 8, 8), 7), vb.ERR_ARG),           # dtype enum
    ):
        assert L.vmoba_partition(ctypes.byref(bad), 0, fake, fake, strides, null, null, null) == code
    # tau outside (0, 1]
    args = [fake] * 5
    for tau in (0.0, -0.1, 1.5, float("nan")):
        rc = L.vmoba_select(ctypes.byref(good), fake, ctypes.c_float(tau), fake, fake, fake, fake, fake, 1024, fake,
                            fake, fake, fake, 1 << 30, null)
        assert rc == vb.ERR_ARG, tau
    # workspace too small
    rc = L.vmoba_select(ctypes.byref(good), fake, ctypes.c_float(0.25), fake, fake, fake, fake, fake, 1024, fake, fake,
                        fake, fake, 16, null)
    assert rc == vb.ERR_WORKSPACE
    rc = L.vmoba_attn_fwd(ctypes.byref(good), fake, fake, fake, fake, fake, fake, fake, 1024, fake, null, fake, fake,
                          fake, 16, null)
    assert rc == vb.ERR_WORKSPACE
