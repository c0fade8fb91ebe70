"""The range-checked build of the library (-DVMOBA_DEBUG, lib/libvmoba_debug.so): every index read from a work list
is checked before use and every workspace slice is followed by a guard zone that is verified after the stage's
kernels.  It stands in for a memory checker: the mid-size parity cases must run through it with the status word
clean, and a planted out-of-range list entry must be reported (and not followed: the access is redirected to
element 0, so nothing faults)."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _debug_env():
    from paper_2506_23858_b200 import build
    return dict(os.environ, VMOBA_LIB=build.ensure_built(debug=True))


def test_mid_size_cases_run_clean_through_the_range_checked_build():
    r = subprocess.run([sys.executable, "-m", "pytest", "tests/test_gpu_layer.py", "tests/test_gpu_stages.py", "-m", "gpu",
                        "-q", "-x", "-p", "no:cacheprovider", "-k",
                        "mid_size or tails or select_matches or sparse_attention_forward_backward or raster or dense_attention"],
                       env=_debug_env(), cwd=ROOT, capture_output=True, text=True, timeout=1200)
    assert r.returncode == 0, r.stdout[-3000:] + r.stderr[-1000:]
    assert " passed" in r.stdout


PLANT = r"""
import numpy as np, torch
from paper_2506_23858_b200 import binding as vb, inputs as gen
from paper_2506_23858_b200.layer import VmobaLayer, default_capacity
w = gen.Workload("mid", 1, 2, 128, 6, 12, 26, (3, 6, 13), 0.25, "bf16", "smooth", 5)
data = gen.make_inputs(w, with_do=False)
shape = vb.shape_of(w)
L = VmobaLayer(shape, capacity=default_capacity(shape, w.tau))
dev = lambda n: torch.from_numpy(data[n + "_bits"].view(np.int16)).cuda().view(torch.bfloat16)
o = torch.empty_like(dev("q"))
L.forward(dev("q"), dev("k"), dev("v"), w.tau, o)
torch.cuda.synchronize()
print("clean", int(L.dev_status.item()))
L.q_idx[3] = w.S + 7            # a query position beyond the head
L.q_idx[11] = -2
L.attn_fwd()
torch.cuda.synchronize()
print("planted", int(L.dev_status.item()))
"""


def test_planted_out_of_range_entry_is_reported_by_the_range_checked_build():
    r = subprocess.run([sys.executable, "-c", PLANT], env=_debug_env(), cwd=ROOT, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stdout[-2000:] + r.stderr[-2000:]
    lines = dict(l.split() for l in r.stdout.strip().splitlines() if l.split()[0] in ("clean", "planted"))
    assert lines["clean"] == "0"
    assert lines["planted"] == "8"          # VMOBA_ERR_BOUNDS
