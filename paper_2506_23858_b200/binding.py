"""ctypes binding of ``libvmoba.so``: the same entry points as ``include/vmoba.h``, taking torch
CUDA tensors and passing their device pointers through.  Argument marshalling only -- every
step of the layer runs in the library's kernels.  There is no CPU fallback: if the library is
missing, or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import math
import os

from . import build as _build

OK, ERR_ARG, ERR_SHAPE, ERR_WORKSPACE, ERR_CAPACITY, ERR_TIMEOUT, ERR_CUDA, ERR_NOT_IMPLEMENTED, ERR_BOUNDS = range(9)
F32, BF16 = 0, 1
STAGE_SCORES, STAGE_SELECT, STAGE_ATTN_FWD, STAGE_ATTN_BWD, STAGE_FULL_FWD, STAGE_FULL_BWD, STAGE_SELECT_ROWNORM = range(7)

EXPORTS = (
    "vmoba_status_string", "vmoba_kernel_launches", "vmoba_workspace_bytes", "vmoba_partition", "vmoba_block_scores",
    "vmoba_block_scores_range", "vmoba_select", "vmoba_select_rule_apply", "vmoba_select_ranged", "vmoba_select_static", "vmoba_select_static_scratch_bytes", "vmoba_attn_fwd",
    "vmoba_attn_fwd_raster", "vmoba_attn_bwd", "vmoba_attn_bwd_raster", "vmoba_full_attn",
    "vmoba_debug_wait_profile", "vmoba_debug_wait_timeout",
)


class VmobaError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__(f"{where}: status {code} ({status_string(code)})")


class Shape(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in ("B", "heads", "head_dim", "T", "H", "W", "bT", "bH", "bW", "dtype")] + [
        ("softmax_scale", ctypes.c_float)]

    @property
    def S(self):
        return self.T * self.H * self.W

    @property
    def n_blocks(self):
        return (self.T // self.bT) * (self.H // self.bH) * (self.W // self.bW)

    @property
    def block_tokens(self):
        return self.bT * self.bH * self.bW

    @property
    def mask_words(self):
        return (self.n_blocks + 31) // 32

    @property
    def scale(self):
        return self.softmax_scale if self.softmax_scale > 0 else 1.0 / math.sqrt(self.head_dim)


def make_shape(B, heads, head_dim, grid, block, dtype, softmax_scale=0.0) -> Shape:
    code = {"f32": F32, "bf16": BF16}[dtype] if isinstance(dtype, str) else int(dtype)
    return Shape(B, heads, head_dim, grid[0], grid[1], grid[2], block[0], block[1], block[2], code, softmax_scale)


def shape_of(w) -> Shape:
    """Shape of an ``inputs.Workload``."""
    return make_shape(w.B, w.heads, w.head_dim, (w.T, w.H, w.W), w.block, w.dtype)


_lib = None


def lib_path() -> str:
    """The in-tree library, or the file VMOBA_LIB names (another build of this same library)."""
    return os.environ.get("VMOBA_LIB") or _build.LIB_PATH


def lib():
    """Loads the C-ABI library (built in-tree by ``build.py``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if path == _build.LIB_PATH:
        _build.ensure_built()   # rebuilds when a source is newer than the library; needs nvcc, raises if the build
                                # fails -- there is no CPU fallback
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: run `python -m paper_2506_23858_b200.build` (no CPU fallback exists)")
    L = ctypes.CDLL(path)
    vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_size_t
    sp = ctypes.POINTER(Shape)
    L.vmoba_status_string.restype = ctypes.c_char_p
    L.vmoba_status_string.argtypes = [ctypes.c_int]
    L.vmoba_kernel_launches.restype = ctypes.c_uint64
    L.vmoba_kernel_launches.argtypes = []
    L.vmoba_workspace_bytes.restype = sz
    L.vmoba_workspace_bytes.argtypes = [sp, ctypes.c_int, i64]
    L.vmoba_partition.restype = ctypes.c_int
    L.vmoba_partition.argtypes = [sp, ctypes.c_int, vp, vp, ctypes.POINTER(i64), vp, vp, vp]
    L.vmoba_block_scores.restype = ctypes.c_int
    L.vmoba_block_scores.argtypes = [sp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.vmoba_block_scores_range.restype = ctypes.c_int
    L.vmoba_block_scores_range.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    L.vmoba_select_ranged.restype = ctypes.c_int
    L.vmoba_select_ranged.argtypes = [sp, vp, vp, ctypes.c_int32, ctypes.c_float, ctypes.c_int32, vp, vp, vp, vp, vp, i64, vp,
                                      vp, vp, vp, sz, vp]
    L.vmoba_select.restype = ctypes.c_int
    L.vmoba_select.argtypes = [sp, vp, ctypes.c_float, vp, vp, vp, vp, vp, i64, vp, vp, vp, vp, sz, vp]
    L.vmoba_select_static.restype = ctypes.c_int
    L.vmoba_select_rule_apply.restype = ctypes.c_int
    L.vmoba_select_rule_apply.argtypes = [sp, vp, ctypes.c_int32, ctypes.c_float, ctypes.c_int32, vp, vp, vp, vp, vp, i64, vp, vp, vp,
                                          vp, sz, vp]
    L.vmoba_select_static.argtypes = [sp, vp, ctypes.c_float, vp, vp, vp, vp, vp, i64, vp, vp, vp, vp]
    L.vmoba_select_static_scratch_bytes.restype = sz
    L.vmoba_select_static_scratch_bytes.argtypes = []
    L.vmoba_attn_fwd.restype = ctypes.c_int
    L.vmoba_attn_fwd.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, sz, vp]
    L.vmoba_attn_bwd.restype = ctypes.c_int
    L.vmoba_attn_bwd.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i64, vp, vp, vp, vp, vp, sz, vp]
    L.vmoba_attn_bwd_raster.restype = ctypes.c_int
    p64 = ctypes.POINTER(ctypes.c_int64)
    L.vmoba_attn_bwd_raster.argtypes = [sp, vp, vp, vp, vp, p64, vp, vp, vp, p64, vp, vp, vp, i64,
                                        vp, vp, vp, p64, vp, vp, vp, sz, vp]
    L.vmoba_attn_fwd_raster.restype = ctypes.c_int
    L.vmoba_attn_fwd_raster.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, i64, vp, p64, vp, vp, vp, vp, vp, sz, vp]
    L.vmoba_debug_wait_timeout.restype = ctypes.c_int
    L.vmoba_debug_wait_timeout.argtypes = [vp, ctypes.c_uint32, vp, vp]
    L.vmoba_debug_wait_profile.restype = None
    L.vmoba_debug_wait_profile.argtypes = [vp]
    L.vmoba_full_attn.restype = ctypes.c_int
    L.vmoba_full_attn.argtypes = [sp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    _lib = L
    return L


def status_string(code: int) -> str:
    return lib().vmoba_status_string(int(code)).decode()


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(code, where):
    if code != OK:
        raise VmobaError(code, where)


def kernel_launches() -> int:
    return int(lib().vmoba_kernel_launches())


def workspace_bytes(shape: Shape, stage: int, capacity: int = 0) -> int:
    return int(lib().vmoba_workspace_bytes(ctypes.byref(shape), stage, capacity))


def _ws_args(ws):
    if ws is None:
        return None, 0
    return _ptr(ws), ws.numel() * ws.element_size()


def vmoba_partition(shape, inverse, src, dst, raster_strides_bsh, perm=None, inv_perm=None, stream=None):
    strides = (ctypes.c_int64 * 3)(*[int(x) for x in raster_strides_bsh])
    _check(lib().vmoba_partition(ctypes.byref(shape), int(inverse), _ptr(src), _ptr(dst), strides, _ptr(perm),
                                 _ptr(inv_perm), _stream(stream)), "vmoba_partition")


def vmoba_block_scores(shape, q_bm, k_bm, centroids, scores, dev_status, ws, stream=None):
    p, n = _ws_args(ws)
    _check(lib().vmoba_block_scores(ctypes.byref(shape), _ptr(q_bm), _ptr(k_bm), _ptr(centroids), _ptr(scores),
                                    _ptr(dev_status), p, n, _stream(stream)), "vmoba_block_scores")


def vmoba_block_scores_range(shape, q_bm, k_bm, centroids, scores, score_range, dev_status, ws, stream=None):
    p, n = _ws_args(ws)
    _check(lib().vmoba_block_scores_range(ctypes.byref(shape), _ptr(q_bm), _ptr(k_bm), _ptr(centroids), _ptr(scores),
                                          _ptr(score_range), _ptr(dev_status), p, n, _stream(stream)),
           "vmoba_block_scores_range")


def vmoba_select_ranged(shape, scores, score_range, rule, tau, topk, mask_bits, kb_ptr, q_idx, q_ptr, q_pairs, capacity,
                        k_per_head, cutoff_per_head, dev_status, ws, stream=None):
    p, n = _ws_args(ws)
    _check(lib().vmoba_select_ranged(ctypes.byref(shape), _ptr(scores), _ptr(score_range), int(rule), float(tau),
                                     int(topk), _ptr(mask_bits), _ptr(kb_ptr), _ptr(q_idx), _ptr(q_ptr), _ptr(q_pairs),
                                     int(capacity), _ptr(k_per_head), _ptr(cutoff_per_head), _ptr(dev_status), p, n,
                                     _stream(stream)), "vmoba_select_ranged")


def vmoba_select(shape, scores, tau, mask_bits, kb_ptr, q_idx, q_ptr, q_pairs, capacity, k_per_head,
                 cutoff_per_head, dev_status, ws, stream=None):
    p, n = _ws_args(ws)
    _check(lib().vmoba_select(ctypes.byref(shape), _ptr(scores), float(tau), _ptr(mask_bits), _ptr(kb_ptr),
                              _ptr(q_idx), _ptr(q_ptr), _ptr(q_pairs), int(capacity), _ptr(k_per_head),
                              _ptr(cutoff_per_head), _ptr(dev_status), p, n, _stream(stream)), "vmoba_select")


SELECT_THRESHOLD_GLOBAL, SELECT_TOPK_GLOBAL, SELECT_THRESHOLD_LOCAL, SELECT_TOPK_LOCAL = 0, 1, 2, 3
SELECT_THRESHOLD_GLOBAL_ROWNORM = 4  # Eq. 4 with per-query softmax normalisation; needs STAGE_SELECT_ROWNORM scratch
SELECT_KEEP_OWN_BLOCK = 0x100      # OR into a rule: every query also keeps the key block it lies in


def vmoba_select_rule_apply(shape, scores, rule, tau, topk, mask_bits, kb_ptr, q_idx, q_ptr, q_pairs, capacity,
                            k_per_head, cutoff_per_head, dev_status, ws, stream=None):
    """vmoba_select with one of the four block-choice rules (threshold / top-k, head-wide / per query)."""
    p, n = _ws_args(ws)
    _check(lib().vmoba_select_rule_apply(ctypes.byref(shape), _ptr(scores), int(rule), float(tau), int(topk),
                                         _ptr(mask_bits), _ptr(kb_ptr), _ptr(q_idx), _ptr(q_ptr), _ptr(q_pairs),
                                         int(capacity), _ptr(k_per_head), _ptr(cutoff_per_head), _ptr(dev_status), p, n,
                                         _stream(stream)), "vmoba_select_rule_apply")


def vmoba_select_static(shape, scores, tau, mask_bits, kb_ptr, q_idx, q_ptr, q_pairs, capacity, k_per_head,
                        cutoff_per_head, dev_status, stream=None):
    """vmoba_select with the library's built-in 16 MiB scratch array instead of a caller workspace: for callers
    that may not allocate device memory.  Calls on one device share that array and must not overlap."""
    _check(lib().vmoba_select_static(ctypes.byref(shape), _ptr(scores), float(tau), _ptr(mask_bits), _ptr(kb_ptr),
                                     _ptr(q_idx), _ptr(q_ptr), _ptr(q_pairs), int(capacity), _ptr(k_per_head),
                                     _ptr(cutoff_per_head), _ptr(dev_status), _stream(stream)), "vmoba_select_static")


def select_static_scratch_bytes() -> int:
    return int(lib().vmoba_select_static_scratch_bytes())


def vmoba_attn_fwd(shape, q_bm, k_bm, v_bm, kb_ptr, q_idx, q_ptr, q_pairs, capacity, o_bm, o_resid, lse, dev_status,
                   ws, stream=None):
    p, n = _ws_args(ws)
    _check(lib().vmoba_attn_fwd(ctypes.byref(shape), _ptr(q_bm), _ptr(k_bm), _ptr(v_bm), _ptr(kb_ptr), _ptr(q_idx),
                                _ptr(q_ptr), _ptr(q_pairs), int(capacity), _ptr(o_bm), _ptr(o_resid), _ptr(lse),
                                _ptr(dev_status), p, n, _stream(stream)), "vmoba_attn_fwd")


def vmoba_attn_bwd(shape, q_bm, k_bm, v_bm, o_bm, o_resid, lse, do_bm, kb_ptr, q_idx, q_ptr, capacity, dq_bm, dk_bm,
                   dv_bm, dev_status, ws, stream=None):
    p, n = _ws_args(ws)
    _check(lib().vmoba_attn_bwd(ctypes.byref(shape), _ptr(q_bm), _ptr(k_bm), _ptr(v_bm), _ptr(o_bm), _ptr(o_resid),
                                _ptr(lse),
                                _ptr(do_bm), _ptr(kb_ptr), _ptr(q_idx), _ptr(q_ptr), int(capacity), _ptr(dq_bm),
                                _ptr(dk_bm), _ptr(dv_bm), _ptr(dev_status), p, n, _stream(stream)), "vmoba_attn_bwd")


def vmoba_attn_fwd_raster(shape, q_bm, k_bm, v_bm, kb_ptr, q_idx, q_ptr, q_pairs, capacity, o, o_strides_bsh, perm,
                          o_resid_bm, lse, dev_status, ws, stream=None):
    p, n = _ws_args(ws)
    os_ = (ctypes.c_int64 * 3)(*[int(x) for x in o_strides_bsh])
    _check(lib().vmoba_attn_fwd_raster(ctypes.byref(shape), _ptr(q_bm), _ptr(k_bm), _ptr(v_bm), _ptr(kb_ptr), _ptr(q_idx),
                                       _ptr(q_ptr), _ptr(q_pairs), int(capacity), _ptr(o), os_, _ptr(perm),
                                       _ptr(o_resid_bm), _ptr(lse), _ptr(dev_status), p, n, _stream(stream)),
           "vmoba_attn_fwd_raster")


def vmoba_attn_bwd_raster(shape, q_bm, k_bm, v_bm, o, o_strides_bsh, o_resid, lse, d_o, do_strides_bsh, kb_ptr, q_idx,
                          q_ptr, capacity, dq, dk, dv, grad_strides_bsh, perm, dev_status, ws, stream=None):
    p, n = _ws_args(ws)
    dos = None if do_strides_bsh is None else (ctypes.c_int64 * 3)(*[int(x) for x in do_strides_bsh])
    os_ = None if o_strides_bsh is None else (ctypes.c_int64 * 3)(*[int(x) for x in o_strides_bsh])
    gs = (ctypes.c_int64 * 3)(*[int(x) for x in grad_strides_bsh])
    _check(lib().vmoba_attn_bwd_raster(ctypes.byref(shape), _ptr(q_bm), _ptr(k_bm), _ptr(v_bm), _ptr(o), os_,
                                       _ptr(o_resid), _ptr(lse), _ptr(d_o), dos, _ptr(kb_ptr), _ptr(q_idx),
                                       _ptr(q_ptr), int(capacity), _ptr(dq), _ptr(dk), _ptr(dv), gs, _ptr(perm),
                                       _ptr(dev_status), p, n, _stream(stream)), "vmoba_attn_bwd_raster")


def vmoba_full_attn(shape, q, k, v, o, lse, do=None, dq=None, dk=None, dv=None, dev_status=None, ws=None,
                    stream=None):
    p, n = _ws_args(ws)
    _check(lib().vmoba_full_attn(ctypes.byref(shape), _ptr(q), _ptr(k), _ptr(v), _ptr(o), _ptr(lse), _ptr(do),
                                 _ptr(dq), _ptr(dk), _ptr(dv), _ptr(dev_status), p, n, _stream(stream)),
           "vmoba_full_attn")


def vmoba_debug_wait_timeout(dev_status, polls, out2=None, stream=None):
    """Runs the one-CTA kernel whose bounded wait is made to run out (see include/vmoba.h)."""
    _check(lib().vmoba_debug_wait_timeout(_ptr(dev_status), int(polls), _ptr(out2), _stream(stream)),
           "vmoba_debug_wait_timeout")


def vmoba_debug_wait_profile(counters=None):
    """Registers a zeroed device tensor of 16 int64 counters for the attention kernels' section timers (None: clears)."""
    if counters is not None and (counters.numel() < 16 or counters.element_size() != 8 or not counters.is_cuda):
        raise ValueError("vmoba_debug_wait_profile: need a CUDA tensor of at least 16 64-bit counters")
    lib().vmoba_debug_wait_profile(_ptr(counters))
