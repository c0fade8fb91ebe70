"""Buffer management and stage sequencing for one VMoBA attention layer on one GPU.

Everything numerical happens inside the C-ABI library; this module only allocates torch
tensors (device memory), passes their pointers to the entry points in order, and exposes the
intermediate buffers so that tests can compare each stage with the oracle.
"""
from __future__ import annotations

import torch

from . import binding as vb


def torch_dtype(shape):
    return torch.bfloat16 if shape.dtype == vb.BF16 else torch.float32


def default_capacity(shape, tau: float, slack: float = 0.02) -> int:
    """Upper bound on the number of selected pairs: the threshold rule keeps at most ceil(tau*P)
    pairs per head (the kept fraction never exceeds tau, Section 4.1), plus exact ties."""
    P = shape.S * shape.n_blocks
    per_head = int(min(P, tau * P * (1.0 + slack) + 1024))
    return min(per_head * shape.B * shape.heads, 2 ** 31 - 1)


class VmobaLayer:
    """Owns the device buffers of one layer shape and runs the stages on the current stream."""

    def __init__(self, shape, capacity: int, device="cuda", with_backward: bool = False):
        self.shape = shape
        self.capacity = int(capacity)
        self.device = torch.device(device)
        s = shape
        dt = torch_dtype(s)
        dev = self.device
        BH, S, d, Nb = s.B * s.heads, s.S, s.head_dim, s.n_blocks
        self.BH, self.S, self.d, self.Nb = BH, S, d, Nb
        bm = lambda: torch.empty((s.B, s.heads, S, d), dtype=dt, device=dev)
        self.q_bm, self.k_bm, self.v_bm, self.o_bm = bm(), bm(), bm(), bm()
        self.centroids = torch.empty((s.B, s.heads, Nb, d), dtype=torch.float32, device=dev)
        self.scores = torch.empty((s.B, s.heads, S, Nb), dtype=torch.float32, device=dev)
        self.mask_bits = torch.empty((BH * S, s.mask_words), dtype=torch.int32, device=dev)
        self.kb_ptr = torch.empty(BH * Nb + 1, dtype=torch.int32, device=dev)
        self.q_idx = torch.empty(self.capacity, dtype=torch.int32, device=dev)
        self.q_ptr = torch.empty(BH * S + 1, dtype=torch.int32, device=dev)
        self.q_pairs = torch.empty(self.capacity, dtype=torch.int32, device=dev)
        self.k_per_head = torch.empty(BH, dtype=torch.int64, device=dev)
        self.cutoff = torch.empty(BH, dtype=torch.float32, device=dev)
        self.score_range = torch.empty((BH, 2), dtype=torch.float32, device=dev)   # per head: smallest, largest score
        self.range_valid = False
        self.lse = torch.empty(BH * S, dtype=torch.float32, device=dev)
        self.perm = torch.empty(S, dtype=torch.int32, device=dev)     # raster token of block-major position p (Eq. 1)
        self.dev_status = torch.zeros(1, dtype=torch.int32, device=dev)
        stages = [vb.STAGE_SCORES, vb.STAGE_SELECT, vb.STAGE_ATTN_FWD]
        if with_backward:
            stages.append(vb.STAGE_ATTN_BWD)
            self.do_bm, self.dq_bm, self.dk_bm, self.dv_bm = bm(), bm(), bm(), bm()
        # rounding residual of o, kept for the backward's rowsum(dO * O) (bf16 training only)
        self.o_resid = bm() if (with_backward and s.dtype == vb.BF16) else None
        ws_bytes = max(vb.workspace_bytes(s, st, self.capacity) for st in stages)
        self.ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        self.with_backward = with_backward
        self.o_raster = None          # the raster-order o of the last attn_fwd_raster, if that is how o was written

    # ---- stage wrappers -----------------------------------------------------------------
    @staticmethod
    def raster_strides(x):
        """Element strides (batch, token, head) of a [B, S, heads, d] tensor."""
        assert x.stride(3) == 1
        return (x.stride(0), x.stride(1), x.stride(2))

    def partition(self, raster, bm, inverse=False, perm=None, inv_perm=None):
        src, dst = (bm, raster) if inverse else (raster, bm)
        vb.vmoba_partition(self.shape, int(inverse), src, dst, self.raster_strides(raster), perm, inv_perm)

    def block_scores(self, with_range=True):
        """Centroids and scores; with_range: the scores kernel also takes each head's smallest and largest score,
        which lets select() skip its own pass for them (valid until self.scores is overwritten by other means)."""
        if with_range:
            vb.vmoba_block_scores_range(self.shape, self.q_bm, self.k_bm, self.centroids, self.scores, self.score_range,
                                        self.dev_status, self.ws)
        else:
            vb.vmoba_block_scores(self.shape, self.q_bm, self.k_bm, self.centroids, self.scores, self.dev_status, self.ws)
        self.range_valid = bool(with_range)

    def select(self, tau, scores=None, use_range=None):
        """Eq. 3 + Eq. 4.  use_range: take the score range the last block_scores() left (default: if it left one and
        the scores are the layer's own)."""
        if use_range is None:
            use_range = self.range_valid and scores is None
        if use_range:
            vb.vmoba_select_ranged(self.shape, self.scores, self.score_range, vb.SELECT_THRESHOLD_GLOBAL, tau, 0,
                                   self.mask_bits, self.kb_ptr, self.q_idx, self.q_ptr, self.q_pairs, self.capacity,
                                   self.k_per_head, self.cutoff, self.dev_status, self.ws)
            return
        vb.vmoba_select(self.shape, self.scores if scores is None else scores, tau, self.mask_bits, self.kb_ptr,
                        self.q_idx, self.q_ptr, self.q_pairs, self.capacity, self.k_per_head, self.cutoff,
                        self.dev_status, self.ws)

    def select_rule(self, rule, tau=0.25, topk=1, scores=None):
        ws = self.ws
        if (rule & 0xff) == vb.SELECT_THRESHOLD_GLOBAL_ROWNORM:
            # this rule keeps a transformed copy of the score matrix in its scratch: allocated on first use
            need = vb.workspace_bytes(self.shape, vb.STAGE_SELECT_ROWNORM, self.capacity)
            if getattr(self, "ws_rownorm", None) is None or self.ws_rownorm.numel() < need:
                self.ws_rownorm = torch.empty(need, dtype=torch.uint8, device=self.ws.device)
            ws = self.ws_rownorm
        vb.vmoba_select_rule_apply(self.shape, self.scores if scores is None else scores, rule, tau, topk, self.mask_bits,
                                   self.kb_ptr, self.q_idx, self.q_ptr, self.q_pairs, self.capacity, self.k_per_head,
                                   self.cutoff, self.dev_status, ws)

    def attn_fwd(self):
        self.o_raster = None
        vb.vmoba_attn_fwd(self.shape, self.q_bm, self.k_bm, self.v_bm, self.kb_ptr, self.q_idx, self.q_ptr,
                          self.q_pairs, self.capacity, self.o_bm, self.o_resid, self.lse, self.dev_status, self.ws)

    def attn_bwd(self):
        vb.vmoba_attn_bwd(self.shape, self.q_bm, self.k_bm, self.v_bm, self.o_bm, self.o_resid, self.lse, self.do_bm,
                          self.kb_ptr, self.q_idx, self.q_ptr, self.capacity, self.dq_bm, self.dk_bm, self.dv_bm,
                          self.dev_status, self.ws)

    def can_fold_inverse(self, dq_out, dk_out, dv_out) -> bool:
        """Whether the backward kernels can write these raster-order gradients themselves."""
        strides = self.raster_strides(dq_out)
        return (self.shape.dtype == vb.BF16 and self.d == 128 and self.raster_strides(dk_out) == strides
                and self.raster_strides(dv_out) == strides)

    def can_fold_o(self) -> bool:
        """Whether the forward kernels can write o in raster order themselves."""
        return self.shape.dtype == vb.BF16 and self.d == 128

    def attn_fwd_raster(self, o_out):
        """Forward writing o straight into the raster-order tensor o_out (needs self.perm from the partition of q).
        The tensor is remembered: a following attn_bwd_raster reads o from it."""
        vb.vmoba_attn_fwd_raster(self.shape, self.q_bm, self.k_bm, self.v_bm, self.kb_ptr, self.q_idx, self.q_ptr,
                                 self.q_pairs, self.capacity, o_out, self.raster_strides(o_out), self.perm,
                                 self.o_resid, self.lse, self.dev_status, self.ws)
        self.o_raster = o_out

    def attn_bwd_raster(self, do_raster_or_none, dq_out, dk_out, dv_out):
        """Backward writing dq, dk, dv in raster order (needs self.perm from the forward's partition of q); dO is
        read in raster order too if given, else from self.do_bm; o is read from the raster-order tensor the last
        attn_fwd_raster wrote, else from self.o_bm."""
        do = self.do_bm if do_raster_or_none is None else do_raster_or_none
        dos = None if do_raster_or_none is None else self.raster_strides(do)
        o = self.o_bm if self.o_raster is None else self.o_raster
        os_ = None if self.o_raster is None else self.raster_strides(o)
        vb.vmoba_attn_bwd_raster(self.shape, self.q_bm, self.k_bm, self.v_bm, o, os_, self.o_resid, self.lse, do,
                                 dos, self.kb_ptr, self.q_idx, self.q_ptr, self.capacity, dq_out,
                                 dk_out, dv_out, self.raster_strides(dq_out), self.perm, self.dev_status, self.ws)

    # ---- whole layer --------------------------------------------------------------------
    def forward(self, q, k, v, tau, o_out, fold_o=None):
        """q, k, v, o_out: [B, S, heads, d] raster-order tensors on the device.

        fold_o: let the forward kernels write o in raster order themselves (bf16, head_dim 128) instead of an inverse
        partition pass; off by default (measured on B200: the scattered 256-byte row writes cost the attention kernel
        more than the pass they save, at 12 heads as at 40).  o_out must then stay alive and unchanged until backward()."""
        self.partition(q, self.q_bm, perm=self.perm)
        self.partition(k, self.k_bm)
        self.partition(v, self.v_bm)
        self.block_scores()
        self.select(tau)
        if fold_o:
            self.attn_fwd_raster(o_out)
            return
        self.attn_fwd()
        self.partition(o_out, self.o_bm, inverse=True)

    def backward(self, do, dq_out, dk_out, dv_out, fold_inverse=None, fold_do=False):
        """Gradients of the last forward(); do and the outputs are raster-order [B, S, heads, d].

        fold_inverse: let the backward kernels write dq, dk, dv in raster order themselves (bf16, head_dim 128,
        outputs with equal strides) instead of three inverse partition passes; default: whenever possible.
        fold_do: also let them read dO in raster order instead of partitioning it first (pays with few heads)."""
        if fold_inverse is None:
            fold_inverse = self.can_fold_inverse(dq_out, dk_out, dv_out)
        if fold_inverse and fold_do:
            self.attn_bwd_raster(do, dq_out, dk_out, dv_out)
            return
        self.partition(do, self.do_bm)
        if fold_inverse:
            self.attn_bwd_raster(None, dq_out, dk_out, dv_out)
            return
        if self.o_raster is not None:      # the block-major backward reads o_bm, which the raster forward did not write
            self.partition(self.o_raster, self.o_bm)
        self.attn_bwd()
        self.partition(dq_out, self.dq_bm, inverse=True)
        self.partition(dk_out, self.dk_bm, inverse=True)
        self.partition(dv_out, self.dv_bm, inverse=True)

    def check_status(self):
        code = int(self.dev_status.item())
        if code != vb.OK:
            raise vb.VmobaError(code, "device status")

    def n_selected(self) -> int:
        return int(self.k_per_head.sum().item())


def dense_step_schedule(n_steps: int, dense_fraction: float = 0.25):
    """Which denoising steps of a sampling run use full attention: the paper's training-free setting runs the
    first 25 % of the steps dense and the rest through VMoBA (Section 4.1, implementation details).  Returns a list
    of n_steps booleans, True = dense; the number of dense steps is ceil(dense_fraction * n_steps)."""
    import math
    if n_steps < 0 or not (0.0 <= dense_fraction <= 1.0):
        raise ValueError("n_steps >= 0 and 0 <= dense_fraction <= 1 required")
    n_dense = min(n_steps, int(math.ceil(dense_fraction * n_steps - 1e-9)))
    return [i < n_dense for i in range(n_steps)]


class SteppedAttention:
    """Host-side switch between the dense path and the sparse layer over the steps of a sampler: step i of
    n_steps calls vmoba_full_attn while dense_step_schedule says so, the VMoBA layer afterwards (forward only:
    this is the inference setting).  Tensors are raster-order [B, S, heads, d] on the device."""

    def __init__(self, layer: VmobaLayer, tau: float, n_steps: int, dense_fraction: float = 0.25):
        self.layer, self.tau = layer, tau
        self.schedule = dense_step_schedule(n_steps, dense_fraction)
        s = layer.shape
        self._lse = torch.empty(s.B * s.heads * s.S, dtype=torch.float32, device=layer.device)

    def forward(self, step: int, q, k, v, o_out) -> str:
        """Runs step `step`; returns which path ran ("dense" or "sparse")."""
        if self.schedule[step]:
            # the dense kernels take [B, heads, S, d] in any one token order
            qd, kd, vd = (x.permute(0, 2, 1, 3).contiguous() for x in (q, k, v))
            od = torch.empty_like(qd)
            vb.vmoba_full_attn(self.layer.shape, qd, kd, vd, od, self._lse, dev_status=self.layer.dev_status)
            o_out.copy_(od.permute(0, 2, 1, 3))
            return "dense"
        self.layer.forward(q, k, v, self.tau, o_out)
        return "sparse"


def lists_from_mask(mask_bh, capacity=None, device="cuda"):
    """Builds kb_ptr / q_idx / q_ptr / q_pairs on the host from a boolean mask [BH, S, Nb]
    (used by tests to feed the attention kernels a selection that did not come from
    vmoba_select).  Pure index bookkeeping."""
    import numpy as np
    BH, S, Nb = mask_bh.shape
    kb_ptr = [0]
    q_idx = []
    pos_of = {}
    for bh in range(BH):
        for j in range(Nb):
            qs = np.nonzero(mask_bh[bh, :, j])[0]
            base = len(q_idx)
            for n, qq in enumerate(qs):
                pos_of[(bh, int(qq), j)] = base + n
            q_idx.extend(qs.tolist())
            kb_ptr.append(len(q_idx))
    q_ptr = [0]
    q_pairs = []
    for bh in range(BH):
        for qq in range(S):
            for j in np.nonzero(mask_bh[bh, qq])[0]:
                q_pairs.append(pos_of[(bh, qq, int(j))])
            q_ptr.append(len(q_pairs))
    n = len(q_idx)
    cap = max(n, 1) if capacity is None else capacity
    pad = lambda a: a + [0] * (cap - len(a))
    mk = lambda a: torch.tensor(a, dtype=torch.int32, device=device)
    return mk(kb_ptr), mk(pad(q_idx)), mk(q_ptr), mk(pad(q_pairs)), n
