"""Seeded synthetic inputs for the VMoBA attention layer.

This module is the one piece shared by the CUDA path's tests/benchmarks and by
the CPU oracle's tests.  It holds none of the method's arithmetic: it only
draws random numbers, shapes them like video-DiT activations (a latent grid of
T x H x W tokens, several heads, head_dim channels) and rounds them to the
storage type.  Token order is raster (t, h, w) with w fastest; tensors are
laid out [B, S, heads, head_dim] (what a DiT's q/k/v projections produce).

Three recipes:

* ``sine``  : x(t,h,w,head,c) = 0.5*sin(2*pi*(t/T + h/H + w/W) + phi_head) + N(0,1),
              phi_head = 2*pi*head/heads; the sine term is shared by q, k and v and by
              all channels; the noise is i.i.d. per element and independent for q, k, v.
* ``white`` : x = N(0,1) only: no locality component at all (the unstructured variant: selection is
              essentially random, the worst case for gathered work lists).
* ``smooth``: x = N(0,1) + f, where f is, per (batch, head), one white N(0,1)
              field of shape [T,H,W,head_dim] blurred along T, H and W (not along
              channels) with a separable Gaussian (sigma = 2 tokens, radius 8,
              periodic wrap, taps normalised; scipy.ndimage.correlate1d) and then
              rescaled to unit standard deviation.  f is shared by q, k and v; the N(0,1) noise is independent.

Draw order per (batch, head), from numpy's PCG64 ``default_rng(seed)`` spawned
per (batch, head) so that any subset of heads can be generated alone:
f (smooth only), noise q, noise k, noise v, dO.
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np


@dataclasses.dataclass(frozen=True)
class Workload:
    """One attention-layer problem: shapes, partition, threshold, input recipe."""
    name: str
    B: int
    heads: int
    head_dim: int
    T: int
    H: int
    W: int
    block: tuple          # (bT, bH, bW) tokens per block along each axis
    tau: float
    dtype: str            # "f32" or "bf16"
    recipe: str           # "sine" or "smooth"
    seed: int

    @property
    def S(self) -> int:
        return self.T * self.H * self.W

    @property
    def n_blocks(self) -> int:
        bT, bH, bW = self.block
        return (self.T // bT) * (self.H // bH) * (self.W // bW)

    @property
    def block_tokens(self) -> int:
        bT, bH, bW = self.block
        return bT * bH * bW

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five benchmark configurations (shapes only; which passes run is the caller's business).
C1 = Workload("c1_tiny", 1, 2, 64, 4, 8, 8, (1, 8, 8), 0.25, "f32", "sine", 0)
C2 = Workload("c2_wan13b_3d", 1, 12, 128, 21, 30, 52, (3, 6, 13), 0.25, "bf16", "smooth", 1)
C3_BLOCKS = {"1d": (1, 30, 52), "2d": (21, 6, 13), "3d": (3, 6, 13)}
C3_TAUS = (0.1, 0.25, 0.5, 1.0)
C4 = Workload("c4_train_3d", 2, 12, 128, 21, 30, 52, (3, 6, 13), 0.25, "bf16", "smooth", 1)
C5_BLOCKS = {"1d": (1, 45, 80), "2d": (21, 9, 10), "3d": (3, 9, 10)}
C5 = Workload("c5_720p", 1, 40, 128, 21, 45, 80, (3, 9, 10), 0.25, "bf16", "smooth", 1)
# The paper's own fine-tuning grid (Table 2 / Table 4: 93x576x1024 video, latent 24x36x64 = 55,296 tokens,
# 8 / 48 / 72 key blocks for the 1D / 2D / 3D layers, tau = 0.25) on Wan-1.3B-sized heads.
T55_BLOCKS = {"1d": (3, 36, 64), "2d": (24, 6, 8), "3d": (8, 12, 8)}
T55 = Workload("t55k_train", 1, 12, 128, 24, 36, 64, (8, 12, 8), 0.25, "bf16", "smooth", 1)
# The paper's second training grid (Table 4: 141x480x832 video, latent 36x30x52 = 56,160 tokens; spatial blocks
# of 5 x 13 tokens -> 24 blocks of 2340 keys, spatio-temporal blocks of 12 x 10 x 13 tokens -> 36 blocks of
# 1560 keys).  The table's temporal entry for this grid is inconsistent (block size 3 but 7 blocks, where
# 36 / 3 = 12); the 1D layer here takes the block size: 12 temporal blocks of 3 frames (4680 keys).
T56_BLOCKS = {"1d": (3, 30, 52), "2d": (36, 5, 13), "3d": (12, 10, 13)}
T56 = Workload("t56k_train", 1, 12, 128, 36, 30, 52, (12, 10, 13), 0.25, "bf16", "smooth", 1)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round-to-nearest-even) and return the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns (uint16) to fp32 exactly."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _gauss_taps(sigma: float, radius: int) -> np.ndarray:
    x = np.arange(-radius, radius + 1, dtype=np.float64)
    w = np.exp(-0.5 * (x / sigma) ** 2)
    return w / w.sum()


def _blur_wrap(f: np.ndarray, axis: int, taps: np.ndarray) -> np.ndarray:
    from scipy.ndimage import correlate1d
    return correlate1d(f, taps, axis=axis, mode="wrap")


def _unit_rng(seed: int, b: int, head: int) -> np.random.Generator:
    return np.random.default_rng([seed, b, head])


def make_head(w: Workload, b: int, head: int, with_do: bool = True):
    """fp32 q, k, v (and dO) of one (batch, head): arrays [S, head_dim] in raster token order."""
    rng = _unit_rng(w.seed, b, head)
    shape = (w.T, w.H, w.W, w.head_dim)
    if w.recipe == "sine":
        t = np.arange(w.T, dtype=np.float64)[:, None, None] / w.T
        h = np.arange(w.H, dtype=np.float64)[None, :, None] / w.H
        x = np.arange(w.W, dtype=np.float64)[None, None, :] / w.W
        phi = 2.0 * math.pi * head / w.heads
        base = (0.5 * np.sin(2.0 * math.pi * (t + h + x) + phi)).astype(np.float32)[..., None]
    elif w.recipe == "smooth":
        f = rng.standard_normal(shape, dtype=np.float32)
        taps = _gauss_taps(2.0, 8)
        for ax in range(3):
            f = _blur_wrap(f, ax, taps)
        base = f / np.float32(f.std())
    elif w.recipe == "white":
        base = np.float32(0.0)
    else:
        raise ValueError(w.recipe)
    out = []
    for _ in range(3):
        out.append((rng.standard_normal(shape, dtype=np.float32) + base).reshape(w.S, w.head_dim))
    if with_do:
        out.append(rng.standard_normal(shape, dtype=np.float32).reshape(w.S, w.head_dim))
    return out


def make_inputs(w: Workload, with_do: bool = True, heads=None):
    """Generate the layer's inputs.

    Returns a dict with fp32 arrays 'q','k','v' (and 'do') of shape
    [B, S, n_heads, head_dim] holding the values exactly as stored (for bf16
    workloads: already rounded to bf16 and widened again), plus, for bf16
    workloads, 'q_bits' etc. with the uint16 bit patterns.  ``heads`` optionally
    restricts generation to a list of head indices (the per-head streams are
    independent, so a subset reproduces the same values).
    """
    from concurrent.futures import ThreadPoolExecutor
    import os
    head_list = list(range(w.heads)) if heads is None else list(heads)
    names = ["q", "k", "v"] + (["do"] if with_do else [])
    arrs = {n: np.empty((w.B, w.S, len(head_list), w.head_dim), dtype=np.float32) for n in names}

    def one(unit):
        b, hi, head = unit
        for n, x in zip(names, make_head(w, b, head, with_do)):
            arrs[n][b, :, hi, :] = x

    units = [(b, hi, head) for b in range(w.B) for hi, head in enumerate(head_list)]
    with ThreadPoolExecutor(max_workers=min(len(units), os.cpu_count() or 1, 32)) as pool:
        list(pool.map(one, units))
    out = {}
    for n in names:
        if w.dtype == "bf16":
            bits = f32_to_bf16_bits(arrs[n])
            out[n + "_bits"] = bits
            out[n] = bf16_bits_to_f32(bits)
        else:
            out[n] = arrs[n]
    return out
