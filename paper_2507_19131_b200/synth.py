"""Seeded synthetic inputs and parameters for the quantized Two-Branch Swin Block (MixA-Q).

This module only DRAWS numbers: feature maps shaped like the paper's COCO-resolution Swin workloads
(800x1333-class images, patch 4, window 7; Section 4.1 "Setup"), random-init weights quantized per output
channel, and closed-form quantizer ranges.  It holds none of the method's arithmetic (no window logic, no
scoring, no LayerNorm, no attention), so both the CUDA library's binding and the CPU oracle's binding can be
fed from it without sharing any of the code under test.  numpy only.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np

F32 = np.float32


@dataclass
class AQ:
    """Per-tensor asymmetric activation quantizer: step size, its reciprocal and the zero point."""
    bits: int
    scale: float
    inv_scale: float
    zp: int


def make_aq(lo: float, hi: float, bits: int) -> AQ:
    qmax = (1 << bits) - 1
    scale = F32((hi - lo) / qmax)
    inv = F32(1.0) / scale
    zp = int(np.clip(np.rint(-lo / float(scale)), 0, qmax))
    return AQ(bits, float(scale), float(F32(inv)), zp)


@dataclass
class Linear:
    codes: np.ndarray   # int8 [out, in], one signed code per byte
    scale: np.ndarray   # float32 [out]
    bits: int


def make_linear(rng: np.random.Generator, out_f: int, in_f: int, bits: int, std: float = 0.02) -> Linear:
    w = rng.standard_normal((out_f, in_f), dtype=F32) * F32(std)
    qmax = (1 << (bits - 1)) - 1
    scale = (np.abs(w).max(axis=1) / qmax).astype(F32)
    codes = np.clip(np.rint(w / scale[:, None]), -qmax, qmax).astype(np.int8)
    return Linear(np.ascontiguousarray(codes), scale, bits)


@dataclass
class Branch:
    ln1_g: np.ndarray
    ln1_b: np.ndarray
    ln2_g: np.ndarray
    ln2_b: np.ndarray
    b_qkv: np.ndarray
    b_proj: np.ndarray
    b_fc1: np.ndarray
    b_fc2: np.ndarray
    qkv_in: AQ
    q: AQ
    k: AQ
    v: AQ
    proj_in: AQ
    fc1_in: AQ
    fc2_in: AQ
    bits: int


@dataclass
class Block:
    dim: int
    heads: int
    window: int
    shift: int
    hidden: int
    qkv: Linear
    proj: Linear
    fc1: Linear
    fc2: Linear
    relpos: np.ndarray          # float32 [(2ws-1)^2, heads]
    hi: Branch
    lo: Branch
    score_inv_scale: float


@dataclass
class Merge:
    ln_g: np.ndarray
    ln_b: np.ndarray
    aq: AQ
    red: Linear                 # [2C, 4C]


@dataclass
class Embed:
    ln_g: np.ndarray
    ln_b: np.ndarray
    bias: np.ndarray
    aq: AQ
    proj: Linear                # [C0, 48]: 4x4 patch of 3 channels, index (ky*4 + kx)*3 + c


def make_embed(rng, c0: int, w_bits: int = 8, bits: int = 8, pixel_range: float = 3.0) -> Embed:
    """Stem parameters: N(0, 0.02^2) projection quantized per output channel, LN gamma/beta as elsewhere, and an input
    quantizer for standardised pixels (ImageNet-style mean/std normalisation puts them in about +-3)."""
    return Embed(_vec(rng, c0, 1.0, 0.02), _vec(rng, c0, 0.0, 0.02), _vec(rng, c0, 0.0, 0.02),
                 make_aq(-pixel_range, pixel_range, bits), make_linear(rng, c0, 48, w_bits))


def input_image(seed: int, B, Hi, Wi) -> np.ndarray:
    """A standardised synthetic image [B][Hi][Wi][3]: smooth blobs plus pixel noise."""
    rng = np.random.default_rng(seed)
    img = rng.standard_normal((B, Hi, Wi, 3), dtype=F32) * F32(0.5)
    for b in range(B):
        img[b] += (2.0 * blob_map(rng, Hi, Wi) - 0.5).astype(F32)[..., None]
    return img


@dataclass
class Backbone:
    dims: List[int]
    depths: List[int]
    heads: List[int]
    blocks: List[Block]
    merges: List[Merge]


def _vec(rng, n, mean, std):
    return (mean + std * rng.standard_normal(n, dtype=F32)).astype(F32)


def make_branch(rng, dim: int, hidden: int, bits: int, biases=None) -> Branch:
    """Closed-form quantizer ranges for a random-init block whose LayerNorm outputs are roughly unit
    variance and whose weights are N(0, 0.02^2): a linear output has std ~ 0.02*sqrt(fan_in)."""
    s_lin = 0.02 * math.sqrt(dim)
    s_hid = 0.02 * math.sqrt(dim)
    if biases is None:
        biases = [_vec(rng, 3 * dim, 0, 0.02), _vec(rng, dim, 0, 0.02), _vec(rng, hidden, 0, 0.02), _vec(rng, dim, 0, 0.02)]
    return Branch(
        ln1_g=_vec(rng, dim, 1.0, 0.02), ln1_b=_vec(rng, dim, 0.0, 0.02),
        ln2_g=_vec(rng, dim, 1.0, 0.02), ln2_b=_vec(rng, dim, 0.0, 0.02),
        b_qkv=biases[0], b_proj=biases[1], b_fc1=biases[2], b_fc2=biases[3],
        qkv_in=make_aq(-6.0, 6.0, bits),
        q=make_aq(-4 * s_lin, 4 * s_lin, bits), k=make_aq(-4 * s_lin, 4 * s_lin, bits),
        v=make_aq(-4 * s_lin, 4 * s_lin, bits),
        proj_in=make_aq(-2 * s_lin, 2 * s_lin, bits),
        fc1_in=make_aq(-6.0, 6.0, bits),
        fc2_in=make_aq(-0.17, 4 * s_hid, bits),
        bits=bits)


def make_block(rng, dim: int, heads: int, shift: int, w_bits: int, hi_bits: int, lo_bits: int,
               score_range: float = 6.0, window: int = 7, share_bias: bool = True,
               relpos_std: float = 2.0) -> Block:
    hidden = 4 * dim
    qkv = make_linear(rng, 3 * dim, dim, w_bits)
    proj = make_linear(rng, dim, dim, w_bits)
    fc1 = make_linear(rng, hidden, dim, w_bits)
    fc2 = make_linear(rng, dim, hidden, w_bits)
    # relative-position bias with trained-model-like magnitude, so that the attention is not uniform
    relpos = (relpos_std * rng.standard_normal(((2 * window - 1) ** 2, heads), dtype=F32)).astype(F32)
    hi = make_branch(rng, dim, hidden, hi_bits)
    # shadow layers share weights and bias (QAT); PTQ keeps the biases independent
    lo = make_branch(rng, dim, hidden, lo_bits,
                     biases=[hi.b_qkv, hi.b_proj, hi.b_fc1, hi.b_fc2] if share_bias else None)
    return Block(dim, heads, window, shift, hidden, qkv, proj, fc1, fc2, relpos, hi, lo,
                 float(F32(127.0 / score_range)))


def make_merge(rng, c_in: int, w_bits: int, bits: int) -> Merge:
    return Merge(_vec(rng, 4 * c_in, 1.0, 0.02), _vec(rng, 4 * c_in, 0.0, 0.02),
                 make_aq(-6.0, 6.0, bits), make_linear(rng, 2 * c_in, 4 * c_in, w_bits))


def make_backbone(seed: int, dims, depths, heads, w_bits: int, hi_bits: int, lo_bits: int,
                  input_range: float = 6.0, share_bias: bool = True) -> Backbone:
    rng = np.random.default_rng(seed)
    blocks, merges = [], []
    for s, (c, dep, nh) in enumerate(zip(dims, depths, heads)):
        if s > 0:
            merges.append(make_merge(rng, dims[s - 1], w_bits, hi_bits))
        # expected magnitude of a stage input: the stem for stage 0, a merge output afterwards
        rng_s = input_range if s == 0 else 6.0 * 0.02 * math.sqrt(4 * dims[s - 1])
        for i in range(dep):
            blocks.append(make_block(rng, c, nh, 0 if i % 2 == 0 else 3, w_bits, hi_bits, lo_bits,
                                     score_range=rng_s, share_bias=share_bias))
    return Backbone(list(dims), list(depths), list(heads), blocks, merges)


# ----------------------------------------------------------------------------------------------
# feature maps
# ----------------------------------------------------------------------------------------------
def input_normal_outliers(seed: int, B, H, W, C, n_out: int = 4, factor: float = 20.0) -> np.ndarray:
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((B, H, W, C), dtype=F32)
    ch = rng.choice(C, size=n_out, replace=False)
    x[..., ch] *= F32(factor)
    return x


def input_student_t(seed: int, B, H, W, C, dof: int = 3) -> np.ndarray:
    rng = np.random.default_rng(seed)
    return rng.standard_t(dof, size=(B, H, W, C)).astype(F32)


def blob_map(rng, H, W, n_lo=3, n_hi=8) -> np.ndarray:
    """Sum of a few Gaussian bumps in [0, 1]: stands in for foreground objects on a quiet background."""
    g = np.zeros((H, W), dtype=np.float64)
    yy, xx = np.mgrid[0:H, 0:W]
    for _ in range(int(rng.integers(n_lo, n_hi + 1))):
        cy, cx = rng.uniform(0, H), rng.uniform(0, W)
        sy = rng.uniform(0.03, 0.10) * H
        sx = rng.uniform(0.03, 0.10) * W
        g = np.maximum(g, np.exp(-0.5 * (((yy - cy) / sy) ** 2 + ((xx - cx) / sx) ** 2)))
    return g


def input_blobs(seed: int, B, H, W, C, bg_std: float = 0.1, gain: float = 9.0) -> np.ndarray:
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((B, H, W, C), dtype=F32) * F32(bg_std)
    for b in range(B):
        x[b] *= (1.0 + gain * blob_map(rng, H, W)).astype(F32)[..., None]
    return x


# ----------------------------------------------------------------------------------------------
# the five workloads (shapes and distributions of the benchmark configurations) + small test cases
# ----------------------------------------------------------------------------------------------
SWIN_T = dict(dims=[96, 192, 384, 768], depths=[2, 2, 6, 2], heads=[3, 6, 12, 24])
SWIN_S = dict(dims=[96, 192, 384, 768], depths=[2, 2, 18, 2], heads=[3, 6, 12, 24])
SWIN_B = dict(dims=[128, 256, 512, 1024], depths=[2, 2, 18, 2], heads=[4, 8, 16, 32])


@dataclass
class Workload:
    name: str
    B: int
    H: int
    W: int
    backbone: Backbone
    x: np.ndarray
    low_ratios: List[float]
    prune_ratios: Optional[List[float]] = None
    note: str = ""


def config1(seed: int = 1000) -> Workload:
    """One W-MSA block, 56x56x96, W8, A8 high / A4 low, ratio 0.5, N(0,1) with 4 outlier channels x20."""
    bb = make_backbone(seed + 1, [96], [1], [3], 8, 8, 4, input_range=6.0)
    x = input_normal_outliers(seed, 1, 56, 56, 96)
    return Workload("cfg1-block-56x56x96", 1, 56, 56, bb, x, [0.5])


def config2(seed: int = 2000, B: int = 2, H: int = 200, W: int = 334) -> Workload:
    """Stage-1 block pair (W-MSA then SW-MSA, shift 3), Student-t(3) activations, W8, A8/A4, ratio 0.3."""
    bb = make_backbone(seed + 1, [96], [2], [3], 8, 8, 4, input_range=8.0)
    x = input_student_t(seed, B, H, W, 96)
    return Workload("cfg2-stage1-pair-200x334x96", B, H, W, bb, x, [0.3])


def config3(seed: int = 3000, ratio: float = 0.5, H: int = 200, W: int = 334) -> Workload:
    """Full Swin-T backbone at 800x1333 (200x334 tokens after the patch-4 stem), W4, A8/A4."""
    bb = make_backbone(seed + 1, **SWIN_T, w_bits=4, hi_bits=8, lo_bits=4, input_range=6.0)
    x = input_blobs(seed, 1, H, W, 96, bg_std=0.3, gain=3.0)
    return Workload("cfg3-swin_t-800x1333", 1, H, W, bb, x, [ratio] * 6)


def config4(seed: int = 4000, B: int = 4, H: int = 256, W: int = 256) -> Workload:
    """Swin-S at 1024x1024, W4, A4 high / A2 low, ratio 0.5, 20 % of the windows pruned."""
    bb = make_backbone(seed + 1, **SWIN_S, w_bits=4, hi_bits=4, lo_bits=2, input_range=6.0)
    x = np.random.default_rng(seed).standard_normal((B, H, W, 96), dtype=F32)
    return Workload("cfg4-swin_s-1024x1024", B, H, W, bb, x, [0.5] * 12, [0.2] * 12)


def config5(seed: int = 5000, ratio: float = 0.5, B: int = 2, H: int = 384, W: int = 384) -> Workload:
    """Swin-B at 1536x1536, W8, A8/A4, clustered high-norm regions over a quiet background."""
    bb = make_backbone(seed + 1, **SWIN_B, w_bits=8, hi_bits=8, lo_bits=4, input_range=2.0)
    x = input_blobs(seed, B, H, W, 128, bg_std=0.1, gain=9.0)
    return Workload("cfg5-swin_b-1536x1536", B, H, W, bb, x, [ratio] * 12)


def tiny_backbone(seed: int = 77, B: int = 2, H: int = 30, W: int = 37, dims=(32, 64, 128), depths=(2, 2, 2),
                  heads=(1, 2, 4), w_bits=4, hi_bits=8, lo_bits=4, ratio=0.4, prune=0.0) -> Workload:
    """A three-stage miniature with ragged (non multiple of 7, odd) sizes for fast end-to-end tests."""
    bb = make_backbone(seed + 1, list(dims), list(depths), list(heads), w_bits, hi_bits, lo_bits)
    x = input_blobs(seed, B, H, W, dims[0], bg_std=0.4, gain=4.0)
    npairs = sum(depths) // 2
    return Workload("tiny", B, H, W, bb, x, [ratio] * npairs, [prune] * npairs if prune > 0 else None)
