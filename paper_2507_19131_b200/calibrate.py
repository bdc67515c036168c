"""Min/max calibration of the activation quantizers (the step in front of the path in the post-training flow).

MixA-Q Section 4.3: one calibration sample; the FULL feature map (all windows, not the windows a branch will later
see) initialises the step sizes of both the high- and the low-precision branch, so that the two branches share their
calibration data and differ only in bit width.  This module runs the floating-point Two-Branch block (every window
through the same weights; LayerNorm parameters of the branch being calibrated) with plain torch operations, on the
GPU when the tensors live there, observes the minimum and maximum at every quantizer site (QKV input, q, k, v, proj
input, fc1 input, fc2 input) and turns them into per-tensor asymmetric quantizers at the two bit widths.

It is a preparation utility, not part of the timed forward: the forward consumes the quantizers it writes.
"""
from __future__ import annotations

import copy
import math
from typing import Dict, List, Tuple

import numpy as np
import torch

from . import synth

SITES = ("qkv_in", "q", "k", "v", "proj_in", "fc1_in", "fc2_in")


def _windows(x: torch.Tensor, ws: int, shift: int):
    """[B,H,W,C] -> (windows [B*nW, ws*ws, C], real-token mask [B*nW, ws*ws], geometry)."""
    B, H, W, C = x.shape
    Hp, Wp = -(-H // ws) * ws, -(-W // ws) * ws
    xp = torch.zeros((B, Hp, Wp, C), dtype=x.dtype, device=x.device)
    xp[:, :H, :W] = x
    real = torch.zeros((B, Hp, Wp), dtype=torch.bool, device=x.device)
    real[:, :H, :W] = True
    if shift:
        xp = torch.roll(xp, (-shift, -shift), (1, 2))
        real = torch.roll(real, (-shift, -shift), (1, 2))

    def part(t):
        t = t.reshape(B, Hp // ws, ws, Wp // ws, ws, *t.shape[3:])
        t = t.permute(0, 1, 3, 2, 4, *range(5, t.dim()))
        return t.reshape(B * (Hp // ws) * (Wp // ws), ws * ws, *t.shape[5:])
    return part(xp), part(real), (B, H, W, Hp, Wp)


def _unwindows(win: torch.Tensor, geo, ws: int, shift: int) -> torch.Tensor:
    B, H, W, Hp, Wp = geo
    C = win.shape[-1]
    t = win.reshape(B, Hp // ws, Wp // ws, ws, ws, C).permute(0, 1, 3, 2, 4, 5).reshape(B, Hp, Wp, C)
    if shift:
        t = torch.roll(t, (shift, shift), (1, 2))
    return t[:, :H, :W].contiguous()


def _shift_mask(geo, ws: int, shift: int, device) -> torch.Tensor:
    B, H, W, Hp, Wp = geo
    if not shift:
        return None

    def region(n, L):
        r = torch.zeros(n, dtype=torch.int64)
        r[L - ws:L - shift] = 1
        r[L - shift:] = 2
        return r
    reg = (region(Hp, Hp)[:, None] * 3 + region(Wp, Wp)[None, :]).to(device)
    reg = reg.reshape(Hp // ws, ws, Wp // ws, ws).permute(0, 2, 1, 3).reshape(-1, ws * ws)
    m = (reg[:, :, None] != reg[:, None, :]).to(torch.float32) * -100.0
    return m.repeat(B, 1, 1)                                   # [B*nW, T, T]


def _relpos(table: torch.Tensor, ws: int, heads: int) -> torch.Tensor:
    idx = torch.arange(ws * ws)
    dy = (idx // ws)[:, None] - (idx // ws)[None, :] + ws - 1
    dx = (idx % ws)[:, None] - (idx % ws)[None, :] + ws - 1
    return table[(dy * (2 * ws - 1) + dx).to(table.device)].permute(2, 0, 1)      # [heads, T, T]


def _deq(lin, device) -> torch.Tensor:
    return torch.from_numpy(lin.codes.astype(np.float32) * lin.scale[:, None]).to(device)


def fp_block(blk, br, x: torch.Tensor, observe=None) -> torch.Tensor:
    """Floating-point block (all windows through one set of LayerNorm parameters / biases `br`).  `observe(site, t)`
    is called with the tensor that the site's quantizer would see."""
    dev = x.device
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(dev)
    ws, C, nh = blk.window, blk.dim, blk.heads
    win, real, geo = _windows(x, ws, blk.shift)
    ln = torch.nn.functional.layer_norm(win, (C,), t(br.ln1_g), t(br.ln1_b), 1e-5) * real[..., None]
    if observe: observe("qkv_in", ln)
    qkv = ln @ _deq(blk.qkv, dev).T + t(br.b_qkv)
    q, k, v = qkv.split(C, dim=-1)
    if observe:
        observe("q", q); observe("k", k); observe("v", v)
    heads = lambda a: a.reshape(a.shape[0], a.shape[1], nh, C // nh).transpose(1, 2)
    logits = heads(q) @ heads(k).transpose(-1, -2) / math.sqrt(C // nh) + _relpos(t(blk.relpos), ws, nh)[None]
    mask = _shift_mask(geo, ws, blk.shift, dev)
    if mask is not None:
        logits = logits + mask[:, None]
    o = (torch.softmax(logits, -1) @ heads(v)).transpose(1, 2).reshape(win.shape)
    if observe: observe("proj_in", o)
    x1 = win + o @ _deq(blk.proj, dev).T + t(br.b_proj)
    ln2 = torch.nn.functional.layer_norm(x1, (C,), t(br.ln2_g), t(br.ln2_b), 1e-5)
    if observe: observe("fc1_in", ln2)
    h = torch.nn.functional.gelu(ln2 @ _deq(blk.fc1, dev).T + t(br.b_fc1))
    if observe: observe("fc2_in", h)
    y = x1 + h @ _deq(blk.fc2, dev).T + t(br.b_fc2)
    return _unwindows(y, geo, ws, blk.shift)


def fp_merge(m, x: torch.Tensor, observe=None) -> torch.Tensor:
    B, H, W, C = x.shape
    dev = x.device
    xp = torch.zeros((B, H + H % 2, W + W % 2, C), dtype=x.dtype, device=dev)
    xp[:, :H, :W] = x
    cat = torch.cat([xp[:, 0::2, 0::2], xp[:, 1::2, 0::2], xp[:, 0::2, 1::2], xp[:, 1::2, 1::2]], -1)
    ln = torch.nn.functional.layer_norm(cat, (4 * C,), torch.from_numpy(m.ln_g).to(dev), torch.from_numpy(m.ln_b).to(dev), 1e-5)
    if observe: observe("in", ln)
    return ln @ _deq(m.red, dev).T


def calibrate_backbone(bb, x0: np.ndarray, device: str = None):
    """Returns a deep copy of `bb` whose activation quantizers (both branches of every block, every merge) come from
    the min/max of the floating-point forward of the calibration sample x0 [B,H,W,C0].  Every block is calibrated on
    the full feature map; the high and the low branch get the same range at their own bit widths.  The sample is
    propagated through the floating-point model with the high branch's LayerNorm parameters and biases."""
    if device is None:
        device = "cuda" if torch.cuda.is_available() else "cpu"
    out = copy.deepcopy(bb)
    x = torch.from_numpy(np.ascontiguousarray(x0, np.float32)).to(device)
    k = 0
    with torch.no_grad():
        for s, d in enumerate(out.depths):
            if s > 0:
                m = out.merges[s - 1]
                rng: Dict[str, Tuple[float, float]] = {}
                x = fp_merge(m, x, lambda site, t: rng.__setitem__(site, (float(t.min()), float(t.max()))))
                m.aq = synth.make_aq(*rng["in"], m.aq.bits)
            for _ in range(d):
                blk = out.blocks[k]
                for name in ("hi", "lo"):
                    br = getattr(blk, name)
                    rng = {}
                    y = fp_block(blk, br, x, lambda site, t: rng.__setitem__(site, (float(t.min()), float(t.max()))))
                    for site in SITES:
                        setattr(br, site, synth.make_aq(rng[site][0], rng[site][1], br.bits))
                    if name == "hi":
                        y_next = y
                # score step: the int8 score codes should span the stage input (the first block of a stage sets it)
                blk.score_inv_scale = float(np.float32(127.0 / max(1e-12, float(x.abs().max()))))
                x = y_next
                k += 1
    return out
