"""Min/max calibration of the activation quantizers (the step in front of the path in the post-training flow).

MixA-Q Section 4.3: one calibration sample; the FULL feature map (all windows, not the windows a branch will later
see) initialises the step sizes of both the high- and the low-precision branch, so that the two branches share their
calibration data and differ only in bit width.

Everything is computed by the library (mixaq_calibrate_block / mixaq_calibrate_merge run the floating-point block with
min/max observers at the seven quantizer sites; mixaq_aq_from_range turns a range into a quantizer).  This module only
walks the backbone, marshals the arguments and copies the results into a parameter object the forward consumes.
It needs the CUDA library and a device, like the rest of the package.
"""
from __future__ import annotations

import copy

import numpy as np
import torch

from . import binding as mq
from . import synth

SITES = ("qkv_in", "q", "k", "v", "proj_in", "fc1_in", "fc2_in")


def _aq(lo: float, hi: float, bits: int) -> synth.AQ:
    scale, inv, zp = mq.aq_from_range(lo, hi, bits)
    return synth.AQ(bits, scale, inv, zp)


def calibrate_backbone(ctx: "mq.Context", bb, x0: np.ndarray):
    """Returns a deep copy of `bb` whose activation quantizers (both branches of every block, every merge) and score
    steps come from the calibration sample x0 [B,H,W,C0].  Every block is calibrated on the full feature map, once
    through each branch's own LayerNorm parameters and biases; the sample is propagated through the floating-point
    model with the high branch's."""
    out = copy.deepcopy(bb)
    dev = mq._Dev(ctx.device)
    x = torch.from_numpy(np.ascontiguousarray(x0, np.float32)).to(ctx.device)
    k = 0
    for s, d in enumerate(out.depths):
        if s > 0:
            m = out.merges[s - 1]
            x, (lo, hi) = mq.calibrate_merge(ctx, mq.fill_merge_struct(dev, m), x)
            m.aq = _aq(lo, hi, m.aq.bits)
        for _ in range(d):
            blk = out.blocks[k]
            bs = mq.fill_block_struct(dev, blk)
            y_next = None
            for branch, name in enumerate(("hi", "lo")):
                br = getattr(blk, name)
                y, rng = mq.calibrate_block(ctx, bs, branch, x)
                for site in SITES:
                    setattr(br, site, _aq(rng[site][0], rng[site][1], br.bits))
                if name == "hi":
                    y_next = y
                    # the int8 score codes span the block's input map
                    blk.score_inv_scale = float(np.float32(127.0 / max(1e-12, max(abs(rng["x_in"][0]), abs(rng["x_in"][1])))))
            x = y_next
            k += 1
    return out
