"""Calibration (Section 4.3: one sample, the full feature map sets the ranges of both branches).

CPU: the walk over a backbone written with the ORACLE's observers (pinned in test_oracle_block.py to a textbook block)
and the properties the calibration must have.  GPU: the library's calibration kernels against those observers."""
import copy

import numpy as np
import pytest

from paper_2507_19131_b200 import synth

F32 = np.float32
SITES = ("qkv_in", "q", "k", "v", "proj_in", "fc1_in", "fc2_in")


def oracle_calibrated_backbone(orc, bb, x0):
    """The reference walk: every block observed once through each branch's own LayerNorm parameters and biases on the
    full map, the sample propagated through the floating-point model with the high branch's."""
    out = copy.deepcopy(bb)
    x, k = np.ascontiguousarray(x0, F32), 0
    for s, d in enumerate(out.depths):
        if s > 0:
            m = out.merges[s - 1]
            x, (lo, hi) = orc.merge_observe_fp(m, x)
            m.aq = synth.make_aq(lo, hi, m.aq.bits)
        for _ in range(d):
            blk = out.blocks[k]
            blk.score_inv_scale = float(F32(127.0 / max(1e-12, float(np.abs(x).max()))))
            y_next = None
            for name in ("hi", "lo"):
                br = getattr(blk, name)
                y, rng = orc.block_observe_fp(blk, name, x)
                for site in SITES:
                    setattr(br, site, synth.make_aq(rng[site][0], rng[site][1], br.bits))
                if name == "hi":
                    y_next = y
            x = y_next
            k += 1
    return out


def poorly_ranged_backbone(wl):
    bad = synth.make_backbone(78, wl.backbone.dims, wl.backbone.depths, wl.backbone.heads, 8, 8, 4)
    for b in bad.blocks:
        # post-training start: the low branch's LayerNorm is a copy of the high branch's
        b.lo.ln1_g, b.lo.ln1_b, b.lo.ln2_g, b.lo.ln2_b = b.hi.ln1_g, b.hi.ln1_b, b.hi.ln2_g, b.hi.ln2_b
        for br in (b.hi, b.lo):
            for site in SITES:
                setattr(br, site, synth.make_aq(-50.0, 50.0, br.bits))
    return bad


def test_calibrated_quantizers_cover_the_sample_and_share_ranges(orc):
    wl = synth.tiny_backbone(ratio=0.4)
    bad = poorly_ranged_backbone(wl)
    cal = oracle_calibrated_backbone(orc, bad, wl.x)
    b0 = cal.blocks[0]
    for site in SITES:
        hi, lo = getattr(b0.hi, site), getattr(b0.lo, site)
        # same observed range, different bit width: scale ratio = (2^8 - 1) / (2^4 - 1)
        assert hi.bits == 8 and lo.bits == 4
        assert lo.scale / hi.scale == pytest.approx(255.0 / 15.0, rel=1e-4)
    # the quantized model with calibrated ranges tracks the floating-point model better than with the poor ranges
    ref = orc.backbone_forward(cal, wl.x, [0.0] * 3, quant=False)

    def sqnr(bb):
        out = orc.backbone_forward(bb, wl.x, [0.0] * 3)
        return [10 * np.log10(float((r.astype(np.float64) ** 2).sum() / ((o.astype(np.float64) - r) ** 2).sum()))
                for o, r in zip(out, ref)]
    s_cal, s_bad = sqnr(cal), sqnr(bad)
    assert all(c > b + 6.0 for c, b in zip(s_cal, s_bad)), (s_cal, s_bad)
    assert s_cal[0] > 20.0


# ------------------------------------------------------------------------------------------------
# the library's calibration kernels (GPU)
# ------------------------------------------------------------------------------------------------
def _rel(a, b, span):
    return abs(a - b) <= 1e-5 * span


@pytest.mark.gpu
@pytest.mark.parametrize("H,W,shift,dim", [(10, 13, 3, 64), (14, 14, 0, 96), (17, 23, 3, 32)])
def test_library_block_observers_equal_the_oracle_fp_mode(orc, H, W, shift, dim):
    torch = pytest.importorskip("torch")
    from paper_2507_19131_b200 import binding as mq
    ctx = mq.Context(0)
    try:
        blk = synth.make_block(np.random.default_rng(H + shift), dim, dim // 32, shift, 4, 8, 4, share_bias=False)
        x = synth.input_blobs(3, 2, H, W, dim, bg_std=0.5, gain=3.0)
        xd = torch.from_numpy(x).cuda()
        dev = mq._Dev(ctx.device)
        bs = mq.fill_block_struct(dev, blk)
        for branch, name in enumerate(("hi", "lo")):
            want_y, want = orc.block_observe_fp(blk, name, x)
            y, got = mq.calibrate_block(ctx, bs, branch, xd)
            y = y.cpu().numpy()
            assert np.abs(y - want_y).max() <= 1e-5 * max(1.0, float(np.abs(want_y).max()))
            assert np.array_equal(y, want_y), "fp block output within tolerance but not bit-identical"
            for site in SITES:
                span = want[site][1] - want[site][0]
                assert _rel(got[site][0], want[site][0], span) and _rel(got[site][1], want[site][1], span), site
                assert got[site] == want[site], f"{site}: within tolerance but not identical"
            assert got["x_in"] == (float(x.min()), float(x.max()))
        m = synth.make_merge(np.random.default_rng(5), dim, 4, 8)
        ms = mq.fill_merge_struct(dev, m)
        want_y, (lo, hi) = orc.merge_observe_fp(m, x)
        ym, (glo, ghi) = mq.calibrate_merge(ctx, ms, xd)
        assert np.array_equal(ym.cpu().numpy(), want_y) and (glo, ghi) == (lo, hi)
        assert ctx.device_status() == 0
    finally:
        ctx.close()


@pytest.mark.gpu
def test_library_calibration_of_a_backbone_and_the_quantizer_definition(orc):
    torch = pytest.importorskip("torch")
    from paper_2507_19131_b200 import binding as mq
    from paper_2507_19131_b200 import calibrate
    # the one definition of "the quantizer that covers a range" against the generator's
    rng = np.random.default_rng(0)
    for _ in range(200):
        lo = float(F32(-abs(rng.standard_normal()) * 10 ** rng.uniform(-2, 2)))
        hi = float(F32(abs(rng.standard_normal()) * 10 ** rng.uniform(-2, 2) + 1e-3))
        for bits in (8, 4, 2):
            want = synth.make_aq(lo, hi, bits)
            assert mq.aq_from_range(lo, hi, bits) == (want.scale, want.inv_scale, want.zp)
    ctx = mq.Context(0)
    try:
        wl = synth.tiny_backbone(ratio=0.4)
        bad = poorly_ranged_backbone(wl)
        cal = calibrate.calibrate_backbone(ctx, bad, wl.x)
        ref = oracle_calibrated_backbone(orc, bad, wl.x)
        for a, b in zip(cal.blocks, ref.blocks):
            assert a.score_inv_scale == b.score_inv_scale
            for name in ("hi", "lo"):
                for site in SITES:
                    assert getattr(getattr(a, name), site) == getattr(getattr(b, name), site), (name, site)
        for a, b in zip(cal.merges, ref.merges):
            assert a.aq == b.aq
        # the calibrated quantizers feed the quantized forward
        want = orc.backbone_forward(cal, wl.x, wl.low_ratios)
        dbb = mq.DeviceBackbone(ctx, cal, wl.B, wl.H, wl.W)
        got = mq.backbone_forward(ctx, dbb, torch.from_numpy(wl.x).cuda(), wl.low_ratios)
        torch.cuda.synchronize()
        for g, w in zip(got, want):
            assert np.array_equal(g.cpu().numpy(), w)
        assert ctx.device_status() == 0
    finally:
        ctx.close()
