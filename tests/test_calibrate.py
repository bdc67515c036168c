"""The calibration utility on CPU: its floating-point block must be the block the oracle runs in fp mode, and the
quantizers it writes must make the quantized model track the floating-point one better than uncalibrated ranges."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

from paper_2507_19131_b200 import calibrate, synth  # noqa: E402

F32 = np.float32


@pytest.mark.parametrize("shift", [0, 3])
def test_fp_block_equals_the_oracle_fp_mode(orc, shift):
    blk = synth.make_block(np.random.default_rng(1 + shift), 64, 2, shift, 8, 8, 4, share_bias=False)
    x = synth.input_blobs(2, 2, 10, 13, 64, bg_std=0.5, gain=3.0)
    for name in ("hi", "lo"):
        low = 0.0 if name == "hi" else 1.0                       # all windows through that branch
        want = orc.block_forward(blk, x, low, quant=False).y
        got = calibrate.fp_block(blk, getattr(blk, name), torch.from_numpy(x)).numpy()
        assert np.abs(got - want).max() < 2e-4 * max(1.0, float(np.abs(want).max()))


def test_fp_merge_equals_the_oracle_fp_mode(orc):
    m = synth.make_merge(np.random.default_rng(3), 32, 8, 8)
    x = synth.input_blobs(4, 2, 9, 11, 32, bg_std=0.5)
    want = orc.merge_forward(m, x, quant=False)
    got = calibrate.fp_merge(m, torch.from_numpy(x)).numpy()
    assert np.abs(got - want).max() < 1e-4


def test_calibrated_quantizers_cover_the_sample_and_share_ranges(orc):
    wl = synth.tiny_backbone(ratio=0.4)
    # start from deliberately poor ranges
    bad = synth.make_backbone(78, wl.backbone.dims, wl.backbone.depths, wl.backbone.heads, 8, 8, 4)
    for b in bad.blocks:
        # post-training start: the low branch's LayerNorm is a copy of the high branch's
        b.lo.ln1_g, b.lo.ln1_b, b.lo.ln2_g, b.lo.ln2_b = b.hi.ln1_g, b.hi.ln1_b, b.hi.ln2_g, b.hi.ln2_b
        for br in (b.hi, b.lo):
            for site in calibrate.SITES:
                setattr(br, site, synth.make_aq(-50.0, 50.0, br.bits))
    cal = calibrate.calibrate_backbone(bad, wl.x, device="cpu")
    b0 = cal.blocks[0]
    for site in calibrate.SITES:
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
