"""Parity of the CUDA library (through the C ABI) against the CPU oracle on the same seeded inputs.
Integer results (scores, selection, packed codes, zero-point-corrected int32 accumulators) must be bit-exact;
binary32 results must agree within 1e-3 of the output's max magnitude (they are expected to be identical)."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_2507_19131_b200 import synth  # noqa: E402

F32 = np.float32
TOL = 1e-3


@pytest.fixture(scope="module")
def mq():
    from paper_2507_19131_b200 import binding
    if not torch.cuda.is_available():
        pytest.fail("GPU test selected but no CUDA device is visible")
    return binding


@pytest.fixture(scope="module")
def ctx(mq):
    c = mq.Context(0)
    yield c
    assert c.device_status() == 0
    c.close()


def dev(x):
    return torch.from_numpy(np.ascontiguousarray(x)).cuda()


def assert_close_rel(got, want, tol=TOL):
    scale = max(float(np.abs(want).max()), 1e-30)
    err = float(np.abs(got.astype(np.float64) - want.astype(np.float64)).max())
    assert err <= tol * scale, f"max abs err {err} > {tol} * {scale}"


def check_taps(orc, blk, ref, got, counts, byte_codes=False):
    """Every intermediate of both branches, bit for bit (byte_codes: the block stores one code per byte)."""
    for name, br, n in (("hi", blk.hi, counts[0]), ("lo", blk.lo, counts[1])):
        r, g = getattr(ref, name), getattr(got, name)
        if n == 0:
            continue
        bits = 8 if byte_codes else br.bits
        for f in ("a_codes", "qkv_codes", "o_codes", "f1_codes", "f2_codes"):
            assert np.array_equal(g.__dict__[f].cpu().numpy(), orc.pack(r.__dict__[f], bits)), f"{name}.{f}"
        for f in ("qkv_acc", "pv_acc", "proj_acc", "fc1_acc", "fc2_acc", "p_codes"):
            assert np.array_equal(g.__dict__[f].cpu().numpy(), r.__dict__[f]), f"{name}.{f}"
        assert_close_rel(g.probs.cpu().numpy(), r.probs)                     # the binary32 softmax, stated tolerance
        assert np.array_equal(g.probs.cpu().numpy(), r.probs), f"{name}.probs not bit-identical"
        assert_close_rel(g.x1.cpu().numpy(), r.x1)
        assert np.array_equal(g.x1.cpu().numpy(), r.x1), f"{name}.x1 not bit-identical"


def run_block_case(orc, mq, ctx, blk, x, low, prune=0.0, reverse=False, stage_energy=False, taps=True, byte_codes=False):
    # the C ABI takes the ratios as binary32: both sides get exactly that value (0.11f * 6000 is below 660)
    low, prune = float(F32(low)), float(F32(prune))
    db = mq.DeviceBlock(ctx, blk, byte_codes=byte_codes)
    xd = dev(x)
    e_ref = e_dev = None
    if stage_energy:
        e_ref = orc.energy(x, blk.score_inv_scale)
        e_dev = mq.stage_energy(ctx, xd, blk.score_inv_scale)
        assert np.array_equal(e_dev.cpu().numpy(), e_ref)
    ref = orc.block_forward(blk, x, low, prune, energy_map=e_ref, reverse=reverse, taps=taps)
    got = mq.block_forward(ctx, db, xd, low, prune, energy=e_dev, reverse=reverse, selection=True, taps=taps)
    torch.cuda.synchronize()
    assert got.counts == ref.counts
    assert np.array_equal(got.scores.cpu().numpy(), ref.scores)
    assert np.array_equal(got.order.cpu().numpy(), ref.order)
    assert np.array_equal(got.cls.cpu().numpy(), ref.cls)
    # per-class window lists in ascending window index: what is unique given the classes
    for c, lst in enumerate((got.idx_hi, got.idx_lo, got.idx_pr)):
        lst = lst.cpu().numpy()
        for b in range(x.shape[0]):
            assert np.array_equal(lst[b], np.flatnonzero(ref.cls[b] == c)), f"class {c} list of image {b}"
    if taps:
        check_taps(orc, blk, ref, got, ref.counts, byte_codes)
    y = got.y.cpu().numpy()
    assert_close_rel(y, ref.y)
    assert np.array_equal(y, ref.y), "outputs are within tolerance but not bit-identical"
    return ref, got


# ------------------------------------------------------------------------------------------------
def test_selection_only_many_shapes(orc, mq, ctx):
    rng = np.random.default_rng(0)
    for (B, H, W, C, shift, low, prune, rev) in [(2, 16, 19, 32, 0, 0.3, 0.0, False), (2, 16, 19, 32, 3, 0.3, 0.2, False),
                                                  (1, 56, 56, 96, 0, 0.5, 0.0, True), (3, 30, 37, 64, 3, 0.7, 0.1, False),
                                                  (1, 7, 7, 32, 0, 0.5, 0.0, False)]:
        blk = synth.make_block(rng, C, C // 32, shift, 8, 8, 4)
        x = synth.input_student_t(int(rng.integers(1 << 30)), B, H, W, C)
        x[:, : H // 2] = np.round(x[:, : H // 2])           # provoke tied scores
        run_block_case(orc, mq, ctx, blk, x, low, prune, reverse=rev, taps=False)


def test_all_equal_scores_break_ties_by_index(orc, mq, ctx):
    blk = synth.make_block(np.random.default_rng(1), 32, 1, 0, 8, 8, 4)
    x = np.ones((1, 21, 28, 32), F32)
    ref, got = run_block_case(orc, mq, ctx, blk, x, 0.5, taps=False)
    assert got.order.cpu().numpy()[0].tolist() == list(range(12))


@pytest.mark.parametrize("shift", [0, 3])
@pytest.mark.parametrize("bits", [(8, 4), (4, 2), (8, 8)])
def test_block_tiny_all_taps(orc, mq, ctx, shift, bits):
    blk = synth.make_block(np.random.default_rng(10 + shift), 64, 2, shift, 4, bits[0], bits[1], share_bias=False)
    x = synth.input_blobs(11, 2, 17, 23, 64, bg_std=0.5, gain=4.0)     # ragged: padded to 21 x 28
    run_block_case(orc, mq, ctx, blk, x, 0.4, stage_energy=bool(shift))


@pytest.mark.parametrize("dim,bits", [(64, (8, 4)), (64, (4, 2)), (384, (8, 4)), (192, (8, 2))])
def test_block_one_code_per_byte_all_taps(orc, mq, ctx, dim, bits):
    """byte_codes = 1: the same code values, stored one per byte whatever the bit width; every tap and the output as
    before (the oracle's codes, here compared unpacked)."""
    blk = synth.make_block(np.random.default_rng(dim + bits[1]), dim, dim // 32, 3, 4, bits[0], bits[1], share_bias=False)
    x = synth.input_blobs(12, 2, 17, 23, dim, bg_std=0.5, gain=4.0)
    run_block_case(orc, mq, ctx, blk, x, 0.4, 0.1, byte_codes=True)


def test_block_config1_all_taps(orc, mq, ctx):
    wl = synth.config1()
    run_block_case(orc, mq, ctx, wl.backbone.blocks[0], wl.x, 0.5)


@pytest.mark.parametrize("low,prune", [(0.0, 0.0), (1.0, 0.0), (0.5, 0.3), (0.0, 1.0), (1.0, 0.5)])
def test_block_degenerate_splits(orc, mq, ctx, low, prune):
    blk = synth.make_block(np.random.default_rng(20), 32, 1, 3, 8, 8, 4)
    x = synth.input_blobs(21, 2, 14, 22, 32, bg_std=0.5, gain=4.0)
    ref, got = run_block_case(orc, mq, ctx, blk, x, low, prune)
    if prune == 1.0:
        assert np.array_equal(got.y.cpu().numpy(), x)                 # everything forwarded unchanged


def test_block_single_window_and_wide_dims(orc, mq, ctx):
    blk = synth.make_block(np.random.default_rng(30), 32, 1, 0, 8, 8, 4)
    run_block_case(orc, mq, ctx, blk, synth.input_blobs(31, 1, 5, 6, 32), 0.0)
    for dim in (128, 192, 384, 512, 768):
        blk = synth.make_block(np.random.default_rng(dim), dim, dim // 32, 3, 4, 8, 4)
        run_block_case(orc, mq, ctx, blk, synth.input_blobs(dim + 1, 1, 14, 15, dim, bg_std=0.5), 0.5)


def test_block_random_shapes_and_settings(orc, mq, ctx):
    """Seeded random sweep: widths, map sizes (ragged), batch, shift, bit-width pairs, ratios, pruning, bias sharing,
    worst-case order.  Every case compares selection, all taps and the output bit for bit."""
    rng = np.random.default_rng(2024)
    dims = [32, 64, 96, 128, 192, 256]
    bit_pairs = [(8, 4), (8, 8), (4, 2), (4, 4), (8, 2), (2, 2)]
    for case in range(14):
        dim = int(rng.choice(dims))
        B = int(rng.integers(1, 4))
        H, W = int(rng.integers(3, 30)), int(rng.integers(3, 30))
        shift = int(rng.choice([0, 3, 1, 6]))
        hb, lb = bit_pairs[int(rng.integers(len(bit_pairs)))]
        low = float(rng.choice([0.0, 0.1, 0.3, 0.5, 0.8, 1.0]))
        prune = float(rng.choice([0.0, 0.0, 0.2, 0.5]))
        blk = synth.make_block(rng, dim, dim // 32, shift, int(rng.choice([4, 8])), hb, lb,
                               share_bias=bool(rng.integers(2)))
        x = synth.input_blobs(int(rng.integers(1 << 30)), B, H, W, dim, bg_std=0.5, gain=4.0)
        run_block_case(orc, mq, ctx, blk, x, low, prune, reverse=bool(rng.integers(2)), stage_energy=bool(rng.integers(2)))


def test_many_windows_per_image_and_the_limit(orc, mq, ctx):
    """A long thin map with 6000 windows in one image (the ranking holds one image's scores in shared memory; the
    limit is 6144 windows), and a map beyond the limit, which must be refused before anything is launched."""
    blk = synth.make_block(np.random.default_rng(60), 32, 1, 3, 8, 8, 4)
    x = synth.input_student_t(61, 1, 7, 7 * 6000, 32)
    run_block_case(orc, mq, ctx, blk, x, 0.37, 0.11, taps=False)
    db = mq.DeviceBlock(ctx, blk)
    big = torch.zeros((1, 7, 7 * 6200, 32), device="cuda")
    with pytest.raises(mq.MixaqError) as e:
        mq.block_forward(ctx, db, big, 0.5)
    assert e.value.status == -2
    assert ctx.device_status() == 0


def test_merge_parity(orc, mq, ctx):
    for (C, B, H, W) in [(32, 2, 9, 11), (96, 1, 20, 34), (192, 1, 13, 8)]:
        m = synth.make_merge(np.random.default_rng(C), C, 4, 8)
        x = synth.input_blobs(C + 5, B, H, W, C, bg_std=0.5)
        dm = mq.DeviceMerge(ctx, m)
        y = mq.merge_forward(ctx, dm, dev(x)).cpu().numpy()
        want = orc.merge_forward(m, x)
        assert_close_rel(y, want)
        assert np.array_equal(y, want)


@pytest.mark.parametrize("prune", [0.0, 0.2])
def test_backbone_tiny(orc, mq, ctx, prune):
    wl = synth.tiny_backbone(ratio=0.4, prune=prune)
    want = orc.backbone_forward(wl.backbone, wl.x, wl.low_ratios, wl.prune_ratios)
    dbb = mq.DeviceBackbone(ctx, wl.backbone, wl.B, wl.H, wl.W)
    got = mq.backbone_forward(ctx, dbb, dev(wl.x), wl.low_ratios, wl.prune_ratios)
    torch.cuda.synchronize()
    for g, w in zip(got, want):
        assert_close_rel(g.cpu().numpy(), w)
        assert np.array_equal(g.cpu().numpy(), w)


def test_backbone_graph_replay_reads_fresh_data(orc, mq, ctx):
    """On a capturable stream the backbone call is captured once and replayed; replays must see new input data."""
    wl = synth.tiny_backbone(ratio=0.4, prune=0.2)
    dbb = mq.DeviceBackbone(ctx, wl.backbone, wl.B, wl.H, wl.W)
    xs = [wl.x, np.ascontiguousarray(wl.x[:, ::-1]), (wl.x * F32(0.5)).astype(F32)]
    xd = dev(xs[0])
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for i, x in enumerate(xs):                                # call 0 captures, calls 1 and 2 replay
            xd.copy_(torch.from_numpy(x), non_blocking=False)
            got = mq.backbone_forward(ctx, dbb, xd, wl.low_ratios, wl.prune_ratios)
            side.synchronize()
            want = orc.backbone_forward(wl.backbone, x, wl.low_ratios, wl.prune_ratios)
            for g, w in zip(got, want):
                assert np.array_equal(g.cpu().numpy(), w), f"call {i}"
    torch.cuda.current_stream().wait_stream(side)


def test_precision_classes_within_a_stage_and_the_elevation_switch(orc, mq):
    """A stage of three pairs with ratios that go down and up: default (classes kept: running maximum) and the
    elevation ablation (every pair its own ratio), each against the oracle in the same mode; with and without the graph."""
    bb = synth.make_backbone(9, [64], [6], [2], 8, 8, 4)
    x = synth.input_blobs(10, 2, 21, 29, 64, bg_std=0.5, gain=4.0)
    ratios, prunes = [0.5, 0.2, 0.4], [0.1, 0.3, 0.0]
    c = mq.Context(0)
    try:
        dbb = mq.DeviceBackbone(c, bb, 2, 21, 29)
        side = torch.cuda.Stream()
        for allow in (False, True):
            c.set_window_elevation(allow)
            want = orc.backbone_forward(bb, x, ratios, prunes, allow_elevation=allow)[0]
            got = mq.backbone_forward(c, dbb, dev(x), ratios, prunes)[0].cpu().numpy()       # default stream: direct launches
            assert np.array_equal(got, want), f"allow={allow}"
            with torch.cuda.stream(side):
                xd = dev(x)
                for _ in range(2):                                                             # capture, then replay
                    got = mq.backbone_forward(c, dbb, xd, ratios, prunes)[0]
                side.synchronize()
                assert np.array_equal(got.cpu().numpy(), want), f"graph, allow={allow}"
        c.set_graph_cache(False)
        with torch.cuda.stream(side):
            got = mq.backbone_forward(c, dbb, dev(x), ratios, prunes)[0]
            side.synchronize()
        assert np.array_equal(got.cpu().numpy(), orc.backbone_forward(bb, x, ratios, prunes, allow_elevation=True)[0])
        # worst-case selection order (Table 4) through the whole backbone
        c.set_reverse_selection(True)
        got = mq.backbone_forward(c, dbb, dev(x), ratios, prunes)[0].cpu().numpy()
        want = orc.backbone_forward(bb, x, ratios, prunes, allow_elevation=True, reverse=True)[0]
        assert np.array_equal(got, want) and not np.array_equal(got, orc.backbone_forward(bb, x, ratios, prunes, allow_elevation=True)[0])
        # NVTX ranges around every launch, stage and block (no tracer attached: the calls must be harmless)
        c.set_nvtx(True)
        again = mq.backbone_forward(c, dbb, dev(x), ratios, prunes)[0].cpu().numpy()
        c.set_nvtx(False)
        assert np.array_equal(again, got)
        assert c.device_status() == 0
    finally:
        c.close()


def test_config2_stage1_pair_full_size(orc, mq, ctx):
    """Block pair at 200x334 (W-MSA then SW-MSA with mask), B=2, Student-t input, ratio 0.3, shared stage energy."""
    wl = synth.config2()
    want = orc.backbone_forward(wl.backbone, wl.x, wl.low_ratios)
    dbb = mq.DeviceBackbone(ctx, wl.backbone, wl.B, wl.H, wl.W)
    got = mq.backbone_forward(ctx, dbb, dev(wl.x), wl.low_ratios)
    torch.cuda.synchronize()
    y = got[0].cpu().numpy()
    assert_close_rel(y, want[0])
    assert np.array_equal(y, want[0])


def _full_backbone_case(orc, mq, ctx, wl):
    """Whole backbone at a benchmark configuration's full size, launched the way bench.py launches it (own stream, so
    the second call replays the captured graph); every stage map against the oracle."""
    want = orc.backbone_forward(wl.backbone, wl.x, wl.low_ratios, wl.prune_ratios)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        xd = dev(wl.x)
        # every block bit-packed, then the storage the benchmark uses (one code per byte from 384 channels on)
        for byte_min in (None, 384):
            dbb = mq.DeviceBackbone(ctx, wl.backbone, wl.B, wl.H, wl.W, byte_codes_min_dim=byte_min)
            for call in range(2):
                got = mq.backbone_forward(ctx, dbb, xd, wl.low_ratios, wl.prune_ratios)
                side.synchronize()
                assert ctx.device_status() == 0
                for st, (g, w) in enumerate(zip(got, want)):
                    g = g.cpu().numpy()
                    assert_close_rel(g, w)
                    assert np.array_equal(g, w), f"stage {st} (call {call}, byte codes from {byte_min}) not bit-identical"
            del dbb
    torch.cuda.current_stream().wait_stream(side)


@pytest.mark.parametrize("ratio", [0.0, 0.25, 0.5, 0.75])
def test_config3_swin_t_800x1333_full_size(orc, mq, ctx, ratio):
    """Swin-T, 200x334 tokens, W4, A8/A4: the benchmark workload at every low-bit ratio the benchmark sweeps."""
    _full_backbone_case(orc, mq, ctx, synth.config3(ratio=ratio))


def test_config4_swin_s_1024_full_size_three_classes(orc, mq, ctx):
    """Swin-S, B=4, 256x256 tokens, W4, A4 high / A2 low, ratio 0.5, 20 % of the windows pruned."""
    _full_backbone_case(orc, mq, ctx, synth.config4())


def test_config5_swin_b_1536_full_size(orc, mq, ctx):
    """Swin-B, B=2, 384x384 tokens, W8, A8/A4, clustered high-norm regions, ratio 0.5."""
    _full_backbone_case(orc, mq, ctx, synth.config5(ratio=0.5))


@pytest.mark.parametrize("B,Hi,Wi,C0", [(2, 16, 20, 32), (1, 13, 18, 96), (1, 7, 5, 32), (1, 800, 1333, 96)])
def test_patch_embed_parity(orc, mq, ctx, B, Hi, Wi, C0):
    """The stem in front of the backbone (image -> x0), including sizes that need zero padding and the full
    800 x 1333 image of the benchmark workload."""
    e = synth.make_embed(np.random.default_rng(C0 + Hi), C0)
    img = synth.input_image(Hi + Wi, B, Hi, Wi)
    de = mq.DeviceEmbed(ctx, e)
    got = mq.embed_forward(ctx, de, dev(img)).cpu().numpy()
    want = orc.patch_embed(e, img)
    assert got.shape == want.shape
    assert_close_rel(got, want)
    assert np.array_equal(got, want)


def test_stage_output_norm_parity(orc, mq, ctx):
    rng = np.random.default_rng(9)
    for (rows_shape, Cc) in [((2, 9, 11), 96), ((1, 25, 42), 768), ((3, 5, 7), 192)]:
        x = (rng.standard_normal(rows_shape + (Cc,), dtype=F32) * F32(3.0) + F32(0.5)).astype(F32)
        g = (1.0 + 0.1 * rng.standard_normal(Cc)).astype(F32)
        b = (0.1 * rng.standard_normal(Cc)).astype(F32)
        got = mq.norm_forward(ctx, dev(g), dev(b), dev(x)).cpu().numpy()
        want = orc.layernorm(x, g, b)
        assert np.array_equal(got, want)


def test_image_to_normed_stage_maps_end_to_end(orc, mq, ctx):
    """image -> stem -> two-branch backbone -> per-stage output norms, against the same chain of oracle calls."""
    wl = synth.tiny_backbone(ratio=0.4, prune=0.2)
    rng = np.random.default_rng(11)
    e = synth.make_embed(rng, wl.backbone.dims[0])
    img = synth.input_image(12, wl.B, 4 * wl.H - 1, 4 * wl.W - 2)          # pads up to (4H, 4W)
    norms = [((1.0 + 0.05 * rng.standard_normal(c)).astype(F32), (0.05 * rng.standard_normal(c)).astype(F32)) for c in wl.backbone.dims]
    x0_ref = orc.patch_embed(e, img)
    want = [orc.layernorm(o, g, b) for o, (g, b) in zip(orc.backbone_forward(wl.backbone, x0_ref, wl.low_ratios, wl.prune_ratios), norms)]
    de = mq.DeviceEmbed(ctx, e)
    x0 = mq.embed_forward(ctx, de, dev(img))
    assert tuple(x0.shape) == (wl.B, wl.H, wl.W, wl.backbone.dims[0])
    dbb = mq.DeviceBackbone(ctx, wl.backbone, wl.B, wl.H, wl.W)
    outs = mq.backbone_forward(ctx, dbb, x0, wl.low_ratios, wl.prune_ratios)
    got = [mq.norm_forward(ctx, dev(g), dev(b), o).cpu().numpy() for o, (g, b) in zip(outs, norms)]
    for gg, ww in zip(got, want):
        assert np.array_equal(gg, ww)


def test_image_to_normed_stage_maps_in_one_backbone_call(orc, mq, ctx):
    """The same chain through ONE mixaq_backbone_forward call (stem and output norms given in the backbone parameters),
    on a capturable stream: first call captures the graph, second replays it."""
    wl = synth.tiny_backbone(ratio=0.4, prune=0.2)
    rng = np.random.default_rng(13)
    e = synth.make_embed(rng, wl.backbone.dims[0])
    Hi, Wi = 4 * wl.H - 1, 4 * wl.W - 2
    img = synth.input_image(14, wl.B, Hi, Wi)
    norms = [((1.0 + 0.05 * rng.standard_normal(c)).astype(F32), (0.05 * rng.standard_normal(c)).astype(F32)) for c in wl.backbone.dims]
    x0_ref = orc.patch_embed(e, img)
    want = [orc.layernorm(o, g, b) for o, (g, b) in zip(orc.backbone_forward(wl.backbone, x0_ref, wl.low_ratios, wl.prune_ratios), norms)]
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        dbb = mq.DeviceBackbone(ctx, wl.backbone, wl.B, Hi, Wi, embed=e, norms=norms)
        imd = dev(img)
        for call in range(2):
            got = mq.backbone_forward(ctx, dbb, imd, wl.low_ratios, wl.prune_ratios)
            side.synchronize()
            for st, (g, w) in enumerate(zip(got, want)):
                assert np.array_equal(g.cpu().numpy(), w), f"stage {st}, call {call}"
    torch.cuda.current_stream().wait_stream(side)
    assert ctx.device_status() == 0


def test_bounded_wait_runs_out_and_the_context_stays_usable(orc, mq):
    """Failure path without a fault: a barrier that nothing signals makes the kernels' bounded wait run out; the status
    word reports it, can be cleared, and the next forward on the same context is correct."""
    c = mq.Context(0)
    try:
        assert c.device_status() == 0
        c.selftest_wait_timeout()
        assert c.device_status() == -5                       # MIXAQ_DEVICE_TIMEOUT
        c.clear_device_status()
        assert c.device_status() == 0
        blk = synth.make_block(np.random.default_rng(50), 32, 1, 3, 8, 8, 4)
        x = synth.input_blobs(51, 1, 14, 15, 32, bg_std=0.5)
        run_block_case(orc, mq, c, blk, x, 0.5)
        assert c.device_status() == 0
    finally:
        c.close()


def test_workspace_guard_zones(orc, mq):
    """The guard zones behind every workspace buffer: untouched by a forward (block with all taps, and a small
    backbone through its graph), and the check itself reports a byte written just past a buffer."""
    c = mq.Context(0)
    try:
        c.set_workspace_guards(True)
        blk = synth.make_block(np.random.default_rng(52), 64, 2, 3, 4, 8, 4)
        x = synth.input_blobs(53, 2, 17, 23, 64, bg_std=0.5, gain=4.0)
        run_block_case(orc, mq, c, blk, x, 0.4, 0.1)
        assert c.device_status() == 0
        wl = synth.tiny_backbone()
        want = orc.backbone_forward(wl.backbone, wl.x, wl.low_ratios, wl.prune_ratios)
        side = torch.cuda.Stream()
        with torch.cuda.stream(side):
            dbb = mq.DeviceBackbone(c, wl.backbone, wl.B, wl.H, wl.W)
            xd = dev(wl.x)
            for _ in range(2):
                got = mq.backbone_forward(c, dbb, xd, wl.low_ratios, wl.prune_ratios)
            side.synchronize()
            for g, w in zip(got, want):
                assert np.array_equal(g.cpu().numpy(), w)
        assert c.device_status() == 0
        c.selftest_workspace_guards(overrun=False)
        assert c.device_status() == 0
        c.selftest_workspace_guards(overrun=True)
        assert c.device_status() == -7                       # MIXAQ_WORKSPACE_OVERRUN
        c.clear_device_status()
        assert c.device_status() == 0
    finally:
        c.close()


def test_mma_issue_rate_microbenchmark(mq, ctx):
    """The library's own tensor-core loop: kind::i8 reaches petaops; kind::f8f6f4 (the path of the 4/6-bit operand
    formats in 8-bit containers) is not faster; kind::mxf4 (block-scaled E2M1, the one narrower path with a higher
    nominal rate) is measured next to them.  The numbers behind the choice of kind::i8 for the low-bit branch."""
    i8 = ctx.measure_mma_peak(0, 2000)
    f8 = ctx.measure_mma_peak(1, 2000)
    mx = ctx.measure_mma_peak(2, 2000)
    assert ctx.device_status() == 0
    assert 1500.0 < i8 < 6000.0 and 1500.0 < f8 < 6000.0 and 1500.0 < mx < 12000.0
    assert f8 < 1.1 * i8
    print(f"mma issue rate TOP/s: i8 {i8:.0f}  f8f6f4 {f8:.0f}  mxf4 {mx:.0f}")


def test_invalid_arguments_are_rejected_before_any_launch(mq, ctx):
    import ctypes as C
    blk = synth.make_block(np.random.default_rng(40), 32, 1, 0, 8, 8, 4)
    db = mq.DeviceBlock(ctx, blk)
    x = torch.zeros((1, 14, 14, 32), device="cuda")
    with pytest.raises(mq.MixaqError) as e:
        mq.block_forward(ctx, db, x, 1.5)
    assert e.value.status == -1
    with pytest.raises(mq.MixaqError) as e:
        mq.block_forward(ctx, db, x, 0.5, y=x)
    assert e.value.status == -1
    L = mq.lib()
    ws = db.workspace(1, 14, 14)
    y = torch.empty_like(x)
    st = L.mixaq_block_forward(ctx.h, C.byref(db.s), C.c_void_p(x.data_ptr()), C.c_void_p(y.data_ptr()), 1, 14, 14,
                               C.c_float(0.5), C.c_float(0.0), None, None, C.c_void_p(ws.data_ptr()), C.c_size_t(16),
                               None, None)
    assert st == -3
    bad = mq.BlockS.from_buffer_copy(db.s)
    bad.window = 8
    st = L.mixaq_block_forward(ctx.h, C.byref(bad), C.c_void_p(x.data_ptr()), C.c_void_p(y.data_ptr()), 1, 14, 14,
                               C.c_float(0.5), C.c_float(0.0), None, None, C.c_void_p(ws.data_ptr()),
                               C.c_size_t(ws.numel()), None, None)
    assert st == -2
    # pointers the kernels could only touch with misaligned accesses are refused on the host: x off by 4 bytes,
    # workspace off by 16, a weight matrix off by 1
    big = torch.zeros(x.numel() + 4, device="cuda")
    for xp, wp in ((big.data_ptr() + 4, ws.data_ptr()), (x.data_ptr(), ws.data_ptr() + 16)):
        st = L.mixaq_block_forward(ctx.h, C.byref(db.s), C.c_void_p(xp), C.c_void_p(y.data_ptr()), 1, 14, 14,
                                   C.c_float(0.5), C.c_float(0.0), None, None, C.c_void_p(wp),
                                   C.c_size_t(ws.numel() - 16), None, None)
        assert st == -1
    bad = mq.BlockS.from_buffer_copy(db.s)
    bad.fc1.codes = bad.fc1.codes + 1
    st = L.mixaq_block_forward(ctx.h, C.byref(bad), C.c_void_p(x.data_ptr()), C.c_void_p(y.data_ptr()), 1, 14, 14,
                               C.c_float(0.5), C.c_float(0.0), None, None, C.c_void_p(ws.data_ptr()),
                               C.c_size_t(ws.numel()), None, None)
    assert st == -1
    assert ctx.device_status() == 0
