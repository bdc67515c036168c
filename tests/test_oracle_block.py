"""Pins of the oracle's block, merging and backbone: the special cases the paper fixes (ratio 0 / ratio 1,
shared shadow weights, pruned windows forwarded unchanged) and a textbook Swin block written on the un-windowed
map in binary64.  CPU only."""
import copy
import math

import numpy as np
import pytest
from scipy.special import erf

from paper_2507_19131_b200 import synth

F32 = np.float32


def small_block(seed=5, dim=32, heads=1, shift=0, w_bits=8, hi=8, lo=4, share_bias=True):
    rng = np.random.default_rng(seed)
    return synth.make_block(rng, dim, heads, shift, w_bits, hi, lo, share_bias=share_bias)


def small_input(seed, B, H, W, C):
    return synth.input_blobs(seed, B, H, W, C, bg_std=0.5, gain=4.0)


# ------------------------------------------------------------------------------------------------
# Section 3.3: the ratio is the proportion of windows in the low branch.  Ratio 0 is the uniform high-bit
# model (Table 1, row "MixA-Q, Act Bit 4"); ratio 1 the uniform low-bit model.
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shift", [0, 3])
def test_ratio0_and_ratio1_reduce_to_uniform_blocks(orc, shift):
    blk = small_block(shift=shift, dim=64, heads=2)
    x = small_input(1, 2, 16, 19, 64)
    y0 = orc.block_forward(blk, x, 0.0).y
    y1 = orc.block_forward(blk, x, 1.0).y
    assert np.array_equal(y0, orc.uniform_block_forward(blk, "hi", x))
    assert np.array_equal(y1, orc.uniform_block_forward(blk, "lo", x))
    assert not np.array_equal(y0, y1)


def test_mixed_ratio_is_a_per_window_mix_of_the_two_uniform_models(orc):
    blk = small_block(shift=0, dim=32, heads=1)
    x = small_input(2, 1, 21, 28, 32)
    r = orc.block_forward(blk, x, 0.5)
    yh = orc.uniform_block_forward(blk, "hi", x)
    yl = orc.uniform_block_forward(blk, "lo", x)
    nwx = 4
    for w in range(12):
        wy, wx = divmod(w, nwx)
        sl = (0, slice(wy * 7, wy * 7 + 7), slice(wx * 7, wx * 7 + 7))
        want = yh[sl] if r.cls[0, w] == 0 else yl[sl]
        assert np.array_equal(r.y[sl], want)
    assert (r.cls[0] == 0).sum() == 6 and (r.cls[0] == 1).sum() == 6


def test_identical_branches_make_the_output_independent_of_the_ratio(orc):
    blk = small_block(shift=3, dim=32, heads=1, hi=8, lo=8)
    blk.lo = copy.deepcopy(blk.hi)                       # same LN, quantizers, bias, bit width
    x = small_input(3, 1, 14, 21, 32)
    ys = [orc.block_forward(blk, x, r).y for r in (0.0, 0.3, 0.7, 1.0)]
    for y in ys[1:]:
        assert np.array_equal(y, ys[0])


def test_pruned_windows_are_forwarded_unchanged(orc):
    blk = small_block(shift=3, dim=32, heads=1)
    x = small_input(4, 2, 15, 22, 32)
    r = orc.block_forward(blk, x, 0.5, prune_ratio=0.25)
    n_hi, n_lo, n_pr = r.counts
    assert n_pr == 3 and n_lo == 4 and n_hi == 5          # 12 windows: 3 pruned, half of the rest low
    changed = np.zeros(x.shape[:3], bool)
    for b in range(2):
        for w in range(12):
            toks = [orc.window_token(15, 22, 7, 3, w, t) for t in range(49)]
            toks = [t for t in toks if t >= 0]
            yy, xx = np.divmod(np.array(toks), 22)
            same = np.array_equal(r.y[b, yy, xx], x[b, yy, xx])
            assert same == (r.cls[b, w] == 2)
            changed[b, yy, xx] = not same
    # the pruned class is the lowest-scored one
    for b in range(2):
        assert r.scores[b][r.cls[b] == 2].max() <= r.scores[b][r.cls[b] != 2].min()


def test_worst_case_selection_swaps_the_roles(orc):
    blk = small_block(shift=0, dim=32, heads=1)
    x = small_input(6, 1, 21, 28, 32)
    a = orc.block_forward(blk, x, 0.5)
    b = orc.block_forward(blk, x, 0.5, reverse=True)
    assert np.array_equal(a.cls[0], 1 - b.cls[0])        # 12 distinct scores, half and half


def test_stage_shared_energy_map_is_used_when_given(orc):
    blk = small_block(shift=3, dim=32, heads=1)
    x = small_input(7, 1, 14, 21, 32)
    other = small_input(8, 1, 14, 21, 32)
    e_other = orc.energy(other, blk.score_inv_scale)
    r = orc.block_forward(blk, x, 0.5, energy_map=e_other)
    assert np.array_equal(r.scores, orc.window_scores(e_other, 7, 3))
    r2 = orc.block_forward(blk, x, 0.5)
    assert np.array_equal(r2.scores, orc.window_scores(orc.energy(x, blk.score_inv_scale), 7, 3))


# ------------------------------------------------------------------------------------------------
# A textbook Swin block on the un-windowed map, binary64, written from global coordinates: token i attends
# token j iff both fall into the same window of the cyclically shifted padded frame and the same mask region.
# ------------------------------------------------------------------------------------------------
def textbook_block(blk, br, x, sites=None):
    """sites (optional dict): filled with (min, max) of what each quantizer site would see, over ALL tokens of the
    padded map (pad tokens pass through the layers like any token; only the final crop drops them)."""
    B, H, W, C = x.shape
    ws, s, nh = blk.window, blk.shift, blk.heads
    d = C // nh
    Hp, Wp = -(-H // ws) * ws, -(-W // ws) * ws

    def ln(v, g, b):
        mu = v.mean(-1, keepdims=True)
        var = ((v - mu) ** 2).mean(-1, keepdims=True)
        return (v - mu) / np.sqrt(var + 1e-5) * g + b

    def lin(v, L, bias):
        return v @ (L.codes.astype(np.float64) * L.scale.astype(np.float64)[:, None]).T + bias

    def see(name, t):
        if sites is not None:
            lo, hi = sites.get(name, (np.inf, -np.inf))
            sites[name] = (min(lo, float(t.min())), max(hi, float(t.max())))

    # coordinates of every padded-frame token in the shifted frame
    yy, xx = np.mgrid[0:Hp, 0:Wp]
    ys, xs = (yy - s) % Hp, (xx - s) % Wp
    win = (ys // ws) * (Wp // ws) + xs // ws
    ti, tj = ys % ws, xs % ws

    def region(p, L):
        return np.where(p < L - ws, 0, np.where(p < L - s, 1, 2)) if s else np.zeros_like(p)

    reg = region(ys, Hp) * 3 + region(xs, Wp)
    win, ti, tj, reg = (a.reshape(-1) for a in (win, ti, tj, reg))
    same_win = win[:, None] == win[None, :]
    masked = reg[:, None] != reg[None, :]
    ridx = (ti[:, None] - ti[None, :] + ws - 1) * (2 * ws - 1) + (tj[:, None] - tj[None, :] + ws - 1)
    out = np.empty_like(x, dtype=np.float64)
    for b in range(B):
        xb = np.zeros((Hp, Wp, C))
        xb[:H, :W] = x[b].astype(np.float64)
        n1 = np.zeros((Hp, Wp, C))
        n1[:H, :W] = ln(xb[:H, :W], br.ln1_g, br.ln1_b)                 # pad tokens are zero AFTER the norm
        see("qkv_in", n1)
        qkv = lin(n1.reshape(-1, C), blk.qkv, br.b_qkv)
        for i, name in enumerate(("q", "k", "v")):
            see(name, qkv[:, i * C:(i + 1) * C])
        att = np.zeros((Hp * Wp, C))
        for h in range(nh):
            q, k, v = (qkv[:, i * C + h * d:i * C + (h + 1) * d] for i in range(3))
            lg = q @ k.T / math.sqrt(d) + blk.relpos[ridx, h].astype(np.float64) + np.where(masked, -100.0, 0.0)
            lg = np.where(same_win, lg, -np.inf)
            p = np.exp(lg - lg.max(-1, keepdims=True))
            p /= p.sum(-1, keepdims=True)
            att[:, h * d:(h + 1) * d] = p @ v
        see("proj_in", att)
        x1 = xb + lin(att, blk.proj, br.b_proj).reshape(Hp, Wp, C)      # a pad token's residual input is zero
        n2 = ln(x1, br.ln2_g, br.ln2_b)
        see("fc1_in", n2)
        hid = lin(n2, blk.fc1, br.b_fc1)
        hid = 0.5 * hid * (1 + erf(hid / math.sqrt(2)))
        see("fc2_in", hid)
        out[b] = (x1 + lin(hid, blk.fc2, br.b_fc2))[:H, :W]
    return out


@pytest.mark.parametrize("H,W,shift,dim,heads", [(10, 12, 0, 32, 1), (10, 12, 3, 32, 1), (14, 14, 3, 64, 2), (8, 9, 3, 32, 1)])
def test_fp_mode_equals_textbook_swin_block(orc, H, W, shift, dim, heads):
    blk = small_block(seed=H * 31 + shift, dim=dim, heads=heads, shift=shift)
    x = small_input(9, 2, H, W, dim)
    got = orc.uniform_block_forward(blk, "hi", x, quant=False)
    want = textbook_block(blk, blk.hi, x)
    assert np.abs(got - want).max() < 2e-4 * max(1.0, np.abs(want).max())
    # and the two-branch bookkeeping in fp mode: identical branches -> same map for any ratio
    blk.lo = copy.deepcopy(blk.hi)
    got2 = orc.block_forward(blk, x, 0.4, quant=False).y
    assert np.array_equal(got2, got)


@pytest.mark.parametrize("H,W,shift,dim,heads", [(10, 12, 3, 32, 1), (14, 14, 0, 64, 2), (8, 9, 3, 32, 1)])
def test_calibration_observer_ranges_equal_the_textbook_blocks(orc, H, W, shift, dim, heads):
    """Section 4.3: the ranges come from the floating-point block on the full feature map.  The oracle's observer
    against the min / max of the same seven tensors of the textbook block (binary64, un-windowed map)."""
    blk = small_block(seed=H + 7 * shift, dim=dim, heads=heads, shift=shift, share_bias=False)
    x = small_input(19, 2, H, W, dim)
    for name in ("hi", "lo"):
        br = getattr(blk, name)
        y, got = orc.block_observe_fp(blk, name, x)
        sites = {}
        want_y = textbook_block(blk, br, x, sites)
        assert np.abs(y - want_y).max() < 2e-4 * max(1.0, np.abs(want_y).max())
        assert np.array_equal(y, orc.uniform_block_forward(blk, name, x, quant=False))
        for site in orc.SITES:
            span = sites[site][1] - sites[site][0]
            assert abs(got[site][0] - sites[site][0]) < 1e-4 * span and abs(got[site][1] - sites[site][1]) < 1e-4 * span, site
    m = synth.make_merge(np.random.default_rng(23), dim, 8, 8)
    ym, (lo, hi) = orc.merge_observe_fp(m, x)
    assert np.array_equal(ym, orc.merge_forward(m, x, quant=False))
    B = x.shape[0]
    xp = np.zeros((B, H + H % 2, W + W % 2, dim), np.float64)
    xp[:, :H, :W] = x
    cat = np.concatenate([xp[:, 0::2, 0::2], xp[:, 1::2, 0::2], xp[:, 0::2, 1::2], xp[:, 1::2, 1::2]], -1)
    mu = cat.mean(-1, keepdims=True)
    n = (cat - mu) / np.sqrt(((cat - mu) ** 2).mean(-1, keepdims=True) + 1e-5) * m.ln_g + m.ln_b
    assert abs(lo - n.min()) < 1e-4 and abs(hi - n.max()) < 1e-4


# ------------------------------------------------------------------------------------------------
# quantized block internals against numpy restatements built from the taps
# ------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("H,W", [(14, 21), (10, 12)])      # 10 x 12 is padded to 14 x 14: pad tokens are keys
def test_quantized_attention_brute_force_from_codes(orc, H, W):
    blk = small_block(seed=12, dim=64, heads=2, shift=3)
    x = small_input(10, 1, H, W, 64)
    r = orc.block_forward(blk, x, 0.5, taps=True)
    T, C, nh, d = 49, 64, 2, 32
    for name, br, n in (("hi", blk.hi, r.counts[0]), ("lo", blk.lo, r.counts[1])):
        tp = getattr(r, name)
        off = 0 if name == "hi" else r.counts[0]
        relb = orc.relpos_bias(blk.relpos, 7, nh).astype(np.float64)
        pmax = (1 << br.bits) - 1
        near_tie = 0
        for j in range(n):
            w = int(r.order[0, off + j])
            mask = orc.shift_mask(H, W, 7, 3, w).astype(np.float64)
            qkv = tp.qkv_codes[j * T:(j + 1) * T].astype(np.int64)
            for h in range(nh):
                q = qkv[:, h * d:(h + 1) * d] - br.q.zp
                k = qkv[:, C + h * d:C + (h + 1) * d] - br.k.zp
                v = qkv[:, 2 * C + h * d:2 * C + (h + 1) * d] - br.v.zp
                lg = (q @ k.T) * (np.float64(F32(br.q.scale)) * np.float64(F32(br.k.scale)) / math.sqrt(d)) + relb[h] + mask
                p = np.exp(lg - lg.max(-1, keepdims=True))
                p /= p.sum(-1, keepdims=True)
                assert np.abs(tp.probs[j, h] - p).max() < 2e-6
                assert np.abs(tp.probs[j, h].sum(-1) - 1).max() < 2e-6
                pc = np.clip(np.rint(p * pmax), 0, pmax)
                diff = pc != tp.p_codes[j, h]
                # a code may differ only where p*pmax sits on a rounding boundary
                frac = np.abs(p * pmax - np.floor(p * pmax) - 0.5)
                assert (frac[diff] < 1e-3).all()
                near_tie += int(diff.sum())
                # dequantized rows sum to 1 within 49 half-steps
                assert np.abs(tp.p_codes[j, h].sum(-1) / pmax - 1).max() <= 49 / (2 * pmax) + 1e-6
                pv = tp.p_codes[j, h].astype(np.int64) @ v
                assert np.array_equal(tp.pv_acc[j * T:(j + 1) * T, h * d:(h + 1) * d], pv)
        assert near_tie <= 3


def numpy_window_map(H, W, ws, shift):
    """[nW][ws*ws] source token (y*W + x) of every window position, -1 for a pad token, from numpy.roll on the padded
    index map: pad to multiples of the window, roll by -shift, cut into windows."""
    Hp, Wp = -(-H // ws) * ws, -(-W // ws) * ws
    idx = -np.ones((Hp, Wp), np.int64)
    idx[:H, :W] = np.arange(H * W).reshape(H, W)
    idx = np.roll(idx, (-shift, -shift), axis=(0, 1))
    return idx.reshape(Hp // ws, ws, Wp // ws, ws).transpose(0, 2, 1, 3).reshape(-1, ws * ws)


@pytest.mark.parametrize("H,W,shift", [(14, 14, 0), (10, 12, 3), (16, 19, 3)])
def test_quantized_block_taps_against_primitives_in_numpy(orc, H, W, shift):
    """Every stage of one quantized window batch restated with numpy from the previous tap: pins the
    wiring (which quantizer, which bias, which residual) rather than the primitives.  On the ragged, shifted maps the
    windows hold pad tokens: their rows must carry the code of zero after LN1 (not the norm of a zero row), take part
    in the layers like any row (residual input zero) and never reach the output map."""
    blk = small_block(seed=13, dim=32, heads=1, shift=shift, share_bias=False)
    x = small_input(11, 1, H, W, 32)
    r = orc.block_forward(blk, x, 0.5, taps=True)
    T, C = 49, 32
    wmap = numpy_window_map(H, W, 7, shift)
    xf = x[0].reshape(H * W, C)
    covered = np.zeros(H * W, int)
    n_pad_rows = 0
    for name, br, off, n in (("hi", blk.hi, 0, r.counts[0]), ("lo", blk.lo, r.counts[0], r.counts[1])):
        tp = getattr(r, name)
        for j in range(n):
            w = int(r.order[0, off + j])
            src = wmap[w]
            real = src >= 0
            n_pad_rows += int((~real).sum())
            xin = np.zeros((T, C), F32)
            xin[real] = xf[src[real]]
            rows = slice(j * T, (j + 1) * T)
            a = np.empty((T, C), np.uint8)
            a[real] = orc.quantize(orc.layernorm(xin[real], br.ln1_g, br.ln1_b), br.qkv_in)
            a[~real] = br.qkv_in.zp                                   # zero AFTER the norm: code of 0.0 is the zero point
            assert np.array_equal(tp.a_codes[rows], a)
            acc = (a.astype(np.int64) - br.qkv_in.zp) @ blk.qkv.codes.astype(np.int64).T
            assert np.array_equal(tp.qkv_acc[rows], acc)
            assert not acc[~real].any()                               # a pad row enters QKV as exact zeros: q, k, v = bias
            yq = (acc.astype(F32) * (F32(br.qkv_in.scale) * blk.qkv.scale)[None]).astype(np.float64) + br.b_qkv
            for i, qz in enumerate((br.q, br.k, br.v)):
                want = np.clip(np.rint(yq[:, i * C:(i + 1) * C] * np.float64(F32(qz.inv_scale))) + qz.zp, 0, (1 << qz.bits) - 1)
                got = tp.qkv_codes[rows, i * C:(i + 1) * C]
                assert (np.abs(want - got) <= 1).all() and (want != got).mean() < 0.01
            so = np.float64(F32(1.0) / F32((1 << br.bits) - 1)) * np.float64(F32(br.v.scale))
            o_want = np.clip(np.rint(tp.pv_acc[rows] * so * np.float64(F32(br.proj_in.inv_scale))) + br.proj_in.zp, 0, (1 << br.bits) - 1)
            assert (np.abs(o_want - tp.o_codes[rows]) <= 1).all() and (o_want != tp.o_codes[rows]).mean() < 0.01
            pacc = (tp.o_codes[rows].astype(np.int64) - br.proj_in.zp) @ blk.proj.codes.astype(np.int64).T
            assert np.array_equal(tp.proj_acc[rows], pacc)
            x1 = xin + pacc * (np.float64(F32(br.proj_in.scale)) * blk.proj.scale.astype(np.float64))[None] + br.b_proj
            assert np.abs(tp.x1[rows] - x1).max() < 1e-5 * max(1, np.abs(x1).max())
            f1 = orc.quantize(orc.layernorm(tp.x1[rows], br.ln2_g, br.ln2_b), br.fc1_in)
            assert np.array_equal(tp.f1_codes[rows], f1)
            a1 = (f1.astype(np.int64) - br.fc1_in.zp) @ blk.fc1.codes.astype(np.int64).T
            assert np.array_equal(tp.fc1_acc[rows], a1)
            hid = a1 * (np.float64(F32(br.fc1_in.scale)) * blk.fc1.scale.astype(np.float64))[None] + br.b_fc1
            hid = 0.5 * hid * (1 + erf(hid / math.sqrt(2)))
            f2 = np.clip(np.rint(hid * np.float64(F32(br.fc2_in.inv_scale))) + br.fc2_in.zp, 0, (1 << br.bits) - 1)
            assert (np.abs(f2 - tp.f2_codes[rows]) <= 1).all() and (f2 != tp.f2_codes[rows]).mean() < 0.01
            a2 = (tp.f2_codes[rows].astype(np.int64) - br.fc2_in.zp) @ blk.fc2.codes.astype(np.int64).T
            assert np.array_equal(tp.fc2_acc[rows], a2)
            yw = tp.x1[rows] + a2 * (np.float64(F32(br.fc2_in.scale)) * blk.fc2.scale.astype(np.float64))[None] + br.b_fc2
            got = r.y[0].reshape(H * W, C)[src[real]]                 # only real tokens are written back
            assert np.abs(got - yw[real]).max() < 1e-5 * max(1, np.abs(yw).max())
            covered[src[real]] += 1
    assert (covered == 1).all()                                        # every token of the map comes from exactly one window row
    Hp, Wp = -(-H // 7) * 7, -(-W // 7) * 7
    assert n_pad_rows == Hp * Wp - H * W


def test_uniform_block_is_written_separately_and_catches_a_planted_pad_mistake(orc):
    """The whole-map uniform block and the window-batch path agree bit for bit on a ragged, shifted map (that is the
    ratio-0 / ratio-1 pin); a plausible mistake -- treating pad tokens as zeros BEFORE the norm, i.e. giving them the
    code of beta instead of the code of zero -- is visible in the taps the agreement rests on."""
    blk = small_block(seed=17, dim=32, heads=1, shift=3)
    x = small_input(18, 1, 10, 12, 32)
    r = orc.block_forward(blk, x, 0.0, taps=True)
    assert np.array_equal(r.y, orc.uniform_block_forward(blk, "hi", x))
    wmap = numpy_window_map(10, 12, 7, 3)
    zero_code = blk.hi.qkv_in.zp
    beta_code = orc.quantize(orc.layernorm(np.zeros((1, 32), F32), blk.hi.ln1_g, blk.hi.ln1_b), blk.hi.qkv_in)[0]
    assert (beta_code != zero_code).any()                              # the two readings differ on this block
    for j in range(r.counts[0]):
        pad = wmap[int(r.order[0, j])] < 0
        assert (r.hi.a_codes[j * 49:(j + 1) * 49][pad] == zero_code).all()


def test_sqnr_rises_with_bit_width(orc):
    """Sanity only: on an outlier-free input the quantized block approaches the fp block as bits grow."""
    x = np.random.default_rng(21).standard_normal((1, 14, 14, 32), dtype=F32)
    sq = []
    for bits in (2, 4, 8):
        blk = small_block(seed=14, dim=32, heads=1, hi=bits, lo=bits)
        ref = orc.uniform_block_forward(blk, "hi", x, quant=False) - x
        got = orc.uniform_block_forward(blk, "hi", x) - x
        sq.append(10 * math.log10((ref ** 2).sum() / ((ref - got) ** 2).sum()))
    assert sq[0] < sq[1] < sq[2] and sq[2] > 15


# ------------------------------------------------------------------------------------------------
# merging and the backbone
# ------------------------------------------------------------------------------------------------
def test_merge_fp_mode_vs_numpy_and_quant_consistency(orc):
    rng = np.random.default_rng(15)
    m = synth.make_merge(rng, 32, 8, 8)
    x = small_input(12, 2, 9, 11, 32)                    # odd sizes: zero padding
    B, H, W, C = x.shape
    xp = np.zeros((B, H + 1, W + 1, C), np.float64)
    xp[:, :H, :W] = x
    cat = np.concatenate([xp[:, 0::2, 0::2], xp[:, 1::2, 0::2], xp[:, 0::2, 1::2], xp[:, 1::2, 1::2]], -1)
    mu = cat.mean(-1, keepdims=True)
    var = ((cat - mu) ** 2).mean(-1, keepdims=True)
    n = (cat - mu) / np.sqrt(var + 1e-5) * m.ln_g + m.ln_b
    want = n @ (m.red.codes.astype(np.float64) * m.red.scale.astype(np.float64)[:, None]).T
    got = orc.merge_forward(m, x, quant=False)
    assert got.shape == (2, 5, 6, 64)
    assert np.abs(got - want).max() < 1e-4
    # quantized: LN -> quantize -> integer GEMM -> one multiply
    gq = orc.merge_forward(m, x)
    a = orc.quantize(orc.layernorm(cat.astype(F32), m.ln_g, m.ln_b), m.aq).reshape(-1, 4 * C)
    acc = orc.int_gemm(a, m.aq.zp, m.red.codes)
    assert np.array_equal(gq.reshape(-1, 64), acc.astype(F32) * (F32(m.aq.scale) * m.red.scale)[None])
    assert np.abs(gq - want).max() < 0.1 * np.abs(want).max()


def test_backbone_is_the_composition_of_merges_and_blocks(orc):
    wl = synth.tiny_backbone(ratio=0.0)
    bb = wl.backbone
    outs = orc.backbone_forward(bb, wl.x, wl.low_ratios)
    # ratio 0 everywhere: the backbone equals uniform high-bit blocks chained with the merges
    cur, k = wl.x, 0
    for s, dep in enumerate(bb.depths):
        if s > 0:
            cur = orc.merge_forward(bb.merges[s - 1], cur)
        for _ in range(dep):
            cur = orc.uniform_block_forward(bb.blocks[k], "hi", cur)
            k += 1
        assert np.array_equal(outs[s], cur)
    assert [o.shape for o in outs] == [(2, 30, 37, 32), (2, 15, 19, 64), (2, 8, 10, 128)]


def test_backbone_shares_the_stage_entry_energy_across_the_stage(orc):
    wl = synth.tiny_backbone(ratio=0.4, prune=0.2)
    bb = wl.backbone
    outs = orc.backbone_forward(bb, wl.x, wl.low_ratios, wl.prune_ratios)
    cur, k = wl.x, 0
    for s, dep in enumerate(bb.depths):
        if s > 0:
            cur = orc.merge_forward(bb.merges[s - 1], cur)
        e = orc.energy(cur, bb.blocks[k].score_inv_scale)            # once, before the first block
        for _ in range(dep):
            cur = orc.block_forward(bb.blocks[k], cur, wl.low_ratios[k // 2], wl.prune_ratios[k // 2], energy_map=e).y
            k += 1
        assert np.array_equal(outs[s], cur)


# ------------------------------------------------------------------------------------------------
# patch embedding (the stem in front of the backbone) and output norms
# ------------------------------------------------------------------------------------------------
def _embed_numpy_fp(e, img):
    """4x4 stride-4 convolution written as a reshape + matmul in binary64, then LayerNorm in binary64."""
    B, Hi, Wi, _ = img.shape
    Hp, Wp = -(-Hi // 4) * 4, -(-Wi // 4) * 4
    pad = np.zeros((B, Hp, Wp, 3), np.float64)
    pad[:, :Hi, :Wi] = img
    patches = pad.reshape(B, Hp // 4, 4, Wp // 4, 4, 3).transpose(0, 1, 3, 2, 4, 5).reshape(B, Hp // 4, Wp // 4, 48)
    w = e.proj.codes.astype(np.float64) * e.proj.scale.astype(np.float64)[:, None]
    t = patches @ w.T + e.bias.astype(np.float64)
    mu = t.mean(-1, keepdims=True)
    var = ((t - mu) ** 2).mean(-1, keepdims=True)
    return (t - mu) / np.sqrt(var + 1e-5) * e.ln_g + e.ln_b


@pytest.mark.parametrize("Hi,Wi", [(16, 20), (13, 18), (7, 5)])
def test_patch_embed_fp_mode_is_a_strided_convolution_plus_layernorm(orc, Hi, Wi):
    e = synth.make_embed(np.random.default_rng(3), 32)
    img = synth.input_image(4, 2, Hi, Wi)
    got = orc.patch_embed(e, img, quant=False)
    want = _embed_numpy_fp(e, img)
    assert got.shape == want.shape == (2, -(-Hi // 4), -(-Wi // 4), 32)
    assert np.abs(got - want).max() < 2e-5


def test_patch_embed_quantized_from_pinned_primitives_and_onehot(orc):
    e = synth.make_embed(np.random.default_rng(5), 32)
    img = synth.input_image(6, 1, 12, 9)                          # 9 -> padded to 12 columns
    got = orc.patch_embed(e, img, quant=True)
    pad = np.zeros((1, 12, 12, 3), F32)
    pad[:, :, :9] = img
    patches = pad.reshape(1, 3, 4, 3, 4, 3).transpose(0, 1, 3, 2, 4, 5).reshape(-1, 48)
    codes = orc.quantize(patches, e.aq)
    acc = orc.int_gemm(codes, e.aq.zp, e.proj.codes)
    t = (acc.astype(F32) * (F32(e.aq.scale) * e.proj.scale)[None, :]).astype(F32) + e.bias[None, :]
    want = orc.layernorm(t.astype(F32), e.ln_g, e.ln_b).reshape(got.shape)
    assert np.array_equal(got, want)
    # close to the floating-point stem at 8 bits
    assert np.abs(got - orc.patch_embed(e, img, quant=False)).max() < 0.15
    # one-hot projection rows: output channel n sees exactly pixel k_n of the patch (dequantized), before the norm
    e2 = synth.make_embed(np.random.default_rng(7), 32)
    e2.proj.codes[:] = 0
    for n in range(32):
        e2.proj.codes[n, n] = 1
    e2.proj.scale[:] = 1.0
    e2.bias[:] = 0.0
    e2.ln_g[:] = 1.0
    e2.ln_b[:] = 0.0
    g2 = orc.patch_embed(e2, img, quant=True).reshape(-1, 32)
    deq = orc.dequantize(codes[:, :32], e2.aq)
    want2 = orc.layernorm(deq, e2.ln_g, e2.ln_b)
    assert np.array_equal(g2, want2)


# ------------------------------------------------------------------------------------------------
# precision classes within a stage (Section 4.4, "Windows Elevation")
# ------------------------------------------------------------------------------------------------
def test_no_elevation_keeps_classes_within_a_stage(orc):
    """One stage of three pairs whose ratios go down and up.  Default: a pair's effective ratio is the largest ratio so
    far in the stage (compressed windows stay compressed), so the forward equals the one with the running-maximum
    ratios; with elevation allowed every pair uses its own ratio."""
    bb = synth.make_backbone(9, [32], [6], [1], 8, 8, 4)
    x = synth.input_blobs(10, 1, 21, 28, 32, bg_std=0.5, gain=4.0)
    ratios = [0.5, 0.2, 0.4]
    dflt = orc.backbone_forward(bb, x, ratios)[0]
    runmax = orc.backbone_forward(bb, x, [0.5, 0.5, 0.5], allow_elevation=True)[0]
    elev = orc.backbone_forward(bb, x, ratios, allow_elevation=True)[0]
    assert np.array_equal(dflt, runmax)
    assert not np.array_equal(dflt, elev)
    # non-decreasing ratios: both policies agree
    up = [0.1, 0.3, 0.6]
    assert np.array_equal(orc.backbone_forward(bb, x, up)[0], orc.backbone_forward(bb, x, up, allow_elevation=True)[0])
    # the running maximum does not leak into the next stage
    bb2 = synth.make_backbone(11, [32, 64], [2, 2], [1, 2], 8, 8, 4)
    a = orc.backbone_forward(bb2, x, [0.6, 0.1])
    b = orc.backbone_forward(bb2, x, [0.6, 0.1], allow_elevation=True)
    assert all(np.array_equal(u, v) for u, v in zip(a, b))
