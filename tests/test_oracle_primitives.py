"""Pins of the oracle's primitives to things other than the oracle: closed forms, binary64 libm/scipy,
numpy brute force, textbook special cases.  CPU only."""
import math

import numpy as np
import pytest
from scipy.special import erf

from paper_2507_19131_b200 import synth

F32 = np.float32


# ---------------------------------------------------------------- ratio -> count (Section 3.3: the ratio is the
# proportion of windows sent to the low-precision branch; 0 = all high, 1 = all low)
def test_low_count_values(orc):
    assert orc.low_count(0.0, 1392) == 0
    assert orc.low_count(1.0, 1392) == 1392
    assert orc.low_count(0.5, 64) == 32
    assert orc.low_count(np.float32(0.3), 1392) == 417
    assert orc.low_count(0.25, 1392) == 348 and orc.low_count(0.25, 360) == 90
    assert orc.low_count(0.25, 96) == 24 and orc.low_count(0.25, 24) == 6
    # tenths (the search space {0, 10, ..., 80 %}) never lose a window to binary rounding
    for n in (10, 20, 30, 1000):
        for k in range(9):
            assert orc.low_count(k / 10.0, n) == k * n // 10


# ---------------------------------------------------------------- quantizer
@pytest.mark.parametrize("bits", [8, 4, 2])
def test_quantizer_grid_roundtrip_zero_saturation(orc, bits):
    aq = synth.make_aq(-1.7, 2.9, bits)
    qmax = (1 << bits) - 1
    codes = np.arange(qmax + 1, dtype=np.uint8)
    grid = orc.dequantize(codes, aq)
    assert np.array_equal(grid, ((codes.astype(np.int64) - aq.zp) * np.float64(F32(aq.scale))).astype(F32))
    assert np.array_equal(orc.quantize(grid, aq), codes)            # on-grid values round-trip
    assert orc.quantize(np.zeros(3, F32), aq).tolist() == [aq.zp] * 3  # 0 maps to the zero point
    assert orc.quantize(np.array([1e9, 1e30], F32), aq).tolist() == [qmax, qmax]
    assert orc.quantize(np.array([-1e9, -1e30], F32), aq).tolist() == [0, 0]


def test_quantizer_round_half_even(orc):
    aq = synth.AQ(8, 1.0, 1.0, 10)
    x = np.array([0.5, 1.5, 2.5, -0.5, -1.5, 0.49999997, 3.5000002], F32)
    assert orc.quantize(x, aq).tolist() == [10, 12, 12, 10, 8, 10, 14]


def test_quantizer_matches_numpy_definition(orc):
    rng = np.random.default_rng(3)
    x = (rng.standard_normal(20000) * 3).astype(F32)
    for bits in (8, 4, 2):
        aq = synth.make_aq(-2.5, 4.0, bits)
        want = np.clip(np.rint(x * F32(aq.inv_scale)) + aq.zp, 0, (1 << bits) - 1).astype(np.uint8)
        assert np.array_equal(orc.quantize(x, aq), want)


@pytest.mark.parametrize("bits,cols", [(8, 96), (4, 96), (2, 96), (4, 32), (2, 128)])
def test_pack_unpack_identity_and_layout(orc, bits, cols):
    rng = np.random.default_rng(bits * 100 + cols)
    codes = rng.integers(0, 1 << bits, size=(13, cols), dtype=np.uint8)
    packed = orc.pack(codes, bits)
    assert packed.shape == (13, cols * bits // 8)
    assert np.array_equal(orc.unpack(packed, cols, bits), codes)
    # little end first: element 0 in the low bits of byte 0
    per = 8 // bits
    b0 = 0
    for e in range(per):
        b0 |= int(codes[0, e]) << (e * bits)
    assert packed[0, 0] == b0


# ---------------------------------------------------------------- LayerNorm
def test_layernorm_vs_float64(orc):
    rng = np.random.default_rng(5)
    for C in (32, 96, 384, 1536):
        x = (rng.standard_t(3, size=(50, C)) * 2).astype(F32)
        g = (1 + 0.1 * rng.standard_normal(C)).astype(F32)
        b = (0.1 * rng.standard_normal(C)).astype(F32)
        xd = x.astype(np.float64)
        mu = xd.mean(-1, keepdims=True)
        var = ((xd - mu) ** 2).mean(-1, keepdims=True)
        want = (xd - mu) / np.sqrt(var + 1e-5) * g + b
        got = orc.layernorm(x, g, b)
        assert np.abs(got - want).max() < 2e-5 * max(1.0, np.abs(want).max())


def test_layernorm_closed_forms(orc):
    C = 96
    g = np.linspace(0.5, 1.5, C).astype(F32)
    b = np.linspace(-1, 1, C).astype(F32)
    # a constant row normalises to beta exactly
    y = orc.layernorm(np.full((1, C), 3.25, F32), g, b)
    assert np.array_equal(y[0], b)
    # a two-valued row (+a on even, -a on odd channels): mean 0, var a^2 -> +-a/sqrt(a^2+eps)
    a = 2.0
    x = np.where(np.arange(C) % 2 == 0, a, -a).astype(F32)[None]
    y = orc.layernorm(x, np.ones(C, F32), np.zeros(C, F32))
    assert np.allclose(np.abs(y), a / math.sqrt(a * a + 1e-5), rtol=0, atol=2e-7)
    assert np.array_equal(np.sign(y[0]), np.sign(x[0]))


# ---------------------------------------------------------------- exp2 / softmax / GELU
def test_exp2_vs_float64(orc):
    t = np.linspace(-125, 0, 400001).astype(F32)
    got = orc.exp2(t).astype(np.float64)
    want = np.exp2(t.astype(np.float64))
    assert np.abs(got / want - 1).max() < 3e-7
    assert orc.exp2(np.array([0.0], F32))[0] == pytest.approx(1.0, abs=2e-7)
    # below the clamp the result is held at 2^-125 (a harmless positive number)
    assert orc.exp2(np.array([-500.0], F32))[0] == pytest.approx(2.0 ** -125, rel=1e-6)


def test_gelu_vs_erf_form_float64(orc):
    x = np.concatenate([np.linspace(-12, 12, 600001), [0.0, -0.0, 50.0, -50.0]]).astype(F32)
    xd = x.astype(np.float64)
    want = 0.5 * xd * (1 + erf(xd / math.sqrt(2)))
    got = orc.gelu(x).astype(np.float64)
    assert np.abs(got - want).max() < 2.5e-6
    assert orc.gelu(np.array([0.0], F32))[0] == 0.0
    # the minimum of GELU (about -0.17 near -0.75) is reproduced
    i = int(np.argmin(got))
    assert abs(x[i] + 0.7518) < 2e-3 and abs(got[i] - want.min()) < 3e-6 and abs(want.min() + 0.16997) < 1e-5


def test_contract_polynomials_are_the_minimax_fits_the_fit_script_derives(orc):
    """The frozen coefficient words of 2^f and log2 Phi(-a) against a fresh Remez run (oracle/fit_contract_polynomials):
    same polynomial up to the last bits of the small coefficients, maximum error within a few percent of the optimum;
    and the oracle evaluates exactly those words (Horner, fused multiply-adds) -- checked through orc.exp2 / orc.gelu."""
    from oracle import fit_contract_polynomials as fit
    res = fit.check()
    assert res["exp2"]["max_rel_coef_diff"] < 2e-6 and res["log2_phi_neg"]["max_rel_coef_diff"] < 2e-4
    for r in res.values():
        assert r["max_err_frozen"] < 1.08 * r["max_err_fitted"]
    # the oracle's exp2 on [-1/2, 1/2] is the frozen polynomial evaluated in binary32
    f = np.linspace(-0.5, 0.5, 1001).astype(F32)
    c = [F32(fit.word_to_float(w)) for w in fit.FROZEN["exp2"]]
    p = np.full_like(f, c[5])
    for k in range(4, -1, -1):
        p = (p.astype(np.float64) * f.astype(np.float64) + np.float64(c[k])).astype(F32)     # one rounding: a fused multiply-add
    assert np.array_equal(orc.exp2(f), p)


def test_softmax_rows(orc):
    rng = np.random.default_rng(11)
    s = (rng.standard_normal((200, 49)) * 4).astype(F32)
    s[7, 5:20] -= 100.0          # masked keys
    p = orc.softmax_rows(s).astype(np.float64)
    sd = s.astype(np.float64)
    e = np.exp(sd - sd.max(-1, keepdims=True))
    want = e / e.sum(-1, keepdims=True)
    assert np.abs(p - want).max() < 5e-7
    assert np.abs(p.sum(-1) - 1).max() < 1e-6
    u = orc.softmax_rows(np.full((1, 49), 0.37, F32))
    assert np.allclose(u, 1.0 / 49.0, rtol=0, atol=1e-8)
    # other row lengths (general window sizes)
    s2 = rng.standard_normal((5, 16)).astype(F32)
    e2 = np.exp(s2.astype(np.float64) - s2.max(-1, keepdims=True))
    assert np.abs(orc.softmax_rows(s2) - e2 / e2.sum(-1, keepdims=True)).max() < 5e-7


# ---------------------------------------------------------------- integer GEMM
def test_int_gemm_vs_int64_and_onehot(orc):
    rng = np.random.default_rng(17)
    a = rng.integers(0, 256, size=(37, 96), dtype=np.uint8)
    w = rng.integers(-127, 128, size=(50, 96)).astype(np.int8)
    za = 131
    want = (a.astype(np.int64) - za) @ w.astype(np.int64).T
    assert np.array_equal(orc.int_gemm(a, za, w), want.astype(np.int32))
    # identity weight codes reproduce (a - z) exactly; a transposed operand would not
    eye = np.eye(96, dtype=np.int8)
    assert np.array_equal(orc.int_gemm(a, za, eye), a.astype(np.int32) - za)
    onehot = np.zeros((3, 96), np.int8)
    onehot[0, 5] = 1
    onehot[1, 95] = -2
    onehot[2, 0] = 7
    got = orc.int_gemm(a, 0, onehot)
    assert np.array_equal(got[:, 0], a[:, 5].astype(np.int32))
    assert np.array_equal(got[:, 1], -2 * a[:, 95].astype(np.int32))
    assert np.array_equal(got[:, 2], 7 * a[:, 0].astype(np.int32))
    # worst-case magnitude fits int32 for the largest reduction used (K = 4096)
    assert 255 * 127 * 4096 < 2 ** 31


# ---------------------------------------------------------------- geometry
def _numpy_window_map(H, W, ws, shift):
    """Standard order: pad to multiples of ws, roll by -shift, cut into windows."""
    Hp, Wp = -(-H // ws) * ws, -(-W // ws) * ws
    ids = -np.ones((Hp, Wp), np.int64)
    ids[:H, :W] = np.arange(H * W).reshape(H, W)
    if shift:
        ids = np.roll(ids, (-shift, -shift), axis=(0, 1))
    return ids.reshape(Hp // ws, ws, Wp // ws, ws).transpose(0, 2, 1, 3).reshape(-1, ws * ws)


@pytest.mark.parametrize("H,W", [(8, 9), (14, 14), (30, 37), (7, 7)])
@pytest.mark.parametrize("shift", [0, 3])
def test_window_partition_is_a_bijection_and_matches_roll(orc, H, W, shift):
    ws = 7
    ref = _numpy_window_map(H, W, ws, shift)
    nW, T = ref.shape
    got = np.array([[orc.window_token(H, W, ws, shift, w, t) for t in range(T)] for w in range(nW)])
    assert np.array_equal(got, ref)
    real = got[got >= 0]
    assert np.array_equal(np.sort(real), np.arange(H * W))            # each real token exactly once
    assert (got < 0).sum() == nW * T - H * W                           # pad count = Hp*Wp - H*W
    # reverse (scatter, un-shift, crop) recovers the map
    x = np.random.default_rng(1).standard_normal(H * W)
    back = np.zeros(H * W)
    back[got[got >= 0]] = x[got[got >= 0]]
    assert np.array_equal(back, x)


def _numpy_shift_mask(H, W, ws, shift):
    Hp, Wp = -(-H // ws) * ws, -(-W // ws) * ws
    img = np.zeros((Hp, Wp))
    cnt = 0
    for hs in (slice(0, -ws), slice(-ws, -shift), slice(-shift, None)):
        for wsl in (slice(0, -ws), slice(-ws, -shift), slice(-shift, None)):
            img[hs, wsl] = cnt
            cnt += 1
    mw = img.reshape(Hp // ws, ws, Wp // ws, ws).transpose(0, 2, 1, 3).reshape(-1, ws * ws)
    diff = mw[:, None, :] - mw[:, :, None]
    return np.where(diff != 0, -100.0, 0.0).astype(F32)


def test_shift_mask_closed_forms_and_reference(orc):
    H, W, ws, s = 21, 28, 7, 3
    nwx = W // ws
    nW = (H // ws) * nwx
    ref = _numpy_shift_mask(H, W, ws, s)
    for w in range(nW):
        m = orc.shift_mask(H, W, ws, s, w)
        assert np.array_equal(m, ref[w])
        masked = int((m != 0).sum())
        wy, wx = divmod(w, nwx)
        last_row, last_col = wy == H // ws - 1, wx == nwx - 1
        if last_row and last_col:
            assert masked == 2401 - (16 ** 2 + 12 ** 2 + 12 ** 2 + 9 ** 2) == 1776
        elif last_row or last_col:
            assert masked == 2 * 28 * 21 == 1176
        else:
            assert masked == 0
        assert set(np.unique(m)) <= {0.0, -100.0}
    assert not orc.shift_mask(H, W, ws, 0, nW - 1).any()              # no shift, no mask
    # ragged map: the mask is defined on the padded frame
    ref2 = _numpy_shift_mask(30, 37, 7, 3)
    for w in (0, 5, 29):
        assert np.array_equal(orc.shift_mask(30, 37, 7, 3, w), ref2[w])


def test_relpos_bias_vs_standard_index(orc):
    ws, heads = 7, 3
    rng = np.random.default_rng(2)
    table = rng.standard_normal(((2 * ws - 1) ** 2, heads)).astype(F32)
    coords = np.stack(np.meshgrid(np.arange(ws), np.arange(ws), indexing="ij")).reshape(2, -1)
    rel = coords[:, :, None] - coords[:, None, :]
    idx = (rel[0] + ws - 1) * (2 * ws - 1) + (rel[1] + ws - 1)
    want = table[idx.reshape(-1)].reshape(ws * ws, ws * ws, heads).transpose(2, 0, 1)
    assert np.array_equal(orc.relpos_bias(table, ws, heads), want)


# ---------------------------------------------------------------- scoring and selection (Section 3.2 / 3.4)
def test_energy_and_window_scores_brute_force(orc):
    rng = np.random.default_rng(23)
    B, H, W, C = 2, 16, 19, 32
    x = (rng.standard_t(3, size=(B, H, W, C)) * 2).astype(F32)
    inv = F32(127 / 6)
    codes = np.clip(np.rint(x * inv), -127, 127).astype(np.int64)
    e_ref = (codes ** 2).sum(-1)
    e = orc.energy(x, inv)
    assert e.dtype == np.int32 and np.array_equal(e, e_ref)
    for shift in (0, 3):
        wm = _numpy_window_map(H, W, 7, shift)
        for b in range(B):
            ef = np.concatenate([e_ref[b].reshape(-1), [0]])           # index -1 -> pad -> 0
            want = ef[wm].sum(-1)
            assert np.array_equal(orc.window_scores(e, 7, shift)[b], want)


def test_selection_order_ties_counts_reverse(orc):
    rng = np.random.default_rng(29)
    scores = rng.integers(0, 50, size=(3, 97)).astype(np.int64)       # many ties
    order, cls, cnt = orc.select(scores, 0.3, 0.2)
    n_pr = math.floor(0.2 * 97 + 1e-6)
    n_lo = math.floor(0.3 * (97 - n_pr) + 1e-6)
    assert cnt == (97 - n_pr - n_lo, n_lo, n_pr)
    for b in range(3):
        want = sorted(range(97), key=lambda w: (-int(scores[b, w]), w))
        assert order[b].tolist() == want
        assert np.array_equal(cls[b, want[:cnt[0]]], np.zeros(cnt[0]))
        assert np.array_equal(cls[b, want[cnt[0]:cnt[0] + cnt[1]]], np.ones(cnt[1]))
        assert np.array_equal(cls[b, want[cnt[0] + cnt[1]:]], np.full(cnt[2], 2))
    # all scores equal: the high set is the lowest indices
    order, cls, cnt = orc.select(np.full((1, 10), 7, np.int64), 0.5)
    assert order[0].tolist() == list(range(10)) and cls[0].tolist() == [0] * 5 + [1] * 5
    # worst-case (reverse) selection ranks by ascending score
    order_r, cls_r, _ = orc.select(scores, 0.3, 0.0, reverse=True)
    for b in range(3):
        assert order_r[b].tolist() == sorted(range(97), key=lambda w: (int(scores[b, w]), w))
    # ratio 0 -> all high; ratio 1 -> all low
    assert not orc.select(scores, 0.0)[1].any()
    assert (orc.select(scores, 1.0)[1] == 1).all()


def test_selection_is_equivariant_under_window_permutation(orc):
    rng = np.random.default_rng(31)
    scores = rng.permutation(200).astype(np.int64)[None]              # distinct scores
    _, cls, _ = orc.select(scores, 0.4, 0.1)
    perm = rng.permutation(200)
    _, cls_p, _ = orc.select(scores[:, perm], 0.4, 0.1)
    assert np.array_equal(cls_p[0], cls[0][perm])


def test_planted_high_norm_blobs_are_selected_high(orc):
    B, H, W, C = 1, 56, 56, 32
    x = (np.random.default_rng(37).standard_normal((B, H, W, C)) * 0.1).astype(F32)
    x[0, 14:21, 28:35] *= 30                                            # exactly window (2, 4)
    x[0, 42:49, 0:7] *= 30                                              # exactly window (6, 0)
    e = orc.energy(x, F32(127 / 6))
    s = orc.window_scores(e, 7, 0)
    _, cls, _ = orc.select(s, 0.9)
    hi = set(np.nonzero(cls[0] == 0)[0].tolist())
    assert {2 * 8 + 4, 6 * 8 + 0} <= hi
