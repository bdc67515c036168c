"""ctypes binding of the CPU oracle (oracle/mixaq_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the CPU-baseline leg of bench.py.
It imports nothing from the CUDA package.  Parameters arrive as plain objects with numpy attributes
(duck-typed; the seeded generators produce them) and are marshalled into the oracle's own C structs.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from types import SimpleNamespace

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SO = os.path.join(_HERE, "libmixaq_oracle.so")
_SRC = os.path.join(_HERE, "mixaq_oracle.cpp")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no fast-math, no contraction; only explicit fmaf fuses)."""
    hdr = os.path.join(_HERE, "mixaq_oracle.h")
    if (not force and os.path.exists(_SO)
            and os.path.getmtime(_SO) >= max(os.path.getmtime(_SRC), os.path.getmtime(hdr))):
        return _SO
    cmd = ["g++", "-O2", "-std=c++17", "-ffp-contract=off", "-mfma", "-fopenmp", "-shared", "-fPIC",
           "-o", _SO, _SRC]
    subprocess.check_call(cmd)
    return _SO


class AQ(C.Structure):
    _fields_ = [("bits", C.c_int), ("scale", C.c_float), ("inv_scale", C.c_float), ("zp", C.c_int)]


class LinearS(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scale", C.c_void_p), ("out_f", C.c_int), ("in_f", C.c_int)]


class BranchS(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("ln1_g", "ln1_b", "ln2_g", "ln2_b", "b_qkv", "b_proj", "b_fc1", "b_fc2")] + \
               [(n, AQ) for n in ("qkv_in", "q", "k", "v", "proj_in", "fc1_in", "fc2_in")] + [("bits", C.c_int)]


class BlockS(C.Structure):
    _fields_ = [("dim", C.c_int), ("heads", C.c_int), ("window", C.c_int), ("shift", C.c_int), ("hidden", C.c_int),
                ("qkv", LinearS), ("proj", LinearS), ("fc1", LinearS), ("fc2", LinearS),
                ("relpos", C.c_void_p), ("hi", BranchS), ("lo", BranchS),
                ("score_inv_scale", C.c_float), ("quant", C.c_int)]


_TAP_FIELDS = ("a_codes", "qkv_acc", "qkv_codes", "probs", "p_codes", "pv_acc", "o_codes", "proj_acc", "x1",
               "f1_codes", "fc1_acc", "f2_codes", "fc2_acc")


class TapsS(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _TAP_FIELDS]


class MergeS(C.Structure):
    _fields_ = [("ln_g", C.c_void_p), ("ln_b", C.c_void_p), ("in_", AQ), ("red", LinearS), ("quant", C.c_int)]


class EmbedS(C.Structure):
    _fields_ = [("ln_g", C.c_void_p), ("ln_b", C.c_void_p), ("bias", C.c_void_p), ("in_", AQ), ("proj", LinearS),
                ("quant", C.c_int)]


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = C.CDLL(_SO)
        _lib.orc_low_count.restype = C.c_int
        _lib.orc_low_count.argtypes = [C.c_double, C.c_int]
        _lib.orc_window_token.restype = C.c_long
        _lib.orc_get_threads.restype = C.c_int
    return _lib


def _p(a):
    return a.ctypes.data_as(C.c_void_p) if a is not None else None


def _aq(q) -> AQ:
    return AQ(int(q.bits), float(q.scale), float(q.inv_scale), int(q.zp))


class _Keep:
    """Owns the contiguous numpy arrays a C struct points into."""

    def __init__(self):
        self.refs = []

    def arr(self, a, dtype):
        a = np.ascontiguousarray(a, dtype=dtype)
        self.refs.append(a)
        return _p(a)


def _linear(keep, L) -> LinearS:
    return LinearS(keep.arr(L.codes, np.int8), keep.arr(L.scale, np.float32), L.codes.shape[0], L.codes.shape[1])


def _branch(keep, b) -> BranchS:
    s = BranchS()
    for n in ("ln1_g", "ln1_b", "ln2_g", "ln2_b", "b_qkv", "b_proj", "b_fc1", "b_fc2"):
        setattr(s, n, keep.arr(getattr(b, n), np.float32))
    for n in ("qkv_in", "q", "k", "v", "proj_in", "fc1_in", "fc2_in"):
        setattr(s, n, _aq(getattr(b, n)))
    s.bits = int(b.bits)
    return s


def block_struct(keep, blk, quant=True) -> BlockS:
    s = BlockS()
    s.dim, s.heads, s.window, s.shift, s.hidden = blk.dim, blk.heads, blk.window, blk.shift, blk.hidden
    s.qkv, s.proj, s.fc1, s.fc2 = (_linear(keep, getattr(blk, n)) for n in ("qkv", "proj", "fc1", "fc2"))
    s.relpos = keep.arr(blk.relpos, np.float32)
    s.hi, s.lo = _branch(keep, blk.hi), _branch(keep, blk.lo)
    s.score_inv_scale = float(blk.score_inv_scale)
    s.quant = 1 if quant else 0
    return s


def merge_struct(keep, m, quant=True) -> MergeS:
    return MergeS(keep.arr(m.ln_g, np.float32), keep.arr(m.ln_b, np.float32), _aq(m.aq), _linear(keep, m.red),
                  1 if quant else 0)


# ------------------------------------------------------------------------------------------------
# primitives
# ------------------------------------------------------------------------------------------------
def low_count(ratio, n):
    return lib().orc_low_count(float(ratio), int(n))


def quantize(x, aq):
    x = np.ascontiguousarray(x, np.float32)
    out = np.empty(x.shape, np.uint8)
    lib().orc_quantize(_p(x), C.c_long(x.size), _aq(aq), _p(out))
    return out


def dequantize(codes, aq):
    codes = np.ascontiguousarray(codes, np.uint8)
    out = np.empty(codes.shape, np.float32)
    lib().orc_dequantize(_p(codes), C.c_long(codes.size), _aq(aq), _p(out))
    return out


def pack(codes, bits):
    codes = np.ascontiguousarray(codes, np.uint8)
    rows, cols = int(np.prod(codes.shape[:-1])), codes.shape[-1]
    per = 8 // bits
    out = np.empty((rows, (cols + per - 1) // per), np.uint8)
    lib().orc_pack(_p(codes), C.c_long(rows), cols, bits, _p(out))
    return out


def unpack(packed, cols, bits):
    packed = np.ascontiguousarray(packed, np.uint8)
    rows = packed.shape[0]
    out = np.empty((rows, cols), np.uint8)
    lib().orc_unpack(_p(packed), C.c_long(rows), cols, bits, _p(out))
    return out


def layernorm(x, g, b):
    x = np.ascontiguousarray(x, np.float32)
    g = np.ascontiguousarray(g, np.float32)
    b = np.ascontiguousarray(b, np.float32)
    y = np.empty_like(x)
    lib().orc_layernorm(_p(x), C.c_long(x.size // x.shape[-1]), x.shape[-1], _p(g), _p(b), _p(y))
    return y


def exp2(t):
    t = np.ascontiguousarray(t, np.float32)
    y = np.empty_like(t)
    lib().orc_exp2(_p(t), C.c_long(t.size), _p(y))
    return y


def gelu(x):
    x = np.ascontiguousarray(x, np.float32)
    y = np.empty_like(x)
    lib().orc_gelu(_p(x), C.c_long(x.size), _p(y))
    return y


def softmax_rows(s):
    s = np.ascontiguousarray(s, np.float32)
    p = np.empty_like(s)
    lib().orc_softmax_rows(_p(s), C.c_long(s.size // s.shape[-1]), s.shape[-1], _p(p))
    return p


def int_gemm(a, za, w):
    a = np.ascontiguousarray(a, np.uint8)
    w = np.ascontiguousarray(w, np.int8)
    acc = np.empty((a.shape[0], w.shape[0]), np.int32)
    lib().orc_int_gemm(_p(a), C.c_long(a.shape[0]), a.shape[1], int(za), _p(w), w.shape[0], _p(acc))
    return acc


def window_token(H, W, ws, shift, w, t):
    return lib().orc_window_token(H, W, ws, shift, w, t)


def shift_mask(H, W, ws, shift, w):
    m = np.empty((ws * ws, ws * ws), np.float32)
    lib().orc_shift_mask(H, W, ws, shift, w, _p(m))
    return m


def relpos_bias(table, ws, heads):
    table = np.ascontiguousarray(table, np.float32)
    out = np.empty((heads, ws * ws, ws * ws), np.float32)
    lib().orc_relpos_bias(_p(table), ws, heads, _p(out))
    return out


def energy(x, inv_scale):
    x = np.ascontiguousarray(x, np.float32)
    B, H, W, Cc = x.shape
    e = np.empty((B, H, W), np.int32)
    lib().orc_energy(_p(x), B, H, W, Cc, C.c_float(inv_scale), _p(e))
    return e


def window_scores(e, ws, shift):
    e = np.ascontiguousarray(e, np.int32)
    B, H, W = e.shape
    nW = -(-H // ws) * -(-W // ws)
    s = np.empty((B, nW), np.int64)
    lib().orc_window_scores(_p(e), B, H, W, ws, shift, _p(s))
    return s


def select(scores, low_ratio, prune_ratio=0.0, reverse=False):
    scores = np.ascontiguousarray(scores, np.int64)
    B, nW = scores.shape
    order = np.empty((B, nW), np.int32)
    cls = np.empty((B, nW), np.uint8)
    cnt = (C.c_int * 3)()
    lib().orc_select(_p(scores), B, nW, C.c_double(low_ratio), C.c_double(prune_ratio), int(reverse),
                     _p(order), _p(cls), cnt)
    return order, cls, tuple(cnt)


# ------------------------------------------------------------------------------------------------
# block / merge / backbone
# ------------------------------------------------------------------------------------------------
def _alloc_taps(M, nwin, Cc, hidden, heads, T):
    t = SimpleNamespace(
        a_codes=np.zeros((M, Cc), np.uint8), qkv_acc=np.zeros((M, 3 * Cc), np.int32),
        qkv_codes=np.zeros((M, 3 * Cc), np.uint8), probs=np.zeros((nwin, heads, T, T), np.float32),
        p_codes=np.zeros((nwin, heads, T, T), np.uint8), pv_acc=np.zeros((M, Cc), np.int32),
        o_codes=np.zeros((M, Cc), np.uint8), proj_acc=np.zeros((M, Cc), np.int32),
        x1=np.zeros((M, Cc), np.float32), f1_codes=np.zeros((M, Cc), np.uint8),
        fc1_acc=np.zeros((M, hidden), np.int32), f2_codes=np.zeros((M, hidden), np.uint8),
        fc2_acc=np.zeros((M, Cc), np.int32))
    s = TapsS()
    for n in _TAP_FIELDS:
        setattr(s, n, _p(getattr(t, n)))
    return t, s


def block_forward(blk, x, low_ratio, prune_ratio=0.0, energy_map=None, reverse=False, taps=False, quant=True):
    """Returns a namespace: y, order, cls, scores, counts and (taps=True) hi / lo intermediates."""
    x = np.ascontiguousarray(x, np.float32)
    B, H, W, Cc = x.shape
    ws = blk.window
    T = ws * ws
    nW = -(-H // ws) * -(-W // ws)
    keep = _Keep()
    bs = block_struct(keep, blk, quant)
    y = np.empty_like(x)
    order = np.empty((B, nW), np.int32)
    cls = np.empty((B, nW), np.uint8)
    scores = np.empty((B, nW), np.int64)
    n_pr = low_count(prune_ratio, nW)
    n_lo = low_count(low_ratio, nW - n_pr)
    n_hi = nW - n_pr - n_lo
    out = SimpleNamespace(y=y, order=order, cls=cls, scores=scores, counts=(n_hi, n_lo, n_pr), hi=None, lo=None)
    th = tl = None
    if taps:
        out.hi, th = _alloc_taps(B * n_hi * T, B * n_hi, Cc, blk.hidden, blk.heads, T)
        out.lo, tl = _alloc_taps(B * n_lo * T, B * n_lo, Cc, blk.hidden, blk.heads, T)
    en = None if energy_map is None else np.ascontiguousarray(energy_map, np.int32)
    lib().orc_block_forward(C.byref(bs), _p(x), _p(y), B, H, W, C.c_double(low_ratio), C.c_double(prune_ratio),
                            _p(en), int(reverse), _p(order), _p(cls), _p(scores),
                            C.byref(th) if th is not None else None, C.byref(tl) if tl is not None else None)
    return out


def uniform_block_forward(blk, branch_name, x, quant=True):
    x = np.ascontiguousarray(x, np.float32)
    B, H, W, _ = x.shape
    keep = _Keep()
    bs = block_struct(keep, blk, quant)
    br = bs.hi if branch_name == "hi" else bs.lo
    y = np.empty_like(x)
    lib().orc_uniform_block_forward(C.byref(bs), C.byref(br), _p(x), _p(y), B, H, W)
    return y


SITES = ("qkv_in", "q", "k", "v", "proj_in", "fc1_in", "fc2_in")


def block_observe_fp(blk, branch_name, x):
    """Floating-point block through one branch's LayerNorm parameters and biases; returns (y, {site: (min, max)})."""
    x = np.ascontiguousarray(x, np.float32)
    B, H, W, _ = x.shape
    keep = _Keep()
    bs = block_struct(keep, blk, quant=False)
    br = bs.hi if branch_name == "hi" else bs.lo
    y = np.empty_like(x)
    r = np.empty(14, np.float32)
    lib().orc_block_observe_fp(C.byref(bs), C.byref(br), _p(x), _p(y), B, H, W, _p(r))
    return y, {s: (float(r[2 * i]), float(r[2 * i + 1])) for i, s in enumerate(SITES)}


def merge_observe_fp(m, x):
    x = np.ascontiguousarray(x, np.float32)
    B, H, W, Cc = x.shape
    keep = _Keep()
    ms = merge_struct(keep, m, quant=False)
    y = np.empty((B, (H + 1) // 2, (W + 1) // 2, m.red.codes.shape[0]), np.float32)
    r = np.empty(2, np.float32)
    lib().orc_merge_observe_fp(C.byref(ms), _p(x), B, H, W, Cc, _p(y), _p(r))
    return y, (float(r[0]), float(r[1]))


def merge_forward(m, x, quant=True):
    x = np.ascontiguousarray(x, np.float32)
    B, H, W, Cc = x.shape
    keep = _Keep()
    ms = merge_struct(keep, m, quant)
    y = np.empty((B, (H + 1) // 2, (W + 1) // 2, m.red.codes.shape[0]), np.float32)
    lib().orc_merge_forward(C.byref(ms), _p(x), B, H, W, Cc, _p(y))
    return y


def backbone_forward(bb, x, low_ratios, prune_ratios=None, quant=True, allow_elevation=False, reverse=False):
    """bb: object with dims, depths, blocks, merges.  Returns the list of stage outputs."""
    x = np.ascontiguousarray(x, np.float32)
    B, H, W, _ = x.shape
    keep = _Keep()
    ns = len(bb.depths)
    blocks = (BlockS * len(bb.blocks))(*[block_struct(keep, b, quant) for b in bb.blocks])
    merges = (MergeS * max(1, len(bb.merges)))(*[merge_struct(keep, m, quant) for m in bb.merges])
    outs, h, w = [], H, W
    for s in range(ns):
        if s > 0:
            h, w = (h + 1) // 2, (w + 1) // 2
        outs.append(np.empty((B, h, w, bb.dims[s]), np.float32))
    ptrs = (C.c_void_p * ns)(*[o.ctypes.data for o in outs])
    depths = (C.c_int * ns)(*bb.depths)
    npairs = len(bb.blocks) // 2 + 1
    lr = (C.c_double * npairs)(*([float(r) for r in low_ratios] + [0.0] * (npairs - len(low_ratios))))
    pr = None
    if prune_ratios is not None:
        pr = (C.c_double * npairs)(*([float(r) for r in prune_ratios] + [0.0] * (npairs - len(prune_ratios))))
    lib().orc_backbone_forward(ns, depths, blocks, merges, _p(x), ptrs, B, H, W, lr, pr, 1 if allow_elevation else 0, 1 if reverse else 0)
    return outs


def patch_embed(e, img, quant=True):
    """e: object with ln_g, ln_b, bias, aq, proj (codes [C0][48], scale).  img: [B][Hi][Wi][3] float32."""
    img = np.ascontiguousarray(img, np.float32)
    B, Hi, Wi, ch = img.shape
    assert ch == 3
    keep = _Keep()
    es = EmbedS(keep.arr(e.ln_g, np.float32), keep.arr(e.ln_b, np.float32), keep.arr(e.bias, np.float32), _aq(e.aq),
                _linear(keep, e.proj), 1 if quant else 0)
    out = np.empty((B, (Hi + 3) // 4, (Wi + 3) // 4, e.proj.codes.shape[0]), np.float32)
    lib().orc_patch_embed(C.byref(es), _p(img), B, Hi, Wi, _p(out))
    return out


def set_threads(n):
    lib().orc_set_threads(int(n))


def get_threads():
    return lib().orc_get_threads()
