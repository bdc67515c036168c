"""Thin Python binding of the C ABI in include/mixaq.h (ctypes).  Argument marshalling only: every step of
the path runs in the library's kernels.  PyTorch supplies device memory and the CUDA stream, nothing else.
There is no fallback: if libmixaq.so is missing or no CUDA device is present, calls raise."""
from __future__ import annotations

import ctypes as C
import os
from types import SimpleNamespace
from typing import List, Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmixaq.so")
_lib = None

EXPORTS = [
    "mixaq_create", "mixaq_destroy", "mixaq_last_error", "mixaq_last_device_status", "mixaq_low_count",
    "mixaq_branch_counts", "mixaq_block_prepared_bytes", "mixaq_block_prepare", "mixaq_merge_prepared_bytes",
    "mixaq_merge_prepare", "mixaq_stage_energy", "mixaq_block_workspace_bytes", "mixaq_block_forward",
    "mixaq_merge_workspace_bytes", "mixaq_merge_forward", "mixaq_backbone_workspace_bytes",
    "mixaq_backbone_forward", "mixaq_last_launch_count", "mixaq_profile_categories", "mixaq_profile_category_name",
    "mixaq_profile_begin", "mixaq_profile_end", "mixaq_merge_forward_static", "mixaq_set_graph_cache",
    "mixaq_embed_prepared_bytes", "mixaq_embed_prepare", "mixaq_embed_workspace_bytes", "mixaq_embed_forward",
    "mixaq_norm_forward", "mixaq_profile_end_records", "mixaq_calibrate_block_workspace_bytes", "mixaq_calibrate_block",
    "mixaq_calibrate_merge_workspace_bytes", "mixaq_calibrate_merge", "mixaq_aq_from_range", "mixaq_clear_device_status", "mixaq_selftest_wait_timeout", "mixaq_measure_mma_peak", "mixaq_set_window_elevation", "mixaq_set_reverse_selection", "mixaq_set_nvtx", "mixaq_set_workspace_guards", "mixaq_selftest_workspace_guards",
]

STATUS = {0: "OK", -1: "INVALID_ARG", -2: "UNSUPPORTED_SHAPE", -3: "WORKSPACE_TOO_SMALL", -4: "CUDA_ERROR",
          -5: "DEVICE_TIMEOUT", -6: "INTERNAL", -7: "WORKSPACE_OVERRUN"}


class MixaqError(RuntimeError):
    def __init__(self, status, msg=""):
        super().__init__(f"mixaq: {STATUS.get(status, status)} {msg}")
        self.status = status


class AQ(C.Structure):
    _fields_ = [("bits", C.c_int), ("scale", C.c_float), ("inv_scale", C.c_float), ("zero_point", C.c_int)]


class LinearS(C.Structure):
    _fields_ = [("codes", C.c_void_p), ("scale", C.c_void_p), ("out_features", C.c_int), ("in_features", C.c_int),
                ("bits", C.c_int)]


class BranchS(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("ln1_g", "ln1_b", "ln2_g", "ln2_b", "b_qkv", "b_proj", "b_fc1", "b_fc2")] + \
               [(n, AQ) for n in ("qkv_in", "q", "k", "v", "proj_in", "fc1_in", "fc2_in")] + [("bits", C.c_int)]


class BlockS(C.Structure):
    _fields_ = [("dim", C.c_int), ("heads", C.c_int), ("window", C.c_int), ("shift", C.c_int), ("hidden", C.c_int),
                ("qkv", LinearS), ("proj", LinearS), ("fc1", LinearS), ("fc2", LinearS),
                ("relpos_table", C.c_void_p), ("hi", BranchS), ("lo", BranchS),
                ("score_inv_scale", C.c_float), ("prepared", C.c_void_p), ("byte_codes", C.c_int)]


class MergeS(C.Structure):
    _fields_ = [("ln_g", C.c_void_p), ("ln_b", C.c_void_p), ("in_", AQ), ("reduction", LinearS),
                ("prepared", C.c_void_p)]


class EmbedS(C.Structure):
    _fields_ = [("ln_g", C.c_void_p), ("ln_b", C.c_void_p), ("bias", C.c_void_p), ("in_", AQ), ("proj", LinearS),
                ("prepared", C.c_void_p)]


class SelectOpts(C.Structure):
    _fields_ = [("energy", C.c_void_p), ("reverse", C.c_int)]


class Selection(C.Structure):
    _fields_ = [("cls", C.c_void_p), ("order", C.c_void_p), ("score", C.c_void_p),
                ("idx_hi", C.c_void_p), ("idx_lo", C.c_void_p), ("idx_pr", C.c_void_p)]


_TAP_FIELDS = ("a_codes", "qkv_acc", "qkv_codes", "probs", "p_codes", "pv_acc", "o_codes", "proj_acc", "x1",
               "f1_codes", "fc1_acc", "f2_codes", "fc2_acc")


class BranchTaps(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _TAP_FIELDS]


class Taps(C.Structure):
    _fields_ = [("hi", BranchTaps), ("lo", BranchTaps)]


class BackboneS(C.Structure):
    _fields_ = [("num_stages", C.c_int), ("depths", C.POINTER(C.c_int)), ("blocks", C.POINTER(BlockS)),
                ("merges", C.POINTER(MergeS)), ("embed", C.POINTER(EmbedS)),
                ("out_norm_g", C.POINTER(C.c_void_p)), ("out_norm_b", C.POINTER(C.c_void_p))]


def lib():
    """Loads libmixaq.so.  Raises if it has not been built: the product has no other code path."""
    global _lib
    if _lib is None:
        if os.path.abspath(LIB_PATH) == os.path.join(_HERE, "libmixaq.so"):
            # (re)build when the library is missing or older than its sources; a box without nvcc uses what is there
            try:
                from . import build as _build
                _build.build_library()
            except Exception as e:                      # noqa: BLE001
                if not os.path.exists(LIB_PATH):
                    raise MixaqError(-4, f"{LIB_PATH} is missing and could not be built: {e}")
        if not os.path.exists(LIB_PATH):
            raise MixaqError(-4, f"{LIB_PATH} is missing: build it with paper_2507_19131_b200/build.py")
        L = C.CDLL(LIB_PATH)
        L.mixaq_last_error.restype = C.c_char_p
        L.mixaq_profile_category_name.restype = C.c_char_p
        for n in ("mixaq_embed_prepared_bytes", "mixaq_embed_workspace_bytes",
                  "mixaq_block_prepared_bytes", "mixaq_merge_prepared_bytes", "mixaq_block_workspace_bytes",
                  "mixaq_merge_workspace_bytes", "mixaq_backbone_workspace_bytes",
                  "mixaq_calibrate_block_workspace_bytes", "mixaq_calibrate_merge_workspace_bytes"):
            getattr(L, n).restype = C.c_size_t
        L.mixaq_low_count.argtypes = [C.c_float, C.c_int]
        _lib = L
    return _lib


def low_count(ratio: float, n: int) -> int:
    return lib().mixaq_low_count(C.c_float(ratio), n)


def branch_counts(H: int, W: int, low_ratio: float, prune_ratio: float = 0.0, window: int = 7):
    cnt = (C.c_int * 3)()
    st = lib().mixaq_branch_counts(H, W, window, C.c_float(low_ratio), C.c_float(prune_ratio), cnt)
    if st != 0:
        raise MixaqError(st)
    return tuple(cnt)


def _stream_ptr() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t: Optional[torch.Tensor]):
    return C.c_void_p(t.data_ptr()) if t is not None else None


class Context:
    """One library context per device (mixaq_create / mixaq_destroy)."""

    def __init__(self, device: int = 0):
        if not torch.cuda.is_available():
            raise MixaqError(-4, "no CUDA device: the library has no CPU path")
        self.device = torch.device("cuda", device)
        torch.cuda.set_device(self.device)
        self.h = C.c_void_p()
        st = lib().mixaq_create(C.byref(self.h), device)
        if st != 0:
            raise MixaqError(st, "mixaq_create")

    def check(self, st: int, what: str = ""):
        if st != 0:
            raise MixaqError(st, what + ": " + lib().mixaq_last_error(self.h).decode())

    def device_status(self) -> int:
        return lib().mixaq_last_device_status(self.h, _stream_ptr())

    def set_workspace_guards(self, enabled: bool):
        """mixaq_set_workspace_guards: fill / compare the guard zones of the block workspace around every block."""
        self.check(lib().mixaq_set_workspace_guards(self.h, 1 if enabled else 0), "set_workspace_guards")

    def selftest_workspace_guards(self, overrun: bool):
        """mixaq_selftest_workspace_guards on a scratch buffer of this context's device."""
        buf = torch.zeros(4096, dtype=torch.uint8, device=self.device)
        self.check(lib().mixaq_selftest_workspace_guards(self.h, _ptr(buf), C.c_size_t(buf.numel()), 1 if overrun else 0,
                                                         _stream_ptr()), "selftest_workspace_guards")

    def set_nvtx(self, enabled: bool):
        """mixaq_set_nvtx: host-side NVTX ranges per kernel family, stage and block."""
        self.check(lib().mixaq_set_nvtx(self.h, 1 if enabled else 0), "set_nvtx")

    def set_reverse_selection(self, reverse: bool):
        self.check(lib().mixaq_set_reverse_selection(self.h, 1 if reverse else 0), "set_reverse_selection")

    def set_window_elevation(self, allow: bool):
        self.check(lib().mixaq_set_window_elevation(self.h, 1 if allow else 0), "set_window_elevation")

    def set_graph_cache(self, enabled: bool):
        self.check(lib().mixaq_set_graph_cache(self.h, 1 if enabled else 0), "set_graph_cache")

    def clear_device_status(self):
        self.check(lib().mixaq_clear_device_status(self.h, _stream_ptr()), "clear_device_status")

    def selftest_wait_timeout(self):
        self.check(lib().mixaq_selftest_wait_timeout(self.h, _stream_ptr()), "selftest_wait_timeout")

    def measure_mma_peak(self, kind: int = 0, groups: int = 2000) -> float:
        """Tensor-core issue rate in TOP/s (kind 0: kind::i8; 1: kind::f8f6f4 with E4M3 operands; 2: kind::mxf4)."""
        scratch = torch.empty(8192, dtype=torch.uint8, device=self.device)
        out = C.c_double()
        self.check(lib().mixaq_measure_mma_peak(self.h, kind, groups, _ptr(scratch), C.c_size_t(8192), C.byref(out),
                                                _stream_ptr()), "measure_mma_peak")
        return float(out.value)

    def launch_count(self) -> int:
        return lib().mixaq_last_launch_count(self.h)

    def profile_begin(self):
        self.check(lib().mixaq_profile_begin(self.h), "profile_begin")

    def profile_end(self):
        """Returns {category: (milliseconds, event pairs)} since profile_begin (synchronises the stream)."""
        n = lib().mixaq_profile_categories()
        ms, cnt = (C.c_float * n)(), (C.c_int * n)()
        self.check(lib().mixaq_profile_end(self.h, _stream_ptr(), ms, cnt), "profile_end")
        return {lib().mixaq_profile_category_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n)}

    def profile_end_records(self, capacity: int = 4096):
        """Returns [(category name, milliseconds)] launch by launch, in issue order, since profile_begin."""
        cat, ms, n = (C.c_int * capacity)(), (C.c_float * capacity)(), C.c_int()
        self.check(lib().mixaq_profile_end_records(self.h, _stream_ptr(), cat, ms, capacity, C.byref(n)), "profile_end_records")
        names = [lib().mixaq_profile_category_name(i).decode() for i in range(lib().mixaq_profile_categories())]
        return [(names[cat[i]], float(ms[i])) for i in range(min(n.value, capacity))]

    def close(self):
        if self.h:
            lib().mixaq_destroy(self.h)
            self.h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def _aq(q) -> AQ:
    return AQ(int(q.bits), float(q.scale), float(q.inv_scale), int(q.zp))


class _Dev:
    """Uploads numpy parameters once and keeps the device tensors alive."""

    def __init__(self, device):
        self.device = device
        self.keep = []

    def up(self, a: np.ndarray, dtype) -> C.c_void_p:
        t = torch.from_numpy(np.ascontiguousarray(a, dtype=dtype)).to(self.device)
        self.keep.append(t)
        return C.c_void_p(t.data_ptr())

    def empty(self, nbytes: int) -> C.c_void_p:
        t = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=self.device)
        self.keep.append(t)
        return C.c_void_p(t.data_ptr())


def _linear(dev: _Dev, L) -> LinearS:
    return LinearS(dev.up(L.codes, np.int8), dev.up(L.scale, np.float32), L.codes.shape[0], L.codes.shape[1], int(L.bits))


def _branch(dev: _Dev, b, cache) -> BranchS:
    s = BranchS()
    for n in ("ln1_g", "ln1_b", "ln2_g", "ln2_b", "b_qkv", "b_proj", "b_fc1", "b_fc2"):
        a = getattr(b, n)
        if id(a) not in cache:          # shared biases are uploaded once and aliased
            cache[id(a)] = dev.up(a, np.float32)
        setattr(s, n, cache[id(a)])
    for n in ("qkv_in", "q", "k", "v", "proj_in", "fc1_in", "fc2_in"):
        setattr(s, n, _aq(getattr(b, n)))
    s.bits = int(b.bits)
    return s


def fill_block_struct(dev: _Dev, blk, byte_codes: bool = False) -> BlockS:
    s = BlockS()
    s.byte_codes = 1 if byte_codes else 0
    s.dim, s.heads, s.window, s.shift, s.hidden = blk.dim, blk.heads, blk.window, blk.shift, blk.hidden
    s.qkv, s.proj, s.fc1, s.fc2 = (_linear(dev, getattr(blk, n)) for n in ("qkv", "proj", "fc1", "fc2"))
    s.relpos_table = dev.up(blk.relpos, np.float32)
    cache = {}
    s.hi, s.lo = _branch(dev, blk.hi, cache), _branch(dev, blk.lo, cache)
    s.score_inv_scale = float(blk.score_inv_scale)
    s.prepared = dev.empty(lib().mixaq_block_prepared_bytes(C.byref(s)))
    return s


def fill_merge_struct(dev: _Dev, m) -> MergeS:
    s = MergeS(dev.up(m.ln_g, np.float32), dev.up(m.ln_b, np.float32), _aq(m.aq), _linear(dev, m.red), None)
    s.prepared = dev.empty(lib().mixaq_merge_prepared_bytes(C.byref(s)))
    return s


class DeviceBlock:
    """Parameters of one Two-Branch Swin Block resident on the device, prepared (mixaq_block_prepare)."""

    def __init__(self, ctx: Context, blk, byte_codes: bool = False):
        self.ctx, self.blk = ctx, blk
        self.dev = _Dev(ctx.device)
        self.s = fill_block_struct(self.dev, blk, byte_codes)
        ctx.check(lib().mixaq_block_prepare(ctx.h, C.byref(self.s), _stream_ptr()), "block_prepare")
        self._ws = None

    def workspace(self, B, H, W) -> torch.Tensor:
        need = lib().mixaq_block_workspace_bytes(C.byref(self.s), B, H, W)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.ctx.device)
        return self._ws


def stage_energy(ctx: Context, x: torch.Tensor, score_inv_scale: float) -> torch.Tensor:
    B, H, W, Cc = x.shape
    e = torch.empty((B, H, W), dtype=torch.int32, device=x.device)
    ctx.check(lib().mixaq_stage_energy(ctx.h, _ptr(x), _ptr(e), B, H, W, Cc, C.c_float(score_inv_scale), _stream_ptr()),
              "stage_energy")
    return e


def _alloc_taps(device, M, slots, Cc, hidden, heads, bits):
    u8, i32, f32 = torch.uint8, torch.int32, torch.float32
    z = lambda shape, dt: torch.zeros(shape, dtype=dt, device=device)
    t = SimpleNamespace(
        a_codes=z((M, Cc * bits // 8), u8), qkv_acc=z((M, 3 * Cc), i32), qkv_codes=z((M, 3 * Cc * bits // 8), u8),
        probs=z((slots, heads, 49, 49), f32), p_codes=z((slots, heads, 49, 49), u8), pv_acc=z((M, Cc), i32), o_codes=z((M, Cc * bits // 8), u8),
        proj_acc=z((M, Cc), i32), x1=z((M, Cc), f32), f1_codes=z((M, Cc * bits // 8), u8),
        fc1_acc=z((M, hidden), i32), f2_codes=z((M, hidden * bits // 8), u8), fc2_acc=z((M, Cc), i32))
    s = BranchTaps()
    for n in _TAP_FIELDS:
        setattr(s, n, _ptr(getattr(t, n)))
    return t, s


def block_forward(ctx: Context, db: DeviceBlock, x: torch.Tensor, low_ratio: float, prune_ratio: float = 0.0,
                  energy: Optional[torch.Tensor] = None, reverse: bool = False, selection: bool = False,
                  taps: bool = False, y: Optional[torch.Tensor] = None):
    """mixaq_block_forward.  x: [B,H,W,C] float32 CUDA tensor.  Returns a namespace with y (and, on request,
    cls / order / scores / counts and the per-branch taps)."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    B, H, W, Cc = x.shape
    if y is None:
        y = torch.empty_like(x)
    ws = db.workspace(B, H, W)
    out = SimpleNamespace(y=y, counts=branch_counts(H, W, low_ratio, prune_ratio))
    nW = -(-H // 7) * -(-W // 7)
    opts = SelectOpts(_ptr(energy), 1 if reverse else 0)
    sel = None
    if selection:
        out.cls = torch.empty((B, nW), dtype=torch.uint8, device=x.device)
        out.order = torch.empty((B, nW), dtype=torch.int32, device=x.device)
        out.scores = torch.empty((B, nW), dtype=torch.int64, device=x.device)
        n_hi, n_lo, n_pr = out.counts
        out.idx_hi, out.idx_lo, out.idx_pr = (torch.empty((B, n), dtype=torch.int32, device=x.device) for n in (n_hi, n_lo, n_pr))
        sel = Selection(_ptr(out.cls), _ptr(out.order), _ptr(out.scores), _ptr(out.idx_hi), _ptr(out.idx_lo), _ptr(out.idx_pr))
    tp = None
    if taps:
        n_hi, n_lo, _ = out.counts
        out.hi, th = _alloc_taps(x.device, B * n_hi * 49, B * n_hi, Cc, db.blk.hidden, db.blk.heads, 8 if db.s.byte_codes else db.blk.hi.bits)
        out.lo, tl = _alloc_taps(x.device, B * n_lo * 49, B * n_lo, Cc, db.blk.hidden, db.blk.heads, 8 if db.s.byte_codes else db.blk.lo.bits)
        tp = Taps(th, tl)
    st = lib().mixaq_block_forward(ctx.h, C.byref(db.s), _ptr(x), _ptr(y), B, H, W, C.c_float(low_ratio),
                                   C.c_float(prune_ratio), C.byref(opts), C.byref(sel) if sel is not None else None,
                                   _ptr(ws), C.c_size_t(ws.numel()), C.byref(tp) if tp is not None else None,
                                   _stream_ptr())
    ctx.check(st, "block_forward")
    return out


class DeviceMerge:
    def __init__(self, ctx: Context, m):
        self.ctx, self.m = ctx, m
        self.dev = _Dev(ctx.device)
        self.s = fill_merge_struct(self.dev, m)
        ctx.check(lib().mixaq_merge_prepare(ctx.h, C.byref(self.s), _stream_ptr()), "merge_prepare")


def merge_forward(ctx: Context, dm: DeviceMerge, x: torch.Tensor) -> torch.Tensor:
    B, H, W, Cc = x.shape
    y = torch.empty((B, (H + 1) // 2, (W + 1) // 2, 2 * Cc), dtype=torch.float32, device=x.device)
    need = lib().mixaq_merge_workspace_bytes(C.byref(dm.s), B, H, W)
    ws = torch.empty(need, dtype=torch.uint8, device=x.device)
    ctx.check(lib().mixaq_merge_forward(ctx.h, C.byref(dm.s), _ptr(x), _ptr(y), B, H, W, _ptr(ws), C.c_size_t(need),
                                        _stream_ptr()), "merge_forward")
    return y


class DeviceEmbed:
    """Stem parameters on the device, prepared (mixaq_embed_prepare)."""

    def __init__(self, ctx: Context, e):
        self.ctx, self.e = ctx, e
        self.dev = _Dev(ctx.device)
        self.s = EmbedS(self.dev.up(e.ln_g, np.float32), self.dev.up(e.ln_b, np.float32), self.dev.up(e.bias, np.float32),
                        _aq(e.aq), _linear(self.dev, e.proj), None)
        self.s.prepared = self.dev.empty(lib().mixaq_embed_prepared_bytes(C.byref(self.s)))
        ctx.check(lib().mixaq_embed_prepare(ctx.h, C.byref(self.s), _stream_ptr()), "embed_prepare")
        self._ws = None


def embed_forward(ctx: Context, de: DeviceEmbed, image: torch.Tensor, x0: Optional[torch.Tensor] = None) -> torch.Tensor:
    """mixaq_embed_forward: image [B,Hi,Wi,3] float32 -> x0 [B,ceil(Hi/4),ceil(Wi/4),C0]."""
    assert image.is_cuda and image.dtype == torch.float32 and image.is_contiguous() and image.shape[-1] == 3
    B, Hi, Wi, _ = image.shape
    c0 = de.e.proj.codes.shape[0]
    if x0 is None:
        x0 = torch.empty((B, (Hi + 3) // 4, (Wi + 3) // 4, c0), dtype=torch.float32, device=image.device)
    need = lib().mixaq_embed_workspace_bytes(C.byref(de.s), B, Hi, Wi)
    if de._ws is None or de._ws.numel() < need:
        de._ws = torch.empty(need, dtype=torch.uint8, device=image.device)
    ctx.check(lib().mixaq_embed_forward(ctx.h, C.byref(de.s), _ptr(image), _ptr(x0), B, Hi, Wi, _ptr(de._ws),
                                        C.c_size_t(de._ws.numel()), _stream_ptr()), "embed_forward")
    return x0


def norm_forward(ctx: Context, gamma: torch.Tensor, beta: torch.Tensor, x: torch.Tensor,
                 y: Optional[torch.Tensor] = None) -> torch.Tensor:
    """mixaq_norm_forward: LayerNorm over the last axis of a float32 tensor (a stage's output map)."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    if y is None:
        y = torch.empty_like(x)
    Cc = x.shape[-1]
    ctx.check(lib().mixaq_norm_forward(ctx.h, _ptr(gamma), _ptr(beta), _ptr(x), _ptr(y), C.c_long(x.numel() // Cc), Cc,
                                       _stream_ptr()), "norm_forward")
    return y


class RangeS(C.Structure):
    _fields_ = [("lo", C.c_float), ("hi", C.c_float)]


CAL_SITES = ("qkv_in", "q", "k", "v", "proj_in", "fc1_in", "fc2_in", "x_in")


class BlockRangesS(C.Structure):
    _fields_ = [(n, RangeS) for n in CAL_SITES]


def aq_from_range(lo: float, hi: float, bits: int):
    """mixaq_aq_from_range: the quantizer of `bits` bits that covers [lo, hi]; returns (scale, inv_scale, zero_point)."""
    q = AQ()
    st = lib().mixaq_aq_from_range(C.c_float(lo), C.c_float(hi), bits, C.byref(q))
    if st != 0:
        raise MixaqError(st, "aq_from_range")
    return float(q.scale), float(q.inv_scale), int(q.zero_point)


def calibrate_block(ctx: Context, block_struct: BlockS, branch: int, x: torch.Tensor, y: torch.Tensor = None):
    """mixaq_calibrate_block: floating-point block through one branch (0 high, 1 low) with the min/max observers.
    Returns (y, {site: (lo, hi)})."""
    assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous()
    B, H, W, _ = x.shape
    if y is None:
        y = torch.empty_like(x)
    need = lib().mixaq_calibrate_block_workspace_bytes(C.byref(block_struct), B, H, W)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
    r = BlockRangesS()
    ctx.check(lib().mixaq_calibrate_block(ctx.h, C.byref(block_struct), branch, _ptr(x), _ptr(y), B, H, W, C.byref(r),
                                          _ptr(ws), C.c_size_t(ws.numel()), _stream_ptr()), "calibrate_block")
    return y, {n: (float(getattr(r, n).lo), float(getattr(r, n).hi)) for n in CAL_SITES}


def calibrate_merge(ctx: Context, merge_struct: MergeS, x: torch.Tensor):
    """mixaq_calibrate_merge: floating-point patch merging; returns (y, (lo, hi)) of its LayerNorm output."""
    B, H, W, Cc = x.shape
    y = torch.empty((B, (H + 1) // 2, (W + 1) // 2, 2 * Cc), dtype=torch.float32, device=x.device)
    need = lib().mixaq_calibrate_merge_workspace_bytes(C.byref(merge_struct), B, H, W)
    ws = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
    r = RangeS()
    ctx.check(lib().mixaq_calibrate_merge(ctx.h, C.byref(merge_struct), _ptr(x), _ptr(y), B, H, W, C.byref(r), _ptr(ws),
                                          C.c_size_t(ws.numel()), _stream_ptr()), "calibrate_merge")
    return y, (float(r.lo), float(r.hi))


STATIC_SCRATCH_BYTES = 8 << 20


def merge_forward_static(ctx: Context, dm: DeviceMerge, x: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
    """mixaq_merge_forward_static: patch merging for callers that cannot allocate device memory where they run
    the network (the intermediate lives in an array built into the library, at most STATIC_SCRATCH_BYTES).
    The caller passes the output tensor; nothing is allocated here or in the library."""
    B, H, W, Cc = x.shape
    assert tuple(y.shape) == (B, (H + 1) // 2, (W + 1) // 2, 2 * Cc) and y.dtype == torch.float32 and y.is_contiguous()
    ctx.check(lib().mixaq_merge_forward_static(ctx.h, C.byref(dm.s), _ptr(x), _ptr(y), B, H, W, _stream_ptr()),
              "merge_forward_static")
    return y


class DeviceBackbone:
    """All parameters of a backbone on the device, prepared; owns the workspace and the stage outputs.
    embed: stem parameters (object with ln_g, ln_b, bias, aq, proj) -- the forward then takes the IMAGE [B,H0,W0,3];
    norms: one (gamma, beta) pair of numpy vectors per stage -- the stage outputs are then LayerNormed.
    byte_codes_min_dim: blocks with at least this many channels keep their intermediate codes one per byte
    (mixaq_block_params.byte_codes); None: every block bit-packs."""

    def __init__(self, ctx: Context, bb, B: int, H0: int, W0: int, embed=None, norms=None, byte_codes_min_dim=None):
        self.ctx, self.bb, self.B, self.H0, self.W0 = ctx, bb, B, H0, W0
        self.dev = _Dev(ctx.device)
        nb = len(bb.blocks)
        self.blocks = (BlockS * nb)(*[fill_block_struct(self.dev, b, byte_codes_min_dim is not None and b.dim >= byte_codes_min_dim)
                                      for b in bb.blocks])
        self.merges = (MergeS * max(1, len(bb.merges)))(*[fill_merge_struct(self.dev, m) for m in bb.merges])
        self.depths = (C.c_int * len(bb.depths))(*bb.depths)
        self.s = BackboneS(len(bb.depths), self.depths, self.blocks, self.merges, None, None, None)
        self.embed = None
        if embed is not None:
            self.embed = DeviceEmbed(ctx, embed)
            self.s.embed = C.pointer(self.embed.s)
        if norms is not None:
            ns = len(bb.depths)
            self.norm_g = (C.c_void_p * ns)(*[self.dev.up(g, np.float32) for g, _ in norms])
            self.norm_b = (C.c_void_p * ns)(*[self.dev.up(b, np.float32) for _, b in norms])
            self.s.out_norm_g, self.s.out_norm_b = self.norm_g, self.norm_b
        for i in range(nb):
            ctx.check(lib().mixaq_block_prepare(ctx.h, C.byref(self.blocks[i]), _stream_ptr()), "block_prepare")
        for i in range(len(bb.merges)):
            ctx.check(lib().mixaq_merge_prepare(ctx.h, C.byref(self.merges[i]), _stream_ptr()), "merge_prepare")
        need = lib().mixaq_backbone_workspace_bytes(C.byref(self.s), B, H0, W0)
        if need == 0:
            raise MixaqError(-1, "backbone_workspace_bytes returned 0")
        self.ws = torch.empty(need, dtype=torch.uint8, device=ctx.device)
        h, w = ((H0 + 3) // 4, (W0 + 3) // 4) if embed is not None else (H0, W0)
        self.outs = []
        for s, c in enumerate(bb.dims):
            if s > 0:
                h, w = (h + 1) // 2, (w + 1) // 2
            self.outs.append(torch.empty((B, h, w, c), dtype=torch.float32, device=ctx.device))
        self.out_ptrs = (C.c_void_p * len(self.outs))(*[o.data_ptr() for o in self.outs])
        self.npairs = (nb + 1) // 2


def backbone_forward(ctx: Context, dbb: DeviceBackbone, x0: torch.Tensor, low_ratios: Sequence[float],
                     prune_ratios: Optional[Sequence[float]] = None) -> List[torch.Tensor]:
    """mixaq_backbone_forward.  Returns the per-stage output tensors owned by `dbb` (overwritten by the next call)."""
    assert x0.is_cuda and x0.dtype == torch.float32 and x0.is_contiguous()
    assert tuple(x0.shape[:3]) == (dbb.B, dbb.H0, dbb.W0)
    lr = (C.c_float * dbb.npairs)(*[float(r) for r in low_ratios][:dbb.npairs])
    pr = None
    if prune_ratios is not None:
        pr = (C.c_float * dbb.npairs)(*[float(r) for r in prune_ratios][:dbb.npairs])
    st = lib().mixaq_backbone_forward(ctx.h, C.byref(dbb.s), _ptr(x0), dbb.out_ptrs, dbb.B, dbb.H0, dbb.W0, lr, pr,
                                      _ptr(dbb.ws), C.c_size_t(dbb.ws.numel()), _stream_ptr())
    ctx.check(st, "backbone_forward")
    return dbb.outs
