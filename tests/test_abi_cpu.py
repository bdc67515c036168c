"""Host-side checks that need no GPU: the C-ABI library loads and exports every symbol the public header
declares, its host helpers agree with the oracle, and sizes behave."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from paper_2507_19131_b200 import build as mq_build
from paper_2507_19131_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    path = mq_build.build_library()
    return C.CDLL(path)


def declared_functions():
    text = open(os.path.join(ROOT, "include", "mixaq.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(mixaq_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(L):
    names = declared_functions()
    assert len(names) >= 18
    for n in names:
        assert hasattr(L, n), f"{n} is declared in include/mixaq.h but not exported"
    from paper_2507_19131_b200 import binding
    assert sorted(binding.EXPORTS) == [n for n in names if n not in ()] or set(binding.EXPORTS) <= set(names)


def test_low_count_matches_the_oracle(L, orc):
    L.mixaq_low_count.argtypes = [C.c_float, C.c_int]
    for n in (1, 7, 24, 25, 49, 64, 96, 100, 196, 360, 361, 784, 1369, 1392, 3025):
        for r in np.linspace(0, 1, 21):
            r32 = float(np.float32(r))
            assert L.mixaq_low_count(r32, n) == orc.low_count(r32, n)


def test_branch_counts_and_argument_checks(L):
    cnt = (C.c_int * 3)()
    assert L.mixaq_branch_counts(200, 334, 7, C.c_float(0.3), C.c_float(0.0), cnt) == 0
    assert tuple(cnt) == (975, 417, 0)                       # 29 x 48 windows per image
    assert L.mixaq_branch_counts(256, 256, 7, C.c_float(0.5), C.c_float(0.2), cnt) == 0
    assert tuple(cnt) == (548, 548, 273) and sum(cnt) == 37 * 37
    assert L.mixaq_branch_counts(56, 56, 8, C.c_float(0.5), C.c_float(0.0), cnt) == -1
    assert L.mixaq_branch_counts(56, 56, 7, C.c_float(1.5), C.c_float(0.0), cnt) == -1
    assert L.mixaq_branch_counts(56, 56, 7, C.c_float(0.5), C.c_float(-0.1), cnt) == -1


def test_workspace_sizes_scale_with_the_problem(L):
    from paper_2507_19131_b200 import binding
    s = binding.BlockS()
    s.dim, s.heads, s.window, s.shift, s.hidden = 96, 3, 7, 0, 384
    s.hi.bits, s.lo.bits = 8, 4
    f = L.mixaq_block_workspace_bytes
    f.restype = C.c_size_t
    a = f(C.byref(s), 1, 56, 56)
    b = f(C.byref(s), 2, 56, 56)
    c = f(C.byref(s), 1, 200, 334)
    assert 0 < a < b < c
    # at least the binary32 residual copy of both branches at the worst split must fit
    assert c >= 2 * 1392 * 49 * 96 * 4
    assert f(None, 1, 56, 56) == 0 and f(C.byref(s), 0, 56, 56) == 0
    g = L.mixaq_block_prepared_bytes
    g.restype = C.c_size_t
    assert g(C.byref(s)) >= 3 * 49 * 49 * 4 + 2 * 2 * (288 + 96 + 384 + 96) * 4


def test_create_needs_a_device_and_never_falls_back(L):
    h = C.c_void_p()
    st = L.mixaq_create(C.byref(h), 0)
    assert st in (0, -4)
    if st == 0:
        assert L.mixaq_destroy(h) == 0
    else:
        assert not h.value
    assert L.mixaq_create(None, 0) == -1
    assert L.mixaq_create(C.byref(h), 4096) == -4


def test_generators_are_seeded_and_shaped_like_the_workloads():
    a, b = synth.config1(), synth.config1()
    assert np.array_equal(a.x, b.x) and np.array_equal(a.backbone.blocks[0].qkv.codes, b.backbone.blocks[0].qkv.codes)
    assert a.x.shape == (1, 56, 56, 96) and a.backbone.blocks[0].hi.bits == 8 and a.backbone.blocks[0].lo.bits == 4
    # four outlier channels, 20x
    std = a.x.reshape(-1, 96).std(0)
    assert (std > 10).sum() == 4
    blk = a.backbone.blocks[0]
    assert np.abs(blk.qkv.codes).max() == 127 and blk.qkv.codes.shape == (288, 96)
    w4 = synth.make_linear(np.random.default_rng(0), 64, 32, 4)
    assert np.abs(w4.codes).max() == 7
