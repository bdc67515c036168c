"""The cost-model helper and the ratio sampler against what the paper prints (tests/golden/paper_cost_model.txt)."""
import os

import numpy as np
import pytest

from paper_2507_19131_b200 import cost_model as cm

HERE = os.path.dirname(os.path.abspath(__file__))


@pytest.fixture(scope="module")
def paper():
    vals = {}
    for line in open(os.path.join(HERE, "golden", "paper_cost_model.txt")):
        line = line.split("#")[0].split()
        if line:
            vals[line[0]] = [float(v) for v in line[1:]]
    return vals


def test_constants_are_the_papers(paper):
    assert list(cm.PAPER_PAIR_GMACS) == paper["pair_gmacs"] and cm.PAPER_FIXED_GMACS == paper["fixed_gmacs"][0]


def test_bops_of_the_uniform_models(paper):
    """Table 1: 88.42 T at 32 bits, 11.05 T at 4 bits, 8.29 T at 3 bits (printed with two decimals)."""
    assert cm.bops_tera(32.0) == pytest.approx(paper["bops_fp32_T"][0], abs=0.015)
    assert cm.bops_tera(4.0) == pytest.approx(paper["bops_a4_T"][0], abs=0.006)
    assert cm.bops_tera(3.0) == pytest.approx(paper["bops_a3_T"][0], abs=0.006)
    assert cm.bops_tera(4.0) / cm.bops_tera(3.0) == pytest.approx(paper["speedup_a3"][0], abs=0.006)
    # all windows high = the uniform model
    assert cm.equivalent_act_bits([0.0] * 6, 4.0) == 4.0
    # all windows low at every pair: half the reducible part remains
    g, c = sum(cm.PAPER_PAIR_GMACS), cm.PAPER_FIXED_GMACS
    assert cm.equivalent_act_bits([1.0] * 6, 4.0) == pytest.approx(4.0 * (g / 2 + c) / (g + c))


def test_printed_equivalent_bits_and_bops_are_consistent(paper):
    """The 8.92 T rows: 8.92 / 11.05 * 4 = 3.23 equivalent bits (printed 3.2* in Table 1, 3.23* in Table 6) and a
    1.24x speedup; a uniform ratio of 0.4 lands there."""
    bits = paper["bops_actbit_3p2_T"][0] / paper["bops_a4_T"][0] * 4.0
    assert bits == pytest.approx(paper["actbit_table6_row"][0], abs=0.006)
    assert cm.bops_tera(bits) == pytest.approx(paper["bops_actbit_3p2_T"][0], abs=0.006)
    assert paper["bops_a4_T"][0] / paper["bops_actbit_3p2_T"][0] == pytest.approx(paper["speedup_actbit_3p2"][0], abs=0.006)
    eq = cm.equivalent_act_bits([0.4] * 6, 4.0)
    assert eq == pytest.approx(3.2278, abs=5e-4)
    assert cm.bops_tera(eq) == pytest.approx(paper["bops_actbit_3p2_T"][0], abs=0.006)
    assert 1.0 / cm.relative_cost([0.4] * 6) == pytest.approx(paper["speedup_actbit_3p2"][0], abs=0.006)
    assert paper["bops_a4_T"][0] / paper["bops_mixaq_1p35_T"][0] == pytest.approx(paper["speedup_mixaq_1p35"][0], abs=0.006)


def test_pruning_rows_of_table_2(paper):
    for bops, speedup, bits in zip(paper["bops_prune_rows_T"], paper["speedup_prune_rows"], paper["actbit_prune_rows"]):
        assert paper["bops_a4_T"][0] / bops == pytest.approx(speedup, abs=0.01)   # 11.05 / 6.63 = 1.667 is printed 1.66
        assert cm.bops_tera(bits) == pytest.approx(bops, abs=0.06)          # Act Bit is printed with one decimal
    # pruning saves the whole window, compression half of it; 30 % pruning everywhere:
    assert cm.equivalent_act_bits([0.3] * 6, 4.0, method="prune") == pytest.approx(
        4.0 * (0.7 * sum(cm.PAPER_PAIR_GMACS) + 3.0) / (sum(cm.PAPER_PAIR_GMACS) + 3.0))
    # combined: (1 - p)(1 - r/2)
    assert cm.cost_fractions([0.5], [0.2]) == [pytest.approx(0.8 * 0.75)]


def test_sum_range_of_the_sampler(paper):
    lo, hi = cm.sum_range(0.65, 0.95, int(paper["n_pairs"][0]))
    assert (lo, hi) == (pytest.approx(paper["sum_range"][0]), pytest.approx(paper["sum_range"][1]))


def test_uniform_sum_sampler_invariants(paper):
    rng = np.random.default_rng(0)
    n, u = int(paper["n_pairs"][0]), paper["upper_bound"][0]
    sums = []
    for _ in range(2000):
        r = cm.sample_ratios(rng, n=n, s_min=paper["sum_range"][0], s_max=paper["sum_range"][1], u=u)
        assert len(r) == n
        t = [round(v * 10) for v in r]
        assert all(abs(v * 10 - k) < 1e-9 and 0 <= k <= round(u * 10) for v, k in zip(r, t))   # tenths, within the bound
        assert 6 <= sum(t) <= 42
        sums.append(sum(t))
    # the SUM is what is uniform (that is the point of the algorithm): every integer sum 6..42 occurs about equally
    counts = np.bincount(sums, minlength=43)[6:43]
    assert counts.min() > 0 and counts.max() < 2.2 * counts.mean()
    # naive per-layer uniform sampling concentrates around 24 instead
    naive = rng.integers(0, 9, size=(2000, n)).sum(1)
    assert np.std(naive) < np.std(sums)


def test_largest_remainder_rounding_keeps_the_sum():
    rng = np.random.default_rng(5)
    for _ in range(200):
        r = cm.sample_ratios(rng, n=6, s_min=2.0, s_max=2.0)
        assert round(sum(r) * 10) == 20


def test_largest_remainder_apportionment_closed_forms():
    lr = cm.largest_remainder
    assert lr([1, 1, 1], 10).tolist() == [4, 3, 3]                 # equal remainders: lowest index first
    assert lr([0.5, 0.3, 0.2], 10).tolist() == [5, 3, 2]           # exact quotas
    assert lr([0.47, 0.33, 0.20], 7).tolist() == [3, 2, 2]         # quotas 3.29, 2.31, 1.40: the 0.40 remainder wins
    assert lr([0.9, 0.05, 0.05], 10, cap=8).tolist() == [8, 1, 1]  # the capped entry's excess moves on
    assert lr([3, 1], 0).tolist() == [0, 0]
    with pytest.raises(ValueError):
        lr([1, 1], 17, cap=8)


def test_real_shape_macs_are_in_the_papers_range():
    """The paper's 14.16 GMACs per stage-3 pair is the linear-layer cost of 4000 tokens; our 800x1333 shape has
    50x84 = 4200 tokens padded to 56x84."""
    pairs, fixed = cm.backbone_pair_gmacs([96, 192, 384, 768], [2, 2, 6, 2], 200, 334)
    assert len(pairs) == 6
    assert pairs[2] == pairs[3] == pairs[4]
    assert 14.0 < pairs[2] < 18.0 and 3.0 < fixed < 4.5
    assert 2 * 4000 * 12 * 384 * 384 / 1e9 == pytest.approx(14.16, abs=0.01)
