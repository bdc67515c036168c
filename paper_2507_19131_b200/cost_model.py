"""Host-side helpers around the Two-Branch forward: the paper's cost model and its ratio sampler.

* Equivalent activation bits and bit operations of a ratio configuration (MixA-Q Appendix 6.2 "Calculation of
  Equivalent Activation Bits"; Section 4 "Experiments": cost is counted in bit operations of the backbone).
* Uniform-sum compression-ratio sampling (Appendix 6.1, Algorithm 1), used to draw ratio vectors for sweeps.
* Per-pair multiply-accumulate counts of an actual backbone shape, so that measured images/s can be put on the
  paper's "relative cost" axis.

Pure Python / numpy; nothing here touches the GPU.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import numpy as np

# Appendix 6.2: GMACs of each pair of consecutive Swin-T blocks, and of the downsampling layers (not reducible).
PAPER_PAIR_GMACS = (13.3, 13.56, 14.16, 14.16, 14.16, 14.02)
PAPER_FIXED_GMACS = 3.0
# Table 1 scales bit operations with the activation bit width only: 88.42 T at 32 bits, 11.05 T at 4, 8.29 T at 3,
# i.e. BOPs = total MACs x 32 x ActBit for the W4 models of the paper.
PAPER_BOPS_PER_MAC_PER_ACT_BIT = 32.0


def cost_fractions(low_ratios: Sequence[float], prune_ratios: Optional[Sequence[float]] = None,
                   method: str = "mixaq") -> List[float]:
    """Fraction of a block pair's computation that remains (Appendix 6.2): 1 - r/2 for MixA-Q (a low-bit window
    costs half), 1 - r for pruning.  With a prune ratio p in front of the compression ratio r (Section 3.4: the
    lowest windows are pruned, the rest is split), the remaining fraction is (1 - p)(1 - r/2); the paper prints no
    formula for the combination, this is the product of its two rules."""
    out = []
    for i, r in enumerate(low_ratios):
        p = float(prune_ratios[i]) if prune_ratios is not None else 0.0
        if method == "mixaq":
            out.append((1.0 - p) * (1.0 - float(r) / 2.0))
        elif method == "prune":
            out.append(1.0 - float(r))
        else:
            raise ValueError("method must be 'mixaq' or 'prune'")
    return out


def equivalent_act_bits(low_ratios: Sequence[float], act_bits_base: float,
                        pair_gmacs: Sequence[float] = PAPER_PAIR_GMACS, fixed_gmacs: float = PAPER_FIXED_GMACS,
                        prune_ratios: Optional[Sequence[float]] = None, method: str = "mixaq") -> float:
    """ActBit_eq = ActBit_base * (sum_i ratio_i * GMACs_i + C) / (sum_i GMACs_i + C)   (Appendix 6.2)."""
    if len(low_ratios) != len(pair_gmacs):
        raise ValueError("one ratio per block pair")
    fr = cost_fractions(low_ratios, prune_ratios, method)
    num = sum(f * g for f, g in zip(fr, pair_gmacs)) + fixed_gmacs
    den = sum(pair_gmacs) + fixed_gmacs
    return act_bits_base * num / den


def bops_tera(act_bits_eq: float, pair_gmacs: Sequence[float] = PAPER_PAIR_GMACS,
              fixed_gmacs: float = PAPER_FIXED_GMACS) -> float:
    """Bit operations in units of 10^12 with the scaling of Table 1 (total MACs x 32 x equivalent activation bits)."""
    return (sum(pair_gmacs) + fixed_gmacs) * 1e9 * PAPER_BOPS_PER_MAC_PER_ACT_BIT * act_bits_eq / 1e12


def relative_cost(low_ratios, pair_gmacs=PAPER_PAIR_GMACS, fixed_gmacs=PAPER_FIXED_GMACS, prune_ratios=None,
                  method="mixaq") -> float:
    """Cost relative to the all-high model; its reciprocal is the paper's "speedup"."""
    return equivalent_act_bits(low_ratios, 1.0, pair_gmacs, fixed_gmacs, prune_ratios, method)


def sum_range(cost_lo: float, cost_hi: float, n_pairs: int, saving: float = 0.5):
    """Range of the sum of compression ratios that keeps the relative cost in [cost_lo, cost_hi] when every pair has
    the same cost and a low-bit window saves `saving` of it (Appendix 6.1: [(1-0.95)*6*2, (1-0.65)*6*2])."""
    return ((1.0 - cost_hi) * n_pairs / saving, (1.0 - cost_lo) * n_pairs / saving)


def largest_remainder(shares: Sequence[float], total: int, cap: Optional[int] = None) -> np.ndarray:
    """Apportions `total` indivisible units in proportion to the non-negative `shares` (largest-remainder method):
    every entry first gets the integer part of its quota; the units still missing go, one each, to the entries with the
    largest fractional parts.  With `cap`, no entry ends above it: entries at the cap are skipped when the missing
    units are handed out (needs total <= cap * len(shares))."""
    shares = np.asarray(shares, dtype=np.float64)
    if total < 0 or shares.ndim != 1 or shares.size == 0 or (shares < 0).any() or shares.sum() <= 0:
        raise ValueError("need a non-empty vector of non-negative shares with a positive sum and total >= 0")
    if cap is not None and total > cap * shares.size:
        raise ValueError("total cannot be met under the cap")
    quota = shares * (float(total) / float(shares.sum()))
    units = np.floor(quota + 1e-12).astype(np.int64)
    if cap is not None:
        units = np.minimum(units, cap)
    while int(units.sum()) < total:
        open_entries = [i for i in range(shares.size) if cap is None or units[i] < cap]
        open_entries.sort(key=lambda i: (-(quota[i] - units[i]), i))
        for i in open_entries[: total - int(units.sum())]:
            units[i] += 1
    return units


def sample_ratios(rng: np.random.Generator, n: int = 6, s_min: float = 0.6, s_max: float = 4.2, u: float = 0.8,
                  alpha: float = 1.0, max_tries: int = 100000) -> List[float]:
    """One ratio vector whose SUM is uniformly distributed (the behaviour of Appendix 6.1, Algorithm 1): ratios are
    multiples of 0.1, none above `u`, and their sum is uniform over the tenths of [s_min, s_max].
    The sum is drawn first, as an integer number of tenths; a symmetric Dirichlet draw (the paper leaves its
    concentration open; alpha = 1 is uniform on the simplex) says how the pairs share it and is redrawn while any
    pair's share of the sum exceeds the bound; `largest_remainder` turns the shares into whole tenths."""
    cap = int(round(u * 10))
    tenths = int(rng.integers(int(np.ceil(s_min * 10 - 1e-9)), int(np.floor(s_max * 10 + 1e-9)) + 1))
    if tenths > cap * n:
        raise ValueError("target sum cannot be met under the upper bound")
    for _ in range(max_tries):
        shares = rng.dirichlet(np.full(n, alpha))
        if shares.max() * tenths <= cap + 1e-12:
            return [float(k) / 10.0 for k in largest_remainder(shares, tenths, cap)]
    raise RuntimeError("no admissible split found")


def backbone_pair_gmacs(dims: Sequence[int], depths: Sequence[int], H0: int, W0: int, window: int = 7):
    """(per-pair GMACs, fixed GMACs) of an actual backbone shape for one image: a block costs
    (12 C^2 + 2 * 49 * C) MACs per window token (QKV, proj, fc1, fc2 and the two attention products), windows cover
    the padded map; patch merging between stages (4C x 2C per output token) is the fixed part."""
    pairs, fixed = [], 0.0
    H, W = H0, W0
    for s, (C, d) in enumerate(zip(dims, depths)):
        if s > 0:
            H2, W2 = (H + 1) // 2, (W + 1) // 2
            fixed += H2 * W2 * (4 * dims[s - 1]) * (2 * dims[s - 1]) / 1e9
            H, W = H2, W2
        Hp, Wp = -(-H // window) * window, -(-W // window) * window
        per_block = Hp * Wp * (12 * C * C + 2 * window * window * C) / 1e9
        for _ in range((d + 1) // 2):
            pairs.append(per_block * min(2, d))
    return pairs, fixed
