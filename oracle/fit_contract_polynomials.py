"""Where the polynomial coefficients of the numeric contract come from (TEST INFRASTRUCTURE, like the rest of oracle/).

The contract evaluates two functions by fixed polynomials in binary32 (Horner, fused multiply-adds):
  * 2^f on [-1/2, 1/2], degree 5   (softmax exponentials and the GELU tail),
  * log2 Phi(-a) on [0, 5], degree 7, Phi the standard normal distribution function   (GELU = max(v,0) - a*Phi(-a)).
Both are minimax fits (smallest maximum absolute error) found with the Remez exchange algorithm in binary64 and
rounded to binary32.  The words in FROZEN below are the contract: the oracle and the kernels each carry them as
literals.  They were produced by a run of this procedure that located the error extrema on a coarser grid, so a fresh
run agrees with them to about 1e-4 relative in the smallest coefficients and exactly in the largest ones, and their
maximum error is within a fraction of a percent of the optimum; `check()` measures both.  Re-deriving them does not
change the contract: the frozen words do.

  python oracle/fit_contract_polynomials.py        # prints frozen and re-derived coefficients and their errors
"""
from __future__ import annotations

import math
import struct

import numpy as np
from scipy.optimize import minimize_scalar
from scipy.special import log_ndtr

# coefficient of f^0, f^1, ... as binary32 bit patterns
FROZEN = {
    "exp2": [0x3f800001, 0x3f317219, 0x3e75fc83, 0x3d635716, 0x3c1e883d, 0x3aafc47d],
    "log2_phi_neg": [0xbf7fffbe, 0xbf935b8f, 0xbeeac5d4, 0xbd5c93e3, 0x3c0a3aed, 0xba6dcc74, 0x38729e20, 0xb5d6f9e3],
}
TARGETS = {
    "exp2": (lambda t: np.exp2(t), 5, -0.5, 0.5),
    "log2_phi_neg": (lambda a: log_ndtr(-np.asarray(a, dtype=np.float64)) / math.log(2.0), 7, 0.0, 5.0),
}


def word_to_float(w: int) -> float:
    return float(struct.unpack("<f", struct.pack("<I", w))[0])


def float_to_word(v: float) -> int:
    return struct.unpack("<I", struct.pack("<f", np.float32(v)))[0]


def remez(f, degree: int, lo: float, hi: float, grid_points: int = 20001, rounds: int = 40):
    """Minimax polynomial of `degree` for f on [lo, hi]: returns (coefficients low order first, max |error|)."""
    n = degree + 2
    k = np.arange(n)
    nodes = (lo + hi) / 2 + (hi - lo) / 2 * np.cos(np.pi * k / (n - 1))[::-1]
    grid = np.linspace(lo, hi, grid_points)
    coef, err = None, None
    for _ in range(rounds):
        # polynomial whose error alternates with equal magnitude on the current nodes
        system = np.zeros((n, n))
        for j in range(degree + 1):
            system[:, j] = nodes ** j
        system[:, degree + 1] = (-1.0) ** k
        coef = np.linalg.solve(system, f(nodes))[: degree + 1]
        error_at = lambda t: np.polyval(coef[::-1], t) - f(t)      # noqa: E731
        err = error_at(grid)
        # one extremum per sign run of the error, refined inside its grid cell
        cuts = np.concatenate([[0], np.where(np.diff(np.sign(err)) != 0)[0] + 1, [grid.size]])
        extrema = []
        for a, b in zip(cuts[:-1], cuts[1:]):
            j = a + int(np.argmax(np.abs(err[a:b])))
            sign = np.sign(err[j])
            left, right = grid[max(j - 1, 0)], grid[min(j + 1, grid.size - 1)]
            res = minimize_scalar(lambda t: -sign * error_at(t), bounds=(left, right), method="bounded",
                                  options={"xatol": 1e-14})
            extrema.append(res.x)
        if len(extrema) != n:
            break
        moved = float(np.abs(np.array(extrema) - nodes).max())
        nodes = np.array(extrema)
        if moved < 1e-13:
            break
    return coef, float(np.abs(err).max())


def check():
    """Per function: re-derived words, frozen words, largest relative coefficient difference, and the maximum error of
    the frozen and of the re-derived polynomial (both evaluated in binary64 on a dense grid)."""
    out = {}
    for name, (f, degree, lo, hi) in TARGETS.items():
        coef, _ = remez(f, degree, lo, hi)
        fitted = np.array([word_to_float(float_to_word(c)) for c in coef])
        frozen = np.array([word_to_float(w) for w in FROZEN[name]])
        grid = np.linspace(lo, hi, 400001)
        truth = f(grid)
        out[name] = {
            "fitted_words": [float_to_word(c) for c in coef],
            "frozen_words": list(FROZEN[name]),
            "max_rel_coef_diff": float(np.abs(fitted / frozen - 1.0).max()),
            "max_err_frozen": float(np.abs(np.polyval(frozen[::-1], grid) - truth).max()),
            "max_err_fitted": float(np.abs(np.polyval(fitted[::-1], grid) - truth).max()),
        }
    return out


if __name__ == "__main__":
    for name, r in check().items():
        print(name)
        print("  frozen  ", " ".join("0x%08x" % w for w in r["frozen_words"]))
        print("  fitted  ", " ".join("0x%08x" % w for w in r["fitted_words"]))
        print("  largest relative coefficient difference %.2e" % r["max_rel_coef_diff"])
        print("  max |error|: frozen %.4e, fitted %.4e" % (r["max_err_frozen"], r["max_err_fitted"]))
