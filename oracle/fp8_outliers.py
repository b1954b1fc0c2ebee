"""CPU oracle of the FP8 option for OutControl's outlier channels (paper Sec. 4.2: the outlier part may be kept in "high
precision (e.g., FP8, BF16)"; the hyper-parameter table lists FP8 as the outlier compute type).

TEST INFRASTRUCTURE ONLY: imported by ``tests/`` and by the oracle's layer functions; the CUDA library never imports it.

PARITY UNPINNED with respect to the paper: the paper gives no FP8 recipe (format, scale granularity, scale rounding), so
the recipe below is this build's own definition. What is pinned is the definition itself (against the E4M3 value table,
exact rational arithmetic and torch's own E4M3 cast), not its agreement with the authors' kernels.

Recipe, for one outlier slice T (X[:, A] or W[:, A], BF16 values):
    amax = max |T|;   e = the smallest integer with amax / 2^e <= 448   (e = 0 for an all-zero slice)
    q    = E4M3(T / 2^e)           OCP E4M3 "FN", round to nearest, ties to the even code (no value exceeds 448)
    T8   = q * 2^e                 the values the FP8 tensor represents
The scale is a power of two, so T / 2^e and q * 2^e are exact and T8 is again exactly representable in BF16 (4 significant
bits): the layer uses T8 wherever the BF16 variant uses T (forward side product, dW[:, A], W-hat[:, A]), and a product of
T8 slices accumulated in FP32 equals the FP8 tensor-core product times the two scales bit for bit.
"""
from __future__ import annotations

import math

import numpy as np

from oracle import nvfp4_oracle as orc

_TABLE = None


def _table() -> np.ndarray:
    """The 127 finite non-negative E4M3 values, ascending (index = byte)."""
    global _TABLE
    if _TABLE is None:
        _TABLE = np.array([orc.e4m3_value(b) for b in range(0x7F)], dtype=np.float64)
    return _TABLE


def scale_exponent(amax: float) -> int:
    """Smallest integer e with amax / 2^e <= 448; 0 for amax == 0."""
    if amax == 0.0:
        return 0
    m, k = math.frexp(amax / 448.0)  # amax / 448 = m * 2^k, 0.5 <= m < 1 (the quotient is only used for its magnitude)
    e = k if m > 0.5 else k - 1  # 2^e >= m 2^k
    # the float quotient may be off by an ulp at an exact power of two: settle it with exact integers
    while math.ldexp(448.0, e) < amax:
        e += 1
    while math.ldexp(448.0, e - 1) >= amax:
        e -= 1
    return e


def e4m3_round(y: np.ndarray) -> np.ndarray:
    """Nearest E4M3 value (ties to the even byte, saturating at 448) of every element, sign kept. float64 in and out."""
    tab = _table()
    a = np.minimum(np.abs(y), 448.0)
    hi = np.searchsorted(tab, a, side="left")  # first index with tab >= a
    hi = np.minimum(hi, len(tab) - 1)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - tab[lo], tab[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    q = np.where(pick_hi, tab[hi], tab[lo])
    return np.copysign(q, y)


def snap(T: np.ndarray):
    """(T8, e): the slice on its scaled E4M3 grid (float32) and the scale exponent."""
    T = np.asarray(T, dtype=np.float32)
    amax = float(np.max(np.abs(T))) if T.size else 0.0
    e = scale_exponent(amax)
    q = e4m3_round(T.astype(np.float64) * math.ldexp(1.0, -e))
    return (q * math.ldexp(1.0, e)).astype(np.float32), e
