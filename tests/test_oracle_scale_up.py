"""Pins for the round-up block-scale variant of stochastic rounding (rounding mode SR_SCALE_UP).

Sec. 2.1 states E[round_S(x)] = x for -6 <= x <= 6. With the block scale rounded to the NEAREST E4M3 value about half of
the blocks get a scale below amax_b / (6 Sg); their largest element then lies beyond 6 on the FP4 grid, is clamped, and
the expectation fails for it. The variant takes the smallest E4M3 value >= amax_b / (6 Sg): these tests pin that
definition with exact rational arithmetic and check the consequence (no clamping, unbiased for every element) against
the statistics of 10^4 seeds.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth

MAGS = [Fraction(v) for v in (0, 0.5, 1, 1.5, 2, 3, 4, 6)]


def table():
    return [Fraction(orc.e4m3_value(b)) for b in range(0x7F)]


def test_encode_up_is_the_ceiling_on_the_e4m3_grid():
    tab = table()
    assert all(tab[i] < tab[i + 1] for i in range(len(tab) - 1))  # bytes are ordered like their values
    for b, v in enumerate(tab):
        f = np.float32(float(v))
        assert orc.e4m3_encode_up(float(f)) == b  # a grid value is its own ceiling
        above = np.nextafter(f, np.float32(np.inf), dtype=np.float32)
        assert orc.e4m3_encode_up(float(above)) == min(b + 1, 0x7E)
        if b > 0:
            below = np.nextafter(f, np.float32(0), dtype=np.float32)
            assert orc.e4m3_encode_up(float(below)) == b
    assert orc.e4m3_encode_up(0.0) == 0
    assert orc.e4m3_encode_up(1e-30) == 1  # the smallest subnormal, 2^-9, where round-to-nearest gives 0
    assert orc.e4m3_encode_up(1000.0) == 0x7E
    rng = np.random.default_rng(5)
    for s in np.exp(rng.uniform(np.log(1e-4), np.log(448), 2000)).astype(np.float32):
        up, rn = orc.e4m3_encode_up(float(s)), orc.e4m3_encode(float(s))
        assert up in (rn, rn + 1)
        assert tab[up] >= Fraction(float(s)) and (up == 0 or tab[up - 1] < Fraction(float(s)))


def unpack(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128])
def test_scales_and_codes_in_exact_arithmetic(gs_mode):
    R, K = 12, 144
    x = synth.gradients(R, K, 31, 1e-3)
    seed, stream = 99, 5
    up = orc.quantize(x, orc.AXIS_ROW, orc.SR_SCALE_UP, gs_mode, seed, stream)
    rn = orc.quantize(x, orc.AXIS_ROW, orc.SR, gs_mode, seed, stream)
    assert np.array_equal(np.asarray(up.gscale), np.asarray(rn.gscale))  # the global scale is not affected
    d = up.sf.astype(int) - rn.sf.astype(int)
    assert set(np.unique(d)) <= {0, 1} and (d == 1).any() and (d == 0).any()
    tab = table()
    codes = unpack(up.codes)
    eps = Fraction(1, 2 ** 20)
    checked = 0
    for r in range(R):
        for b in range(K // 16):
            blk = x[r, 16 * b:16 * b + 16]
            Sg = Fraction(float(up.gscale[0] if gs_mode == orc.GS_TENSOR else up.gscale[r] if gs_mode == orc.GS_ROW
                                else up.gscale[r, b // 8]))
            sb = int(up.sf[r, b])
            Sb = tab[sb]
            amax_b = max(abs(Fraction(float(v))) for v in blk)
            s_exact = amax_b / Sg / 6
            # smallest grid value >= s (up to the two float roundings of t and s)
            assert Sb >= s_exact * (1 - eps)
            assert sb == 0 or tab[sb - 1] < s_exact * (1 + eps)
            for i, xv in enumerate(blk):
                a = abs(Fraction(float(xv))) / (Sg * Sb)
                assert a <= 6 * (1 + eps)  # nothing beyond the grid: the clamp never bites
                m = int(codes[r, 16 * b + i]) & 7
                lo = max(j for j, q in enumerate(MAGS) if q <= min(a, Fraction(6)))
                if lo == 7:
                    assert m == 7
                    continue
                f = (a - MAGS[lo]) / (MAGS[lo + 1] - MAGS[lo])
                v = (Fraction(orc.sr_bits(seed, stream, r * K + 16 * b + i)) + Fraction(1, 2)) / 65536
                if abs(v - f) > eps * 8:
                    assert m == (lo + 1 if v < f else lo), (r, b, i)
                    checked += 1
    assert checked > 0.9 * R * K


def test_every_element_is_unbiased_where_the_nearest_scale_is_not():
    """10^4 seeds. SR_SCALE_UP: every element's mean is within the sampling error of its value. Plain SR on the same
    input: the clamped block maxima (scale rounded down) have a mean that is too small by the clamped amount."""
    x = synth.gradients(4, 64, 56, 1e-3)
    n = 10_000
    mags = np.array([float(m) for m in MAGS])

    def run(mode):
        base = orc.quantize(x, orc.AXIS_ROW, mode, orc.GS_ROW, seed=1, stream_id=3)
        step = np.array([[orc.e4m3_value(b) for b in row] for row in base.sf]).repeat(16, axis=1) * base.gscale[:, None]
        acc = np.zeros(x.shape, dtype=np.float64)
        for s in range(n):
            op = orc.quantize(x, orc.AXIS_ROW, mode, orc.GS_ROW, seed=s * 7919 + 1, stream_id=3)
            acc += orc.dequantize(op)
        return acc / n, step

    mean_up, step_up = run(orc.SR_SCALE_UP)
    a = np.abs(x.astype(np.float64)) / step_up
    assert a.max() <= 6 * (1 + 1e-6)
    lo = np.searchsorted(mags, np.minimum(a, 6), side="right") - 1
    q1, q2 = mags[lo], mags[np.minimum(lo + 1, 7)]
    var = np.maximum((q2 - a) * (a - q1), 0)
    sigma = step_up * np.sqrt(var) / np.sqrt(n)
    free = var > 1e-6
    z = (mean_up - x)[free] / sigma[free]
    assert free.sum() > 200
    assert np.abs(z).max() < 5.0 and 0.7 < np.mean(z ** 2) < 1.4 and abs(z.mean()) < 4.0 / np.sqrt(free.sum())
    assert np.allclose(mean_up[~free], x[~free], rtol=0, atol=1e-12 + 1e-3 * step_up[~free])

    mean_rn, step_rn = run(orc.SR)
    a_rn = np.abs(x.astype(np.float64)) / step_rn
    clamped = a_rn > 6 * (1 + 1e-3)
    assert clamped.sum() >= 3  # some block maxima fall beyond the grid with the nearest scale
    # their mean is exactly the clamp, 6 steps, short of |x| by (a - 6) steps
    assert np.allclose(np.abs(mean_rn[clamped]), 6 * step_rn[clamped], rtol=1e-12)
    assert np.all(np.abs(x[clamped]) - np.abs(mean_rn[clamped]) > 1e-3 * 6 * step_rn[clamped])
    # and the variant removes exactly that bias
    zc = (mean_up - x)[clamped] / np.maximum(sigma[clamped], 1e-300)
    assert np.all(np.abs(zc[var[clamped] > 1e-6]) < 5.0)
