"""Pins for the oracle's number formats, random generator and element rounding.

Nothing here re-types the oracle's own formulas: expected values come from the paper's printed value set
(Sec. 2.1), from the published Philox known-answer vectors, from torch's float8_e4m3fn cast (an independent
library routine), and from exact rational arithmetic.
"""
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")

# Sec. 2.1 "NVFP4 Format": FP4Values = {0, +-0.5, +-1, +-1.5, +-2, +-3, +-4, +-6}
PAPER_FP4_VALUES = {0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0, -0.5, -1.0, -1.5, -2.0, -3.0, -4.0, -6.0}


def test_e2m1_table_is_the_papers_value_set():
    vals = [orc.e2m1_value(c) for c in range(16)]
    assert set(vals) == PAPER_FP4_VALUES  # -0.0 == 0.0 collapses, leaving the 15 distinct values
    # magnitude index is monotone, sign is bit 3, and the encoding is 1 sign / 2 exponent / 1 mantissa bit
    for c in range(8):
        assert vals[c] >= 0 and vals[c + 8] == -vals[c]
        if c:
            assert vals[c] > vals[c - 1]
        e, m = c >> 1, c & 1
        expect = Fraction(m, 2) if e == 0 else Fraction(2) ** (e - 1) * (1 + Fraction(m, 2))
        assert Fraction(vals[c]) == expect
    assert np.signbit(vals[8])


def test_e4m3_table_matches_library_float8():
    bytes_ = torch.arange(256, dtype=torch.uint8)
    ref = bytes_.view(torch.float8_e4m3fn).to(torch.float64).numpy()
    ours = np.array([orc.e4m3_value(b) for b in range(256)])
    assert np.array_equal(np.isnan(ref), np.isnan(ours))
    ok = ~np.isnan(ref)
    assert np.array_equal(ref[ok], ours[ok])
    assert np.isnan(ours[0x7F]) and np.isnan(ours[0xFF])
    finite = ours[:0x7F]
    assert len(finite) == 127 and finite.max() == 448.0 and ours[0x7E] == 448.0  # Sec. 2.2: range +-448
    assert np.all(np.diff(finite) > 0)  # non-negative bytes are monotone in value


def test_e4m3_encode_rn_even_at_every_midpoint_and_saturates():
    vals = [Fraction(orc.e4m3_value(b)) for b in range(0x7F)]
    for b in range(0x7E):
        lo, hi = vals[b], vals[b + 1]
        mid = (lo + hi) / 2
        midf = float(mid)
        assert Fraction(midf) == mid  # midpoints of adjacent E4M3 values are float32-representable
        even = b if b % 2 == 0 else b + 1
        assert orc.e4m3_encode(midf) == even
        below = np.nextafter(np.float32(midf), np.float32(0))
        above = np.nextafter(np.float32(midf), np.float32(1e9))
        assert orc.e4m3_encode(float(below)) == b
        assert orc.e4m3_encode(float(above)) == b + 1
        assert orc.e4m3_encode(float(lo)) == b
    for big in (448.0, 449.0, 464.0, 480.0, 1e4, 3.0e38):
        assert orc.e4m3_encode(big) == 0x7E
    assert orc.e4m3_encode(0.0) == 0


def test_e4m3_encode_agrees_with_library_cast_below_saturation():
    rng = np.random.default_rng(11)
    x = np.concatenate([
        np.exp(rng.uniform(np.log(2.0 ** -12), np.log(447.9), 4000)),
        rng.uniform(0, 2.0 ** -6, 500),
    ]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    ours = np.array([orc.e4m3_encode(v) for v in x], dtype=np.uint8)
    assert np.array_equal(ref, ours)


def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 3
    for r in rows:
        v = [int(t, 16) for t in r]
        out = orc.philox4x32_10(v[0:4], v[4:6])
        assert [int(o) for o in out] == v[6:10]


def test_sr_bits_addressing():
    """Element idx takes the 16-bit field (idx % 8) of the Philox block with counter idx // 8, key = seed."""
    seed, stream = 0x0123456789ABCDEF, 5
    for idx in (0, 1, 7, 8, 9, 1023, (1 << 32) + 3, (1 << 35) + 6):
        j = idx // 8
        w = orc.philox4x32_10([j & 0xFFFFFFFF, j >> 32, stream, 0], [seed & 0xFFFFFFFF, seed >> 32])
        fields = [int(w[i // 2]) >> (16 * (i % 2)) & 0xFFFF for i in range(8)]
        assert orc.sr_bits(seed, stream, idx) == fields[idx % 8]
    # a different stream id or seed gives a different block
    a = [orc.sr_bits(1, 3, i) for i in range(64)]
    assert a != [orc.sr_bits(1, 4, i) for i in range(64)]
    assert a != [orc.sr_bits(2, 3, i) for i in range(64)]


MAGS = [Fraction(v) for v in (0, 0.5, 1, 1.5, 2, 3, 4, 6)]


def brute_nearest(a: Fraction) -> int:
    """argmin_q |a - q| over the paper's magnitudes in exact arithmetic; an exact tie goes to the even index."""
    errs = [abs(a - q) for q in MAGS]
    best = min(errs)
    cands = [i for i, e in enumerate(errs) if e == best]
    return cands[0] if len(cands) == 1 else [i for i in cands if i % 2 == 0][0]


def test_rtn_is_nearest_value_bruteforce():
    rng = np.random.default_rng(3)
    xs = list(rng.uniform(0, 6, 3000).astype(np.float32))
    ties = [0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]
    for t in ties:
        xs += [np.float32(t), np.nextafter(np.float32(t), np.float32(0)), np.nextafter(np.float32(t), np.float32(9))]
    xs += [np.float32(float(q)) for q in MAGS]
    for a in xs:
        assert orc.round_rtn_mag(float(a)) == brute_nearest(Fraction(float(a)))
    # the seven ties named one by one: 0.25->0, 0.75->1, 1.25->1, 1.75->2, 2.5->2, 3.5->4, 5->4
    assert [float(MAGS[orc.round_rtn_mag(t)]) for t in ties] == [0.0, 1.0, 1.0, 2.0, 2.0, 4.0, 4.0]


def test_rounding_fixes_representable_values():
    for i, q in enumerate(MAGS):
        assert orc.round_rtn_mag(float(q)) == i
        for u in (0, 1, 32767, 32768, 65535):
            assert orc.round_sr_mag(float(q), u) == i
    assert orc.round_sr_mag(6.0, 65535) == 7


def test_sr_rounds_to_bracket_and_is_unbiased_over_all_u():
    """Exhaustive over the 65536 draws: P(up) is within 2^-17 of f = (a - q1)/(q2 - q1), i.e. the expected
    rounded value is within (q2 - q1) * 2^-17 of a  (the paper's E[round_S(x)] = x, Sec. 2.1)."""
    rng = np.random.default_rng(5)
    samples = [0.1, 0.25, 0.4999, 0.75, 1.3, 1.9, 2.0001, 2.7, 3.99, 4.5, 5.999] + list(rng.uniform(0, 6, 6))
    for a in samples:
        a32 = float(np.float32(a))
        lo = max(i for i, q in enumerate(MAGS) if q <= Fraction(a32))
        q1, q2 = MAGS[lo], MAGS[lo + 1]
        f = (Fraction(a32) - q1) / (q2 - q1)
        ups = 0
        for u in range(65536):
            m = orc.round_sr_mag(a32, u)
            assert m in (lo, lo + 1)
            ups += m == lo + 1
        assert abs(Fraction(ups, 65536) - f) <= Fraction(1, 1 << 17)
        mean = q1 + (q2 - q1) * Fraction(ups, 65536)
        assert abs(mean - Fraction(a32)) <= (q2 - q1) * Fraction(1, 1 << 17)
    # monotone in u: small u rounds up, large u rounds down (the draw is compared from below)
    assert orc.round_sr_mag(2.5, 0) == 5 and orc.round_sr_mag(2.5, 65535) == 4
    assert orc.round_sr_mag(2.5, 32767) == 5 and orc.round_sr_mag(2.5, 32768) == 4
