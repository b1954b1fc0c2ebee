"""Pins for the oracle's double-block quantizer (Sec. 2.2) against facts that do not come from the oracle:
hand-derived worked blocks, exact rational arithmetic on its outputs, structural invariants, symmetries and
the unbiasedness of stochastic rounding.
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
MAGS = [Fraction(v) for v in (0, 0.5, 1, 1.5, 2, 3, 4, 6)]
E4M3 = None


def e4m3_table():
    global E4M3
    if E4M3 is None:
        E4M3 = [Fraction(orc.e4m3_value(b)) for b in range(0x7F)]
    return E4M3


def unpack(codes: np.ndarray) -> np.ndarray:
    """[R, K/2] bytes -> [R, K] 4-bit codes, low nibble first."""
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def group_scale(op: orc.Operand, r: int, k: int) -> float:
    if op.gs_mode == orc.GS_TENSOR:
        return float(op.gscale[0])
    if op.gs_mode == orc.GS_ROW:
        return float(op.gscale[r])
    return float(op.gscale[r, k // 128])


def load_blocks():
    rows = []
    for line in open(os.path.join(GOLDEN, "quantize_blocks.txt")):
        if not line.strip() or line[0] == "#":
            continue
        v, s, c = line.split("|")
        rows.append(([float(t) for t in v.split()], int(s.strip(), 16), [int(t) for t in c.split()]))
    return rows


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128])
def test_hand_derived_blocks(gs_mode):
    blocks = load_blocks()
    x = np.array([v for b in blocks for v in b[0]], dtype=np.float32).reshape(1, 64)
    op = orc.quantize(x, orc.AXIS_ROW, orc.RTN, gs_mode)
    assert np.all(op.gscale == 1.0)  # 2688 / (448 * 6)
    assert list(op.sf[0]) == [b[1] for b in blocks]
    assert list(unpack(op.codes)[0]) == [c for b in blocks for c in b[2]]
    # reconstruction X ~ P * S_global * S_block, worked by hand for a few entries
    deq = orc.dequantize(op)[0]
    assert deq[0] == 6 * 448 and deq[1] == 2 * 448 and deq[2] == -1 * 448 and deq[6] == 1 * 448
    assert deq[16] == 6 and deq[17] == 4 and deq[26] == -4 and deq[25] == 0.5
    assert deq[32] == 6 * 3.25 and deq[33] == 3 * 3.25 and deq[34] == -2 * 3.25 and deq[35] == 0.5 * 3.25
    assert np.all(deq[48:] == 0)
    # nibble order: low nibble holds the even k
    assert op.codes[0, 0] == (7 | (4 << 4)) and op.codes[0, 1] == (10 | (0 << 4))


def check_against_exact_arithmetic(x: np.ndarray, op: orc.Operand, rounding_is_rtn: bool, uof=None):
    """Verify every output of a quantize call from the paper's formulas in exact rational arithmetic.
    float32 rounding inside the pinned operation sequence can only matter within a few ulp of a decision
    threshold; such borderline cases are skipped (they are covered by the hand-derived blocks)."""
    tab = e4m3_table()
    R, K = x.shape
    codes = unpack(op.codes)
    eps = Fraction(1, 1 << 20)
    checked = 0
    for r in range(R):
        for b in range((K + 15) // 16):
            blk = x[r, 16 * b: min(16 * b + 16, K)]
            Sg = Fraction(group_scale(op, r, 16 * b))
            # global scale = amax / 2688, correctly rounded to float32 (half-ulp bound via 2^-24 relative)
            if op.gs_mode == orc.GS_TENSOR:
                amax_g = Fraction(float(np.abs(x).max()))
            elif op.gs_mode == orc.GS_ROW:
                amax_g = Fraction(float(np.abs(x[r]).max()))
            else:
                g0 = (16 * b) // 128 * 128
                amax_g = Fraction(float(np.abs(x[r, g0: min(g0 + 128, K)]).max()))
            if amax_g == 0:
                assert Sg == 1
            else:
                assert abs(Sg - amax_g / 2688) <= (amax_g / 2688) * Fraction(1, 1 << 24)
            amax_b = Fraction(float(np.abs(blk).max()))
            s_exact = amax_b / Sg / 6
            sb = int(op.sf[r, b])
            Sb = tab[sb]
            # S_block: the nearest E4M3 value to amax_b / S_global / 6 (saturating)
            if s_exact >= 448:
                assert sb == 0x7E
            else:
                lo = max(i for i, v in enumerate(tab) if v <= s_exact)
                mid = (tab[lo] + tab[lo + 1]) / 2
                if abs(s_exact - mid) > mid * eps:
                    assert sb == (lo if s_exact < mid else lo + 1), (r, b, float(s_exact))
            for i, xv in enumerate(blk):
                code = int(codes[r, 16 * b + i])
                assert (code >> 3) == int(np.signbit(xv))
                m = code & 7
                if Sb == 0:
                    assert m == 0
                    continue
                a = min(abs(Fraction(float(xv))) / (Sg * Sb), Fraction(6))
                if rounding_is_rtn:
                    errs = [abs(a - q) for q in MAGS]
                    order = sorted(range(8), key=lambda j: errs[j])
                    if errs[order[1]] - errs[order[0]] > eps * 8:
                        assert m == order[0], (r, b, i, float(a), m)
                        checked += 1
                    else:
                        assert m in order[:2]
                else:
                    lo = max(j for j, q in enumerate(MAGS) if q <= a)
                    if lo == 7:
                        assert m == 7
                        continue
                    assert m in (lo, lo + 1) or abs(a - MAGS[lo]) < eps * 8, (r, b, i, float(a), m)
                    if uof is not None:
                        f = (a - MAGS[lo]) / (MAGS[lo + 1] - MAGS[lo])
                        v = (Fraction(uof(r, 16 * b + i)) + Fraction(1, 2)) / 65536
                        if abs(v - f) > eps * 8:
                            assert m == (lo + 1 if v < f else lo)
                            checked += 1
    return checked


def small_inputs(seed, R=16, K=16, outliers=True):
    x, _ = synth.activations(R, K, seed, n_outlier=2 if outliers and K >= 4 else 0, factor=50.0)
    return x


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128])
@pytest.mark.parametrize("shape", [(16, 16), (5, 48), (3, 144), (2, 272), (4, 40)])
def test_rtn_bruteforce_exact_arithmetic(gs_mode, shape):
    x = small_inputs(100 + shape[1], *shape)
    op = orc.quantize(x, orc.AXIS_ROW, orc.RTN, gs_mode)
    n = check_against_exact_arithmetic(x, op, True)
    assert n > 0.9 * x.size * 0.9
    K16 = (shape[1] + 15) // 16 * 16
    assert op.codes.shape == (shape[0], K16 // 2) and op.sf.shape == (shape[0], K16 // 16)
    if shape[1] % 16:  # padding nibbles are zero
        assert np.all(unpack(op.codes)[:, shape[1]:] == 0)


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_BLOCK128])
def test_sr_bruteforce_exact_arithmetic(gs_mode):
    x = synth.gradients(16, 48, 77, 1e-3)
    seed, stream = 1234, 3
    op = orc.quantize(x, orc.AXIS_ROW, orc.SR, gs_mode, seed, stream)
    n = check_against_exact_arithmetic(x, op, False, uof=lambda r, k: orc.sr_bits(seed, stream, r * 48 + k))
    assert n > 0.5 * x.size


def test_block_scale_closed_form():
    """If 448 * amax_b / amax_g is itself an E4M3 value, S_block equals it exactly (Sec. 2.2 closed form)."""
    tab = e4m3_table()
    x = np.zeros((1, 16 * 20), dtype=np.float32)
    x[0, 0] = 2688.0  # S_global = 1
    picks = [0x7E, 0x78, 0x70, 0x45, 0x38, 0x30, 0x21, 0x10, 0x08, 0x07, 0x03, 0x01]
    for j, byte in enumerate(picks):
        x[0, 16 * (j + 1) + 3] = -float(tab[byte] * 6)  # amax_b / 6 = the E4M3 value
    op = orc.quantize(x, orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR)
    assert op.gscale[0] == 1.0 and op.sf[0, 0] == 0x7E
    assert list(op.sf[0, 1: len(picks) + 1]) == picks
    assert np.all(op.sf[0, len(picks) + 1:] == 0)
    # and the block maximum maps to magnitude 6 with its sign
    c = unpack(op.codes)[0]
    for j in range(len(picks)):
        assert c[16 * (j + 1) + 3] == 15


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128])
def test_invariants_max_scale_and_max_code(gs_mode):
    rng = np.random.default_rng(9)
    x = synth.round_to_bf16((rng.standard_normal((64, 384)) * np.exp(rng.uniform(-8, 8, (64, 1)))).astype(np.float32))
    op = orc.quantize(x, orc.AXIS_ROW, orc.RTN, gs_mode)
    codes = unpack(op.codes)
    sf = op.sf
    # every outer group with a non-zero element holds a block whose scale is the E4M3 maximum 448
    if gs_mode == orc.GS_TENSOR:
        assert (sf == 0x7E).any()
    elif gs_mode == orc.GS_ROW:
        assert np.all((sf == 0x7E).any(axis=1))
    else:
        assert np.all((sf.reshape(64, 3, 8) == 0x7E).any(axis=2))
    # every block with a normal E4M3 scale (>= 2^-6, byte >= 0x08) has a largest magnitude of 6 (index 7)
    mags = (codes & 7).reshape(64, 24, 16).max(axis=2)
    assert np.all(mags[sf >= 0x08] == 7)
    # error bound where the block scale is a normal E4M3 (relative rounding error <= 1/17): |x - x_hat| is
    # at most half the widest grid gap (1.0) times the step; the clamp excess is at most 0.375 * step
    deq = orc.dequantize(op)
    step = np.array([[orc.e4m3_value(b) for b in row] for row in sf]).repeat(16, axis=1)
    gs = {orc.GS_TENSOR: lambda: np.full(x.shape, op.gscale[0]), orc.GS_ROW: lambda: op.gscale[:, None].repeat(384, 1),
          orc.GS_BLOCK128: lambda: op.gscale.repeat(128, axis=1)}[gs_mode]()
    bound = 1.0 * step * gs * (1 + 1e-6)
    ok = sf.repeat(16, axis=1) >= 0x08
    assert np.all(np.abs(x.astype(np.float64) - deq)[ok] <= bound[ok])


def canonical(R, K, seed, scale_exp=-3):
    """Lossless inputs: E2M1 grid values times 448 * 2^e, a +-6 in every 16-block of rows AND columns."""
    rng = np.random.default_rng(seed)
    q = np.array([float(m) for m in MAGS])[rng.integers(0, 8, (R, K))] * rng.choice([-1.0, 1.0], (R, K))
    i, j = np.meshgrid(np.arange(R), np.arange(K), indexing="ij")
    six = (i + j) % 2 == 0
    q[six] = 6.0 * rng.choice([-1.0, 1.0], (R, K))[six]
    return (q * 448.0 * 2.0 ** scale_exp).astype(np.float32), q


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128])
@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR])
@pytest.mark.parametrize("axis", [orc.AXIS_ROW, orc.AXIS_COL])
def test_idempotent_on_canonical_inputs(gs_mode, rounding, axis):
    x, q = canonical(32, 272, 21)
    assert np.array_equal(synth.round_to_bf16(x), x)
    op = orc.quantize(x, axis, rounding, gs_mode, seed=5, stream_id=4)
    xt = x if axis == orc.AXIS_ROW else x.T
    assert np.all(op.gscale == 2.0 ** -3)
    assert np.all(op.sf == 0x7E)
    assert np.array_equal(orc.dequantize(op)[:, : xt.shape[1]], xt.astype(np.float64))
    assert np.array_equal(orc.rematerialize_f32(op), xt)
    op2 = orc.quantize(orc.rematerialize_f32(op), orc.AXIS_ROW, rounding, gs_mode, seed=99, stream_id=6)
    assert np.array_equal(op2.codes, op.codes) and np.array_equal(op2.sf, op.sf) and np.array_equal(op2.gscale, op.gscale)


@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR])
def test_scaling_and_sign_equivariance(rounding):
    x = small_inputs(31, 24, 160)
    a = orc.quantize(x, orc.AXIS_ROW, rounding, orc.GS_BLOCK128, seed=8, stream_id=3)
    b = orc.quantize(x * np.float32(2.0 ** 5), orc.AXIS_ROW, rounding, orc.GS_BLOCK128, seed=8, stream_id=3)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.sf, b.sf)
    assert np.array_equal(a.gscale * np.float32(32), b.gscale)
    c = orc.quantize(-x, orc.AXIS_ROW, rounding, orc.GS_BLOCK128, seed=8, stream_id=3)
    assert np.array_equal(a.codes ^ 0x88, c.codes) and np.array_equal(a.sf, c.sf) and np.array_equal(a.gscale, c.gscale)


def test_column_axis_is_row_axis_of_the_transpose():
    x = small_inputs(41, 48, 80)
    a = orc.quantize(x, orc.AXIS_COL, orc.SR, orc.GS_ROW, seed=3, stream_id=5)
    b = orc.quantize(np.ascontiguousarray(x.T), orc.AXIS_ROW, orc.SR, orc.GS_ROW, seed=3, stream_id=5)
    assert a.R == 80 and a.K == 48
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.sf, b.sf) and np.array_equal(a.gscale, b.gscale)
    # groups really run down the source columns: scaling one source column changes only that operand row
    y = x.copy()
    y[:, 7] *= 64
    c = orc.quantize(y, orc.AXIS_COL, orc.RTN, orc.GS_ROW)
    d = orc.quantize(x, orc.AXIS_COL, orc.RTN, orc.GS_ROW)
    changed = np.nonzero((c.gscale != d.gscale))[0]
    assert list(changed) == [7]
    assert np.array_equal(np.delete(c.codes, 7, 0), np.delete(d.codes, 7, 0))


def test_zero_groups_and_underflowing_blocks():
    x = np.zeros((3, 256), dtype=np.float32)
    x[1, 5] = 1000.0
    x[1, 40] = 1e-6  # block amax / group amax far below the smallest E4M3 step -> scale 0 -> codes 0
    x[1, 41] = -1e-6
    for mode in (orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128):
        op = orc.quantize(x, orc.AXIS_ROW, orc.SR, mode, seed=1, stream_id=3)
        c = unpack(op.codes)
        assert op.sf[1, 0] == 0x7E and op.sf[1, 2] == 0 and np.all(op.sf[0] == 0) and np.all(op.sf[2] == 0)
        assert c[1, 5] == 7 and c[1, 40] == 0 and c[1, 41] == 8  # sign survives a zero magnitude
        assert np.all(c[0] == 0) and np.all(c[2] == 0)
        if mode == orc.GS_ROW:
            assert op.gscale[0] == 1.0 and op.gscale[2] == 1.0
        if mode == orc.GS_BLOCK128:
            assert op.gscale[1, 1] == 1.0 and op.gscale[0, 0] == 1.0
    z = orc.quantize(np.array([[-0.0] * 16], dtype=np.float32), orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR)
    assert np.all(unpack(z.codes) == 8) and z.gscale[0] == 1.0


def test_sr_is_unbiased_monte_carlo():
    """10^4 independent seeds: the mean of the dequantized draws is within 3 sigma of the input
    (per element |z| < 5 for all, and the z-scores have unit mean square), excluding clamped elements."""
    x = synth.gradients(4, 32, 55, 1e-3)
    n = 10_000
    acc = np.zeros(x.shape, dtype=np.float64)
    base = orc.quantize(x, orc.AXIS_ROW, orc.RTN, orc.GS_ROW)
    step = np.array([[orc.e4m3_value(b) for b in row] for row in base.sf]).repeat(16, axis=1) * base.gscale[:, None]
    for s in range(n):
        op = orc.quantize(x, orc.AXIS_ROW, orc.SR, orc.GS_ROW, seed=s * 7919 + 1, stream_id=3)
        assert np.array_equal(op.sf, base.sf)  # scales do not depend on the rounding mode
        acc += orc.dequantize(op)
    mean = acc / n
    a = np.abs(x.astype(np.float64)) / step
    mags = np.array([float(m) for m in MAGS])
    lo = np.searchsorted(mags, np.minimum(a, 6), side="right") - 1
    q1 = mags[lo]
    q2 = mags[np.minimum(lo + 1, 7)]
    var = (q2 - a) * (a - q1)
    free = (a < 6) & (var > 1e-6)
    sigma = step * np.sqrt(np.maximum(var, 0)) / np.sqrt(n)
    z = (mean - x)[free] / sigma[free]
    assert free.sum() > 80
    assert np.abs(z).max() < 5.0
    assert 0.6 < np.mean(z ** 2) < 1.5
    assert abs(z.mean()) < 4.0 / np.sqrt(free.sum())
    exact = ~free & (a <= 6)
    assert np.allclose(mean[exact], x[exact], rtol=0, atol=1e-12 + 1e-3 * step[exact])


def test_tensor_mode_closed_form_for_the_aligned_tensor():
    """amax of the dequantized tensor equals float32(2688 * S_global): the block holding the maximum has
    scale 448 and magnitude 6."""
    for seed in range(5):
        x = small_inputs(seed, 32, 64)
        op = orc.quantize(x, orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR)
        xh = orc.rematerialize_f32(op)
        assert np.abs(xh).max() == np.float32(2688.0) * op.gscale[0]


def test_rematerialize_is_one_float32_rounding_of_the_exact_product():
    x = small_inputs(3, 8, 48)
    op = orc.quantize(x, orc.AXIS_ROW, orc.RTN, orc.GS_ROW)
    xh = orc.rematerialize_f32(op)
    exact = orc.dequantize(op)[:, :48]  # exact in float64 (<= 6 + 24 significant bits)
    assert np.array_equal(xh, exact.astype(np.float32))
    assert xh.dtype == np.float32
