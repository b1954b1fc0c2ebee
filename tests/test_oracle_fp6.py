"""Pins for the oracle of the simulated FP6 x FP4 layer (paper Sec. 5.4, "Precision Switching in Final Stage"; the FP6
recipe is this build's own definition, see oracle/fp6_sim.py): the E2M3 value table against the format's defining facts and
against an independent library type, both rounding rules against exact rational arithmetic, every scale and code of whole
operands re-derived with fractions, invariants of the quantizer, and the three products on lossless inputs."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import fp6_sim as f6
from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.test_oracle_quantize import canonical

E4M3 = [orc.e4m3_value(b) for b in range(127)]


def test_e2m3_table_against_the_format_and_a_library_type():
    m = [f6.e2m3_value(c) for c in range(32)]
    assert m[0] == 0 and m[1] == 0.125 and m[7] == 0.875  # subnormals: multiples of 1/8
    assert m[8] == 1.0 and m[31] == 7.5                   # smallest normal, largest value
    assert all(b > a for a, b in zip(m, m[1:]))
    steps = sorted(set(b - a for a, b in zip(m, m[1:])))
    assert steps == [0.125, 0.25, 0.5]
    e2m1 = [orc.e2m1_value(c) for c in range(8)]
    assert set(e2m1) <= set(m)  # two more mantissa bits: every FP4 value is an FP6 value
    ml = pytest.importorskip("ml_dtypes")
    lib_vals = sorted(set(abs(float(v)) for v in np.arange(64, dtype=np.uint8).view(ml.float6_e2m3fn)))
    assert lib_vals == m


def exact_nearest(a: Fraction):
    best = min(range(32), key=lambda c: (abs(Fraction(f6.e2m3_value(c)) - a), c % 2))  # nearest, then the even code
    return best


def test_round_to_nearest_against_exact_fractions_and_the_library_cast():
    rng = np.random.default_rng(1)
    vals = list(rng.uniform(0, 7.5, 400).astype(np.float32).astype(np.float64))
    mids = [(f6.e2m3_value(c) + f6.e2m3_value(c + 1)) / 2 for c in range(31)]
    vals += mids + [float(np.nextafter(np.float32(v), np.float32(0))) for v in mids] + [float(np.nextafter(np.float32(v), np.float32(9))) for v in mids] + [0.0, 7.5]
    got = f6.round_rtn_mag(np.array(vals))
    for v, g in zip(vals, got):
        assert int(g) == exact_nearest(Fraction(v)), v
    for c in range(31):  # all 31 ties go to the even code
        assert int(f6.round_rtn_mag(np.array([mids[c]]))[0]) == (c if c % 2 == 0 else c + 1)
    ml = pytest.importorskip("ml_dtypes")
    cast = np.array(vals, dtype=np.float32).astype(ml.float6_e2m3fn).astype(np.float32)
    assert np.array_equal(cast, f6.MAGS[got].astype(np.float32))


def test_stochastic_rounding_rule_exhaustively_over_the_draws():
    u = np.arange(65536, dtype=np.uint32)
    for a in [0.0, 0.01, 0.124, 0.126, 0.99, 1.0, 1.3, 2.1, 3.9, 4.0, 5.3, 7.49, 7.5]:
        codes = f6.round_sr_mag(np.full(65536, a), u)
        lo = max(c for c in range(32) if f6.e2m3_value(c) <= a)
        hi = min(lo + 1, 31)
        assert set(np.unique(codes)) <= {lo, hi}
        q1, q2 = Fraction(f6.e2m3_value(lo)), Fraction(f6.e2m3_value(hi))
        frac = (Fraction(a) - q1) / (q2 - q1) if hi > lo else Fraction(0)
        ups = int((codes == hi).sum()) if hi > lo else 0
        expect = sum(1 for k in (0, 1, 2, 65535) if Fraction(2 * k + 1, 131072) < frac)  # spot check of the rule itself
        assert sum(1 for k in (0, 1, 2, 65535) if codes[k] == hi and hi > lo) == expect
        assert abs(Fraction(ups, 65536) - frac) <= Fraction(1, 131072)  # P(up) = frac up to the 16-bit grid


def rederive(x, op, rounding, seed, stream_id):
    """Every scale and code of an operand from exact rational arithmetic on the float32 inputs (independent of the oracle's
    float code path except for the E4M3 value table and the Philox draws, which have pins of their own)."""
    R, K = x.shape
    f32 = np.float32
    for r in range(R):
        if op.gs_mode == orc.GS_TENSOR:
            amax_g = np.max(np.abs(x))
            Sg = op.gscale[0]
        else:
            amax_g = np.max(np.abs(x[r]))
            Sg = op.gscale[r]
        assert Sg == (f32(1) if amax_g == 0 else f32(f32(amax_g) / f32(3360)))
        for b in range(op.K16 // 16):
            blk = np.zeros(16, dtype=np.float32)
            n = max(0, min(16, K - 16 * b))
            blk[:n] = x[r, 16 * b:16 * b + n]
            s = f32(f32(np.max(np.abs(blk)) / Sg) / f32(7.5))
            # nearest E4M3 value of s (exact fractions; ties to the even byte; 448 the ceiling)
            sb = min(range(127), key=lambda c: (abs(Fraction(E4M3[c]) - Fraction(float(s))), c % 2))
            assert op.sf[r, b] == sb
            d = f32(Sg * f32(E4M3[sb]))
            rcp = f32(0) if sb == 0 else f32(f32(1) / d)
            for i in range(16):
                y = f32(blk[i] * rcp)
                a = min(Fraction(float(abs(y))), Fraction(15, 2))
                if rounding == orc.RTN:
                    want = exact_nearest(a)
                else:
                    lo = max(c for c in range(32) if Fraction(f6.e2m3_value(c)) <= a)
                    hi = min(lo + 1, 31)
                    u = orc.sr_bits(seed, stream_id, r * op.K16 + 16 * b + i)
                    up = hi > lo and Fraction(2 * u + 1, 131072) < (a - Fraction(f6.e2m3_value(lo))) / Fraction(f6.e2m3_value(hi) - f6.e2m3_value(lo))
                    want = hi if up else lo
                assert (op.codes[r, 16 * b + i] & 31) == want
                assert (op.codes[r, 16 * b + i] >> 5) == int(np.signbit(blk[i]))


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_ROW])
@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR])
def test_every_scale_and_code_rederived_exactly(gs_mode, rounding):
    x = synth.gradients(5, 40, 77, 1e-3)
    x[2, :] = 0  # an all-zero row: global scale 1 in ROW mode, zero block scales
    op = f6.quantize(x, orc.AXIS_ROW, rounding, gs_mode, seed=11, stream_id=3)
    assert op.codes.shape == (5, 48) and op.sf.shape == (5, 3)
    rederive(x, op, rounding, 11, 3)
    assert np.all(op.codes[:, 40:] == 0) and np.all(f6.block_values(op)[2] == 0)


def canonical6(R, K, seed, scale_exp=-3):
    """Lossless inputs of the FP6 quantizer: E2M3 grid values times 448 * 2^e, a +-7.5 in every 16-block of rows and columns."""
    rng = np.random.default_rng(seed)
    q = f6.MAGS[rng.integers(0, 32, (R, K))] * rng.choice([-1.0, 1.0], (R, K))
    i, j = np.meshgrid(np.arange(R), np.arange(K), indexing="ij")
    top = (i + j) % 2 == 0
    q[top] = 7.5 * rng.choice([-1.0, 1.0], (R, K))[top]
    return (q * 448.0 * 2.0 ** scale_exp).astype(np.float32), q


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_ROW])
@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR])
@pytest.mark.parametrize("axis", [orc.AXIS_ROW, orc.AXIS_COL])
def test_idempotent_on_lossless_inputs(gs_mode, rounding, axis):
    x, q = canonical6(32, 80, 5)
    assert np.array_equal(synth.round_to_bf16(x), x)  # 8 significant bits: BF16 inputs
    op = f6.quantize(x, axis, rounding, gs_mode, seed=9, stream_id=6)
    xt = x if axis == orc.AXIS_ROW else x.T
    assert np.all(op.gscale == 2.0 ** -3) and np.all(op.sf == 0x7E)
    assert np.array_equal(f6.dequantize(op)[:, : xt.shape[1]], xt.astype(np.float64))
    assert np.array_equal(f6.rematerialize_f32(op), xt)
    assert np.array_equal(synth.round_to_bf16(f6.block_values(op)), f6.block_values(op))  # P * S_block fits BF16


def test_invariants_error_bound_and_unbiasedness():
    x, _ = synth.activations(24, 96, 31, n_outlier=2, factor=30.0)
    for gs_mode in (orc.GS_TENSOR, orc.GS_ROW):
        op = f6.quantize(x, orc.AXIS_ROW, orc.RTN, gs_mode)
        assert (op.sf == 0x7E).any(axis=1).all() if gs_mode == orc.GS_ROW else (op.sf == 0x7E).any()
        assert (op.codes & 31).max() >= 30  # the largest element lands on 7 or 7.5
        deq = f6.dequantize(op)[:, :96]
        step = np.repeat(np.array([orc.e4m3_value(int(b)) for b in op.sf.ravel()]).reshape(op.sf.shape), 16, axis=1)[:, :96]
        g = (op.gscale[0] if gs_mode == orc.GS_TENSOR else op.gscale[:, None]).astype(np.float64)
        # half of the widest cell (0.5) inside the grid; elements beyond 7.5 (block scale rounded down) lose at most 7 %
        inside = np.abs(x) <= 7.5 * step * g
        assert np.all(np.abs(x - deq)[inside] <= 0.25 * (step * g * np.ones_like(deq))[inside] * (1 + 1e-6))
    # the FP6 grid refines the FP4 grid: with the same input the FP6 error is smaller on average
    e6 = np.abs(x - f6.dequantize(f6.quantize(x))[:, :96]).mean()
    e4 = np.abs(x - orc.dequantize(orc.quantize(x))[:, :96]).mean()
    assert e6 < 0.5 * e4
    # stochastic rounding: the mean over seeds approaches the input (elements inside the grid)
    xs = synth.gradients(4, 32, 3, 1e-3)
    acc = np.zeros((4, 32))
    n = 400
    for seed in range(n):
        acc += f6.dequantize(f6.quantize(xs, orc.AXIS_ROW, orc.SR, orc.GS_ROW, seed=seed, stream_id=3))[:, :32]
    one = f6.quantize(xs, orc.AXIS_ROW, orc.RTN, orc.GS_ROW)
    cell = 0.5 * np.repeat(np.array([orc.e4m3_value(int(b)) for b in one.sf.ravel()]).reshape(one.sf.shape), 16, axis=1) * one.gscale[:, None]
    inside = np.abs(xs) <= 7.5 * 2 * cell
    assert np.all(np.abs(acc / n - xs)[inside] <= 3.0 * cell[inside] / np.sqrt(n) + 1e-12)


def test_column_axis_is_row_axis_of_the_transpose():
    x = synth.gradients(40, 24, 8, 1e-2)
    a = f6.quantize(x, orc.AXIS_COL, orc.SR, orc.GS_ROW, seed=3, stream_id=6)
    b = f6.quantize(np.ascontiguousarray(x.T), orc.AXIS_ROW, orc.SR, orc.GS_ROW, seed=3, stream_id=6)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.sf, b.sf) and np.array_equal(a.gscale, b.gscale)


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_ROW])
def test_the_three_products_are_exact_on_lossless_inputs(gs_mode):
    """X on the FP6 grid, W on the FP4 grid; the gradient on the FP6 grid for dX and on the FP4 grid for dW (the formulas
    quantize it to FP6 in one product and to FP4 in the other). Every quantizer is then lossless and each product an
    exactly known matrix: this pins which operand is quantized how, along which axis, and that backward reads X-hat / W-hat."""
    X, _ = canonical6(32, 64, 1, -3)
    W, _ = canonical(48, 64, 2, -9)
    dY6, _ = canonical6(32, 48, 3, -14)
    dY4, _ = canonical(32, 48, 4, -14)
    Y, saved = f6.linear_fwd(X, W, gs_mode)
    assert Y.shape == (32, 48) and np.array_equal(Y, X.astype(np.float64) @ W.astype(np.float64).T)
    dX, q3, q4 = f6.linear_bwd_dx(dY6, saved, seed=5, gs_mode=gs_mode)
    assert dX.shape == (32, 64) and np.array_equal(dX, dY6.astype(np.float64) @ W.astype(np.float64))
    assert isinstance(q3, f6.Fp6Operand) and isinstance(q4, orc.Operand) and (q4.R, q4.K) == (64, 48)
    dW, q5, q6 = f6.linear_bwd_dw(dY4, saved, seed=5, gs_mode=gs_mode)
    assert dW.shape == (48, 64) and np.array_equal(dW, dY4.astype(np.float64).T @ X.astype(np.float64))
    assert isinstance(q5, orc.Operand) and isinstance(q6, f6.Fp6Operand) and (q6.R, q6.K) == (64, 32)
    # a gradient that is NOT on the FP4 grid makes dW differ from the unquantized product, while dX (FP6) stays exact
    dWx, _, _ = f6.linear_bwd_dw(dY6, saved, seed=5, gs_mode=gs_mode)
    assert not np.array_equal(dWx, dY6.astype(np.float64).T @ X.astype(np.float64))
