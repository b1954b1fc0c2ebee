"""Pins for the 16x16 weight-block recipe (oracle/w16x16.py): the comparison recipe of the paper's weight-block ablation
(Sec. 2.3, third difference; appendix on the overhead of the 1x16 weight scaling)."""
from fractions import Fraction

import numpy as np
import pytest

from oracle import nvfp4_oracle as orc
from oracle import w16x16
from paper_2510_27527_b200 import synth

MAGS = [Fraction(v) for v in (0, 0.5, 1, 1.5, 2, 3, 4, 6)]


def unpack(codes):
    out = np.empty((codes.shape[0], codes.shape[1] * 2), dtype=np.uint8)
    out[:, 0::2] = codes & 15
    out[:, 1::2] = codes >> 4
    return out


def test_array_rounding_is_the_scalar_rounding():
    a = np.concatenate([np.linspace(0, 6, 4801), np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]),
                        np.nextafter(np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]), 10),
                        np.nextafter(np.array([0.25, 0.75, 1.25, 1.75, 2.5, 3.5, 5.0]), -10)])
    want = np.array([orc.round_rtn_mag(float(np.float32(v))) for v in a])
    assert np.array_equal(w16x16.rtn_mag(a.astype(np.float32).astype(np.float64)), want)


@pytest.mark.parametrize("shape", [(16, 16), (48, 80), (40, 72), (17, 33)])
def test_scales_and_codes_in_exact_arithmetic(shape):
    W = synth.weights(shape[0], shape[1], 5 + shape[1]) * np.float32(3.0)
    W[3 % shape[0], 5 % shape[1]] *= np.float32(40.0)  # one dominant square
    op = w16x16.quantize(W)
    C, D = shape
    assert op.codes.shape == (C, (D + 15) // 16 * 8) and op.sf.shape == (C, (D + 15) // 16)
    tab = [Fraction(orc.e4m3_value(b)) for b in range(0x7F)]
    Sg = Fraction(float(op.gscale[0]))
    assert op.gscale[0] == np.float32(np.abs(W).max() / np.float32(2688.0))
    codes = unpack(op.codes)
    eps = Fraction(1, 2 ** 20)
    checked = 0
    for r0 in range(0, C, 16):
        for b in range((D + 15) // 16):
            blk = W[r0:r0 + 16, 16 * b:16 * b + 16]
            sb = int(op.sf[r0, b])
            assert np.all(op.sf[r0:r0 + 16, b] == sb)  # the rows of a square repeat its scale
            amax_b = max(abs(Fraction(float(v))) for v in blk.reshape(-1))
            s_exact = amax_b / Sg / 6
            lo = max(i for i, v in enumerate(tab) if v <= s_exact)
            if lo < 0x7E:
                mid = (tab[lo] + tab[lo + 1]) / 2
                if abs(s_exact - mid) > mid * eps:
                    assert sb == (lo if s_exact < mid else lo + 1)
            Sb = tab[sb]
            for (i, j), w in np.ndenumerate(blk):
                code = int(codes[r0 + i, 16 * b + j])
                assert (code >> 3) == int(np.signbit(w))
                if Sb == 0:
                    assert code & 7 == 0
                    continue
                a = min(abs(Fraction(float(w))) / (Sg * Sb), Fraction(6))
                errs = sorted(range(8), key=lambda q: abs(a - MAGS[q]))
                if abs(a - MAGS[errs[1]]) - abs(a - MAGS[errs[0]]) > eps * 8:
                    assert code & 7 == errs[0]
                    checked += 1
    assert checked > 0.9 * C * D
    # the square that holds the tensor maximum has scale 448 and a magnitude-6 element
    assert op.sf.max() == 0x7E and (codes & 7).max() == 7
    if D % 16:
        assert np.all(codes[:, D:] == 0)


def test_reduces_to_the_1x16_quantizer_when_the_rows_of_a_square_agree():
    base = synth.weights(4, 96, 11)
    W = np.repeat(base, 16, axis=0)  # 64 x 96: every 16-row group holds one row 16 times
    a, b = w16x16.quantize(W), orc.quantize(W, orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.sf, b.sf) and np.array_equal(a.gscale, b.gscale)


@pytest.mark.parametrize("shape", [(32, 48), (48, 16), (40, 72), (17, 33)])
def test_transposing_the_operand_is_quantizing_the_transpose(shape):
    W = synth.weights(shape[0], shape[1], 31 + shape[0])
    q = w16x16.quantize(W)
    t = w16x16.transpose_operand(q)
    qt = w16x16.quantize(np.ascontiguousarray(W.T))
    assert t.R == shape[1] and t.K == shape[0]
    assert np.array_equal(t.codes, qt.codes) and np.array_equal(t.sf, qt.sf) and np.array_equal(t.gscale, qt.gscale)
    assert np.array_equal(orc.dequantize(t)[:, : shape[0]], orc.dequantize(q)[:, : shape[1]].T)


def test_layer_backward_uses_the_forward_codes_without_requantization():
    X, W, dY, _ = synth.layer_inputs(8, 96, 80, 48, n_outlier=0, factor=1.0, grad_scale=1e-3)
    cfg = orc.LayerConfig(gs_mode=orc.GS_TENSOR, seed=6, w_block16=True, rht=True)
    Y, saved = orc.linear_fwd(X, W, cfg)
    W_hat = orc.dequantize(saved.qw)[:, :80]
    assert np.allclose(Y, orc.dequantize(saved.qx)[:, :80] @ W_hat.T, rtol=1e-12, atol=1e-300)
    q3 = orc.quantize(dY, orc.AXIS_ROW, orc.SR, orc.GS_TENSOR, 6, orc.STREAM_Q3)
    dX = orc.linear_bwd_dx(dY, saved, cfg)
    assert np.allclose(dX, orc.dequantize(q3)[:, :48] @ W_hat, rtol=1e-11, atol=1e-300)
    # the recipe is coarser than 1x16 blocks on the same weights
    e16 = np.linalg.norm(W_hat - W)
    e1 = np.linalg.norm(orc.dequantize(orc.quantize(W, orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR))[:, :80] - W)
    assert e16 > e1
