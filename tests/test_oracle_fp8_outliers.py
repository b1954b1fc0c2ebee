"""Pins for the FP8 outlier-channel option (oracle/fp8_outliers.py). The recipe is this build's own (the paper names FP8 as
the outlier compute type, Sec. 4.2 and its hyper-parameter table, without a recipe): the pins fix the definition against
the E4M3 value table, exact rational arithmetic and torch's E4M3 cast."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import fp8_outliers as f8
from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth


def test_scale_exponent_is_the_smallest_power_of_two_that_fits():
    rng = np.random.default_rng(3)
    vals = list(np.exp(rng.uniform(np.log(1e-6), np.log(1e6), 300)).astype(np.float32))
    vals += [448.0, 448.0 * 2, 448.0 / 4, np.nextafter(np.float32(448), np.float32(1e9)), np.nextafter(np.float32(448), np.float32(0)),
             1.0, 3.5, 7.0, 2.0 ** -20, 1.75 * 2.0 ** 13]
    for a in vals:
        e = f8.scale_exponent(float(a))
        fa = Fraction(float(a))
        assert fa / Fraction(2) ** e <= 448
        assert fa / Fraction(2) ** (e - 1) > 448
    assert f8.scale_exponent(0.0) == 0
    assert f8.scale_exponent(448.0) == 0 and f8.scale_exponent(449.0) == 1 and f8.scale_exponent(224.0) == -1


def test_e4m3_round_matches_the_table_and_torch():
    tab = [orc.e4m3_value(b) for b in range(0x7F)]
    # grid values are fixed points, midpoints go to the even byte, everything beyond 448 saturates
    g = np.array(tab)
    assert np.array_equal(f8.e4m3_round(g), g) and np.array_equal(f8.e4m3_round(-g), -g)
    for b in range(0x7E):
        mid = (tab[b] + tab[b + 1]) / 2
        want = tab[b] if b % 2 == 0 else tab[b + 1]
        assert f8.e4m3_round(np.array([mid]))[0] == want, b
        assert f8.e4m3_round(np.array([np.nextafter(mid, 1e9)]))[0] == tab[b + 1]
        assert f8.e4m3_round(np.array([np.nextafter(mid, -1e9)]))[0] == tab[b]
    assert f8.e4m3_round(np.array([1e9, -500.0]))[0] == 448.0 and f8.e4m3_round(np.array([1e9, -500.0]))[1] == -448.0
    # torch's own cast (round to nearest even) on in-range values
    rng = np.random.default_rng(9)
    y = (rng.standard_normal(20000) * np.exp(rng.uniform(-8, 6, 20000))).astype(np.float32)
    y = y[np.abs(y) <= 448]
    want = torch.from_numpy(y).to(torch.float8_e4m3fn).to(torch.float32).numpy()
    assert np.array_equal(f8.e4m3_round(y.astype(np.float64)).astype(np.float32), want)


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_snap_properties(seed):
    x, _ = synth.activations(64, 24, seed, n_outlier=3, factor=50.0)
    x = x * np.float32(10.0 ** (seed - 2))
    t8, e = f8.snap(x)
    # the largest element lands inside (224, 448] on the grid, nothing saturates
    assert 224 < np.abs(x).max() / 2.0 ** e <= 448
    # idempotent, BF16-exact, sign- and zero-preserving
    assert np.array_equal(f8.snap(t8)[0], t8)
    bits = t8.view(np.uint32)
    assert np.all((bits & 0xFFFF) == 0)
    assert np.array_equal(np.signbit(t8[t8 != 0]), np.signbit(x[t8 != 0])) and np.all(t8[x == 0] == 0)
    # relative error of a normal E4M3 value is at most 2^-4; below the normal range the step is 2^-9 of the scaled grid
    y = np.abs(x.astype(np.float64)) / 2.0 ** e
    err = np.abs(t8.astype(np.float64) - x) / 2.0 ** e
    normal = y >= 2.0 ** -6
    assert np.all(err[normal] <= y[normal] * 2.0 ** -4 * (1 + 1e-12))
    assert np.all(err[~normal] <= 2.0 ** -10 * (1 + 1e-12))
    # same thing through torch's cast
    want = (torch.from_numpy((x.astype(np.float64) / 2.0 ** e).astype(np.float32)).to(torch.float8_e4m3fn).to(torch.float32).numpy()
            * np.float32(2.0 ** e))
    assert np.array_equal(t8, want)
    assert f8.snap(np.zeros((4, 4), dtype=np.float32))[1] == 0


def test_layer_uses_the_snapped_slices_everywhere():
    """With outlier_fp8 the layer equals the BF16-outlier layer run on inputs whose outlier columns were snapped first."""
    X, W, dY, ch = synth.layer_inputs(5, 96, 80, 48, n_outlier=5, factor=40.0, grad_scale=1e-3)
    cfg8 = orc.LayerConfig(gs_mode=orc.GS_ROW, seed=4, outliers=ch, outlier_fp8=True)
    cfg16 = orc.LayerConfig(gs_mode=orc.GS_ROW, seed=4, outliers=ch)
    Xs, Ws = X.copy(), W.copy()
    Xs[:, ch], Ws[:, ch] = f8.snap(X[:, ch])[0], f8.snap(W[:, ch])[0]
    Y8, s8 = orc.linear_fwd(X, W, cfg8)
    Y16, s16 = orc.linear_fwd(Xs, Ws, cfg16)
    assert np.array_equal(Y8, Y16)
    assert np.array_equal(orc.linear_bwd_dx(dY, s8, cfg8), orc.linear_bwd_dx(dY, s16, cfg16))
    assert np.array_equal(orc.linear_bwd_dw(dY, s8, cfg8), orc.linear_bwd_dw(dY, s16, cfg16))
    # and it differs from keeping the outliers in BF16
    Yb, _ = orc.linear_fwd(X, W, cfg16)
    assert not np.array_equal(Y8, Yb)
