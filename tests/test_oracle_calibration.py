"""Pins for the calibration oracle (Sec. 4.2: accumulated per-channel l2-norms, top-p % channels): closed forms,
numpy's own norm routine, a brute-force rank count, and recovery of planted outlier channels."""
import numpy as np

from oracle import calibration as cal
from paper_2510_27527_b200 import synth


def test_accumulate_closed_forms_and_library_norm():
    N, D = 37, 9
    X = np.zeros((N, D))
    X[:, 0] = 3.0  # constant column: |c| sqrt(N)
    X[:, 1] = -2.0
    X[5, 2] = 7.0  # one-hot: |v|
    X[:, 3] = np.arange(N)  # sqrt(sum k^2) = sqrt((N-1)N(2N-1)/6)
    acc = cal.accumulate(np.zeros(D), X)
    assert np.isclose(acc[0], 3.0 * np.sqrt(N)) and np.isclose(acc[1], 2.0 * np.sqrt(N))
    assert acc[2] == 7.0 and np.isclose(acc[3], np.sqrt((N - 1) * N * (2 * N - 1) / 6.0)) and acc[4] == 0.0
    rng = np.random.default_rng(0)
    Y = rng.standard_normal((N, D))
    acc2 = cal.accumulate(acc, Y)
    assert np.allclose(acc2 - acc, np.linalg.norm(Y, axis=0))
    # norms add across steps; they are not the norm of the stacked window (pins "accumulate the norms")
    both = cal.accumulate(cal.accumulate(np.zeros(D), Y), 2.0 * Y)
    assert np.allclose(both, 3.0 * np.linalg.norm(Y, axis=0))
    assert not np.allclose(both, np.linalg.norm(np.vstack([Y, 2.0 * Y]), axis=0))


def test_select_against_brute_force_rank_and_ties():
    rng = np.random.default_rng(1)
    acc = rng.integers(0, 6, 40).astype(np.float64)  # many ties
    for n_out in (0, 1, 7, 39, 40):
        outl, keep, cmap = cal.select(acc, n_out)
        # brute force: d is chosen iff fewer than n_out channels beat it (larger value, or equal value and lower index)
        want = [d for d in range(40) if sum(1 for j in range(40) if acc[j] > acc[d] or (acc[j] == acc[d] and j < d)) < n_out]
        assert outl.tolist() == want and len(outl) == n_out
        assert sorted(outl.tolist() + keep.tolist()) == list(range(40))
        assert np.all(np.diff(outl) > 0) and np.all(np.diff(keep) > 0)
        assert np.all(cmap[outl] == -1) and cmap[keep].tolist() == list(range(40 - n_out))
    # every chosen value >= every kept value
    outl, keep, _ = cal.select(acc, 7)
    assert acc[outl].min() >= acc[keep].max()


def test_planted_outlier_channels_are_recovered():
    acc = np.zeros(512)
    truth = None
    for step in range(5):
        X, ch = synth.activations(256, 512, 100 + step, n_outlier=6, factor=30.0, channel_seed=7)
        truth = ch if truth is None else truth
        assert np.array_equal(ch, truth)
        acc = cal.accumulate(acc, X)
    outl, _, _ = cal.select(acc, 6)
    assert outl.tolist() == sorted(truth.tolist())
