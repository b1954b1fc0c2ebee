"""Pins for the OsciReset oracle (Algorithms 1 and 2): a hand-computed oscillating element, path lengths recomputed in
float64, the paper's claim that a reset leaves the quantized weights unchanged, and the selectivity of the reset."""
import numpy as np
import pytest

from oracle import nvfp4_oracle as orc
from oracle import oscireset as osc
from paper_2510_27527_b200 import synth

MODES = [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128]


def test_bf16_cast_agrees_with_an_independent_implementation_and_ties_go_to_even():
    rng = np.random.default_rng(0)
    w = (rng.standard_normal(4096) * np.exp(rng.uniform(-20, 20, 4096))).astype(np.float32)
    assert np.array_equal(osc.bf16_round(w), synth.round_to_bf16(w))
    # 1 + 2^-8 is exactly between 1 and 1 + 2^-7: even mantissa wins (1.0); 1 + 3*2^-8 -> 1 + 2^-6
    assert osc.bf16_round(np.array([1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8], dtype=np.float32)).tolist() == [1.0, 1.0 + 2.0 ** -6]


@pytest.mark.parametrize("gs_mode", MODES)
def test_hand_computed_oscillating_element(gs_mode):
    """One 16-block whose largest element is 2688: S_global = 1, S_block = 448, so Q(w) = 448 * nearest E2M1 value of
    w / 448. Element 3 alternates between 0.2 * 448 (-> 0) and 0.3 * 448 (-> 0.5 * 448 = 224); element 5 drifts inside
    one bin. After n steps: D_Q[3] = 224 n exactly, D_M[3] ~ 44.8 n, D_Q[5] = 0."""
    base = np.zeros((1, 16), dtype=np.float32)
    base[0, 0] = 2688.0
    base[0, 5] = 448.0 * 1.1
    st = osc.Stats(base.shape)
    lo, hi = np.float32(0.2 * 448), np.float32(0.3 * 448)
    n = 6
    for t in range(n + 1):
        W = base.copy()
        W[0, 3] = lo if t % 2 == 0 else hi
        W[0, 5] += np.float32(0.5 * t)
        osc.update_stats(W, st, t, gs_mode)
    assert st.D_Q[0, 3] == 224.0 * n and st.D_Q[0, 5] == 0.0 and st.D_Q[0, 0] == 0.0
    assert np.isclose(st.D_M[0, 3], float(hi - lo) * n, rtol=1e-6) and np.isclose(st.D_M[0, 5], 0.5 * n, rtol=1e-5)
    assert st.D_M[0, 0] == 0.0
    # risk of element 3 = 224 / 44.8 = 5: reset with tau = 4, not with tau = 6; element 5 (risk 0) and 0 (0/0) never
    W_now = base.copy()
    W_now[0, 3] = lo  # t = n is even
    W_now[0, 5] += np.float32(0.5 * n)
    out, mask = osc.suppress(W_now, st, 4.0, gs_mode)
    assert mask.sum() == 1 and mask[0, 3] and out[0, 3] == 0.0  # bin centre of 0.2 * 448 is 0
    assert np.array_equal(np.delete(out, 3), np.delete(W_now, 3))
    out6, mask6 = osc.suppress(W_now, st, 6.0, gs_mode)
    assert mask6.sum() == 0 and np.array_equal(out6, W_now)


@pytest.mark.parametrize("gs_mode", MODES)
def test_path_lengths_and_reset_invariants_on_a_synthetic_trajectory(gs_mode):
    traj, planted = synth.weight_trajectory(48, 272, 8, seed=3)
    st = osc.Stats(traj[0].shape)
    for t, W in enumerate(traj):
        osc.update_stats(W, st, t, gs_mode)
    # path lengths recomputed in float64 from the definition
    dm = sum(np.abs(traj[t].astype(np.float64) - traj[t - 1]) for t in range(1, len(traj)))
    qs = [osc.quant_dequant(W, gs_mode).astype(np.float64) for W in traj]
    dq = sum(np.abs(qs[t] - qs[t - 1]) for t in range(1, len(traj)))
    assert np.allclose(st.D_M, dm, rtol=1e-5, atol=1e-12) and np.allclose(st.D_Q, dq, rtol=1e-5, atol=1e-12)
    assert np.array_equal(st.W_prev, traj[-1])
    # tau = 8: a small share of the elements (those whose quantized value flipped while the master barely moved)
    out, mask = osc.suppress(traj[-1], st, 8.0, gs_mode)
    assert 0.01 < mask.mean() < 0.2 and np.all(dq[mask] > 0) and np.all(dq[mask] >= 7.99 * dm[mask])
    assert np.all(dq[~mask] <= 8.01 * dm[~mask])
    # only the selected elements change, and they move to their own quantized value
    assert np.array_equal(out[~mask], traj[-1][~mask])
    assert np.array_equal(out[mask], osc.quant_dequant(traj[-1], gs_mode)[mask])
    # the paper's claim: the quantized weights are not affected right after the reset (codes, scales, global scales)
    a = orc.quantize(osc.bf16_round(traj[-1]), orc.AXIS_ROW, orc.RTN, gs_mode)
    b = orc.quantize(osc.bf16_round(out), orc.AXIS_ROW, orc.RTN, gs_mode)
    assert np.array_equal(a.codes, b.codes) and np.array_equal(a.sf, b.sf) and np.array_equal(a.gscale, b.gscale)
    # resetting everything (tau = 0 selects every element that moved) is idempotent under Q as well
    out_all, mask_all = osc.suppress(traj[-1], st, 0.0, gs_mode)
    assert mask_all.mean() > 0.99
    assert np.array_equal(osc.quant_dequant(out_all, gs_mode), osc.quant_dequant(traj[-1], gs_mode))


def test_step_zero_clears_the_statistics():
    traj, _ = synth.weight_trajectory(8, 64, 3, seed=5)
    st = osc.Stats(traj[0].shape)
    for t, W in enumerate(traj):
        osc.update_stats(W, st, t, orc.GS_TENSOR)
    assert st.D_M.any()
    osc.update_stats(traj[1], st, 0, orc.GS_TENSOR)
    assert not st.D_M.any() and not st.D_Q.any() and np.array_equal(st.W_prev, traj[1])


def test_sensitivity_on_a_hand_built_block():
    """S_global = 1, S_block = 448 (largest element 2688): w / 448 = y sits at a known place in its bin.
    y = 0.24 rounds to 0 (bin width 0.5): s = 0.48; y = 2.4 rounds to 2 (width 0.75): s = 0.4 / 0.75;
    y = 3.0 exactly: s = 0; y = 4.9 rounds to 4 (width 1.5): s = 0.6; y = 5.5 rounds to 6 (width 2): s = 0.25."""
    W = np.zeros((1, 16), dtype=np.float32)
    W[0, 0] = 2688.0
    ys = {1: 0.24, 2: 2.4, 3: 3.0, 4: 4.9, 5: 5.5, 6: -1.2}
    for k, y in ys.items():
        W[0, k] = np.float32(y * 448.0)
    s = osc.sensitivity(W, orc.GS_TENSOR)
    yb = {k: float(osc.bf16_round(np.array([W[0, k]]))[0]) / 448.0 for k in ys}  # what the quantizer sees
    assert yb[1] < 0.25 and abs(s[0, 1] - abs(ys[1]) / 0.5) < 2e-3
    assert abs(s[0, 2] - 0.4 / 0.75) < 2e-3 and s[0, 3] == 0.0
    assert abs(s[0, 4] - 0.9 / 1.5) < 2e-3 and abs(s[0, 5] - 0.5 / 2.0) < 2e-3
    assert abs(s[0, 6] - 0.2 / 0.5) < 2e-3 and s[0, 0] == 0.0 and s[0, 7] == 0.0
    # scores never exceed ~2/3 (the wider side of the asymmetric bins of 2 and 4), up to the BF16 cast of the input
    traj, _ = synth.weight_trajectory(32, 256, 0, seed=2)
    for gs in MODES:
        sm = osc.sensitivity(traj[0], gs)
        assert np.all(sm >= 0) and sm.max() < 0.68 and np.all(np.isfinite(sm))


def test_select_tracked_is_top_k_with_index_ties():
    s = np.array([[0.1, 0.5, 0.5, 0.2], [0.5, 0.0, 0.3, 0.5]], dtype=np.float32)
    assert osc.select_tracked(s, 3).tolist() == [1, 2, 4]  # three of the four 0.5 scores, lowest indices
    assert osc.select_tracked(s, 5).tolist() == [1, 2, 4, 6, 7]
    assert osc.select_tracked(s, 0).tolist() == []
    rng = np.random.default_rng(0)
    big = rng.random((7, 33)).astype(np.float32)
    idx = osc.select_tracked(big, 20)
    assert len(idx) == 20 and np.all(np.diff(idx) > 0)
    assert big.reshape(-1)[idx].min() >= np.delete(big.reshape(-1), idx).max()


@pytest.mark.parametrize("gs_mode", MODES)
def test_sparse_statistics_equal_the_dense_ones_on_the_tracked_elements(gs_mode):
    """Algorithm 3 restricted to idx is Algorithm 2 restricted to idx (same snapshots, same sums)."""
    traj, _ = synth.weight_trajectory(24, 144, 6, seed=8)
    dense = osc.Stats(traj[0].shape)
    n_track = 24 * 144 // 10
    sp = osc.SparseStats(n_track)
    for t, W in enumerate(traj):
        osc.update_stats(W, dense, t, gs_mode)
        osc.update_stats_sparse(W, sp, t, gs_mode)
    assert np.array_equal(sp.D_M, dense.D_M.reshape(-1)[sp.idx]) and np.array_equal(sp.D_Q, dense.D_Q.reshape(-1)[sp.idx])
    # the tracked tenth is strongly enriched in the elements that the dense statistics flag at tau = 8 (base rate 0.1)
    _, mask = osc.suppress(traj[-1], dense, 8.0, gs_mode)
    flagged = np.nonzero(mask.reshape(-1))[0]
    assert len(flagged) > 0 and np.isin(flagged, sp.idx).mean() > 0.3
    out_s, hit = osc.suppress_sparse(traj[-1], sp, 8.0, gs_mode)
    out_d, _ = osc.suppress(traj[-1], dense, 8.0, gs_mode)
    changed = np.nonzero((out_s != traj[-1]).reshape(-1))[0]
    assert np.all(np.isin(changed, sp.idx)) and np.array_equal(out_s.reshape(-1)[sp.idx], out_d.reshape(-1)[sp.idx])
