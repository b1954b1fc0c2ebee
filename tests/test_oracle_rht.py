"""Pins for the oracle's random Hadamard transformation (Sec. 4.1): the Hadamard matrix from its textbook definition
(Kronecker powers of H_2, via numpy), orthogonality, the product identity A B^T = (A S H)(B S H)^T, the sign
addressing against the Philox known-answer block, and the layer's backward products staying unbiased."""
import numpy as np
import pytest

from oracle import nvfp4_oracle as orc

H2 = np.array([[1.0, 1.0], [1.0, -1.0]])
# the paper's recursive definition H_2d = H_2 (x) H_d with the 1/sqrt(2) per level collected: (1/sqrt 2)^4 = 1/4
H16 = np.kron(np.kron(H2, H2), np.kron(H2, H2)) / 4.0


def signs(seed, stream, K):
    return np.array([-1.0 if orc.rht_sign_bit(seed, stream, k) else 1.0 for k in range(K)])


def test_matches_the_kronecker_definition_on_integers():
    rng = np.random.default_rng(0)
    x = rng.integers(-64, 65, (5, 48)).astype(np.float32)  # small integers: every float32 sum is exact
    y = orc.rht16(x, seed=9, stream_id=7)
    s = signs(9, 7, 48)
    want = np.concatenate([(x[:, g:g + 16] * s[g:g + 16]) @ H16 for g in range(0, 48, 16)], axis=1)
    assert np.array_equal(y.astype(np.float64), want)
    assert np.allclose(H16 @ H16.T, np.eye(16))
    # unit vectors give the rows of H_16: entries +-1/4, first column all +
    e = np.eye(16, dtype=np.float32)
    rows = orc.rht16(e, seed=0, stream_id=99) * signs(0, 99, 16)[:, None]
    assert np.array_equal(np.abs(rows), np.full((16, 16), 0.25)) and np.all(rows[:, 0] > 0)


def test_sign_addressing_uses_the_published_philox_block():
    # counter (0, 0, stream, 0x5348), key (seed lo, seed hi): bits of the four words, LSB first
    w = orc.philox4x32_10([0, 0, 7, 0x5348], [123, 0])
    for k in (0, 1, 31, 32, 77, 127):
        assert orc.rht_sign_bit(123, 7, k) == (int(w[k // 32]) >> (k % 32)) & 1
    w2 = orc.philox4x32_10([3, 0, 7, 0x5348], [123, 0])
    assert orc.rht_sign_bit(123, 7, 3 * 128 + 5) == (int(w2[0]) >> 5) & 1
    s = signs(5, 8, 512)
    assert 0.35 < (s < 0).mean() < 0.65
    assert not np.array_equal(s, signs(5, 7, 512)) and not np.array_equal(s, signs(6, 8, 512))


def test_product_identity_is_exact_on_integers_and_padding_is_zero_extension():
    rng = np.random.default_rng(1)
    A = rng.integers(-8, 9, (7, 40)).astype(np.float32)
    B = rng.integers(-8, 9, (5, 40)).astype(np.float32)
    A2, B2 = orc.rht16(A, 3, 7), orc.rht16(B, 3, 7)
    assert A2.shape == (7, 48)
    assert np.array_equal(orc.gemm_tn(A2, B2), orc.gemm_tn(A, B))  # (A S H)(B S H)^T = A B^T
    # different sign diagonals on the two operands break the identity
    assert not np.array_equal(orc.gemm_tn(A2, orc.rht16(B, 3, 8)), orc.gemm_tn(A, B))
    # energy is preserved (orthogonal transform)
    assert np.allclose((A2.astype(np.float64) ** 2).sum(axis=1), (A.astype(np.float64) ** 2).sum(axis=1))


def test_general_inputs_are_within_float32_rounding_of_the_exact_transform():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((9, 64)).astype(np.float32) * np.exp(rng.uniform(-5, 5, (9, 64))).astype(np.float32)
    y = orc.rht16(x, 11, 8)
    s = signs(11, 8, 64)
    want = np.concatenate([(x[:, g:g + 16].astype(np.float64) * s[g:g + 16]) @ H16 for g in range(0, 64, 16)], axis=1)
    scale = np.abs(x).reshape(9, 4, 16).sum(axis=2).repeat(16, axis=1)
    assert np.all(np.abs(y - want) <= 4 * 2.0 ** -24 * scale + 1e-30)


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_BLOCK128])
def test_backward_products_with_rht_stay_unbiased(gs_mode):
    """Averaged over seeds, dX and dW approach dY W-hat and dY^T X-hat: both operands of each product must carry the
    same S H (a transform on one side only, or different signs, would leave an O(1) error)."""
    from paper_2510_27527_b200 import synth

    X, W, dY, _ = synth.layer_inputs(1, 64, 128, 96, n_outlier=2, factor=30.0, grad_scale=1e-3)
    cfg0 = orc.LayerConfig(gs_mode=gs_mode, seed=0, rht=True)
    _, saved = orc.linear_fwd(X, W, cfg0)
    Wh = orc.rematerialize_f32(saved.qw).astype(np.float64)
    Xh = orc.rematerialize_f32(saved.qx).astype(np.float64)
    exact_dx, exact_dw = dY.astype(np.float64) @ Wh, dY.astype(np.float64).T @ Xh
    n = 48
    acc_dx, acc_dw = np.zeros_like(exact_dx), np.zeros_like(exact_dw)
    one = None
    for sd in range(n):
        cfg = orc.LayerConfig(gs_mode=gs_mode, seed=1000 + sd, rht=True)
        dx, dw = orc.linear_bwd_dx(dY, saved, cfg), orc.linear_bwd_dw(dY, saved, cfg)
        one = one if one is not None else (dx, dw)
        acc_dx += dx
        acc_dw += dw
    rel = lambda a, b: np.linalg.norm(a - b) / np.linalg.norm(b)
    e1_dx, e1_dw = rel(one[0], exact_dx), rel(one[1], exact_dw)
    en_dx, en_dw = rel(acc_dx / n, exact_dx), rel(acc_dw / n, exact_dw)
    assert e1_dx < 0.5 and e1_dw < 0.5
    # the error of the mean shrinks like 1/sqrt(n) (up to the small clamp bias): at least 3.5x for n = 48
    assert en_dx < e1_dx / 3.5 and en_dw < e1_dw / 3.5
