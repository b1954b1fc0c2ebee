"""Pins for the oracle's matrix products and for the layer composition (Sec. 2.3, Sec. 4.2): brute-force
triple loops, numpy's matmul as an independent library routine, and inputs built so that every quantizer is
lossless, which makes each of Y, dX, dW an exactly known integer-valued matrix."""
import numpy as np
import pytest

from oracle import nvfp4_oracle as orc
from tests.test_oracle_quantize import canonical


def test_gemm_tn_bruteforce_and_library():
    rng = np.random.default_rng(0)
    for (M, N, K) in [(1, 1, 1), (3, 5, 7), (16, 16, 16), (17, 9, 128)]:
        A = rng.integers(-8, 9, (M, K)).astype(np.float64)
        B = rng.integers(-8, 9, (N, K)).astype(np.float64)
        C = orc.gemm_tn(A, B)
        brute = [[sum(A[m, k] * B[n, k] for k in range(K)) for n in range(N)] for m in range(M)]
        assert np.array_equal(C, np.array(brute))  # integers: exact, order-free
        assert np.array_equal(C, A @ B.T)
    A = rng.standard_normal((33, 200))
    B = rng.standard_normal((21, 200))
    C = orc.gemm_tn(A, B)
    assert np.allclose(C, A @ B.T, rtol=1e-12, atol=1e-12)
    assert C.shape == (33, 21)
    assert not np.allclose(C[:21, :21], (B @ A.T)[:21, :21])  # a transposed-operand mistake would show
    ms = np.array([0, 5, 32, 7])
    ns = np.array([0, 20, 3, 7])
    v, va = orc.gemm_tn_samples(A, B, ms, ns)
    assert np.array_equal(v, C[ms, ns])
    assert np.allclose(va, (np.abs(A[ms]) * np.abs(B[ns])).sum(axis=1))


def test_operand_product_on_hand_example():
    """Two 1x16 operands whose dequantized values are known by hand (Sec. 2.2 last equation)."""
    a = np.zeros((1, 16), dtype=np.float32)
    b = np.zeros((1, 16), dtype=np.float32)
    a[0, :3] = [2688, 1344, -448]  # Sg = 1, Sb = 448, codes 6, 3, -1
    b[0, :3] = [6, 6, 3]  # Sg = 6/2688, Sb = 448 -> values 6, 6, 3 up to the float32 rounding of Sg
    qa = orc.quantize(a)
    qb = orc.quantize(b)
    sgb = np.float32(6.0) / np.float32(2688.0)
    expect = (2688 * 6 + 1344 * 6 - 448 * 3) * (448.0 * float(sgb))
    assert orc.gemm_operands(qa, qb)[0, 0] == pytest.approx(expect, rel=1e-15)


def lossless_layer(N=32, D=64, C=48, seed=0):
    X, _ = canonical(N, D, seed + 1, -3)
    W, _ = canonical(C, D, seed + 2, -9)
    dY, _ = canonical(N, C, seed + 3, -14)
    return X, W, dY


@pytest.mark.parametrize("gs_mode", [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128])
def test_layer_is_exact_on_lossless_inputs(gs_mode):
    X, W, dY = lossless_layer()
    cfg = orc.LayerConfig(gs_mode=gs_mode, seed=3)
    Y, saved = orc.linear_fwd(X, W, cfg)
    X64, W64, dY64 = X.astype(np.float64), W.astype(np.float64), dY.astype(np.float64)
    assert Y.shape == (32, 48) and np.array_equal(Y, X64 @ W64.T)
    dX = orc.linear_bwd_dx(dY, saved, cfg)
    assert dX.shape == (32, 64) and np.array_equal(dX, dY64 @ W64)
    dW = orc.linear_bwd_dw(dY, saved, cfg)
    assert dW.shape == (48, 64) and np.array_equal(dW, dY64.T @ X64)


@pytest.mark.parametrize("outliers", [[5], [0, 1, 17, 63], list(range(3, 64, 7))])
def test_outcontrol_split_is_exact_algebra_on_lossless_inputs(outliers):
    """With lossless quantizers, Y = X_keep W_keep^T + X_out W_out^T is the unsplit product (Sec. 4.2), also
    when the kept columns no longer fill whole 16-blocks; dW columns land at their original positions."""
    X, W, dY = lossless_layer(seed=10)
    # outlier channels may hold arbitrary high-precision values: they never pass a quantizer in fwd / dW
    rng = np.random.default_rng(1)
    X[:, outliers] = rng.integers(-200, 200, (32, len(outliers))).astype(np.float32)
    cfg = orc.LayerConfig(gs_mode=orc.GS_ROW, seed=1, outliers=np.array(outliers))
    Y, saved = orc.linear_fwd(X, W, cfg)
    X64, W64, dY64 = X.astype(np.float64), W.astype(np.float64), dY.astype(np.float64)
    assert np.array_equal(Y, X64 @ W64.T)
    assert saved.qx.K == 64 - len(outliers) and saved.qw.K == 64 - len(outliers)
    dW = orc.linear_bwd_dw(dY, saved, cfg)
    assert np.array_equal(dW, dY64.T @ X64)
    dX = orc.linear_bwd_dx(dY, saved, cfg)  # W's outlier columns are canonical too, so Q4 stays lossless
    assert np.array_equal(dX, dY64 @ W64)


def test_backward_uses_the_aligned_forward_operands():
    """Perturb X and W below the rounding thresholds: forward sees the canonical grid values, and backward must
    re-quantize THOSE (X-hat, W-hat of Sec. 2.3), not the raw inputs."""
    Xc, Wc, dY = lossless_layer(seed=20)
    rng = np.random.default_rng(2)

    def perturb(a):
        p = a * (1 + rng.uniform(-0.01, 0.01, a.shape)).astype(np.float32)
        big = np.abs(a) == np.abs(a).max()
        p[big] = a[big]  # keep the +-6 entries so that every scale is unchanged
        return p.astype(np.float32)

    X, W = perturb(Xc), perturb(Wc)
    assert not np.array_equal(X, Xc)
    cfg = orc.LayerConfig(gs_mode=orc.GS_BLOCK128, seed=7)
    Y, saved = orc.linear_fwd(X, W, cfg)
    Xc64, Wc64, dY64 = Xc.astype(np.float64), Wc.astype(np.float64), dY.astype(np.float64)
    assert np.array_equal(Y, Xc64 @ Wc64.T)
    assert np.array_equal(orc.linear_bwd_dx(dY, saved, cfg), dY64 @ Wc64)
    assert np.array_equal(orc.linear_bwd_dw(dY, saved, cfg), dY64.T @ Xc64)
    assert not np.array_equal(dY64 @ Wc64, dY64 @ W.astype(np.float64))


def test_default_rounding_assignment_and_stream_independence():
    """Forward is deterministic (seed-free); the backward draws differ between seeds and between operands."""
    from paper_2510_27527_b200 import synth

    X, W, dY, _ = synth.layer_inputs(1, 32, 64, 48, n_outlier=2, factor=50.0, grad_scale=1e-3)
    a = orc.LayerConfig(seed=1)
    b = orc.LayerConfig(seed=2)
    assert a.rounding == (orc.RTN, orc.RTN, orc.SR, orc.SR, orc.SR, orc.SR)
    Ya, sa = orc.linear_fwd(X, W, a)
    Yb, sb = orc.linear_fwd(X, W, b)
    assert np.array_equal(Ya, Yb)
    dXa, dXb = orc.linear_bwd_dx(dY, sa, a), orc.linear_bwd_dx(dY, sb, b)
    assert not np.array_equal(dXa, dXb)
    assert np.array_equal(dXa, orc.linear_bwd_dx(dY, sa, a))  # replayable
    # quantized products stay close to the exact ones (a sanity bound, not a precision claim)
    exact = dY.astype(np.float64) @ W.astype(np.float64)
    assert np.linalg.norm(dXa - exact) / np.linalg.norm(exact) < 0.3
    exactY = X.astype(np.float64) @ W.astype(np.float64).T
    assert np.linalg.norm(Ya - exactY) / np.linalg.norm(exactY) < 0.2
