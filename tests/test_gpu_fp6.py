"""GPU parity of the simulated FP6 x FP4 products (paper Sec. 5.4, "Precision Switching in Final Stage") against the oracle
(oracle/fp6_sim.py), through the C ABI: the dense operands P * S_block and the global scales bit for bit (stochastic
rounding included, same seed), the products element by element within 1e-3 of the FP64 sums of the same dequantized
operands."""
import numpy as np
import pytest
import torch

from oracle import fp6_sim as f6
from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.gpu_util import assert_operand_equal, bf16_ulp_close, rel_fro, to_dev_bf16

pytestmark = pytest.mark.gpu


def B():
    from paper_2510_27527_b200 import binding

    return binding


def dense_values(d):
    """Device dense operand -> (float32 [R, ld] values, float32 global scale)."""
    torch.cuda.synchronize()
    return d.vals.float().cpu().numpy(), float(d.gscale.cpu().numpy()[0])


def assert_dense_equal(d, ref, what, values):
    vals, g = dense_values(d)
    want = values(ref)  # float32 [R, K16]
    assert d.R == ref.R and d.K == ref.K and vals.shape[1] % 64 == 0 and vals.shape[1] >= want.shape[1]
    assert np.float32(g) == ref.gscale[0], f"{what}: global scale {g} != {ref.gscale[0]}"
    bad = np.argwhere(vals[:, : want.shape[1]] != want)
    assert bad.size == 0, f"{what}: {len(bad)} values differ, first at {bad[0]}: {vals[tuple(bad[0])]} != {want[tuple(bad[0])]}"
    assert np.all(vals[:, want.shape[1]:] == 0), f"{what}: padding columns are not zero"
    # the sign of a zero magnitude is the input's sign, as in the oracle
    assert np.array_equal(np.signbit(vals[:, : want.shape[1]]), np.signbit(want)), f"{what}: signs of zeros differ"


@pytest.mark.parametrize("shape", [(1, 16), (5, 40), (130, 272), (64, 1000), (300, 64)])
@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR])
def test_fp6_row_quantizer_bit_exact(shape, rounding):
    b = B()
    x = synth.gradients(shape[0], shape[1], 50 + shape[1], 1e-3) if rounding == orc.SR else synth.activations(
        shape[0], shape[1], 50 + shape[1], n_outlier=min(2, shape[1] // 8), factor=40.0)[0]
    ref = f6.quantize(x, orc.AXIS_ROW, rounding, orc.GS_TENSOR, seed=4242, stream_id=3)
    cols8 = (shape[1] + 7) // 8 * 8
    full = np.zeros((shape[0], cols8), dtype=np.float32)
    full[:, : shape[1]] = x
    src = to_dev_bf16(full)[:, : shape[1]]
    out = b.alloc_dense(shape[0], shape[1], poison=True)
    b.nvfp4_fp6_quantize(src, rounding, 4242, 3, out=out)
    assert_dense_equal(out, ref, f"fp6 rows {shape} r{rounding}", f6.block_values)


@pytest.mark.parametrize("shape", [(16, 4), (200, 72), (130, 272), (1000, 36)])
@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR])
def test_fp6_transposing_requantizer_bit_exact(shape, rounding):
    """Q6_S(X-hat^T): the dense forward operand of X, re-quantized along the tokens."""
    b = B()
    x, _ = synth.activations(shape[0], shape[1], 9 + shape[0], n_outlier=1, factor=30.0)
    fwd_ref = f6.quantize(x, orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR, stream_id=1)
    ref = f6.quantize(f6.rematerialize_f32(fwd_ref), orc.AXIS_COL, rounding, orc.GS_TENSOR, seed=77, stream_id=6)
    cols8 = (shape[1] + 7) // 8 * 8  # rows of the source start on 16-byte boundaries
    full = np.zeros((shape[0], cols8), dtype=np.float32)
    full[:, : shape[1]] = x
    fwd = b.nvfp4_fp6_quantize(to_dev_bf16(full)[:, : shape[1]], orc.RTN, 0, 1)
    assert_dense_equal(fwd, fwd_ref, "forward operand", f6.block_values)
    out = b.alloc_dense(shape[1], shape[0], poison=True)
    b.nvfp4_fp6_requantize_t(fwd, rounding, 77, 6, out=out)
    assert_dense_equal(out, ref, f"fp6 requantize_t {shape} r{rounding}", f6.block_values)


@pytest.mark.parametrize("layout", [0, 1])
def test_expanded_fp4_operand_is_p_times_block_scale(layout):
    b = B()
    x, _ = synth.activations(130, 200, 3, n_outlier=2, factor=50.0)
    ref = orc.quantize(x, orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR)
    q = b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_ROW, b.ROUND_RTN, 0, 1, b.GS_TENSOR, layout)
    assert_operand_equal(q, ref, "fp4 operand")
    d = b.alloc_dense(130, 200, poison=True)
    b.nvfp4_expand_operand(q, out=d)
    assert_dense_equal(d, ref, "expanded FP4 operand", f6.fp4_block_values)


def check_product(got: torch.Tensor, A64, B64, bf16_out, what):
    torch.cuda.synchronize()
    want = orc.gemm_tn(A64, B64)
    absdot = np.abs(A64) @ np.abs(B64).T
    g = got.float().cpu().numpy().astype(np.float64)
    assert g.shape == want.shape
    if bf16_out:
        assert np.all(bf16_ulp_close(g, want, 1.0, 1e-5 * absdot)), what
    else:
        assert np.all(np.abs(g - want) <= 1e-3 * absdot + 1e-30), what
        assert rel_fro(g, want) <= 1e-5, what


@pytest.mark.parametrize("shape", [(32, 64, 48), (256, 512, 384), (300, 200, 136), (1100, 136, 264)])
def test_simulated_layer_matches_the_oracle(shape):
    """Forward and both backward products of the simulated layer: every operand bit-exact, every product within tolerance.
    Shapes: (tokens, D, C); the last two are ragged in every dimension (tiles, 64-wide k tiles, 16-blocks)."""
    b = B()
    N, D, C = shape
    X, W, dY, _ = synth.layer_inputs(1, N, D, C, n_outlier=2, factor=30.0, grad_scale=1e-3)
    Yo, so = f6.linear_fwd(X, W)
    Xd, Wd, dYd = b.upload_bf16(X), b.upload_bf16(W), b.upload_bf16(dY)
    Y, saved = b.fp6_linear_fwd(Xd, Wd, b.DT_F32)
    assert_dense_equal(saved[0], so.qx6, "Q6_D(X)", f6.block_values)
    assert_operand_equal(saved[1], so.qw, "Q4_D(W)")
    check_product(Y, f6.dequantize(so.qx6), orc.dequantize(so.qw), False, "Y")
    dX, dW, (q3, q4, q5, q6) = b.fp6_linear_bwd(dYd, saved, seed=123, dx_dtype=b.DT_F32)
    dXo, q3o, q4o = f6.linear_bwd_dx(dY, so, seed=123)
    dWo, q5o, q6o = f6.linear_bwd_dw(dY, so, seed=123)
    assert_dense_equal(q3, q3o, "Q6_S(dY)", f6.block_values)
    assert_operand_equal(q4, q4o, "Q4_S(W-hat^T)")
    assert_operand_equal(q5, q5o, "Q4_S(dY^T)")
    assert_dense_equal(q6, q6o, "Q6_S(X-hat^T)", f6.block_values)
    check_product(dX, f6.dequantize(q3o), orc.dequantize(q4o), False, "dX")
    check_product(dW, orc.dequantize(q5o), f6.dequantize(q6o), False, "dW")
    assert rel_fro(dX.float().cpu().numpy(), dXo) <= 1e-5 and rel_fro(dW.float().cpu().numpy(), dWo) <= 1e-5
    # BF16 outputs: one rounding of the same sums
    Y16, _ = b.fp6_linear_fwd(Xd, Wd, b.DT_BF16)
    check_product(Y16, f6.dequantize(so.qx6), orc.dequantize(so.qw), True, "Y bf16")


def test_fp6_calls_refuse_bad_arguments_before_any_launch():
    b = B()
    x = to_dev_bf16(np.ones((16, 32), dtype=np.float32))
    out = b.alloc_dense(16, 32)
    with pytest.raises(b.Nvfp4Error):
        b.nvfp4_fp6_quantize(x, b.ROUND_SR_SCALE_UP, 0, 1, out=out)  # rounding outside the simulation
    odd = to_dev_bf16(np.ones((16, 36), dtype=np.float32))  # 72-byte rows: not 16-byte aligned
    with pytest.raises(b.Nvfp4Error):
        b.nvfp4_fp6_quantize(odd, b.ROUND_RTN, 0, 1)
    wrong = b.alloc_dense(16, 48)
    with pytest.raises(b.Nvfp4Error):
        b.nvfp4_fp6_quantize(x, b.ROUND_RTN, 0, 1, out=wrong)  # shape mismatch
    row = b.nvfp4_quantize(x, b.AXIS_ROW, b.ROUND_RTN, 0, 1, b.GS_ROW)
    with pytest.raises(b.Nvfp4Error):
        b.nvfp4_expand_operand(row)  # only TENSOR-mode operands are part of the simulation
    a, c = b.alloc_dense(16, 32), b.alloc_dense(16, 48)
    with pytest.raises(b.Nvfp4Error):
        b.nvfp4_dense_gemm(a, c)  # K mismatch
