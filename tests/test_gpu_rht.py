"""GPU parity of the random Hadamard transformation in the backward quantizers (Sec. 4.1): the CUDA quantizers with a
sign stream must give, bit for bit, the oracle's quantization of the oracle's transformed matrix; the layer's backward
products with the transformation must match the oracle's to the product tolerance."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.gpu_util import assert_operand_equal, rel_fro, to_dev_bf16, to_dev_i32

pytestmark = pytest.mark.gpu
MODES = [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128]


def B():
    from paper_2510_27527_b200 import binding

    return binding


@pytest.mark.parametrize("shape", [(1, 16), (3, 48), (50, 200), (129, 272), (300, 1000), (64, 4096 + 64), (1100, 136)])
@pytest.mark.parametrize("gs_mode", MODES)
@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR])
def test_row_axis_with_rht_bit_exact(shape, gs_mode, rounding):
    b = B()
    x = synth.gradients(shape[0], shape[1], 31 + shape[1], 1e-3)
    ref = orc.quantize(orc.rht16(x, 77, 7), orc.AXIS_ROW, rounding, gs_mode, seed=77, stream_id=3)
    for layout in (b.SF_LINEAR, b.SF_TILED128x4):
        out = b.alloc_operand(shape[0], shape[1], gs_mode, layout, poison=True)
        b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_ROW, rounding, 77, 3, gs_mode, layout, out=out, rht_stream_id=7)
        assert_operand_equal(out, ref, f"rht row {shape} gs{gs_mode} r{rounding} layout{layout}", k_extended=True)


# (column counts that are multiples of 4 take the register-transposing kernels and their own amax pre-pass; 1000, 700 and
# 1040 rows end inside a 16-block, a lane's 64 rows and a CTA's 512)
@pytest.mark.parametrize("shape", [(16, 1), (48, 5), (272, 129), (1000, 72), (200, 333), (130, 64), (700, 68), (1040, 132)])
@pytest.mark.parametrize("gs_mode", MODES)
@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR])
def test_col_axis_with_rht_bit_exact(shape, gs_mode, rounding):
    """Q5: the transformation runs along the source rows (the operand's K)."""
    b = B()
    cols8 = (shape[1] + 7) // 8 * 8
    full = synth.gradients(shape[0], cols8, 13 + shape[0], 1e-3)
    x = np.ascontiguousarray(full[:, : shape[1]])
    ref = orc.quantize(orc.rht16(np.ascontiguousarray(x.T), 5, 8), orc.AXIS_ROW, rounding, gs_mode, seed=5, stream_id=5)
    out = b.alloc_operand(shape[1], shape[0], gs_mode, b.SF_TILED128x4, poison=True)
    b.nvfp4_quantize(to_dev_bf16(full)[:, : shape[1]], b.AXIS_COL, rounding, 5, 5, gs_mode, out=out, rht_stream_id=8)
    assert_operand_equal(out, ref, f"rht col {shape} gs{gs_mode} r{rounding}", k_extended=True)


@pytest.mark.parametrize("shape", [(16, 16), (130, 272), (256, 512), (520, 200)])
@pytest.mark.parametrize("gs_mode", MODES)
def test_requantize_transposed_with_rht_bit_exact(shape, gs_mode):
    """Q4 / Q6: transform the transposed aligned tensor, then quantize (no closed-form tensor scale any more)."""
    b = B()
    x, _ = synth.activations(shape[0], shape[1], 21 + shape[0], n_outlier=2, factor=30.0)
    fwd_ref = orc.quantize(x, orc.AXIS_ROW, orc.RTN, gs_mode)
    xt = np.ascontiguousarray(orc.rematerialize_f32(fwd_ref).T)
    ref = orc.quantize(orc.rht16(xt, 5, 8), orc.AXIS_ROW, orc.SR, gs_mode, seed=5, stream_id=6)
    fwd = b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode)
    out = b.alloc_operand(shape[1], shape[0], gs_mode, poison=True)
    b.nvfp4_requantize_t(fwd, b.ROUND_SR, 5, 6, out=out, rht_stream_id=8)
    assert_operand_equal(out, ref, f"rht requantize_t {shape} gs{gs_mode}", k_extended=True)


def test_same_stream_on_both_operands_preserves_the_product():
    """A B^T ~ Q(A S H) Q(B S H)^T: through the CUDA quantizers and the FP4 product, the transformed pair estimates the
    same matrix as the plain pair (within quantization noise), while mismatched sign streams do not."""
    b = B()
    A = synth.gradients(256, 512, 1, 1.0)
    Bm = synth.gradients(128, 512, 2, 1.0)
    exact = orc.gemm_tn(A, Bm)
    def prod(sa, sb):
        qa = b.nvfp4_quantize(to_dev_bf16(A), b.AXIS_ROW, b.ROUND_RTN, 3, 3, b.GS_BLOCK128, rht_stream_id=sa)
        qb = b.nvfp4_quantize(to_dev_bf16(Bm), b.AXIS_ROW, b.ROUND_RTN, 3, 4, b.GS_BLOCK128, rht_stream_id=sb)
        out = b.nvfp4_gemm(qa, qb)
        torch.cuda.synchronize()
        return out.float().cpu().numpy()
    assert rel_fro(prod(7, 7), exact) < 0.2
    assert rel_fro(prod(0, 0), exact) < 0.2
    assert rel_fro(prod(7, 8), exact) > 0.7


def run_bwd(b, X, W, dY, gs_mode, outliers, seed):
    cfg = b.LayerConfig(gs_mode=gs_mode, seed=seed, outliers=outliers, y_dtype=b.DT_F32, dx_dtype=b.DT_F32, dw_dtype=b.DT_F32,
                        rht=True)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    Y, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    dX = b.nvfp4_linear_bwd_dx(dYd, saved, cfg)
    dW = b.nvfp4_linear_bwd_dw(dYd, saved, cfg)
    torch.cuda.synchronize()
    return Y.float().cpu().numpy(), dX.float().cpu().numpy(), dW.float().cpu().numpy()


@pytest.mark.parametrize("gs_mode", MODES)
@pytest.mark.parametrize("outcontrol", [False, True])
@pytest.mark.parametrize("dims", [(256, 512, 512), (200, 272, 136)])
def test_layer_backward_with_rht(gs_mode, outcontrol, dims):
    b = B()
    N_tok, D, C = dims
    X, W, dY, ch = synth.layer_inputs(4, N_tok, D, C, n_outlier=4, factor=50.0, grad_scale=1e-3)
    outl = ch if outcontrol else None
    ocfg = orc.LayerConfig(gs_mode=gs_mode, seed=11, outliers=outl, rht=True)
    Yo, so = orc.linear_fwd(X, W, ocfg)
    dXo, dWo = orc.linear_bwd_dx(dY, so, ocfg), orc.linear_bwd_dw(dY, so, ocfg)
    Y, dX, dW = run_bwd(b, X, W, dY, gs_mode, outl, 11)
    assert rel_fro(Y, Yo) <= 2e-5  # forward is untouched by the flag
    assert rel_fro(dX, dXo) <= 2e-5, rel_fro(dX, dXo)
    assert rel_fro(dW, dWo) <= 2e-5, rel_fro(dW, dWo)
    # and the flag does change the backward operands
    ocfg0 = orc.LayerConfig(gs_mode=gs_mode, seed=11, outliers=outl, rht=False)
    assert rel_fro(dX, orc.linear_bwd_dx(dY, so, ocfg0)) > 1e-3
