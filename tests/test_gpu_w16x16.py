"""GPU parity of the 16x16 weight-block recipe: the quantizer and the operand transposition bit for bit, the layer's
forward / dX / dW against the oracle."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from oracle import w16x16
from paper_2510_27527_b200 import synth
from tests.gpu_util import assert_operand_equal, rel_fro, to_dev_bf16

pytestmark = pytest.mark.gpu


def B():
    from paper_2510_27527_b200 import binding

    return binding


@pytest.mark.parametrize("shape", [(16, 16), (48, 80), (40, 72), (17, 40), (256, 512), (130, 264), (512, 1024)])
@pytest.mark.parametrize("layout", [0, 1])
def test_quantizer_and_transposition_bit_exact(shape, layout):
    b = B()
    W = synth.weights(shape[0], shape[1], 40 + shape[0]) * np.float32(2.5)
    W[5 % shape[0], 7 % shape[1]] *= np.float32(30.0)
    W = torch.from_numpy(W).to(torch.bfloat16).float().numpy()  # the device sees BF16
    ref = w16x16.quantize(W)
    out = b.alloc_operand(shape[0], shape[1], b.GS_TENSOR, layout, poison=True)
    b.nvfp4_quantize_w16x16(to_dev_bf16(W), layout, out=out)
    assert_operand_equal(out, ref, f"w16x16 {shape} layout{layout}")
    ref_t = w16x16.transpose_operand(ref)
    out_t = b.alloc_operand(shape[1], shape[0], b.GS_TENSOR, b.SF_TILED128x4, poison=True)
    b.nvfp4_transpose_operand16(out, out=out_t)
    assert_operand_equal(out_t, ref_t, f"transpose {shape} layout{layout}")


def test_zero_matrix_and_zero_squares():
    b = B()
    W = synth.weights(64, 96, 3)
    W[16:32, 32:64] = 0.0
    ref = w16x16.quantize(W)
    out = b.alloc_operand(64, 96, b.GS_TENSOR, b.SF_TILED128x4, poison=True)
    b.nvfp4_quantize_w16x16(to_dev_bf16(W), out=out)
    assert_operand_equal(out, ref, "zero squares")
    Z = np.zeros((32, 48), dtype=np.float32)
    out = b.alloc_operand(32, 48, b.GS_TENSOR, b.SF_TILED128x4, poison=True)
    b.nvfp4_quantize_w16x16(to_dev_bf16(Z), out=out)
    assert_operand_equal(out, w16x16.quantize(Z), "all zero")


@pytest.mark.parametrize("rht", [False, True])
@pytest.mark.parametrize("shape", [(256, 512, 384), (200, 272, 136)])
def test_layer_with_16x16_weight_blocks(rht, shape):
    b = B()
    N_tok, D, C = shape
    X, W, dY, _ = synth.layer_inputs(14, N_tok, D, C, n_outlier=2, factor=20.0, grad_scale=1e-3)
    ocfg = orc.LayerConfig(gs_mode=orc.GS_TENSOR, seed=9, w_block16=True, rht=rht)
    Yo, so = orc.linear_fwd(X, W, ocfg)
    dXo, dWo = orc.linear_bwd_dx(dY, so, ocfg), orc.linear_bwd_dw(dY, so, ocfg)
    cfg = b.LayerConfig(gs_mode=b.GS_TENSOR, seed=9, w_block16=True, rht=rht, y_dtype=b.DT_F32, dx_dtype=b.DT_F32, dw_dtype=b.DT_F32)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    Y, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    assert_operand_equal(saved.qw, so.qw, "Q2 (16x16)")
    dX, dW = b.nvfp4_linear_bwd(dYd, saved, cfg)
    dX2 = b.nvfp4_linear_bwd_dx(dYd, saved, cfg)
    torch.cuda.synchronize()
    assert rel_fro(Y.float().cpu().numpy(), Yo) <= 2e-5
    assert rel_fro(dX.float().cpu().numpy(), dXo) <= 2e-5
    assert rel_fro(dW.float().cpu().numpy(), dWo) <= 2e-5
    assert torch.equal(dX, dX2)


def test_16x16_needs_tensor_scales_and_no_outliers():
    b = B()
    X, W, _, ch = synth.layer_inputs(1, 64, 64, 32, n_outlier=2, factor=20.0, grad_scale=1e-3)
    for cfg in (b.LayerConfig(gs_mode=b.GS_ROW, w_block16=True), b.LayerConfig(gs_mode=b.GS_TENSOR, w_block16=True, outliers=ch)):
        with pytest.raises(b.Nvfp4Error):
            b.nvfp4_linear_fwd(to_dev_bf16(X), to_dev_bf16(W), cfg)
