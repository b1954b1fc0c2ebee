"""Parity of the remaining BASELINE configurations at their full sizes, through the entry points and in the launch
configuration bench.py times (nvfp4_linear_fwd + nvfp4_linear_bwd, tiled scales, BF16 Y / dX, FP32 dW):
  - config 2: the O projection (1024 -> 1024, tokens 8192);
  - config 3: the SwiGLU MLP (1024 -> 2816 and 2816 -> 1024, tokens 8192; K = 2816 = 11 k tiles, C = 2816 = 22 n tiles);
  - config 4: tokens 16384 (dW with K = 16384), one attention and one MLP linear of the 24-layer model;
  - the per-row scale mode and OutControl with 10 % outlier channels (the paper's setting) at size.
Operands bit for bit (all six quantizers), products on sampled entries and tiles the oracle computes one by one."""
import pytest

from tests.gpu_util import check_layer_at_size

pytestmark = pytest.mark.gpu


def B():
    from paper_2510_27527_b200 import binding

    return binding


def test_config2_o_projection_full_size():
    check_layer_at_size(B(), 2, 8192, 1024, 1024, 0, weight_id=11, rng_seed=20, name="cfg2 o")


@pytest.mark.parametrize("gs_mode", [0, 2])
def test_config3_gate_projection_full_size(gs_mode):
    check_layer_at_size(B(), 3, 8192, 1024, 2816, gs_mode, weight_id=10, rng_seed=30 + gs_mode, name="cfg3 gate")


@pytest.mark.parametrize("gs_mode", [0, 2])
def test_config3_down_projection_full_size(gs_mode):
    check_layer_at_size(B(), 3, 8192, 2816, 1024, gs_mode, weight_id=12, swiglu=True, rng_seed=32 + gs_mode, name="cfg3 down")


def test_config4_qkv_tokens_16384():
    check_layer_at_size(B(), 4, 16384, 1024, 3072, 0, weight_id=10, rng_seed=40, name="cfg4 qkv")


def test_config4_down_projection_tokens_16384():
    check_layer_at_size(B(), 4, 16384, 2816, 1024, 0, weight_id=14, swiglu=True, rng_seed=41, name="cfg4 down")


def test_row_scale_mode_full_size():
    check_layer_at_size(B(), 2, 8192, 1024, 3072, 1, weight_id=10, rng_seed=50, name="cfg2 qkv ROW")


@pytest.mark.parametrize("gs_mode", [0, 1, 2])
def test_outcontrol_ten_percent_qkv_full_size(gs_mode):
    """D = 1024, 102 outlier channels (Kh = 128): the side product fused in the forward product, the two-pass W-hat^T, the
    ragged 922-column tiles of Q4 / Q6, the BF16 side product of dW with its token splits and the assembling pass."""
    check_layer_at_size(B(), 2, 8192, 1024, 3072, gs_mode, weight_id=10, n_out=102, rng_seed=60 + gs_mode, name="cfg2 qkv OutControl")


def test_outcontrol_ten_percent_down_projection_full_size():
    """D = 2816, 282 outlier channels (Kh = 320: two slabs of the BF16 side product of dW)."""
    check_layer_at_size(B(), 3, 8192, 2816, 1024, 0, weight_id=12, swiglu=True, n_out=282, rng_seed=70, name="cfg3 down OutControl")


def test_paper_recipe_full_size():
    """1 x 128 outer-block scales + random Hadamard transformation + 10 % outlier channels on the MLP up projection."""
    check_layer_at_size(B(), 3, 8192, 1024, 2816, 2, weight_id=11, n_out=102, rht=True, rng_seed=80, name="cfg3 up full recipe")
