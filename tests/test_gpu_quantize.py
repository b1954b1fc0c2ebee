"""GPU parity: the CUDA quantizers, called through the C ABI, must reproduce the oracle's packed codes, E4M3 scales
and FP32 global scales bit for bit (stochastic rounding included, same seed)."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.gpu_util import assert_operand_equal, to_dev_bf16, to_dev_i32

pytestmark = pytest.mark.gpu

SHAPES = [(1, 16), (3, 48), (127, 144), (129, 272), (256, 512), (300, 1000), (64, 4096 + 64)]
MODES = [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128]


def B():
    from paper_2510_27527_b200 import binding

    return binding


def make(shape, seed, kind="act"):
    if kind == "act":
        x, _ = synth.activations(shape[0], shape[1], seed, n_outlier=min(3, shape[1] // 8), factor=50.0)
        return x
    return synth.gradients(shape[0], shape[1], seed, 1e-3)


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("gs_mode", MODES)
@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR, orc.SR_SCALE_UP])
def test_row_axis_bit_exact(shape, gs_mode, rounding):
    b = B()
    x = make(shape, 7 + shape[1], "act" if rounding == orc.RTN else "grad")
    ref = orc.quantize(x, orc.AXIS_ROW, rounding, gs_mode, seed=1234567, stream_id=3)
    for layout in (b.SF_LINEAR, b.SF_TILED128x4):
        out = b.alloc_operand(shape[0], shape[1], gs_mode, layout, poison=True)
        b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_ROW, rounding, 1234567, 3, gs_mode, layout, out=out)
        assert_operand_equal(out, ref, f"row {shape} gs{gs_mode} r{rounding} layout{layout}")


# (rows, columns) of the source; the operand is its transpose. Column counts that are multiples of 4 take the kernels that
# transpose in registers (ragged token counts: 1000, 700, 1040 end inside a 16-block, a lane's 64 rows, a warp's 128 and a
# CTA's 512; 68 and 132 columns leave most lanes of the last CTA without work); the others take the staged kernels.
@pytest.mark.parametrize("shape", [(16, 1), (48, 5), (144, 127), (272, 129), (512, 256), (1000, 72), (200, 333), (700, 68),
                                   (1040, 132), (64, 4)])
@pytest.mark.parametrize("gs_mode", MODES)
@pytest.mark.parametrize("rounding", [orc.RTN, orc.SR, orc.SR_SCALE_UP])
def test_col_axis_bit_exact(shape, gs_mode, rounding):
    b = B()
    cols8 = (shape[1] + 7) // 8 * 8  # leading dimension must be a multiple of 8 elements
    full = make((shape[0], cols8), 11 + shape[0], "grad")
    x = np.ascontiguousarray(full[:, : shape[1]])
    ref = orc.quantize(x, orc.AXIS_COL, rounding, gs_mode, seed=99, stream_id=5)
    src = to_dev_bf16(full)[:, : shape[1]]
    for layout in (b.SF_TILED128x4, b.SF_LINEAR):
        out = b.alloc_operand(shape[1], shape[0], gs_mode, layout, poison=True)
        b.nvfp4_quantize(src, b.AXIS_COL, rounding, 99, 5, gs_mode, layout, out=out)
        assert_operand_equal(out, ref, f"col {shape} gs{gs_mode} r{rounding} layout{layout}")


@pytest.mark.parametrize("gs_mode", MODES)
def test_keep_cols_compaction(gs_mode):
    b = B()
    x = make((130, 512), 3)
    outl = np.array([0, 17, 100, 511])
    keep = np.setdiff1d(np.arange(512), outl)
    ref = orc.quantize(x[:, keep], orc.AXIS_ROW, orc.RTN, gs_mode)
    out = b.alloc_operand(130, 508, gs_mode, poison=True)
    b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode, keep_cols=to_dev_i32(keep), out=out)
    assert_operand_equal(out, ref, "keep_cols")


@pytest.mark.parametrize("shape", [(16, 16), (130, 272), (256, 512), (520, 200)])
@pytest.mark.parametrize("gs_mode", MODES)
@pytest.mark.parametrize("in_layout", [0, 1])
@pytest.mark.parametrize("rounding", [orc.SR, orc.SR_SCALE_UP])
def test_requantize_transposed_bit_exact(shape, gs_mode, in_layout, rounding):
    """Q4 / Q6: re-quantize the aligned tensor X-hat along the other axis, from the forward operand's codes."""
    b = B()
    x = make(shape, 21 + shape[0])
    fwd_ref = orc.quantize(x, orc.AXIS_ROW, orc.RTN, gs_mode)
    ref = orc.quantize(orc.rematerialize_f32(fwd_ref), orc.AXIS_COL, rounding, gs_mode, seed=5, stream_id=6)
    fwd = b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode, in_layout)
    assert_operand_equal(fwd, fwd_ref, "fwd operand")
    out = b.alloc_operand(shape[1], shape[0], gs_mode, poison=True)
    b.nvfp4_requantize_t(fwd, rounding, 5, 6, out=out)
    assert_operand_equal(out, ref, f"requantize_t {shape} gs{gs_mode} r{rounding}")


@pytest.mark.parametrize("gs_mode", MODES)
def test_requantize_with_row_map_mixes_high_precision_columns(gs_mode):
    """OutControl's W-hat: kept columns from the forward operand, outlier columns from the BF16 tensor."""
    b = B()
    C, D = 200, 272
    w = synth.weights(C, D, 5)
    outl = np.array([3, 64, 65, 200, 271])
    w[:, outl] *= 40
    w = synth.round_to_bf16(w)
    keep = np.setdiff1d(np.arange(D), outl)
    fwd_ref = orc.quantize(w[:, keep], orc.AXIS_ROW, orc.RTN, gs_mode)
    w_hat = orc.aligned_full(fwd_ref, keep, outl, w[:, outl], D)
    ref = orc.quantize(w_hat, orc.AXIS_COL, orc.SR, gs_mode, seed=8, stream_id=4)
    wd = to_dev_bf16(w)
    fwd = b.nvfp4_quantize(wd, b.AXIS_ROW, b.ROUND_RTN, 0, 2, gs_mode, keep_cols=to_dev_i32(keep))
    cmap = np.full(D, -1, dtype=np.int32)
    cmap[keep] = np.arange(len(keep))
    out = b.alloc_operand(D, C, gs_mode, poison=True)
    b.nvfp4_requantize_t(fwd, b.ROUND_SR, 8, 4, hp=wd, row_map=to_dev_i32(cmap), out=out)
    assert_operand_equal(out, ref, "requantize_t row_map")


def test_edge_values_zero_rows_negative_zero_and_underflow():
    b = B()
    x = np.zeros((5, 256), dtype=np.float32)
    x[1, 5] = 1000.0
    x[1, 40] = 1e-6
    x[1, 41] = -1e-6
    x[2, :] = -0.0
    x[3, 128:] = synth.round_to_bf16(np.linspace(-3, 3, 128).astype(np.float32))
    x = synth.round_to_bf16(x)
    for mode in MODES:
        for rounding in (orc.RTN, orc.SR):
            ref = orc.quantize(x, orc.AXIS_ROW, rounding, mode, seed=1, stream_id=3)
            out = b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_ROW, rounding, 1, 3, mode)
            assert_operand_equal(out, ref, f"edge rows gs{mode} r{rounding}")
            ref = orc.quantize(x, orc.AXIS_COL, rounding, mode, seed=1, stream_id=3)
            out = b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_COL, rounding, 1, 3, mode)
            assert_operand_equal(out, ref, f"edge cols gs{mode} r{rounding}")


def test_all_seven_rtn_ties_and_saturation_on_device():
    """The hand-derived blocks of tests/golden (exact ties, scale rounded down -> clamp) through the CUDA path."""
    import os

    rows = []
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "quantize_blocks.txt")):
        if line.strip() and line[0] != "#":
            v, s, c = line.split("|")
            rows.append(([float(t) for t in v.split()], int(s.strip(), 16), [int(t) for t in c.split()]))
    x = np.array([v for r in rows for v in r[0]], dtype=np.float32).reshape(1, 64)
    xb = synth.round_to_bf16(x)
    b = B()
    out = b.nvfp4_quantize(to_dev_bf16(xb), b.AXIS_ROW, b.ROUND_RTN, 0, 0, b.GS_TENSOR, b.SF_LINEAR)
    ref = orc.quantize(xb, orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR)
    assert_operand_equal(out, ref, "golden blocks (bf16-rounded)")
    torch.cuda.synchronize()
    sf = out.sf_linear()[0, :4]
    assert list(sf) == [r[1] for r in rows]
    # block 0 and block 2 consist of BF16-representable values: their codes are the hand-derived ones
    codes = out.codes.cpu().numpy()[:32]
    nib = np.stack([codes & 15, codes >> 4], axis=1).reshape(-1)
    assert list(nib[0:16]) == rows[0][2] and list(nib[32:48]) == rows[2][2]


@pytest.mark.parametrize("shape", [(128, 128), (129, 128), (127, 128), (64, 256), (65, 256), (512, 256), (513, 256), (16, 1024),
                                   (17, 1024), (1024, 128), (96, 384), (2048, 128 * 3)])
@pytest.mark.parametrize("gs_mode", MODES)
def test_row_axis_cta_boundaries(shape, gs_mode):
    """Shapes around the 1024-block CTA granularity with K a multiple of 128: interior CTAs take the unchecked copy of
    the kernel body, the last CTA the checked one; both must agree with the oracle bit for bit."""
    b = B()
    x = make(shape, 100 + shape[0], "grad")
    for rounding in (orc.RTN, orc.SR):
        ref = orc.quantize(x, orc.AXIS_ROW, rounding, gs_mode, seed=31, stream_id=3)
        out = b.alloc_operand(shape[0], shape[1], gs_mode, b.SF_TILED128x4, poison=True)
        b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_ROW, rounding, 31, 3, gs_mode, out=out)
        assert_operand_equal(out, ref, f"cta boundary {shape} gs{gs_mode} r{rounding}")


def test_randomised_shapes_modes_and_axes():
    """Forty random (shape, axis, rounding, scale mode, transformation) combinations with a fixed seed."""
    b = B()
    rng = np.random.default_rng(2024)
    for case in range(40):
        rows, cols = int(rng.integers(1, 700)), int(rng.integers(1, 90)) * 8
        axis = int(rng.integers(0, 2))
        rounding = int(rng.integers(0, 3))
        gs_mode = int(rng.integers(0, 3))
        rht = int(rng.integers(0, 2)) * 7
        x = make((rows, cols), 500 + case, "grad")
        seed = int(rng.integers(0, 2 ** 40))
        if axis == orc.AXIS_ROW:
            src = orc.rht16(x, seed, rht) if rht else x
            R, K = rows, cols
        else:
            xt = np.ascontiguousarray(x.T)
            src = orc.rht16(xt, seed, rht) if rht else xt
            R, K = cols, rows
        ref = orc.quantize(src, orc.AXIS_ROW, rounding, gs_mode, seed=seed, stream_id=3)
        out = b.alloc_operand(R, K, gs_mode, b.SF_TILED128x4, poison=True)
        b.nvfp4_quantize(to_dev_bf16(x), axis, rounding, seed, 3, gs_mode, out=out, rht_stream_id=rht)
        assert_operand_equal(out, ref, f"case {case}: {rows}x{cols} axis{axis} r{rounding} gs{gs_mode} rht{rht}", k_extended=bool(rht))
