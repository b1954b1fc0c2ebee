"""Parity at the benchmark's full sizes, in the launch configuration bench.py times (tiled scales, BF16 / FP32
outputs, same entry points): quantizers bit-exact on the whole tensor, GEMM outputs on sampled entries and tiles
that the oracle computes one by one (FP64 dot products of the dequantized operands)."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.gpu_util import assert_operand_equal, check_sampled, to_dev_bf16

pytestmark = pytest.mark.gpu


def B():
    from paper_2510_27527_b200 import binding

    return binding


@pytest.mark.parametrize("gs_mode", [0, 2])
def test_attention_projection_qkv_full_size(gs_mode):
    """BASELINE config 2, the QKV linear: tokens 8192, 1024 -> 3072; forward, dX, dW through the layer entry points."""
    b = B()
    c = synth.CONFIGS[2]
    T, D, C = c["tokens"], 1024, 3072
    X, W, dY, _ = synth.layer_inputs(2, T, D, C, n_outlier=c["n_outlier"], factor=c["factor"], grad_scale=c["grad_scale"],
                                     weight_id=10)
    cfg = b.LayerConfig(gs_mode=gs_mode, seed=0, y_dtype=b.DT_BF16, dx_dtype=b.DT_BF16, dw_dtype=b.DT_F32)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    Y, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    dX = b.nvfp4_linear_bwd_dx(dYd, saved, cfg)
    dW = b.nvfp4_linear_bwd_dw(dYd, saved, cfg)
    torch.cuda.synchronize()
    rng = np.random.default_rng(0)
    # oracle operands (whole tensors), compared bit for bit where the device exposes them
    q1 = orc.quantize(X, orc.AXIS_ROW, orc.RTN, gs_mode, 0, 1)
    q2 = orc.quantize(W, orc.AXIS_ROW, orc.RTN, gs_mode, 0, 2)
    assert_operand_equal(saved.qx, q1, "Q1(X) full size")
    assert_operand_equal(saved.qw, q2, "Q2(W) full size")
    check_sampled(Y, orc.dequantize(q1), orc.dequantize(q2), rng, True, "Y")
    q3 = orc.quantize(dY, orc.AXIS_ROW, orc.SR, gs_mode, 0, 3)
    q4 = orc.quantize(orc.rematerialize_f32(q2), orc.AXIS_COL, orc.SR, gs_mode, 0, 4)
    check_sampled(dX, orc.dequantize(q3), orc.dequantize(q4), rng, True, "dX")
    q5 = orc.quantize(dY, orc.AXIS_COL, orc.SR, gs_mode, 0, 5)
    q6 = orc.quantize(orc.rematerialize_f32(q1), orc.AXIS_COL, orc.SR, gs_mode, 0, 6)
    check_sampled(dW, orc.dequantize(q5), orc.dequantize(q6), rng, False, "dW")
    # the backward operands themselves, bit for bit, through the operand-level entry points
    g3 = b.nvfp4_quantize(dYd, b.AXIS_ROW, b.ROUND_SR, 0, 3, gs_mode)
    assert_operand_equal(g3, q3, "Q3(dY) full size")
    g5 = b.nvfp4_quantize(dYd, b.AXIS_COL, b.ROUND_SR, 0, 5, gs_mode)
    assert_operand_equal(g5, q5, "Q5(dY^T) full size")
    g4 = b.nvfp4_requantize_t(saved.qw, b.ROUND_SR, 0, 4)
    assert_operand_equal(g4, q4, "Q4(W-hat) full size")
    g6 = b.nvfp4_requantize_t(saved.qx, b.ROUND_SR, 0, 6)
    assert_operand_equal(g6, q6, "Q6(X-hat) full size")


def test_largest_sweep_shape_quantize_and_gemm():
    """BASELINE config 5, the largest shape: M = 16384, N = K = 8192 (BF16 ~N(0,1), 0.5 % channels x100)."""
    b = B()
    M, N, K = 16384, 8192, 8192
    A, _ = synth.activations(M, K, synth.seed_of(5, 1), n_outlier=41, factor=100.0)
    Bm, _ = synth.activations(N, K, synth.seed_of(5, 2), n_outlier=41, factor=100.0)
    Ad, Bd = to_dev_bf16(A), to_dev_bf16(Bm)
    qa = b.nvfp4_quantize(Ad, b.AXIS_ROW, b.ROUND_RTN, 0, 1, b.GS_TENSOR)
    qb = b.nvfp4_quantize(Bd, b.AXIS_ROW, b.ROUND_SR, 7, 2, b.GS_TENSOR)
    oa = orc.quantize(A, orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR, 0, 1)
    ob = orc.quantize(Bm, orc.AXIS_ROW, orc.SR, orc.GS_TENSOR, 7, 2)
    assert_operand_equal(qa, oa, "A 16384x8192 RTN")
    assert_operand_equal(qb, ob, "B 8192x8192 SR")
    C = b.nvfp4_gemm(qa, qb, b.DT_BF16)
    torch.cuda.synchronize()
    check_sampled(C, orc.dequantize(oa), orc.dequantize(ob), np.random.default_rng(1), True, "C 16384x8192x8192")
    del C
    # the transposed (column-axis) quantizer at the same size, bit for bit
    qt = b.nvfp4_quantize(Bd, b.AXIS_COL, b.ROUND_SR, 9, 5, b.GS_BLOCK128)
    ot = orc.quantize(Bm, orc.AXIS_COL, orc.SR, orc.GS_BLOCK128, 9, 5)
    assert_operand_equal(qt, ot, "B^T 8192x8192 SR block128")


def test_attention_projection_with_rht_full_size():
    """The paper's base recipe at the benchmark's size: 1x128 outer-block scales, random Hadamard transformation in the
    four backward quantizers, through the combined backward entry point that bench.py times."""
    b = B()
    c = synth.CONFIGS[2]
    T, D, C = c["tokens"], 1024, 3072
    gs_mode = orc.GS_BLOCK128
    X, W, dY, _ = synth.layer_inputs(2, T, D, C, n_outlier=c["n_outlier"], factor=c["factor"], grad_scale=c["grad_scale"],
                                     weight_id=10)
    cfg = b.LayerConfig(gs_mode=gs_mode, seed=0, y_dtype=b.DT_BF16, dx_dtype=b.DT_BF16, dw_dtype=b.DT_F32, rht=True)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    _, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    dX, dW = b.nvfp4_linear_bwd(dYd, saved, cfg)
    torch.cuda.synchronize()
    rng = np.random.default_rng(3)
    q1 = orc.quantize(X, orc.AXIS_ROW, orc.RTN, gs_mode, 0, 1)
    q2 = orc.quantize(W, orc.AXIS_ROW, orc.RTN, gs_mode, 0, 2)
    q3 = orc.quantize(orc.rht16(dY, 0, orc.STREAM_RHT_DX), orc.AXIS_ROW, orc.SR, gs_mode, 0, 3)
    q4 = orc.quantize(orc.rht16(np.ascontiguousarray(orc.rematerialize_f32(q2).T), 0, orc.STREAM_RHT_DX), orc.AXIS_ROW, orc.SR,
                      gs_mode, 0, 4)
    check_sampled(dX, orc.dequantize(q3), orc.dequantize(q4), rng, True, "dX with RHT")
    q5 = orc.quantize(orc.rht16(np.ascontiguousarray(dY.T), 0, orc.STREAM_RHT_DW), orc.AXIS_ROW, orc.SR, gs_mode, 0, 5)
    q6 = orc.quantize(orc.rht16(np.ascontiguousarray(orc.rematerialize_f32(q1).T), 0, orc.STREAM_RHT_DW), orc.AXIS_ROW, orc.SR,
                      gs_mode, 0, 6)
    check_sampled(dW, orc.dequantize(q5), orc.dequantize(q6), rng, False, "dW with RHT")
    g3 = b.nvfp4_quantize(dYd, b.AXIS_ROW, b.ROUND_SR, 0, 3, gs_mode, rht_stream_id=7)
    assert_operand_equal(g3, q3, "Q3(dY S H) full size", k_extended=True)
    g5 = b.nvfp4_quantize(dYd, b.AXIS_COL, b.ROUND_SR, 0, 5, gs_mode, rht_stream_id=8)
    assert_operand_equal(g5, q5, "Q5(dY^T S H) full size", k_extended=True)
    g6 = b.nvfp4_requantize_t(saved.qx, b.ROUND_SR, 0, 6, rht_stream_id=8)
    assert_operand_equal(g6, q6, "Q6(X-hat^T S H) full size", k_extended=True)


def test_oscireset_and_calibration_at_model_size():
    """A 4096 x 4096 FP32 weight matrix through two statistics steps (dense and memory-efficient) and the reset, and a
    8192 x 4096 activation through the calibration: bit-exact / within the float32 tolerance against the oracle."""
    from oracle import calibration as cal
    from oracle import oscireset as osc

    b = B()
    C, D = 4096, 4096
    traj, _ = synth.weight_trajectory(C, D, 2, seed=77)
    gs = orc.GS_BLOCK128
    ref, sref = osc.Stats((C, D)), osc.SparseStats(C * D // 20)
    st = b.alloc_osci_state(torch.from_numpy(traj[0]).cuda())
    sp = b.alloc_osci_sparse_state(C * D // 20)
    for t, Wt in enumerate(traj):
        Wd = torch.from_numpy(Wt).cuda()
        osc.update_stats(Wt, ref, t, gs)
        osc.update_stats_sparse(Wt, sref, t, gs)
        b.nvfp4_osci_update(Wd, st, t, gs)
        b.nvfp4_osci_sparse_update(Wd, sp, t, gs)
    torch.cuda.synchronize()
    u32 = lambda a: np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    assert np.array_equal(u32(st.D_M.cpu().numpy()), u32(ref.D_M)) and np.array_equal(u32(st.D_Q.cpu().numpy()), u32(ref.D_Q))
    assert np.array_equal(sp.idx.cpu().numpy().astype(np.int64), sref.idx)
    assert np.array_equal(u32(sp.D_M.cpu().numpy()), u32(sref.D_M)) and np.array_equal(u32(sp.D_Q.cpu().numpy()), u32(sref.D_Q))
    want, mask = osc.suppress(traj[-1], ref, 8.0, gs)
    Wd = torch.from_numpy(traj[-1]).cuda()
    n = torch.zeros(1, dtype=torch.int64, device="cuda")
    b.nvfp4_osci_suppress(Wd, st, 8.0, gs, n_reset=n)
    torch.cuda.synchronize()
    assert np.array_equal(u32(Wd.cpu().numpy()), u32(want)) and int(n.item()) == int(mask.sum())
    X, ch = synth.activations(8192, 4096, 5, n_outlier=20, factor=30.0)
    acc = torch.zeros(4096, dtype=torch.float32, device="cuda")
    b.nvfp4_outlier_accumulate(to_dev_bf16(X), acc)
    want_acc = cal.accumulate(np.zeros(4096), X)
    torch.cuda.synchronize()
    got = acc.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - want_acc) <= 1e-5 * want_acc)
    outl, _, _ = b.nvfp4_outlier_select(acc, 20)
    assert outl.cpu().numpy().tolist() == sorted(ch.tolist())


def test_variants_at_the_qkv_size():
    """The options added around the hot path at the benchmark's QKV size (tokens 8192, 1024 -> 3072), in the launch
    configuration bench.py times: rounded-up block scales in Q3 / Q5, FP8 outlier channels, 16x16 weight squares."""
    from oracle import fp8_outliers as f8
    from oracle import w16x16

    b = B()
    c = synth.CONFIGS[2]
    T, D, C = c["tokens"], 1024, 3072
    X, W, dY, ch = synth.layer_inputs(2, T, D, C, n_outlier=c["n_outlier"], factor=c["factor"], grad_scale=c["grad_scale"],
                                      weight_id=10)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    rng = np.random.default_rng(1)
    # rounded-up block scales, whole operands
    q3 = orc.quantize(dY, orc.AXIS_ROW, orc.SR_SCALE_UP, orc.GS_TENSOR, 0, 3)
    assert_operand_equal(b.nvfp4_quantize(dYd, b.AXIS_ROW, b.ROUND_SR_SCALE_UP, 0, 3, b.GS_TENSOR), q3, "Q3 scale-up full size")
    q5 = orc.quantize(dY, orc.AXIS_COL, orc.SR_SCALE_UP, orc.GS_TENSOR, 0, 5)
    assert_operand_equal(b.nvfp4_quantize(dYd, b.AXIS_COL, b.ROUND_SR_SCALE_UP, 0, 5, b.GS_TENSOR), q5, "Q5 scale-up full size")
    # 16x16 weight squares: quantizer and transposition bit for bit, dX on sampled entries
    qw = w16x16.quantize(W)
    cfg = b.LayerConfig(gs_mode=b.GS_TENSOR, seed=0, w_block16=True, y_dtype=b.DT_BF16, dx_dtype=b.DT_BF16, dw_dtype=b.DT_F32)
    Y, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    assert_operand_equal(saved.qw, qw, "Q2 16x16 full size")
    assert_operand_equal(b.nvfp4_transpose_operand16(saved.qw), w16x16.transpose_operand(qw), "W-hat^T 16x16 full size")
    dX, _ = b.nvfp4_linear_bwd(dYd, saved, cfg)
    torch.cuda.synchronize()
    q3p = orc.quantize(dY, orc.AXIS_ROW, orc.SR, orc.GS_TENSOR, 0, 3)
    check_sampled(dX, orc.dequantize(q3p), orc.dequantize(w16x16.transpose_operand(qw)), rng, True, "dX 16x16")
    # FP8 outlier channels (10 % of the channels, as bench.py --outliers 0.1 --outlier-fp8): side operands bit for bit
    outl = synth.outlier_channels(D, 102, 77)
    cfg8 = b.LayerConfig(gs_mode=b.GS_TENSOR, seed=0, outliers=outl, outlier_fp8=True, y_dtype=b.DT_BF16, dx_dtype=b.DT_BF16,
                         dw_dtype=b.DT_F32)
    Y8, saved8 = b.nvfp4_linear_fwd(Xd, Wd, cfg8)
    torch.cuda.synchronize()
    assert np.array_equal(saved8.X_out.float().cpu().numpy()[:, :102], f8.snap(X[:, outl])[0])
    assert np.array_equal(saved8.W_out.float().cpu().numpy()[:, :102], f8.snap(W[:, outl])[0])
    keep = np.setdiff1d(np.arange(D), outl)
    q1 = orc.quantize(X[:, keep], orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR, 0, 1)
    q2 = orc.quantize(W[:, keep], orc.AXIS_ROW, orc.RTN, orc.GS_TENSOR, 0, 2)
    A64 = np.concatenate([orc.dequantize(q1), f8.snap(X[:, outl])[0].astype(np.float64)], axis=1)
    B64 = np.concatenate([orc.dequantize(q2), f8.snap(W[:, outl])[0].astype(np.float64)], axis=1)
    check_sampled(Y8, A64, B64, rng, True, "Y with FP8 outlier channels")


@pytest.mark.parametrize("case", [
    # (source rows = operand k, source columns = operand rows, scale mode, source scale layout, rounding)
    (4100, 2100, 0, 1, 1),   # 8.6 M elements, 128 x 128 CTA tiles; ragged in rows (inside a 16-block) and in columns (not a multiple of 8)
    (4100, 2100, 1, 0, 2),   # ROW scales of source and result, linear source scale layout, rounded-up block scales
    (16400, 9300, 0, 1, 1),  # 153 M elements: 512 x 128 CTA tiles, ragged in both directions
    (16400, 9300, 1, 1, 1),
])
def test_register_transposing_requantizer_on_large_ragged_operands(case):
    """Q4 / Q6 from 8 M elements on take the kernel that transposes in registers (smaller operands keep the staged kernel, which
    the small-shape tests cover): both of its tile sizes, both scale modes it handles, bit for bit."""
    b = B()
    rows, cols, gs_mode, in_layout, rounding = case
    x, _ = synth.activations(rows, cols, 400 + rows, n_outlier=5, factor=40.0)
    cols8 = (cols + 7) // 8 * 8
    full = np.zeros((rows, cols8), dtype=np.float32)
    full[:, :cols] = x
    fwd_ref = orc.quantize(x, orc.AXIS_ROW, orc.RTN, gs_mode)
    ref = orc.quantize(orc.rematerialize_f32(fwd_ref), orc.AXIS_COL, rounding, gs_mode, seed=17, stream_id=6)
    fwd = b.nvfp4_quantize(to_dev_bf16(full)[:, :cols], b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode, in_layout)
    assert_operand_equal(fwd, fwd_ref, f"forward operand {case}")
    out = b.alloc_operand(cols, rows, gs_mode, poison=True)
    b.nvfp4_requantize_t(fwd, rounding, 17, 6, out=out)
    assert_operand_equal(out, ref, f"requantize_t {case}")
