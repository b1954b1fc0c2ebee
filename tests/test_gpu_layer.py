"""GPU parity of the whole layer (forward, dX, dW; with and without OutControl) on the small configuration:
X 256x512 ~N(0,1) with 4 outlier channels x50, W 512x512 ~N(0,0.02), dY 256x512 Student-t(3) x 1e-3, seed 0."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.gpu_util import assert_operand_equal, bf16_ulp_close, rel_fro, to_dev_bf16

pytestmark = pytest.mark.gpu


def B():
    from paper_2510_27527_b200 import binding

    return binding


def run_layer(b, X, W, dY, gs_mode, outliers, f32_out=True, seed=0):
    cfg = b.LayerConfig(gs_mode=gs_mode, seed=seed, outliers=outliers, y_dtype=b.DT_F32 if f32_out else b.DT_BF16,
                        dx_dtype=b.DT_F32 if f32_out else b.DT_BF16, dw_dtype=b.DT_F32)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    Y, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    dX = b.nvfp4_linear_bwd_dx(dYd, saved, cfg)
    dW = b.nvfp4_linear_bwd_dw(dYd, saved, cfg)
    torch.cuda.synchronize()
    return Y.float().cpu().numpy(), dX.float().cpu().numpy(), dW.float().cpu().numpy(), saved


@pytest.mark.parametrize("gs_mode", [0, 1, 2])
@pytest.mark.parametrize("outcontrol", [False, True])
def test_config1_layer(gs_mode, outcontrol):
    b = B()
    c = synth.CONFIGS[1]
    (_, D, C), = c["linears"]
    X, W, dY, ch = synth.layer_inputs(1, c["tokens"], D, C, n_outlier=c["n_outlier"], factor=c["factor"],
                                      grad_scale=c["grad_scale"])
    outl = ch if outcontrol else None
    ocfg = orc.LayerConfig(gs_mode=gs_mode, seed=0, outliers=outl)
    Yo, so = orc.linear_fwd(X, W, ocfg)
    dXo = orc.linear_bwd_dx(dY, so, ocfg)
    dWo = orc.linear_bwd_dw(dY, so, ocfg)
    Y, dX, dW, saved = run_layer(b, X, W, dY, gs_mode, outl)
    assert_operand_equal(saved.qx, so.qx, "Q1(X)")
    assert_operand_equal(saved.qw, so.qw, "Q2(W)")
    for name, got, want in (("Y", Y, Yo), ("dX", dX, dXo), ("dW", dW, dWo)):
        assert got.shape == want.shape
        assert rel_fro(got, want) <= 1e-3, name
        assert rel_fro(got, want) <= 2e-5, (name, rel_fro(got, want))
    # BF16 outputs: one rounding of the same FP32 result
    Y16, dX16, _, _ = run_layer(b, X, W, dY, gs_mode, outl, f32_out=False)
    # (noise term: FP32 accumulation error where a sum cancels, scaled by the output's typical magnitude)
    assert np.all(bf16_ulp_close(Y16, Yo, 1.0, 1e-4 * np.abs(Yo).mean()))
    assert np.all(bf16_ulp_close(dX16, dXo, 1.0, 1e-4 * np.abs(dXo).mean()))


def test_layer_is_replayable_and_seed_dependent():
    b = B()
    X, W, dY, _ = synth.layer_inputs(1, 256, 512, 512, n_outlier=4, factor=50.0, grad_scale=1e-3)
    a = run_layer(b, X, W, dY, 0, None, seed=5)
    a2 = run_layer(b, X, W, dY, 0, None, seed=5)
    c = run_layer(b, X, W, dY, 0, None, seed=6)
    assert np.array_equal(a[0], c[0])  # forward is deterministic rounding
    assert np.array_equal(a[1], a2[1]) and np.array_equal(a[2], a2[2])
    assert not np.array_equal(a[1], c[1]) and not np.array_equal(a[2], c[2])


def test_ragged_layer_shapes():
    """Tokens / features that are not multiples of the tile sizes (partial 16-blocks, partial 128-row tiles)."""
    b = B()
    N_tok, D, C = 200, 272, 136
    X, W, dY, ch = synth.layer_inputs(9, N_tok, D, C, n_outlier=3, factor=40.0, grad_scale=1e-3)
    for outl in (None, ch):
        for gs_mode in (0, 1, 2):
            ocfg = orc.LayerConfig(gs_mode=gs_mode, seed=3, outliers=outl)
            Yo, so = orc.linear_fwd(X, W, ocfg)
            dXo, dWo = orc.linear_bwd_dx(dY, so, ocfg), orc.linear_bwd_dw(dY, so, ocfg)
            Y, dX, dW, _ = run_layer(b, X, W, dY, gs_mode, outl, seed=3)
            assert rel_fro(Y, Yo) <= 2e-5 and rel_fro(dX, dXo) <= 2e-5 and rel_fro(dW, dWo) <= 2e-5


@pytest.mark.parametrize("gs_mode", [0, 1, 2])
@pytest.mark.parametrize("outcontrol", [False, True])
@pytest.mark.parametrize("rht", [False, True])
def test_combined_backward_is_bit_identical_to_the_two_calls(gs_mode, outcontrol, rht):
    """nvfp4_linear_bwd = bwd_dx then bwd_dw; sharing the per-tensor amax of dY changes no bit."""
    b = B()
    N_tok, D, C = 200, 272, 136
    X, W, dY, ch = synth.layer_inputs(9, N_tok, D, C, n_outlier=3, factor=40.0, grad_scale=1e-3)
    cfg = b.LayerConfig(gs_mode=gs_mode, seed=3, outliers=ch if outcontrol else None, dx_dtype=b.DT_BF16, dw_dtype=b.DT_F32, rht=rht)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    _, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    dX1 = b.nvfp4_linear_bwd_dx(dYd, saved, cfg)
    dW1 = b.nvfp4_linear_bwd_dw(dYd, saved, cfg)
    dX2, dW2 = b.nvfp4_linear_bwd(dYd, saved, cfg)
    torch.cuda.synchronize()
    assert torch.equal(dX1, dX2) and torch.equal(dW1, dW2)


@pytest.mark.parametrize("gs_mode", [0, 1, 2])
@pytest.mark.parametrize("outcontrol", [False, True])
@pytest.mark.parametrize("rht", [False, True])
def test_backward_with_rounded_up_block_scales(gs_mode, outcontrol, rht):
    """The strictly unbiased variant (block scale rounded up) in all four backward quantizers, through the layer calls."""
    b = B()
    N_tok, D, C = 200, 272, 136
    X, W, dY, ch = synth.layer_inputs(12, N_tok, D, C, n_outlier=3, factor=40.0, grad_scale=1e-3)
    outl = ch if outcontrol else None
    rounding = (orc.RTN, orc.RTN, orc.SR_SCALE_UP, orc.SR_SCALE_UP, orc.SR_SCALE_UP, orc.SR_SCALE_UP)
    ocfg = orc.LayerConfig(gs_mode=gs_mode, seed=8, outliers=outl, rounding=rounding, rht=rht)
    _, so = orc.linear_fwd(X, W, ocfg)
    dXo, dWo = orc.linear_bwd_dx(dY, so, ocfg), orc.linear_bwd_dw(dY, so, ocfg)
    plain = orc.LayerConfig(gs_mode=gs_mode, seed=8, outliers=outl, rht=rht)
    assert rel_fro(orc.linear_bwd_dx(dY, so, plain), dXo) > 1e-3  # the variant is a different quantizer
    cfg = b.LayerConfig(gs_mode=gs_mode, seed=8, outliers=outl, rounding=rounding, rht=rht, y_dtype=b.DT_F32, dx_dtype=b.DT_F32,
                        dw_dtype=b.DT_F32)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    _, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    dX, dW = b.nvfp4_linear_bwd(dYd, saved, cfg)
    torch.cuda.synchronize()
    assert rel_fro(dX.float().cpu().numpy(), dXo) <= 2e-5
    assert rel_fro(dW.float().cpu().numpy(), dWo) <= 2e-5


@pytest.mark.parametrize("gs_mode", [0, 1, 2])
@pytest.mark.parametrize("rht", [False, True])
def test_fp8_outlier_channels(gs_mode, rht):
    """OutControl with the outlier channels on their per-tensor power-of-two scaled E4M3 grids: the side operands are the
    oracle's bit for bit, and forward / dX / dW follow."""
    from oracle import fp8_outliers as f8

    b = B()
    N_tok, D, C = 200, 272, 136
    X, W, dY, ch = synth.layer_inputs(21, N_tok, D, C, n_outlier=5, factor=40.0, grad_scale=1e-3)
    ocfg = orc.LayerConfig(gs_mode=gs_mode, seed=2, outliers=ch, rht=rht, outlier_fp8=True)
    Yo, so = orc.linear_fwd(X, W, ocfg)
    dXo, dWo = orc.linear_bwd_dx(dY, so, ocfg), orc.linear_bwd_dw(dY, so, ocfg)
    cfg = b.LayerConfig(gs_mode=gs_mode, seed=2, outliers=ch, rht=rht, outlier_fp8=True, y_dtype=b.DT_F32, dx_dtype=b.DT_F32,
                        dw_dtype=b.DT_F32)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    Y, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    dX, dW = b.nvfp4_linear_bwd(dYd, saved, cfg)
    torch.cuda.synchronize()
    n = len(ch)
    X8 = saved.X_out.float().cpu().numpy()
    W8 = saved.W_out.float().cpu().numpy()
    assert np.array_equal(X8[:, :n], f8.snap(X[:, ch])[0]) and np.all(X8[:, n:] == 0)
    assert np.array_equal(W8[:, :n], f8.snap(W[:, ch])[0]) and np.all(W8[:, n:] == 0)
    assert not np.array_equal(X8[:, :n], X[:, ch])  # the option does something on these inputs
    assert rel_fro(Y.float().cpu().numpy(), Yo) <= 2e-5
    assert rel_fro(dX.float().cpu().numpy(), dXo) <= 2e-5
    assert rel_fro(dW.float().cpu().numpy(), dWo) <= 2e-5


def test_fp8_outlier_snap_extremes():
    """Scale exponents far from zero, an all-zero slice, exact powers of two and values that fall below the E4M3 grid."""
    from oracle import fp8_outliers as f8

    b = B()
    rng = np.random.default_rng(77)
    for scale in (2.0 ** -40, 1.0, 448.0, 2.0 ** 30, 0.0):
        X = (rng.standard_normal((64, 32)) * scale).astype(np.float32)
        X[:, 3] *= np.float32(2.0 ** -12)  # a column that lands in the subnormal range of the scaled grid or below it
        X = torch.from_numpy(X).to(torch.bfloat16).float().numpy()
        W = torch.from_numpy((rng.standard_normal((16, 32)) * 0.02).astype(np.float32)).to(torch.bfloat16).float().numpy()
        ch = np.array([1, 3, 8, 30])
        cfg = b.LayerConfig(gs_mode=0, seed=0, outliers=ch, outlier_fp8=True, y_dtype=b.DT_F32)
        _, saved = b.nvfp4_linear_fwd(to_dev_bf16(X), to_dev_bf16(W), cfg)
        torch.cuda.synchronize()
        assert np.array_equal(saved.X_out.float().cpu().numpy()[:, :4], f8.snap(X[:, ch])[0]), scale
        assert np.array_equal(saved.W_out.float().cpu().numpy()[:, :4], f8.snap(W[:, ch])[0]), scale


@pytest.mark.parametrize("outcontrol", [False, True])
def test_graph_replay_and_second_stream_give_the_eager_bits(outcontrol):
    """A captured step (fork / join of the library's side stream included) replays to the eager results bit for bit, and so
    does a call issued on a user stream that is not the current one's default."""
    b = B()
    X, W, dY, ch = synth.layer_inputs(31, 256, 512, 384, n_outlier=4, factor=50.0, grad_scale=1e-3)
    cfg = b.LayerConfig(gs_mode=0, seed=11, outliers=ch if outcontrol else None, y_dtype=b.DT_BF16, dx_dtype=b.DT_BF16, dw_dtype=b.DT_F32)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    cfg.prepare(512)
    saved = b.alloc_saved(Xd, Wd, cfg)
    Y = torch.empty((256, 384), dtype=torch.bfloat16, device="cuda")
    dX = torch.empty((256, 512), dtype=torch.bfloat16, device="cuda")
    dW = torch.empty((384, 512), dtype=torch.float32, device="cuda")
    ws_f = b.linear_workspace(b.OP_FWD, 256, 512, 384, cfg, Xd.device)
    ws_b = b.linear_workspace(b.OP_BWD, 256, 512, 384, cfg, Xd.device)

    def step():
        b.nvfp4_linear_fwd(Xd, Wd, cfg, Y=Y, saved=saved, workspace=ws_f)
        b.nvfp4_linear_bwd(dYd, saved, cfg, dX=dX, dW=dW, workspace=ws_b)

    step()  # eager (also creates the side stream outside any capture)
    torch.cuda.synchronize()
    want = (Y.clone(), dX.clone(), dW.clone())
    for t in (Y, dX, dW):
        t.zero_()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        step()
    for t in (Y, dX, dW):
        t.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert all(torch.equal(a, w) for a, w in zip((Y, dX, dW), want))
    for t in (Y, dX, dW):
        t.zero_()
    s2 = torch.cuda.Stream()
    s2.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s2):
        step()
    s2.synchronize()
    assert all(torch.equal(a, w) for a, w in zip((Y, dX, dW), want))


def test_randomised_layer_configurations():
    """Twenty random (shape, scale mode, OutControl, Hadamard, outlier format, rounding variant) layer configurations with a
    fixed seed, forward / dX / dW against the oracle."""
    b = B()
    rng = np.random.default_rng(4242)
    for case in range(20):
        N_tok = int(rng.integers(1, 40)) * 8 + int(rng.integers(0, 8))
        D = int(rng.integers(3, 60)) * 8
        C = int(rng.integers(1, 40)) * 8
        gs_mode = int(rng.integers(0, 3))
        rht = bool(rng.integers(0, 2))
        n_outl = int(rng.integers(0, 4)) * int(rng.integers(1, 6))
        n_outl = min(n_outl, D - 16)
        fp8 = bool(rng.integers(0, 2)) and n_outl > 0
        scale_up = bool(rng.integers(0, 2))
        w16 = gs_mode == 0 and n_outl == 0 and bool(rng.integers(0, 2))
        X, W, dY, _ = synth.layer_inputs(100 + case, N_tok, D, C, n_outlier=min(3, D // 8), factor=30.0, grad_scale=1e-3)
        outl = synth.outlier_channels(D, n_outl, 900 + case) if n_outl else None
        sr = orc.SR_SCALE_UP if scale_up else orc.SR
        rounding = (orc.RTN, orc.RTN, sr, sr, sr, sr)
        ocfg = orc.LayerConfig(gs_mode=gs_mode, seed=case, outliers=outl, rht=rht, outlier_fp8=fp8, rounding=rounding, w_block16=w16)
        Yo, so = orc.linear_fwd(X, W, ocfg)
        dXo, dWo = orc.linear_bwd_dx(dY, so, ocfg), orc.linear_bwd_dw(dY, so, ocfg)
        cfg = b.LayerConfig(gs_mode=gs_mode, seed=case, outliers=outl, rht=rht, outlier_fp8=fp8, rounding=rounding, w_block16=w16,
                            y_dtype=b.DT_F32, dx_dtype=b.DT_F32, dw_dtype=b.DT_F32)
        Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
        Y, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
        dX, dW = b.nvfp4_linear_bwd(dYd, saved, cfg)
        torch.cuda.synchronize()
        tag = f"case {case}: {N_tok}x{D}->{C} gs{gs_mode} rht{rht} outl{n_outl} fp8{fp8} up{scale_up} w16{w16}"
        assert rel_fro(Y.float().cpu().numpy(), Yo) <= 2e-5, tag
        assert rel_fro(dX.float().cpu().numpy(), dXo) <= 2e-5, tag
        assert rel_fro(dW.float().cpu().numpy(), dWo) <= 2e-5, tag
