"""GPU parity of OutControl's calibration kernels (Sec. 4.2): accumulated per-channel l2-norms within the float32
tolerance, selection identical to the oracle's wherever the float32 values order the channels the same way."""
import numpy as np
import pytest
import torch

from oracle import calibration as cal
from paper_2510_27527_b200 import synth
from tests.gpu_util import to_dev_bf16

pytestmark = pytest.mark.gpu
# float32 sum of n squares (fused multiply-add, at most ~8192/8 terms per partial, partials added in order) and one
# correctly rounded square root: relative error well under sqrt(n) * 2^-24 ~ 5e-6 for n = 8192
RTOL = 1e-5


def B():
    from paper_2510_27527_b200 import binding

    return binding


@pytest.mark.parametrize("shape", [(1, 8), (7, 24), (130, 272), (1000, 520), (4096, 1024), (300, 1000)])
def test_accumulate_matches_oracle_over_three_steps(shape):
    b = B()
    N, D = shape
    acc_ref = np.zeros(D)
    acc = torch.zeros(D, dtype=torch.float32, device="cuda")
    for step in range(3):
        X, _ = synth.activations(N, (D + 7) // 8 * 8, 50 + step, n_outlier=min(3, D // 8), factor=40.0, channel_seed=1)
        Xd = to_dev_bf16(X)[:, :D]
        acc_ref = cal.accumulate(acc_ref, X[:, :D])
        b.nvfp4_outlier_accumulate(Xd, acc)
    torch.cuda.synchronize()
    got = acc.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(got - acc_ref) <= RTOL * acc_ref + 1e-30), np.max(np.abs(got - acc_ref) / np.maximum(acc_ref, 1e-30))


def test_accumulate_is_bit_reproducible_and_handles_zero_and_constant_columns():
    b = B()
    N, D = 513, 264
    X = np.zeros((N, D), dtype=np.float32)
    X[:, 1] = 3.0
    X[7, 2] = -5.0
    X[:, 3:] = synth.gradients(N, D - 3, 3, 1.0)
    X = synth.round_to_bf16(X)
    outs = []
    for _ in range(2):
        acc = torch.zeros(D, dtype=torch.float32, device="cuda")
        b.nvfp4_outlier_accumulate(to_dev_bf16(X), acc)
        torch.cuda.synchronize()
        outs.append(acc.cpu().numpy())
    assert np.array_equal(outs[0], outs[1])
    assert outs[0][0] == 0.0 and outs[0][2] == 5.0 and abs(outs[0][1] - 3.0 * np.sqrt(N)) <= 1e-5 * 3.0 * np.sqrt(N)


@pytest.mark.parametrize("D,n_out", [(8, 0), (8, 8), (40, 7), (1000, 100), (1024, 10), (5000, 500), (16384, 1638)])
def test_select_is_identical_on_float32_inputs(D, n_out):
    """The selection is integer work on given float32 values: bit-exact against the oracle, ties included."""
    b = B()
    rng = np.random.default_rng(D)
    acc = rng.integers(0, max(4, D // 3), D).astype(np.float32)  # plenty of ties
    outl_o, keep_o, cmap_o = cal.select(acc.astype(np.float64), n_out)
    outl, keep, cmap = b.nvfp4_outlier_select(torch.from_numpy(acc).cuda(), n_out)
    torch.cuda.synchronize()
    assert np.array_equal(outl.cpu().numpy(), outl_o)
    assert np.array_equal(keep.cpu().numpy(), keep_o)
    assert np.array_equal(cmap.cpu().numpy(), cmap_o)


def test_calibrated_set_drives_the_layer():
    """Window of 4 steps -> select -> the arrays are what the layer's OutControl configuration takes."""
    b = B()
    N, D, C = 256, 512, 256
    acc = torch.zeros(D, dtype=torch.float32, device="cuda")
    acc_ref = np.zeros(D)
    for step in range(4):
        X, ch = synth.activations(N, D, 200 + step, n_outlier=5, factor=30.0, channel_seed=9)
        b.nvfp4_outlier_accumulate(to_dev_bf16(X), acc)
        acc_ref = cal.accumulate(acc_ref, X)
    outl, keep, cmap = b.nvfp4_outlier_select(acc, 5)
    torch.cuda.synchronize()
    assert outl.cpu().numpy().tolist() == sorted(ch.tolist()) == cal.select(acc_ref, 5)[0].tolist()
    cfg = b.LayerConfig(gs_mode=b.GS_TENSOR, outliers=outl.cpu().numpy(), y_dtype=b.DT_F32)
    cfg.prepare(D)
    assert torch.equal(cfg._keep, keep) and torch.equal(cfg._map, cmap) and torch.equal(cfg._outl, outl)
