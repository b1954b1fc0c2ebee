"""Helpers of the GPU parity tests: host<->device plumbing and operand comparison (no arithmetic of the method)."""
import numpy as np
import torch

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth


def to_dev_bf16(x: np.ndarray) -> torch.Tensor:
    bits = synth.to_bf16_bits(x)
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).cuda()


def to_dev_i32(a) -> torch.Tensor:
    return torch.from_numpy(np.asarray(a, dtype=np.int32)).cuda()


def assert_operand_equal(gpu_op, ref: orc.Operand, what="", k_extended=False):
    """Bit-exact comparison of a device operand with an oracle operand: codes, scales, global scales; and the
    padding the device layout adds (K up to 128) must be zero. `k_extended`: the reference was computed on a matrix
    already zero-extended to a multiple of 16 columns (the Hadamard-transformed operands), the device operand keeps K."""
    torch.cuda.synchronize()
    assert gpu_op.R == ref.R and (gpu_op.K == ref.K or (k_extended and (gpu_op.K + 15) // 16 * 16 == ref.K)), what
    Kp = gpu_op.Kp
    K16 = ref.K16
    codes = gpu_op.codes.cpu().numpy()[: ref.R * (Kp // 2)].reshape(ref.R, Kp // 2)
    bad = np.argwhere(codes[:, : K16 // 2] != ref.codes)
    assert len(bad) == 0, f"{what}: {len(bad)} code bytes differ, first at {bad[:5].tolist()}"
    assert not codes[:, K16 // 2:].any(), f"{what}: code padding not zero"
    sf = gpu_op.sf_linear()
    bad = np.argwhere(sf[:, : K16 // 16] != ref.sf)
    assert len(bad) == 0, f"{what}: {len(bad)} scale bytes differ, first at {bad[:5].tolist()}: gpu {sf[tuple(bad[0])]} ref {ref.sf[tuple(bad[0])]}"
    assert not sf[:, K16 // 16:].any(), f"{what}: scale padding not zero"
    n = {0: 1, 1: ref.R, 2: ref.R * (Kp // 128)}[ref.gs_mode]
    gs = gpu_op.gscale.cpu().numpy()[:n]
    if ref.gs_mode == 2:
        gs = gs.reshape(ref.R, Kp // 128)[:, : ref.gscale.shape[1]]
    assert np.array_equal(gs.reshape(ref.gscale.shape).view(np.uint32), ref.gscale.view(np.uint32)), f"{what}: global scales differ"


def rel_fro(a: np.ndarray, b: np.ndarray) -> float:
    return float(np.linalg.norm(a.astype(np.float64) - b) / max(np.linalg.norm(b), 1e-300))


def upload_operand(ref: orc.Operand, binding, sf_layout=None):
    """Oracle operand -> device operand in the library's layout (padding and index shuffling only)."""
    b = binding
    sf_layout = b.SF_TILED128x4 if sf_layout is None else sf_layout
    R, K = ref.R, ref.K
    Kp = b.lib.nvfp4_padded_k(K)
    K16 = ref.K16
    codes = np.zeros((R, Kp // 2), dtype=np.uint8)
    codes[:, : K16 // 2] = ref.codes
    nb = Kp // 16
    if sf_layout == b.SF_LINEAR:
        sf = np.zeros((R, nb), dtype=np.uint8)
        sf[:, : K16 // 16] = ref.sf
    else:
        nbp = (nb + 15) // 16 * 16
        Rp = (R + 127) // 128 * 128
        sf = np.zeros(Rp * nbp, dtype=np.uint8)
        r = np.arange(R)[:, None]
        kb = np.arange(K16 // 16)[None, :]
        off = ((r >> 7) * (nbp >> 2) + (kb >> 2)) * 512 + (r & 31) * 16 + ((r >> 5) & 3) * 4 + (kb & 3)
        sf[off] = ref.sf
    if ref.gs_mode == 2:
        gs = np.ones((R, Kp // 128), dtype=np.float32)
        gs[:, : ref.gscale.shape[1]] = ref.gscale
    else:
        gs = ref.gscale
    op = b.Operand(torch.from_numpy(codes.reshape(-1)).cuda(), torch.from_numpy(sf.reshape(-1)).cuda(),
                   torch.from_numpy(np.ascontiguousarray(gs).reshape(-1)).cuda(), R, K, ref.gs_mode, sf_layout)
    return op


def bf16_ulp_close(got: np.ndarray, want64: np.ndarray, ulps=1.0, noise=0.0):
    """|got - want| <= ulps * (BF16 spacing at |want|) + noise, elementwise. `noise` is the absolute FP32
    accumulation error allowed before the single BF16 rounding (it matters where the sum cancels to ~0)."""
    mag = np.maximum(np.abs(want64), 1e-300)
    spacing = 2.0 ** (np.floor(np.log2(mag)) - 7)
    return np.abs(got.astype(np.float64) - want64) <= ulps * spacing + noise + 1e-300


# ------------------------------------------------------------------------------------------------------------
# products at sizes the oracle cannot multiply in full: sampled entries and tiles, FP64 dot products one by one
# ------------------------------------------------------------------------------------------------------------
def sample_positions(M, N, rng, n_scatter=4096, n_tiles=4, tile=32):
    ms = [rng.integers(0, M, n_scatter)]
    ns = [rng.integers(0, N, n_scatter)]
    for _ in range(n_tiles):
        m0, n0 = rng.integers(0, M - tile + 1), rng.integers(0, N - tile + 1)
        mm, nn = np.meshgrid(np.arange(m0, m0 + tile), np.arange(n0, n0 + tile), indexing="ij")
        ms.append(mm.ravel())
        ns.append(nn.ravel())
    # always include the corners and the last row / column
    ms.append(np.array([0, 0, M - 1, M - 1]))
    ns.append(np.array([0, N - 1, 0, N - 1]))
    return np.concatenate(ms).astype(np.int64), np.concatenate(ns).astype(np.int64)


def check_sampled(got: torch.Tensor, A64, B64, rng, bf16_out, name):
    M, N = got.shape
    ms, ns = sample_positions(M, N, rng)
    want, absdot = orc.gemm_tn_samples(A64, B64, ms, ns)
    g = got[torch.from_numpy(ms).cuda(), torch.from_numpy(ns).cuda()].float().cpu().numpy().astype(np.float64)
    tol = 1e-3 * absdot  # |err| <= 1e-3 * sum_k |a_k b_k| elementwise
    if bf16_out:
        tol = tol + np.abs(want) * 2.0 ** -8  # one BF16 rounding of the result
    bad = np.abs(g - want) > tol + 1e-300
    assert not bad.any(), (name, int(bad.sum()), float(np.abs(g - want).max()))
    rel = np.linalg.norm(g - want) / np.linalg.norm(want)
    assert rel <= (4e-3 if bf16_out else 1e-3), (name, rel)


def check_layer_at_size(b, cfg_id, T, D, C, gs_mode, *, weight_id, swiglu=False, n_out=0, rng_seed=0, rht=False, name=""):
    """One linear of a BASELINE configuration at its full size through nvfp4_linear_fwd + nvfp4_linear_bwd (the calls bench.py
    times): all six operands bit for bit against the oracle (Q3..Q6 read back from the backward workspace), Y / dX / dW on
    sampled entries and tiles; with OutControl (n_out outlier channels) also the side operands and dW's outlier columns."""
    c = synth.CONFIGS[cfg_id]
    X, W, dY, _ = synth.layer_inputs(cfg_id, T, D, C, n_outlier=max(1, D // 100), factor=c["factor"], grad_scale=c["grad_scale"],
                                     weight_id=weight_id, swiglu=swiglu)
    outl = synth.outlier_channels(D, n_out, synth.seed_of(cfg_id, 50)) if n_out else None
    cfg = b.LayerConfig(gs_mode=gs_mode, seed=0, y_dtype=b.DT_BF16, dx_dtype=b.DT_BF16, dw_dtype=b.DT_F32, outliers=outl, rht=rht)
    Xd, Wd, dYd = to_dev_bf16(X), to_dev_bf16(W), to_dev_bf16(dY)
    Y, saved = b.nvfp4_linear_fwd(Xd, Wd, cfg)
    ws = b.linear_workspace(b.OP_BWD, T, D, C, cfg)
    dX, dW = b.nvfp4_linear_bwd(dYd, saved, cfg, workspace=ws)
    torch.cuda.synchronize()
    rng = np.random.default_rng(rng_seed)
    keep = np.arange(D) if outl is None else np.setdiff1d(np.arange(D), outl)
    outl_idx = np.zeros(0, dtype=np.int64) if outl is None else np.asarray(outl)
    q1 = orc.quantize(X[:, keep], orc.AXIS_ROW, orc.RTN, gs_mode, 0, 1)
    q2 = orc.quantize(W[:, keep], orc.AXIS_ROW, orc.RTN, gs_mode, 0, 2)
    assert_operand_equal(saved.qx, q1, f"{name} Q1(X)")
    assert_operand_equal(saved.qw, q2, f"{name} Q2(W)")
    A64, B64 = orc.dequantize(q1), orc.dequantize(q2)
    if n_out:
        assert np.array_equal(saved.X_out.float().cpu().numpy()[:, :n_out], X[:, outl_idx])
        assert np.array_equal(saved.W_out.float().cpu().numpy()[:, :n_out], W[:, outl_idx])
        assert not saved.X_out[:, n_out:].any() and not saved.W_out[:, n_out:].any()
        A64 = np.concatenate([A64, X[:, outl_idx].astype(np.float64)], axis=1)
        B64 = np.concatenate([B64, W[:, outl_idx].astype(np.float64)], axis=1)
    check_sampled(Y, A64, B64, rng, True, f"{name} Y")
    del A64, B64
    # dX = Q3(dY) Q4(W-hat^T)
    W_hat = orc.aligned_full(q2, keep, outl_idx, W[:, outl_idx], D)
    a3, a4 = dY, np.ascontiguousarray(W_hat.T)
    if rht:
        a3, a4 = orc.rht16(a3, 0, orc.STREAM_RHT_DX), orc.rht16(a4, 0, orc.STREAM_RHT_DX)
    q3 = orc.quantize(a3, orc.AXIS_ROW, orc.SR, gs_mode, 0, 3)
    q4 = orc.quantize(a4, orc.AXIS_ROW, orc.SR, gs_mode, 0, 4)
    assert_operand_equal(b.nvfp4_linear_bwd_operand(b.OP_BWD, 3, T, D, C, cfg, ws), q3, f"{name} Q3(dY)", k_extended=rht)
    assert_operand_equal(b.nvfp4_linear_bwd_operand(b.OP_BWD, 4, T, D, C, cfg, ws), q4, f"{name} Q4(W-hat^T)", k_extended=rht)
    check_sampled(dX, orc.dequantize(q3), orc.dequantize(q4), rng, True, f"{name} dX")
    del q3, q4, a3, a4
    # dW[:, keep] = Q5(dY^T) Q6(X-hat^T[keep]); dW[:, outl] = dY^T X[:, outl]
    a5, a6 = np.ascontiguousarray(dY.T), np.ascontiguousarray(orc.rematerialize_f32(q1).T)
    if rht:
        a5, a6 = orc.rht16(a5, 0, orc.STREAM_RHT_DW), orc.rht16(a6, 0, orc.STREAM_RHT_DW)
    q5 = orc.quantize(a5, orc.AXIS_ROW, orc.SR, gs_mode, 0, 5)
    q6 = orc.quantize(a6, orc.AXIS_ROW, orc.SR, gs_mode, 0, 6)
    assert_operand_equal(b.nvfp4_linear_bwd_operand(b.OP_BWD, 5, T, D, C, cfg, ws), q5, f"{name} Q5(dY^T)", k_extended=rht)
    assert_operand_equal(b.nvfp4_linear_bwd_operand(b.OP_BWD, 6, T, D, C, cfg, ws), q6, f"{name} Q6(X-hat^T)", k_extended=rht)
    dW_keep = dW if not n_out else dW[:, torch.from_numpy(keep).cuda()]
    check_sampled(dW_keep, orc.dequantize(q5), orc.dequantize(q6), rng, False, f"{name} dW")
    if n_out:
        got = dW[:, torch.from_numpy(outl_idx).cuda()].cpu().numpy().astype(np.float64)
        g64, x64 = dY.astype(np.float64), X[:, outl_idx].astype(np.float64)
        want = g64.T @ x64
        absdot = np.abs(g64).T @ np.abs(x64)
        assert np.all(np.abs(got - want) <= 1e-3 * absdot + 1e-300), f"{name} dW outlier columns"
        assert np.linalg.norm(got - want) <= 1e-5 * np.linalg.norm(want)
