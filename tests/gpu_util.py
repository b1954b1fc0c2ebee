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
