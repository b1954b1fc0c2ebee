"""CPU oracle of the 16x16 weight-block recipe that the paper compares its 1x16 weight blocks with (Sec. 2.3, the list of
differences to NVIDIA's recipe, third item; appendix "overhead of the 1x16 weight scaling scheme": the 16x16 baseline
"does not require weight re-quantization" in backward).

TEST INFRASTRUCTURE ONLY: imported by ``tests/`` and by the oracle's layer functions; the CUDA library never imports it.

What the paper fixes: the weight scale group is a 16x16 square instead of 1x16, so W and W^T carry the same quantized
values and dX = Q3(dY) x W-hat uses the forward codes as they are (no Q4, hence no rounding and no Hadamard factor on
that product).  Readings where it is silent:
  * the FP32 global scale is per tensor (a per-row or per-1x128 scale would differ between W and W^T);
  * the block scale follows the same pinned binary32 sequence as the 1x16 quantizer (Sec. 2.2) with amax_b taken over
    the 16x16 square:  Sg = amax_t / 2688;  t = amax_b / Sg;  s = t / 6;  Sb = e4m3(s);  d = Sg Sb;  r = 1 / d;  y = w r;
    round to nearest, ties to the even code;  squares at the ragged edge of the matrix cover the rows / columns that exist;
  * the operand keeps the ordinary layout (one scale byte per row and 16 columns): the 16 rows of a square repeat it.
"""
from __future__ import annotations

import numpy as np

from oracle import nvfp4_oracle as orc


_MAGS = np.array([0.0, 0.5, 1.0, 1.5, 2.0, 3.0, 4.0, 6.0])


def rtn_mag(a: np.ndarray) -> np.ndarray:
    """Index of the nearest E2M1 magnitude of every a in [0, 6], ties to the even index (the definition, on arrays;
    checked against the scalar routine of the main oracle in the tests)."""
    hi = np.minimum(np.searchsorted(_MAGS, a, side="left"), 7)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - _MAGS[lo], _MAGS[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    return np.where(pick_hi, hi, lo).astype(np.uint8)


def quantize(W: np.ndarray) -> orc.Operand:
    """Q2 with 16x16 blocks: operand [C, D] (groups along D), per-tensor global scale, RTN."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    C, D = W.shape
    D16 = (D + 15) // 16 * 16
    codes = np.zeros((C, D16 // 2), dtype=np.uint8)
    sf = np.zeros((C, D16 // 16), dtype=np.uint8)
    amax_t = np.float32(np.max(np.abs(W))) if W.size else np.float32(0)
    Sg = np.float32(1.0) if amax_t == 0 else np.float32(amax_t / np.float32(2688.0))
    nib = np.zeros((C, D16), dtype=np.uint8)
    for r0 in range(0, C, 16):
        for b in range(D16 // 16):
            blk = W[r0:r0 + 16, 16 * b:16 * b + 16]
            if blk.size == 0:
                continue
            amax_b = np.float32(np.max(np.abs(blk)))
            t = np.float32(amax_b / Sg)
            s = np.float32(t / np.float32(6.0))
            sb = orc.e4m3_encode(float(s))
            Sbf = np.float32(orc.e4m3_value(sb))
            sf[r0:r0 + 16, b] = sb
            d = np.float32(Sg * Sbf)
            rcp = np.float32(0.0) if Sbf == 0 else np.float32(np.float32(1.0) / d)
            y = (blk * rcp).astype(np.float32)  # one binary32 multiply per element
            m = rtn_mag(np.minimum(np.abs(y.astype(np.float64)), 6.0))
            nib[r0:r0 + blk.shape[0], 16 * b:16 * b + blk.shape[1]] = np.where(np.signbit(blk), 8, 0).astype(np.uint8) | m
    codes[:, :] = nib[:, 0::2] | (nib[:, 1::2] << 4)
    return orc.Operand(codes, sf, np.array([Sg], dtype=np.float32), C, D, orc.GS_TENSOR)


def transpose_operand(op: orc.Operand) -> orc.Operand:
    """The operand of W-hat^T, [D, C] with groups along C, from the 16x16-block operand of W: codes transposed, the scale
    of (row d, block c/16) is the square's scale. No arithmetic."""
    C, D = op.R, op.K
    C16 = (C + 15) // 16 * 16
    nib = np.zeros((C, op.K16), dtype=np.uint8)
    nib[:, 0::2] = op.codes & 15
    nib[:, 1::2] = op.codes >> 4
    tn = np.zeros((D, C16), dtype=np.uint8)
    tn[:, :C] = nib[:, :D].T
    codes = (tn[:, 0::2] | (tn[:, 1::2] << 4)).astype(np.uint8)
    sf = np.zeros((D, C16 // 16), dtype=np.uint8)
    for cb in range(C16 // 16):
        sf[:, cb] = np.repeat(op.sf[16 * cb, :], 16)[:D]  # any row of the group holds the group's scales
    return orc.Operand(codes, sf, op.gscale.copy(), D, C, orc.GS_TENSOR)
