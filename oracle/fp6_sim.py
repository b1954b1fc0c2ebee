"""CPU oracle of the simulated FP6 x FP4 linear layer of the paper's precision-switching study (Sec. 5.4, paragraph
"Precision Switching in Final Stage"):

    Y  = Q6_D(X)    x Q4_D(W^T)                       (D: deterministic rounding, S: stochastic rounding)
    dX = Q6_S(dY)   x Q4_S(W-hat)
    dW = Q4_S(dY^T) x Q6_S(X-hat)                     X-hat = dequantized Q6_D(X), W-hat = dequantized Q4_D(W)

TEST INFRASTRUCTURE ONLY: imported by ``tests/``; the CUDA library never imports it.

PARITY UNPINNED with respect to the paper: it names "FP6" and gives the three products above, nothing else. This build's
own definition of the FP6 quantizer, chosen as the smallest change to the paper's FP4 quantizer (Sec. 2.1 - 2.2):
  * element format E2M3 (sign, 2 exponent bits with bias 1, 3 mantissa bits; 32 magnitudes 0, 1/8, ..., 7/8 (subnormal),
    1 ... 1.875 (step 1/8), 2 ... 3.75 (step 1/4), 4 ... 7.5 (step 1/2); no infinities, no NaN) -- E2M1 with two more
    mantissa bits, so every E2M1 value is an E2M3 value;
  * the same double-block scaling with Q_max = 7.5 in place of 6:  Sg = amax_g / 3360 (= 448 * 7.5; 1 for an all-zero
    group);  t = amax_b / Sg;  s = t / 7.5;  Sb = e4m3(s);  d = Sg Sb;  r = 1 / d (0 if Sb = 0);  y = x r, each one binary32
    operation, then |y| is clamped to 7.5;
  * round to nearest with ties to the even code; stochastic rounding with the same 16-bit draws, the same Philox
    addressing (element idx = row * K16 + k of the operand, 16 bits per element) and the same rule as the FP4 quantizer:
    round the magnitude up iff (u + 0.5) / 65536 < (a - q1) / (q2 - q1);
  * per-tensor (TENSOR) or per-row (ROW) FP32 scales; the 1x128 outer block is not part of the simulation;
  * FP4 operands are this repository's ordinary ones (oracle/nvfp4_oracle.py); products are FP64 sums of the dequantized
    operands, like everywhere else; no OutControl, no Hadamard transformation (the paper's formulas show neither).
Stream ids: Q6_D(X) 1, Q4_D(W) 2, Q6_S(dY) 3, Q4_S(W-hat^T) 4, Q4_S(dY^T) 5, Q6_S(X-hat^T) 6 -- the ids of the quantizers
they replace.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

from oracle import nvfp4_oracle as orc

QMAX = 7.5


def e2m3_value(code: int) -> float:
    """Magnitude of the 5-bit code (exponent = code >> 3, mantissa = code & 7)."""
    e, m = code >> 3, code & 7
    return m / 8.0 if e == 0 else 2.0 ** (e - 1) * (1.0 + m / 8.0)


MAGS = np.array([e2m3_value(c) for c in range(32)], dtype=np.float64)


def round_rtn_mag(a: np.ndarray) -> np.ndarray:
    """Code of the nearest magnitude for every a in [0, 7.5]; a tie goes to the even code."""
    hi = np.minimum(np.searchsorted(MAGS, a, side="left"), 31)
    lo = np.maximum(hi - 1, 0)
    d_lo, d_hi = a - MAGS[lo], MAGS[hi] - a
    pick_hi = (d_hi < d_lo) | ((d_hi == d_lo) & (hi % 2 == 0))
    return np.where(pick_hi, hi, lo).astype(np.uint8)


def round_sr_mag(a: np.ndarray, u: np.ndarray) -> np.ndarray:
    """Stochastic rounding of magnitudes a in [0, 7.5] with 16-bit draws u: q1 <= a < q2 neighbouring magnitudes, up iff
    (u + 0.5) / 65536 < (a - q1) / (q2 - q1). All quantities are dyadic rationals that binary64 holds exactly."""
    lo = np.clip(np.searchsorted(MAGS, a, side="right") - 1, 0, 31)
    hi = np.minimum(lo + 1, 31)
    q1, q2 = MAGS[lo], MAGS[hi]
    width = np.where(hi > lo, q2 - q1, 1.0)
    frac = (a - q1) / width  # exact: a - q1 is exact, the width is a power of two
    up = (hi > lo) & ((u.astype(np.float64) + 0.5) / 65536.0 < frac)
    return np.where(up, hi, lo).astype(np.uint8)


@dataclass
class Fp6Operand:
    codes: np.ndarray   # uint8 [R, K16]: sign << 5 | magnitude code
    sf: np.ndarray      # uint8 [R, K16 / 16] E4M3 block scales
    gscale: np.ndarray  # float32 [1] (TENSOR) or [R] (ROW)
    R: int
    K: int
    gs_mode: int

    @property
    def K16(self) -> int:
        return self.codes.shape[1]


def _draws(seed: int, stream_id: int, idx0: int, n: int) -> np.ndarray:
    return np.array([orc.sr_bits(seed, stream_id, idx0 + i) for i in range(n)], dtype=np.uint32)


def quantize(x: np.ndarray, axis: int = orc.AXIS_ROW, rounding: int = orc.RTN, gs_mode: int = orc.GS_TENSOR, seed: int = 0,
             stream_id: int = 0) -> Fp6Operand:
    """The FP6 double-block quantizer; ``axis = AXIS_COL`` is, by definition, the quantizer applied to the transposed matrix."""
    assert gs_mode in (orc.GS_TENSOR, orc.GS_ROW) and rounding in (orc.RTN, orc.SR)
    x = np.asarray(x, dtype=np.float32)
    if axis == orc.AXIS_COL:
        x = x.T
    x = np.ascontiguousarray(x)
    R, K = x.shape
    K16 = (K + 15) // 16 * 16
    xp = np.zeros((R, K16), dtype=np.float32)
    xp[:, :K] = x
    codes = np.zeros((R, K16), dtype=np.uint8)
    sf = np.zeros((R, K16 // 16), dtype=np.uint8)
    f32 = np.float32
    if gs_mode == orc.GS_TENSOR:
        amax_t = f32(np.max(np.abs(x))) if x.size else f32(0)
        g_all = np.full(R, f32(1.0) if amax_t == 0 else f32(amax_t / f32(3360.0)), dtype=np.float32)
        gscale = g_all[:1].copy() if R else np.ones(1, dtype=np.float32)
    else:
        amax_r = np.max(np.abs(x), axis=1) if K else np.zeros(R, dtype=np.float32)
        g_all = np.where(amax_r == 0, f32(1.0), (amax_r / f32(3360.0)).astype(np.float32)).astype(np.float32)
        gscale = g_all.copy()
    for r in range(R):
        Sg = g_all[r]
        for b in range(K16 // 16):
            blk = xp[r, 16 * b:16 * b + 16]
            amax_b = f32(np.max(np.abs(blk)))
            t = f32(amax_b / Sg)
            s = f32(t / f32(7.5))
            sb = orc.e4m3_encode(float(s))
            Sbf = f32(orc.e4m3_value(sb))
            sf[r, b] = sb
            d = f32(Sg * Sbf)
            rcp = f32(0.0) if Sbf == 0 else f32(f32(1.0) / d)
            y = (blk * rcp).astype(np.float32)  # one binary32 multiply per element
            a = np.minimum(np.abs(y.astype(np.float64)), QMAX)
            if rounding == orc.RTN:
                m = round_rtn_mag(a)
            else:
                m = round_sr_mag(a, _draws(seed, stream_id, r * K16 + 16 * b, 16))
            codes[r, 16 * b:16 * b + 16] = np.where(np.signbit(blk), 32, 0).astype(np.uint8) | m
    return Fp6Operand(codes, sf, gscale, R, K, gs_mode)


def block_values(op: Fp6Operand) -> np.ndarray:
    """P * S_block as float32 [R, K16]: exact (at most 8 significant bits), and exactly representable in BF16."""
    mag = MAGS[op.codes & 31]
    sign = np.where(op.codes & 32, -1.0, 1.0)
    sb = np.array([orc.e4m3_value(int(b)) for b in range(256)], dtype=np.float64)[op.sf]
    return (sign * mag * np.repeat(sb, 16, axis=1)).astype(np.float32)


def _row_scale(op) -> np.ndarray:
    return (np.full(op.R, op.gscale[0], dtype=np.float32) if op.gs_mode == orc.GS_TENSOR else op.gscale.astype(np.float32))


def dequantize(op: Fp6Operand) -> np.ndarray:
    """Exact values P * S_block * S_global as float64 [R, K16]."""
    return block_values(op).astype(np.float64) * _row_scale(op).astype(np.float64)[:, None]


def rematerialize_f32(op: Fp6Operand) -> np.ndarray:
    """The aligned tensor the backward re-quantizer reads: float32((P * S_block) * S_global), [R, K]."""
    v = (block_values(op) * _row_scale(op)[:, None]).astype(np.float32)  # one binary32 multiply per element
    return np.ascontiguousarray(v[:, : op.K])


def fp4_block_values(op: orc.Operand) -> np.ndarray:
    """P * S_block of an ordinary FP4 operand as float32 [R, K16] (what the simulated products read as BF16)."""
    one = orc.Operand(op.codes, op.sf, np.ones_like(op.gscale), op.R, op.K, op.gs_mode)
    return orc.dequantize(one).astype(np.float32)


@dataclass
class Saved:
    qx6: Fp6Operand
    qw: orc.Operand


def linear_fwd(X: np.ndarray, W: np.ndarray, gs_mode: int = orc.GS_TENSOR):
    """Y = Q6_D(X) x Q4_D(W)^T, FP64 accumulation of the dequantized operands."""
    qx6 = quantize(X, orc.AXIS_ROW, orc.RTN, gs_mode, stream_id=1)
    qw = orc.quantize(W, orc.AXIS_ROW, orc.RTN, gs_mode, stream_id=2)
    Y = orc.gemm_tn(dequantize(qx6), orc.dequantize(qw))
    return Y[:, : W.shape[0]], Saved(qx6, qw)


def linear_bwd_dx(dY: np.ndarray, saved: Saved, seed: int = 0, gs_mode: int = orc.GS_TENSOR):
    """dX = Q6_S(dY) x Q4_S(W-hat^T)^T: both operands quantized along C. Returns (dX, Q6_S(dY), Q4_S(W-hat^T))."""
    q3 = quantize(dY, orc.AXIS_ROW, orc.SR, gs_mode, seed, 3)
    q4 = orc.quantize(orc.rematerialize_f32(saved.qw), orc.AXIS_COL, orc.SR, gs_mode, seed, 4)
    return orc.gemm_tn(dequantize(q3), orc.dequantize(q4)), q3, q4


def linear_bwd_dw(dY: np.ndarray, saved: Saved, seed: int = 0, gs_mode: int = orc.GS_TENSOR):
    """dW = Q4_S(dY^T) x Q6_S(X-hat^T)^T: both operands quantized along the tokens. Returns (dW, Q4_S(dY^T), Q6_S(X-hat^T))."""
    q5 = orc.quantize(dY, orc.AXIS_COL, orc.SR, gs_mode, seed, 5)
    q6 = quantize(rematerialize_f32(saved.qx6), orc.AXIS_COL, orc.SR, gs_mode, seed, 6)
    return orc.gemm_tn(orc.dequantize(q5), dequantize(q6)), q5, q6
