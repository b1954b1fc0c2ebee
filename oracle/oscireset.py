"""CPU oracle of OsciReset's per-element statistics and reset (paper Sec. 3.2-3.3; Algorithm 1 "OscillationSuppress",
Algorithm 2 "UpdateOscillationStats" of the appendix).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, the smoke check and the bench's cpu_baseline / reference legs; the
CUDA library never imports it and it imports nothing from the CUDA path.

What the paper states, for every element w of a quantized weight matrix over a tracking interval:
    dist_M(w) = sum_t |w(t) - w(t-1)|                 (master weight path length)
    dist_Q(w) = sum_t |Q(w(t)) - Q(w(t-1))|           (quantized weight path length; Q = FP4 quant-dequant)
    OsciRisk(w) = dist_Q(w) / dist_M(w);  if OsciRisk(w) >= tau:  w <- w_FP4 * scale   (the centre of its bin)
Algorithm 2 keeps D_M, D_Q and a snapshot W' of the previous step's weights: at t0 = 0 it clears D_M, D_Q and sets
W' <- W; afterwards D_M += |W - W'|, D_Q += |Q(W) - Q(W')|, W' <- W.

Readings where the paper is silent:
  * master weights, the snapshot and both statistics are float32 matrices; every operation is one binary32 operation
    (subtract, absolute value, add; divide and compare for the risk), so results are defined bit for bit;
  * Q(W) is what the layer's forward weight quantizer represents: the master weights are cast to BF16 (round to
    nearest even), double-block quantized along the input-feature axis with round-to-nearest in the configured
    global-scale mode (Sec. 2.2), and dequantized as float32((P * S_block) * S_global);
  * "w_FP4 * scale" is that same dequantized value;
  * 0 / 0 (an element that never moved) is not >= tau: no reset; x / 0 with x > 0 cannot occur (Q moves only if w does);
  * the statistics are left as they are by the reset (the trainer clears them at the next t0 = 0).
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import nvfp4_oracle as orc


def bf16_round(w: np.ndarray) -> np.ndarray:
    """float32 -> nearest BF16 (ties to even), returned as float32; torch's CPU cast is the library primitive used."""
    t = torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32))
    return t.to(torch.bfloat16).to(torch.float32).numpy()


def quant_dequant(W: np.ndarray, gs_mode: int) -> np.ndarray:
    """Q(W): the values the forward weight operand represents, float32 [C, D]."""
    op = orc.quantize(bf16_round(W), orc.AXIS_ROW, orc.RTN, gs_mode)
    return orc.rematerialize_f32(op)


class Stats:
    """State of Algorithm 2 for one weight matrix."""

    def __init__(self, shape):
        self.W_prev = np.zeros(shape, dtype=np.float32)
        self.D_M = np.zeros(shape, dtype=np.float32)
        self.D_Q = np.zeros(shape, dtype=np.float32)


def update_stats(W: np.ndarray, st: Stats, t0: int, gs_mode: int) -> None:
    """Algorithm 2 for one matrix (in place on ``st``)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    if t0 == 0:
        st.D_M[...] = 0.0
        st.D_Q[...] = 0.0
        st.W_prev[...] = W
        return
    q_now = quant_dequant(W, gs_mode)
    q_prev = quant_dequant(st.W_prev, gs_mode)
    st.D_M = (st.D_M + np.abs(W - st.W_prev)).astype(np.float32)
    st.D_Q = (st.D_Q + np.abs(q_now - q_prev)).astype(np.float32)
    st.W_prev = W.copy()


def suppress(W: np.ndarray, st: Stats, tau: float, gs_mode: int):
    """Algorithm 1 for one matrix: returns (new W, boolean mask of the reset elements)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    q = quant_dequant(W, gs_mode)
    with np.errstate(divide="ignore", invalid="ignore"):
        risk = (st.D_Q / st.D_M).astype(np.float32)
    mask = risk >= np.float32(tau)  # NaN compares false
    out = W.copy()
    out[mask] = q[mask]
    return out, mask
