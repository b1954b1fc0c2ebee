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


# ----------------------------------------------------------------------------------------------------------------
# Memory-efficient statistics (appendix Algorithm 3, "UpdateOscillationStats_MemoryEfficient"): only the elements
# closest to a rounding threshold at t0 = 0 are tracked.
#
# What the paper states: at t0 = 0 the sensitivity score s = |W - Q(W)| / binwidth(Q(W)) is computed, idx = indices of
# the top-p_sample % elements of s; D_M~ = D_Q~ = 0 and the snapshots W'_M~ = W[idx], W'_Q~ = Q(W)[idx] are taken.
# Afterwards, per step: D_M~ += |W[idx] - W'_M~|, D_Q~ += |Q(W)[idx] - W'_Q~|, snapshots <- current values.
#
# Readings where the paper is silent:
#   * binwidth(q) for q = P * S_block * S_global is (upper - lower rounding threshold of the E2M1 value P) * S_block *
#     S_global, thresholds being the midpoints between neighbouring values: widths 0.5, 0.5, 0.5, 0.5, 0.75, 1, 1.5 for
#     |P| = 0, 0.5, 1, 1.5, 2, 3, 4 (the bin of 0 is [-0.25, 0.25]) and 2 for |P| = 6 (the bin [5, 6] mirrored at 6, so
#     that a value at the threshold 5 scores 0.5 like every other threshold approached from its wider side);
#     a block whose scale is 0 (all magnitudes 0) scores 0;
#   * the number of tracked elements n_track is given by the caller (its rounding of p_sample % of the size);
#   * ties in s go to the lower linear index r * D + c; idx is stored sorted ascending;
#   * float32 throughout, one binary32 operation each: s = float32(|w - q|) / float32(width * float32(Sg * Sb_value));
#     the master value (not its BF16 cast) enters |W - Q(W)|;
#   * the reset (Algorithm 1) over the tracked subset: W[idx[i]] <- Q(W)[idx[i]] where D_Q~[i] / D_M~[i] >= tau.
# ----------------------------------------------------------------------------------------------------------------
_BINWIDTH = np.array([0.5, 0.5, 0.5, 0.5, 0.75, 1.0, 1.5, 2.0], dtype=np.float32)  # by magnitude index of P


def sensitivity(W: np.ndarray, gs_mode: int) -> np.ndarray:
    """s = |W - Q(W)| / binwidth(Q(W)), float32 [C, D]."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    C, D = W.shape
    op = orc.quantize(bf16_round(W), orc.AXIS_ROW, orc.RTN, gs_mode)
    q = orc.rematerialize_f32(op)
    K16 = op.K16
    lo = (op.codes & 0x0F).astype(np.int64)
    hi = (op.codes >> 4).astype(np.int64)
    codes = np.empty((C, K16), dtype=np.int64)
    codes[:, 0::2] = lo
    codes[:, 1::2] = hi
    mag = (codes & 7)[:, :D]
    sb = np.array([orc.e4m3_value(int(b)) for b in range(256)], dtype=np.float32)[op.sf]  # [C, K16/16]
    sb = np.repeat(sb, 16, axis=1)[:, :D]
    if gs_mode == orc.GS_TENSOR:
        sg = np.full((C, D), op.gscale[0], dtype=np.float32)
    elif gs_mode == orc.GS_ROW:
        sg = np.repeat(op.gscale.reshape(C, 1), D, axis=1).astype(np.float32)
    else:
        sg = np.repeat(op.gscale.reshape(C, -1), 128, axis=1)[:, :D].astype(np.float32)
    d = (sg * sb).astype(np.float32)  # float32(Sg * Sb)
    width = (_BINWIDTH[mag] * d).astype(np.float32)
    err = np.abs(W - q).astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        s = (err / width).astype(np.float32)
    s[d == 0.0] = 0.0
    return s


def select_tracked(s: np.ndarray, n_track: int) -> np.ndarray:
    """Linear indices (sorted ascending, int64) of the n_track largest scores; ties to the lower index."""
    flat = s.reshape(-1)
    order = np.lexsort((np.arange(flat.size), -flat.astype(np.float64)))  # primary: score descending; secondary: index
    return np.sort(order[:n_track]).astype(np.int64)


class SparseStats:
    def __init__(self, n_track: int):
        self.idx = np.zeros(n_track, dtype=np.int64)
        self.WM_prev = np.zeros(n_track, dtype=np.float32)
        self.WQ_prev = np.zeros(n_track, dtype=np.float32)
        self.D_M = np.zeros(n_track, dtype=np.float32)
        self.D_Q = np.zeros(n_track, dtype=np.float32)


def update_stats_sparse(W: np.ndarray, st: SparseStats, t0: int, gs_mode: int) -> None:
    """Algorithm 3 for one matrix (in place on ``st``)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    q = quant_dequant(W, gs_mode)
    if t0 == 0:
        st.idx = select_tracked(sensitivity(W, gs_mode), len(st.idx))
        st.D_M[...] = 0.0
        st.D_Q[...] = 0.0
        st.WM_prev = W.reshape(-1)[st.idx].copy()
        st.WQ_prev = q.reshape(-1)[st.idx].copy()
        return
    wm = W.reshape(-1)[st.idx]
    wq = q.reshape(-1)[st.idx]
    st.D_M = (st.D_M + np.abs(wm - st.WM_prev)).astype(np.float32)
    st.D_Q = (st.D_Q + np.abs(wq - st.WQ_prev)).astype(np.float32)
    st.WM_prev = wm.copy()
    st.WQ_prev = wq.copy()


def suppress_sparse(W: np.ndarray, st: SparseStats, tau: float, gs_mode: int):
    """Algorithm 1 over the tracked subset: returns (new W, boolean mask over the tracked elements)."""
    W = np.ascontiguousarray(W, dtype=np.float32)
    q = quant_dequant(W, gs_mode)
    with np.errstate(divide="ignore", invalid="ignore"):
        risk = (st.D_Q / st.D_M).astype(np.float32)
    hit = risk >= np.float32(tau)
    out = W.copy()
    flat = out.reshape(-1)
    flat[st.idx[hit]] = q.reshape(-1)[st.idx[hit]]
    return out, hit
