"""CPU oracle of OutControl's outlier-channel calibration (paper Sec. 4.2, the paragraph that defines the index set A).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, the smoke check and the bench's cpu_baseline / reference legs; the
CUDA library never imports it and it imports nothing from the CUDA path.

What the paper states: the activation l2-norms of every channel are accumulated over a short calibration window
(e.g. 50 steps), and the top p % channels by the accumulated statistic form the outlier set A; the complement is the
set of kept channels.

Readings where the paper is silent:
  * per step and per channel d the statistic is the l2-norm over that step's tokens, sqrt(sum_t X[t, d]^2), and the
    window accumulates these norms by addition;
  * |A| = n_out is given by the caller (round(p * D) is the caller's business);
  * ties at the selection boundary go to the lower channel index (a total order: value descending, index ascending);
  * outputs: A sorted ascending, its sorted complement, and the map channel -> position among the kept (-1 for A).
Everything is float64 here; the CUDA path accumulates in float32 and is compared within the tolerance that implies.
"""
from __future__ import annotations

import numpy as np


def accumulate(acc: np.ndarray, X: np.ndarray) -> np.ndarray:
    """acc[d] + ||X[:, d]||_2 for one step's activations X [N_tok, D] (float64 result)."""
    X = np.asarray(X, dtype=np.float64)
    acc = np.asarray(acc, dtype=np.float64)
    assert X.ndim == 2 and acc.shape == (X.shape[1],)
    norms = np.zeros(X.shape[1], dtype=np.float64)
    for d in range(X.shape[1]):
        col = X[:, d]
        norms[d] = np.sqrt(float(np.sum(col * col)))
    return acc + norms


def select(acc: np.ndarray, n_out: int):
    """Top-n_out channels of acc (value descending, index ascending on ties).
    Returns (outlier_cols sorted, keep_cols sorted, col_map) as int32 arrays."""
    acc = np.asarray(acc, dtype=np.float64)
    D = acc.shape[0]
    assert 0 <= n_out <= D
    # rank of d = number of channels that come before it in the total order
    order = sorted(range(D), key=lambda d: (-acc[d], d))
    chosen = np.zeros(D, dtype=bool)
    chosen[order[:n_out]] = True
    outl = np.nonzero(chosen)[0].astype(np.int32)
    keep = np.nonzero(~chosen)[0].astype(np.int32)
    col_map = np.full(D, -1, dtype=np.int32)
    col_map[keep] = np.arange(len(keep), dtype=np.int32)
    return outl, keep, col_map
