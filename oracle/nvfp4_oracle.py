"""ctypes front-end and layer-level composition for the CPU oracle (``nvfp4_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the bench's cpu_baseline /
reference legs. The CUDA library and its Python binding never import this module, and this module imports
nothing from them.

The arithmetic lives in the C file; this module only (a) builds and loads it, (b) marshals numpy arrays, and
(c) strings the quantizers and products together in the order the paper's linear-layer equations give
(Sec. 2.3 for the six quantizers and three products, Sec. 4.2 for the OutControl split). Transposes, column
gathers and scatters are pure data movement done with numpy indexing.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

RTN, SR = 0, 1
SR_SCALE_UP = 2  # stochastic rounding with the block scale rounded up to E4M3 (strictly unbiased variant)
GS_TENSOR, GS_ROW, GS_BLOCK128 = 0, 1, 2
AXIS_ROW, AXIS_COL = 0, 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nvfp4_oracle.c")
_LIB = os.path.join(_HERE, "libnvfp4_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no CUDA involved). Returns the path of the shared object."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC", _SRC, "-o", tmp, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        c_i64, c_u64, c_u32, c_int = ctypes.c_int64, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int
        vp = ctypes.c_void_p
        L.orc_e2m1_value.restype = ctypes.c_double
        L.orc_e2m1_value.argtypes = [c_int]
        L.orc_e4m3_value.restype = ctypes.c_double
        L.orc_e4m3_value.argtypes = [c_int]
        L.orc_e4m3_encode.restype = c_int
        L.orc_e4m3_encode.argtypes = [ctypes.c_float]
        L.orc_e4m3_encode_up.restype = c_int
        L.orc_e4m3_encode_up.argtypes = [ctypes.c_float]
        L.orc_philox4x32_10.restype = None
        L.orc_philox4x32_10.argtypes = [vp, vp, vp]
        L.orc_sr_bits.restype = c_u32
        L.orc_sr_bits.argtypes = [c_u64, c_u32, c_u64]
        L.orc_round_rtn_mag.restype = c_int
        L.orc_round_rtn_mag.argtypes = [ctypes.c_float]
        L.orc_round_sr_mag.restype = c_int
        L.orc_round_sr_mag.argtypes = [ctypes.c_float, c_u32]
        L.orc_quantize.restype = None
        L.orc_quantize.argtypes = [vp, c_i64, c_i64, c_int, c_int, c_u64, c_u32, vp, vp, vp]
        L.orc_dequantize.restype = None
        L.orc_dequantize.argtypes = [vp, vp, vp, c_i64, c_i64, c_int, vp]
        L.orc_rematerialize_f32.restype = None
        L.orc_rematerialize_f32.argtypes = [vp, vp, vp, c_i64, c_i64, c_int, vp]
        L.orc_rht_sign_bit.restype = c_int
        L.orc_rht_sign_bit.argtypes = [c_u64, c_u32, c_u64]
        L.orc_rht16.restype = None
        L.orc_rht16.argtypes = [vp, c_i64, c_i64, c_u64, c_u32, vp]
        L.orc_gemm_tn_f64.restype = None
        L.orc_gemm_tn_f64.argtypes = [vp, vp, c_i64, c_i64, c_i64, vp]
        L.orc_gemm_tn_f64_samples.restype = None
        L.orc_gemm_tn_f64_samples.argtypes = [vp, vp, c_i64, vp, vp, c_i64, vp, vp]
        _lib = L
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def threads() -> int:
    """Number of OpenMP threads the C loops use (OMP_NUM_THREADS, else the affinity mask)."""
    env = os.environ.get("OMP_NUM_THREADS")
    return int(env) if env else len(os.sched_getaffinity(0))


# ------------------------------------------------------------------------------------------------------------
# scalar helpers
# ------------------------------------------------------------------------------------------------------------
def e2m1_value(code: int) -> float:
    return lib().orc_e2m1_value(int(code))


def e4m3_value(byte: int) -> float:
    return lib().orc_e4m3_value(int(byte))


def e4m3_encode(s: float) -> int:
    return lib().orc_e4m3_encode(float(s))


def e4m3_encode_up(s: float) -> int:
    """Byte of the smallest E4M3 value >= s (0x7E if none): the block scale of the SR_SCALE_UP variant."""
    return lib().orc_e4m3_encode_up(float(s))


def philox4x32_10(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().orc_philox4x32_10(_p(c), _p(k), _p(out))
    return out


def sr_bits(seed: int, stream_id: int, idx: int) -> int:
    return lib().orc_sr_bits(int(seed), int(stream_id), int(idx))


def round_rtn_mag(a: float) -> int:
    return lib().orc_round_rtn_mag(float(a))


def round_sr_mag(a: float, u: int) -> int:
    return lib().orc_round_sr_mag(float(a), int(u))


# ------------------------------------------------------------------------------------------------------------
# quantized operand
# ------------------------------------------------------------------------------------------------------------
@dataclass
class Operand:
    """A quantized matrix in operand orientation [R, K] (groups along K). K16 = K rounded up to 16."""

    codes: np.ndarray  # uint8 [R, K16/2], low nibble = even k
    sf: np.ndarray  # uint8 [R, K16/16], E4M3
    gscale: np.ndarray  # float32 [1] | [R] | [R, ceil(K/128)]
    R: int
    K: int
    gs_mode: int

    @property
    def K16(self) -> int:
        return (self.K + 15) // 16 * 16


def quantize(x: np.ndarray, axis: int = AXIS_ROW, rounding: int = RTN, gs_mode: int = GS_TENSOR, seed: int = 0,
             stream_id: int = 0) -> Operand:
    """Double-block quantization (Sec. 2.2). ``axis=AXIS_COL`` is, by definition, the quantizer applied to the
    transposed matrix: the result has shape [cols, rows]."""
    x = np.asarray(x, dtype=np.float32)
    if axis == AXIS_COL:
        x = x.T
    x = np.ascontiguousarray(x)
    R, K = x.shape
    K16 = (K + 15) // 16 * 16
    codes = np.zeros((R, K16 // 2), dtype=np.uint8)
    sf = np.zeros((R, K16 // 16), dtype=np.uint8)
    ng = (K + 127) // 128
    gshape = {GS_TENSOR: (1,), GS_ROW: (R,), GS_BLOCK128: (R, ng)}[gs_mode]
    gscale = np.zeros(gshape, dtype=np.float32)
    lib().orc_quantize(_p(x), R, K, rounding, gs_mode, seed, stream_id, _p(codes), _p(sf), _p(gscale))
    return Operand(codes, sf, gscale, R, K, gs_mode)


def dequantize(op: Operand) -> np.ndarray:
    """Exact values P * S_block * S_global as float64 [R, K16] (padding columns are 0)."""
    out = np.zeros((op.R, op.K16), dtype=np.float64)
    lib().orc_dequantize(_p(op.codes), _p(op.sf), _p(op.gscale), op.R, op.K, op.gs_mode, _p(out))
    return out


def rematerialize_f32(op: Operand) -> np.ndarray:
    """The aligned tensor the backward quantizers read: float32 [R, K] (padding dropped)."""
    out = np.zeros((op.R, op.K16), dtype=np.float32)
    lib().orc_rematerialize_f32(_p(op.codes), _p(op.sf), _p(op.gscale), op.R, op.K, op.gs_mode, _p(out))
    return np.ascontiguousarray(out[:, : op.K])


def rht_sign_bit(seed: int, stream_id: int, k: int) -> int:
    return lib().orc_rht_sign_bit(int(seed), int(stream_id), int(k))


def rht16(x: np.ndarray, seed: int, stream_id: int) -> np.ndarray:
    """Random Hadamard transformation along k (Sec. 4.1, block size 16): (x * s) H_16 per 16 consecutive k.
    Returns float32 [R, K16]."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    R, K = x.shape
    K16 = (K + 15) // 16 * 16
    out = np.zeros((R, K16), dtype=np.float32)
    lib().orc_rht16(_p(x), R, K, seed, stream_id, _p(out))
    return out


def gemm_tn(A: np.ndarray, B: np.ndarray) -> np.ndarray:
    """C[m, n] = sum_k A[m, k] B[n, k] in float64."""
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    M, K = A.shape
    N, K2 = B.shape
    assert K == K2
    C = np.zeros((M, N), dtype=np.float64)
    lib().orc_gemm_tn_f64(_p(A), _p(B), M, N, K, _p(C))
    return C


def gemm_tn_samples(A: np.ndarray, B: np.ndarray, ms: np.ndarray, ns: np.ndarray):
    """The same product at positions (ms[i], ns[i]) only. Returns (values, sum_k |a_k b_k|)."""
    A = np.ascontiguousarray(A, dtype=np.float64)
    B = np.ascontiguousarray(B, dtype=np.float64)
    ms = np.ascontiguousarray(ms, dtype=np.int64)
    ns = np.ascontiguousarray(ns, dtype=np.int64)
    assert A.shape[1] == B.shape[1]
    out = np.zeros(len(ms), dtype=np.float64)
    out_abs = np.zeros(len(ms), dtype=np.float64)
    lib().orc_gemm_tn_f64_samples(_p(A), _p(B), A.shape[1], _p(ms), _p(ns), len(ms), _p(out), _p(out_abs))
    return out, out_abs


def gemm_operands(a: Operand, b: Operand) -> np.ndarray:
    """Block-scaled product of two quantized operands: dequantize, then accumulate in float64."""
    return gemm_tn(dequantize(a), dequantize(b))


# ------------------------------------------------------------------------------------------------------------
# the linear layer (Sec. 2.3) with the optional OutControl split (Sec. 4.2, without the Hadamard factors)
# ------------------------------------------------------------------------------------------------------------
STREAM_Q3, STREAM_Q4, STREAM_Q5, STREAM_Q6 = 3, 4, 5, 6
STREAM_RHT_DX, STREAM_RHT_DW = 7, 8  # sign diagonals S_C (dX product) and S_N (dW product)


@dataclass
class LayerConfig:
    gs_mode: int = GS_TENSOR
    seed: int = 0
    # rounding of Q1..Q6; the paper's assignment is deterministic in forward, stochastic in backward
    rounding: tuple = (RTN, RTN, SR, SR, SR, SR)
    outliers: np.ndarray | None = None  # sorted channel indices of the set A (columns of X / W), or None
    rht: bool = False  # random Hadamard transformation of both operands of the two backward products (Sec. 4.1)
    # outlier channels on a per-tensor power-of-two scaled E4M3 grid instead of BF16 (oracle/fp8_outliers.py: this
    # build's own FP8 recipe, the paper gives none)
    outlier_fp8: bool = False
    # weights in 16x16 scale squares (the recipe the paper compares its 1x16 blocks with; oracle/w16x16.py): per-tensor
    # global scale only, no outlier channels; dX then uses the forward codes as they are (no Q4, no Hadamard factor)
    w_block16: bool = False


@dataclass
class Saved:
    """What forward leaves for backward: the two forward operands (over the kept columns) and, under
    OutControl, the high-precision columns."""

    qx: Operand  # Q1(X[:, keep])    [N_tok, Dk]
    qw: Operand  # Q2(W[:, keep])    [C, Dk]
    keep: np.ndarray  # kept (non-outlier) column indices, sorted
    outl: np.ndarray  # outlier column indices, sorted
    X_out: np.ndarray  # X[:, outl]  (bf16 values in float32)
    W_out: np.ndarray  # W[:, outl]
    D: int


def _split(D: int, outliers):
    outl = np.zeros(0, dtype=np.int64) if outliers is None else np.asarray(outliers, dtype=np.int64)
    assert np.all(np.diff(outl) > 0), "outlier indices must be sorted and unique"
    mask = np.ones(D, dtype=bool)
    mask[outl] = False
    return np.nonzero(mask)[0], outl


def linear_fwd(X: np.ndarray, W: np.ndarray, cfg: LayerConfig):
    """Y = Q1_D(X_keep) Q2_D(W_keep)^T  +  X_out W_out^T (high precision). X [N_tok, D], W [C, D]."""
    X = np.asarray(X, dtype=np.float32)
    W = np.asarray(W, dtype=np.float32)
    D = X.shape[1]
    keep, outl = _split(D, cfg.outliers)
    qx = quantize(X[:, keep], AXIS_ROW, cfg.rounding[0], cfg.gs_mode, cfg.seed, 1)
    if cfg.w_block16:
        from oracle import w16x16  # (imports this module)

        assert cfg.gs_mode == GS_TENSOR and len(outl) == 0 and cfg.rounding[1] == RTN
        qw = w16x16.quantize(W)
    else:
        qw = quantize(W[:, keep], AXIS_ROW, cfg.rounding[1], cfg.gs_mode, cfg.seed, 2)
    Y = gemm_operands(qx, qw)
    X_out = np.ascontiguousarray(X[:, outl])
    W_out = np.ascontiguousarray(W[:, outl])
    if len(outl) and cfg.outlier_fp8:
        from oracle import fp8_outliers  # (imports this module)

        X_out, W_out = fp8_outliers.snap(X_out)[0], fp8_outliers.snap(W_out)[0]
    if len(outl):
        Y = Y + gemm_tn(X_out, W_out)
    return Y, Saved(qx, qw, keep, outl, X_out, W_out, D)


def aligned_full(op: Operand, keep: np.ndarray, outl: np.ndarray, hp_cols: np.ndarray, D: int) -> np.ndarray:
    """X-hat / W-hat over all D columns: kept columns from the dequantized forward operand (float32, one
    rounding), outlier columns straight from the high-precision tensor."""
    full = np.zeros((op.R, D), dtype=np.float32)
    full[:, keep] = rematerialize_f32(op)
    full[:, outl] = hp_cols
    return full


def linear_bwd_dx(dY: np.ndarray, saved: Saved, cfg: LayerConfig) -> np.ndarray:
    """dX = Q3_S(dY) Q4_S(W-hat): one FP4 product over all D columns. dY [N_tok, C] -> dX [N_tok, D]."""
    dY = np.asarray(dY, dtype=np.float32)
    if cfg.w_block16:
        from oracle import w16x16

        q3 = quantize(dY, AXIS_ROW, cfg.rounding[2], cfg.gs_mode, cfg.seed, STREAM_Q3)
        return gemm_operands(q3, w16x16.transpose_operand(saved.qw))
    W_hat = aligned_full(saved.qw, saved.keep, saved.outl, saved.W_out, saved.D)  # [C, D]
    A, B = dY, np.ascontiguousarray(W_hat.T)  # [N_tok, C], [D, C]: both along the contraction axis C
    if cfg.rht:
        A, B = rht16(A, cfg.seed, STREAM_RHT_DX), rht16(B, cfg.seed, STREAM_RHT_DX)
    q3 = quantize(A, AXIS_ROW, cfg.rounding[2], cfg.gs_mode, cfg.seed, STREAM_Q3)
    q4 = quantize(B, AXIS_ROW, cfg.rounding[3], cfg.gs_mode, cfg.seed, STREAM_Q4)
    return gemm_operands(q3, q4)


def linear_bwd_dw(dY: np.ndarray, saved: Saved, cfg: LayerConfig) -> np.ndarray:
    """dW[:, keep] = Q5_S(dY^T) Q6_S(X-hat[:, keep]);  dW[:, outl] = dY^T X_out (high precision). -> [C, D]."""
    dY = np.asarray(dY, dtype=np.float32)
    C = dY.shape[1]
    X_hat_keep = rematerialize_f32(saved.qx)  # [N_tok, Dk]
    A, B = np.ascontiguousarray(dY.T), np.ascontiguousarray(X_hat_keep.T)  # [C, N_tok], [Dk, N_tok]: along tokens
    if cfg.rht:
        A, B = rht16(A, cfg.seed, STREAM_RHT_DW), rht16(B, cfg.seed, STREAM_RHT_DW)
    q5 = quantize(A, AXIS_ROW, cfg.rounding[4], cfg.gs_mode, cfg.seed, STREAM_Q5)
    q6 = quantize(B, AXIS_ROW, cfg.rounding[5], cfg.gs_mode, cfg.seed, STREAM_Q6)
    dW = np.zeros((C, saved.D), dtype=np.float64)
    dW[:, saved.keep] = gemm_operands(q5, q6)
    if len(saved.outl):
        dW[:, saved.outl] = gemm_tn(dY.T, saved.X_out.T)
    return dW
