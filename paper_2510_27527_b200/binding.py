"""Thin ctypes binding of the C-ABI library (``include/nvfp4.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels of ``libnvfp4_b200.so``. PyTorch is
used for device memory and streams, nothing else. There is no fallback: importing this module raises if the
shared library has not been built (``python -m paper_2510_27527_b200.build``).
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libnvfp4_b200.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2510_27527_b200.build` (no fallback exists)")
_lib = ctypes.CDLL(LIB_PATH)

# enums of include/nvfp4.h
OK = 0
ROUND_RTN, ROUND_SR = 0, 1
ROUND_SR_SCALE_UP = 2  # stochastic rounding, block scale rounded up to E4M3 (every element within +-6)
AXIS_ROW, AXIS_COL = 0, 1
GS_TENSOR, GS_ROW, GS_BLOCK128 = 0, 1, 2
SF_LINEAR, SF_TILED128x4 = 0, 1
DT_BF16, DT_F32 = 0, 1
OP_FWD, OP_BWD_DX, OP_BWD_DW, OP_BWD = 0, 1, 2, 3
GEMM_AUTO, GEMM_TILE128, GEMM_PAIR256, GEMM_PAIR192 = 0, 1, 2, 3
ERR_TIMEOUT = 8

c_i64, c_i32, c_u64, c_u32, c_vp, c_sz = (ctypes.c_int64, ctypes.c_int32, ctypes.c_uint64, ctypes.c_uint32,
                                          ctypes.c_void_p, ctypes.c_size_t)


class COperand(ctypes.Structure):
    _fields_ = [("codes", c_vp), ("sf", c_vp), ("gscale", c_vp), ("R", c_i64), ("K", c_i64), ("gs_mode", c_i32),
                ("sf_layout", c_i32)]


class CLayerCfg(ctypes.Structure):
    _fields_ = [("gs_mode", c_i32), ("rounding", c_i32 * 6), ("seed", c_u64), ("y_dtype", c_i32), ("dx_dtype", c_i32),
                ("dw_dtype", c_i32), ("n_out", c_i64), ("outlier_cols", c_vp), ("keep_cols", c_vp), ("col_map", c_vp),
                ("dev_status", c_vp), ("rht", c_i32), ("outlier_format", c_i32), ("weight_block", c_i32),
                ("side_stream", c_vp), ("ev_fork", c_vp), ("ev_join", c_vp), ("ev_aux", c_vp)]


class CGemmOpts(ctypes.Structure):
    _fields_ = [("variant", c_i32), ("starve_first_stage", c_i32), ("wait_limit_cycles", c_i64)]


class CDenseOperand(ctypes.Structure):
    _fields_ = [("vals", c_vp), ("gscale", c_vp), ("R", c_i64), ("K", c_i64), ("ld", c_i64)]


class CSaved(ctypes.Structure):
    _fields_ = [("qx", COperand), ("qw", COperand), ("X", c_vp), ("W", c_vp), ("ldx", c_i64), ("ldw", c_i64),
                ("N_tok", c_i64), ("D", c_i64), ("C", c_i64), ("X_out", c_vp), ("W_out", c_vp)]


EXPORTS = {
    "nvfp4_padded_k": (c_i64, [c_i64]),
    "nvfp4_outlier_pad": (c_i64, [c_i64]),
    "nvfp4_operand_codes_bytes": (c_sz, [c_i64, c_i64]),
    "nvfp4_operand_sf_bytes": (c_sz, [c_i64, c_i64, c_i32]),
    "nvfp4_operand_gscale_count": (c_sz, [c_i64, c_i64, c_i32]),
    "nvfp4_status_string": (ctypes.c_char_p, [c_i32]),
    "nvfp4_quantize_workspace_bytes": (c_sz, [c_i64, c_i32]),
    "nvfp4_quantize": (c_i32, [c_vp, c_i64, c_i64, c_i64, c_i32, c_i32, c_u64, c_u32, c_u32, c_vp, c_i64,
                               ctypes.POINTER(COperand), c_vp, c_sz, c_vp]),
    "nvfp4_quantize_static_max_rows": (c_i64, []),
    "nvfp4_quantize_static": (c_i32, [c_vp, c_i64, c_i64, c_i64, c_i32, c_i32, c_u64, c_u32, c_vp, c_i64,
                                      ctypes.POINTER(COperand), c_vp]),
    "nvfp4_requantize_t": (c_i32, [ctypes.POINTER(COperand), c_vp, c_i64, c_vp, c_i64, c_i32, c_u64, c_u32, c_u32,
                                   ctypes.POINTER(COperand), c_vp, c_sz, c_vp]),
    "nvfp4_quantize_w16x16": (c_i32, [c_vp, c_i64, c_i64, c_i64, ctypes.POINTER(COperand), c_vp, c_sz, c_vp]),
    "nvfp4_transpose_operand16": (c_i32, [ctypes.POINTER(COperand), ctypes.POINTER(COperand), c_vp]),
    "nvfp4_gemm_workspace_bytes": (c_sz, [c_i64, c_i64, c_i64]),
    "nvfp4_gemm": (c_i32, [ctypes.POINTER(COperand), ctypes.POINTER(COperand), c_vp, c_i32, c_i64, c_i32, c_vp, c_vp,
                           c_sz, c_vp]),
    "nvfp4_gemm_ex": (c_i32, [ctypes.POINTER(COperand), ctypes.POINTER(COperand), c_vp, c_i32, c_i64, c_i32, c_vp,
                              ctypes.POINTER(CGemmOpts), c_vp, c_sz, c_vp]),
    "nvfp4_linear_workspace_bytes": (c_sz, [c_i32, c_i64, c_i64, c_i64, c_i64, c_i32]),
    "nvfp4_linear_bwd_operand": (c_i32, [c_i32, c_i32, c_i64, c_i64, c_i64, c_i64, c_i32, c_vp, c_sz, ctypes.POINTER(COperand)]),
    "nvfp4_linear_fwd": (c_i32, [c_vp, c_i64, c_vp, c_i64, c_i64, c_i64, c_i64, ctypes.POINTER(CLayerCfg), c_vp, c_i64,
                                 ctypes.POINTER(CSaved), c_vp, c_sz, c_vp]),
    "nvfp4_linear_bwd_dx": (c_i32, [c_vp, c_i64, ctypes.POINTER(CSaved), ctypes.POINTER(CLayerCfg), c_vp, c_i64, c_vp,
                                    c_sz, c_vp]),
    "nvfp4_linear_bwd_dw": (c_i32, [c_vp, c_i64, ctypes.POINTER(CSaved), ctypes.POINTER(CLayerCfg), c_vp, c_i64, c_vp,
                                    c_sz, c_vp]),
    "nvfp4_linear_bwd": (c_i32, [c_vp, c_i64, ctypes.POINTER(CSaved), ctypes.POINTER(CLayerCfg), c_vp, c_i64, c_vp, c_i64, c_vp,
                                 c_sz, c_vp]),
    "nvfp4_outlier_accumulate_workspace_bytes": (c_sz, [c_i64, c_i64]),
    "nvfp4_outlier_accumulate": (c_i32, [c_vp, c_i64, c_i64, c_i64, c_vp, c_vp, c_sz, c_vp]),
    "nvfp4_outlier_select": (c_i32, [c_vp, c_i64, c_i64, c_vp, c_vp, c_vp, c_vp]),
    "nvfp4_osci_workspace_bytes": (c_sz, [c_i64, c_i32]),
    "nvfp4_osci_update": (c_i32, [c_vp, c_i64, c_i64, c_i64, c_i32, c_i32, c_vp, c_vp, c_vp, c_vp, c_sz, c_vp]),
    "nvfp4_osci_suppress": (c_i32, [c_vp, c_i64, c_i64, c_i64, c_i32, c_vp, c_vp, ctypes.c_float, c_vp, c_vp, c_sz, c_vp]),
    "nvfp4_osci_sparse_workspace_bytes": (c_sz, [c_i64, c_i64, c_i32, c_i64, c_i32]),
    "nvfp4_osci_sparse_update": (c_i32, [c_vp, c_i64, c_i64, c_i64, c_i32, c_i32, c_i64, c_vp, c_vp, c_vp, c_vp, c_vp, c_vp, c_sz,
                                         c_vp]),
    "nvfp4_dense_ld": (c_i64, [c_i64]),
    "nvfp4_fp6_workspace_bytes": (c_sz, []),
    "nvfp4_fp6_quantize": (c_i32, [c_vp, c_i64, c_i64, c_i64, c_i32, c_u64, c_u32, ctypes.POINTER(CDenseOperand), c_vp, c_sz, c_vp]),
    "nvfp4_fp6_requantize_t": (c_i32, [ctypes.POINTER(CDenseOperand), c_i32, c_u64, c_u32, ctypes.POINTER(CDenseOperand), c_vp, c_sz,
                                       c_vp]),
    "nvfp4_expand_operand": (c_i32, [ctypes.POINTER(COperand), ctypes.POINTER(CDenseOperand), c_vp]),
    "nvfp4_dense_gemm": (c_i32, [ctypes.POINTER(CDenseOperand), ctypes.POINTER(CDenseOperand), c_vp, c_i32, c_i64, c_vp, c_vp]),
    "nvfp4_osci_sparse_suppress": (c_i32, [c_vp, c_i64, c_i64, c_i64, c_i32, c_i64, c_vp, c_vp, c_vp, ctypes.c_float, c_vp, c_vp,
                                           c_sz, c_vp]),
}
# measurement aids (include/nvfp4_measure.h): the launch counter lives in the main library, the tensor-core issue loop in
# a library of its own that only the benchmark and its test load
MEASURE_EXPORTS = {
    "nvfp4_launch_count": (ctypes.c_longlong, []),
    "nvfp4_mma_issue_probe": (c_i32, [c_i32, c_vp, ctypes.POINTER(ctypes.c_double), c_vp]),
    "nvfp4_mma_issue_probe_n": (c_i32, [c_i32, c_i32, c_i32, c_i32, c_i32, c_i32, c_vp, c_vp, ctypes.POINTER(ctypes.c_double), c_vp]),
}
for _name, (_res, _args) in list(EXPORTS.items()) + [("nvfp4_launch_count", MEASURE_EXPORTS["nvfp4_launch_count"])]:
    _f = getattr(_lib, _name)
    _f.restype = _res
    _f.argtypes = _args

lib = _lib
MEASURE_LIB_PATH = os.path.join(_HERE, "libnvfp4_measure.so")
_measure_lib = None


def measure_lib():
    """The measurement-aid library (tensor-core issue loop), loaded on first use."""
    global _measure_lib
    if _measure_lib is None:
        if not os.path.exists(MEASURE_LIB_PATH):
            raise ImportError(f"{MEASURE_LIB_PATH} is missing: build it with `python -m paper_2510_27527_b200.build`")
        _measure_lib = ctypes.CDLL(MEASURE_LIB_PATH)
        for name in ("nvfp4_mma_issue_probe", "nvfp4_mma_issue_probe_n"):
            res, args = MEASURE_EXPORTS[name]
            getattr(_measure_lib, name).restype = res
            getattr(_measure_lib, name).argtypes = args
    return _measure_lib


class Nvfp4Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {_lib.nvfp4_status_string(status).decode()} (status {status})")


def _check(status: int, where: str):
    if status != OK:
        raise Nvfp4Error(status, where)


def _stream_ptr() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


# ------------------------------------------------------------------------------------------------------------
# device-memory holders
# ------------------------------------------------------------------------------------------------------------
@dataclass
class Operand:
    """Device buffers of one quantized operand [R, K] (see nvfp4_operand in the header)."""

    codes: torch.Tensor  # uint8 [R, Kp/2]
    sf: torch.Tensor  # uint8, flat
    gscale: torch.Tensor  # float32, flat
    R: int
    K: int
    gs_mode: int
    sf_layout: int

    def c(self) -> COperand:
        return COperand(_ptr(self.codes), _ptr(self.sf), _ptr(self.gscale), self.R, self.K, self.gs_mode, self.sf_layout)

    @property
    def Kp(self) -> int:
        return _lib.nvfp4_padded_k(self.K)

    def sf_linear(self) -> np.ndarray:
        """Scales as a host array [R, Kp/16] whatever the device layout (index shuffling only)."""
        nb = self.Kp // 16
        raw = self.sf.cpu().numpy()
        if self.sf_layout == SF_LINEAR:
            return raw.reshape(self.R, nb)
        nbp = (nb + 15) // 16 * 16
        r = np.arange(self.R)[:, None]
        kb = np.arange(nb)[None, :]
        off = ((r >> 7) * (nbp >> 2) + (kb >> 2)) * 512 + (r & 31) * 16 + ((r >> 5) & 3) * 4 + (kb & 3)
        return raw[off]


def alloc_operand(R: int, K: int, gs_mode: int, sf_layout: int = SF_TILED128x4, device="cuda", poison: bool = False) -> Operand:
    fill = 0xA5 if poison else 0
    codes = torch.full((max(_lib.nvfp4_operand_codes_bytes(R, K), 1),), fill, dtype=torch.uint8, device=device)
    sf = torch.full((max(_lib.nvfp4_operand_sf_bytes(R, K, sf_layout), 1),), fill, dtype=torch.uint8, device=device)
    gs = torch.zeros(max(_lib.nvfp4_operand_gscale_count(R, K, gs_mode), 1), dtype=torch.float32, device=device)
    return Operand(codes, sf, gs, R, K, gs_mode, sf_layout)


def _matrix(rows: int, cols: int, dtype_code: int, device) -> torch.Tensor:
    """Row-major output whose rows start on 16-byte boundaries (leading dimension padded to 8 elements)."""
    ld = (cols + 7) // 8 * 8
    buf = torch.empty((rows, ld), dtype=torch.float32 if dtype_code == DT_F32 else torch.bfloat16, device=device)
    return buf[:, :cols]


def upload_bf16(x: np.ndarray, device="cuda") -> torch.Tensor:
    """float32 host array holding BF16-representable values -> bfloat16 device tensor (bit copy)."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    bits = (x.view(np.uint32) >> 16).astype(np.uint16)
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(device)


def _workspace(nbytes: int, device="cuda") -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


# ------------------------------------------------------------------------------------------------------------
# entry points (same names as the C ABI)
# ------------------------------------------------------------------------------------------------------------
def nvfp4_quantize(src: torch.Tensor, axis: int = AXIS_ROW, rounding: int = ROUND_RTN, seed: int = 0, stream_id: int = 0,
                   gs_mode: int = GS_TENSOR, sf_layout: int = SF_TILED128x4, keep_cols: torch.Tensor | None = None,
                   out: Operand | None = None, workspace: torch.Tensor | None = None, rht_stream_id: int = 0) -> Operand:
    assert src.dtype == torch.bfloat16 and src.dim() == 2 and src.stride(1) == 1
    rows, cols = src.shape
    kept = cols if keep_cols is None else int(keep_cols.numel())
    R, K = (rows, kept) if axis == AXIS_ROW else (kept, rows)
    if out is None:
        out = alloc_operand(R, K, gs_mode, sf_layout, src.device)
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_quantize_workspace_bytes(R, gs_mode), src.device)
    co = out.c()
    _check(_lib.nvfp4_quantize(_ptr(src), rows, cols, src.stride(0), axis, rounding, seed, stream_id, rht_stream_id,
                               _ptr(keep_cols), kept, ctypes.byref(co), _ptr(ws), ws.numel(), _stream_ptr()), "nvfp4_quantize")
    return out


def nvfp4_quantize_static(src: torch.Tensor, axis: int = AXIS_ROW, rounding: int = ROUND_RTN, seed: int = 0,
                          stream_id: int = 0, gs_mode: int = GS_TENSOR, sf_layout: int = SF_TILED128x4,
                          keep_cols: torch.Tensor | None = None, out: Operand | None = None) -> Operand:
    """nvfp4_quantize for callers that cannot hand over scratch memory: the amax cells live inside the library.
    `out` should be passed by such callers (allocating it here is a convenience for tests)."""
    assert src.dtype == torch.bfloat16 and src.dim() == 2 and src.stride(1) == 1
    rows, cols = src.shape
    kept = cols if keep_cols is None else int(keep_cols.numel())
    R, K = (rows, kept) if axis == AXIS_ROW else (kept, rows)
    if out is None:
        out = alloc_operand(R, K, gs_mode, sf_layout, src.device)
    co = out.c()
    _check(_lib.nvfp4_quantize_static(_ptr(src), rows, cols, src.stride(0), axis, rounding, seed, stream_id, _ptr(keep_cols),
                                      kept, ctypes.byref(co), _stream_ptr()), "nvfp4_quantize_static")
    return out


def nvfp4_requantize_t(inp: Operand, rounding: int = ROUND_SR, seed: int = 0, stream_id: int = 0, gs_mode: int | None = None,
                       sf_layout: int = SF_TILED128x4, hp: torch.Tensor | None = None, row_map: torch.Tensor | None = None,
                       out: Operand | None = None, workspace: torch.Tensor | None = None, rht_stream_id: int = 0) -> Operand:
    gs_mode = inp.gs_mode if gs_mode is None else gs_mode
    D = inp.K if row_map is None else int(row_map.numel())
    if out is None:
        out = alloc_operand(D, inp.R, gs_mode, sf_layout, inp.codes.device)
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_quantize_workspace_bytes(D, gs_mode), inp.codes.device)
    ci, co = inp.c(), out.c()
    _check(_lib.nvfp4_requantize_t(ctypes.byref(ci), _ptr(hp), 0 if hp is None else hp.stride(0), _ptr(row_map), D, rounding,
                                   seed, stream_id, rht_stream_id, ctypes.byref(co), _ptr(ws), ws.numel(), _stream_ptr()),
           "nvfp4_requantize_t")
    return out


def nvfp4_quantize_w16x16(W: torch.Tensor, sf_layout: int = SF_TILED128x4, out: Operand | None = None,
                          workspace: torch.Tensor | None = None) -> Operand:
    """Q2 of the 16x16 weight-block recipe: one E4M3 scale per 16x16 square, per-tensor global scale, round to nearest."""
    C, D = W.shape
    if out is None:
        out = alloc_operand(C, D, GS_TENSOR, sf_layout, W.device)
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_quantize_workspace_bytes(C, GS_TENSOR), W.device)
    co = out.c()
    _check(_lib.nvfp4_quantize_w16x16(_ptr(W), C, D, W.stride(0), ctypes.byref(co), _ptr(ws), ws.numel(), _stream_ptr()),
           "nvfp4_quantize_w16x16")
    return out


def nvfp4_transpose_operand16(inp: Operand, sf_layout: int = SF_TILED128x4, out: Operand | None = None) -> Operand:
    """Operand of W-hat^T from the 16x16-block operand of W (codes transposed, scales re-indexed; no arithmetic)."""
    if out is None:
        out = alloc_operand(inp.K, inp.R, GS_TENSOR, sf_layout, inp.codes.device)
    ci, co = inp.c(), out.c()
    _check(_lib.nvfp4_transpose_operand16(ctypes.byref(ci), ctypes.byref(co), _stream_ptr()), "nvfp4_transpose_operand16")
    return out


def nvfp4_gemm(A: Operand, B: Operand, c_dtype: int = DT_F32, out: torch.Tensor | None = None, accumulate: bool = False,
               dev_status: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> torch.Tensor:
    if out is None:
        out = _matrix(A.R, B.R, c_dtype, A.codes.device)
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_gemm_workspace_bytes(A.R, B.R, A.K), A.codes.device)
    ca, cb = A.c(), B.c()
    _check(_lib.nvfp4_gemm(ctypes.byref(ca), ctypes.byref(cb), _ptr(out), c_dtype, out.stride(0), int(accumulate),
                           _ptr(dev_status), _ptr(ws), ws.numel(), _stream_ptr()), "nvfp4_gemm")
    return out


def nvfp4_gemm_ex(A: Operand, B: Operand, c_dtype: int = DT_F32, out: torch.Tensor | None = None, accumulate: bool = False,
                  dev_status: torch.Tensor | None = None, variant: int = GEMM_AUTO, wait_limit_cycles: int = 0,
                  starve_first_stage: bool = False, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """nvfp4_gemm with an explicit kernel variant, wait bound and the test hook of the bounded waits."""
    if out is None:
        out = _matrix(A.R, B.R, c_dtype, A.codes.device)
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_gemm_workspace_bytes(A.R, B.R, A.K), A.codes.device)
    ca, cb = A.c(), B.c()
    opts = CGemmOpts(variant, int(starve_first_stage), wait_limit_cycles)
    _check(_lib.nvfp4_gemm_ex(ctypes.byref(ca), ctypes.byref(cb), _ptr(out), c_dtype, out.stride(0), int(accumulate),
                              _ptr(dev_status), ctypes.byref(opts), _ptr(ws), ws.numel(), _stream_ptr()), "nvfp4_gemm_ex")
    return out


def nvfp4_outlier_accumulate(X: torch.Tensor, acc: torch.Tensor, workspace: torch.Tensor | None = None) -> torch.Tensor:
    """acc[d] += ||X[:, d]||_2 (one step of OutControl's calibration window); acc is float32 [D] on the device."""
    assert X.dtype == torch.bfloat16 and X.dim() == 2 and X.stride(1) == 1
    assert acc.dtype == torch.float32 and acc.is_contiguous() and acc.numel() == X.shape[1]
    N_tok, D = X.shape
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_outlier_accumulate_workspace_bytes(N_tok, D), X.device)
    _check(_lib.nvfp4_outlier_accumulate(_ptr(X), X.stride(0), N_tok, D, _ptr(acc), _ptr(ws), ws.numel(), _stream_ptr()),
           "nvfp4_outlier_accumulate")
    return acc


def nvfp4_outlier_select(acc: torch.Tensor, n_out: int):
    """Top-n_out channels of acc -> (outlier_cols, keep_cols, col_map), int32 device tensors."""
    assert acc.dtype == torch.float32 and acc.is_contiguous()
    D = acc.numel()
    outl = torch.empty(max(n_out, 1), dtype=torch.int32, device=acc.device)[:n_out]
    keep = torch.empty(max(D - n_out, 1), dtype=torch.int32, device=acc.device)[: D - n_out]
    cmap = torch.empty(max(D, 1), dtype=torch.int32, device=acc.device)[:D]
    _check(_lib.nvfp4_outlier_select(_ptr(acc), D, n_out, _ptr(outl), _ptr(keep), _ptr(cmap), _stream_ptr()), "nvfp4_outlier_select")
    return outl, keep, cmap


def nvfp4_mma_issue_probe(iters: int, dev_status: torch.Tensor | None = None, n: int = 256, side_warps: int = 0,
                          side_kind: int = 0, random_data: bool = False, dev_bytes_moved: torch.Tensor | None = None,
                          loop_kind: int = 0) -> float:
    """Enqueues the tensor-core issue loop (instructions of M = 128, N = n, K = 64; loop_kind 0 = only MMAs, 1 = with the
    scale copies of a GEMM, 2 = and a commit per group, 3 / 4 = a five-stage ring walked the straightforward way / as the
    library's GEMMs walk it; side_warps further warps per SM storing to shared memory (side_kind 0), loading the accumulator
    (1), bulk-copying from L2 into shared memory (2) or from shared memory to global (3) meanwhile; random_data = hashed
    operand codes and scales instead of 1.0). dev_bytes_moved: int64[2] device counters, [0] += side bytes, [1] = loop
    cycles. Returns the FP4 flops the launch performs."""
    fl = ctypes.c_double(0.0)
    _check(measure_lib().nvfp4_mma_issue_probe_n(iters, n, loop_kind, side_warps, side_kind, int(random_data), _ptr(dev_status),
                                                 _ptr(dev_bytes_moved), ctypes.byref(fl), _stream_ptr()), "nvfp4_mma_issue_probe_n")
    return fl.value


@dataclass
class OsciState:
    """State of the oscillation statistics for one weight matrix (float32 [C, D] each, device)."""

    W_prev: torch.Tensor
    D_M: torch.Tensor
    D_Q: torch.Tensor


def alloc_osci_state(W: torch.Tensor) -> OsciState:
    mk = lambda: torch.empty(W.shape, dtype=torch.float32, device=W.device)
    return OsciState(mk(), mk(), mk())


def nvfp4_osci_update(W: torch.Tensor, state: OsciState, t0: int, gs_mode: int = GS_TENSOR, workspace: torch.Tensor | None = None) -> None:
    assert W.dtype == torch.float32 and W.dim() == 2 and W.stride(1) == 1
    C, D = W.shape
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_osci_workspace_bytes(C, gs_mode), W.device)
    _check(_lib.nvfp4_osci_update(_ptr(W), W.stride(0), C, D, gs_mode, t0, _ptr(state.W_prev), _ptr(state.D_M), _ptr(state.D_Q),
                                  _ptr(ws), ws.numel(), _stream_ptr()), "nvfp4_osci_update")


def nvfp4_osci_suppress(W: torch.Tensor, state: OsciState, tau: float, gs_mode: int = GS_TENSOR, n_reset: torch.Tensor | None = None,
                        workspace: torch.Tensor | None = None) -> None:
    """Resets, in place, the elements of W whose oscillation risk D_Q / D_M is at least tau."""
    assert W.dtype == torch.float32 and W.dim() == 2 and W.stride(1) == 1
    assert n_reset is None or (n_reset.dtype == torch.int64 and n_reset.numel() == 1)
    C, D = W.shape
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_osci_workspace_bytes(C, gs_mode), W.device)
    _check(_lib.nvfp4_osci_suppress(_ptr(W), W.stride(0), C, D, gs_mode, _ptr(state.D_M), _ptr(state.D_Q), float(tau), _ptr(n_reset),
                                    _ptr(ws), ws.numel(), _stream_ptr()), "nvfp4_osci_suppress")


@dataclass
class OsciSparseState:
    """State of the memory-efficient oscillation statistics: n_track tracked elements of one weight matrix."""

    idx: torch.Tensor  # int32, linear indices, sorted
    WM_prev: torch.Tensor
    WQ_prev: torch.Tensor
    D_M: torch.Tensor
    D_Q: torch.Tensor


def alloc_osci_sparse_state(n_track: int, device="cuda") -> OsciSparseState:
    mk = lambda dt: torch.empty(max(n_track, 1), dtype=dt, device=device)[:n_track]
    return OsciSparseState(mk(torch.int32), mk(torch.float32), mk(torch.float32), mk(torch.float32), mk(torch.float32))


def nvfp4_osci_sparse_update(W: torch.Tensor, state: OsciSparseState, t0: int, gs_mode: int = GS_TENSOR,
                             workspace: torch.Tensor | None = None) -> None:
    assert W.dtype == torch.float32 and W.dim() == 2 and W.stride(1) == 1
    C, D = W.shape
    n = state.idx.numel()
    ws = workspace if workspace is not None else _workspace(
        _lib.nvfp4_osci_sparse_workspace_bytes(C, D, gs_mode, n, 0 if t0 == 0 else 1), W.device)
    _check(_lib.nvfp4_osci_sparse_update(_ptr(W), W.stride(0), C, D, gs_mode, t0, n, _ptr(state.idx), _ptr(state.WM_prev),
                                         _ptr(state.WQ_prev), _ptr(state.D_M), _ptr(state.D_Q), _ptr(ws), ws.numel(), _stream_ptr()),
           "nvfp4_osci_sparse_update")


def nvfp4_osci_sparse_suppress(W: torch.Tensor, state: OsciSparseState, tau: float, gs_mode: int = GS_TENSOR,
                               n_reset: torch.Tensor | None = None, workspace: torch.Tensor | None = None) -> None:
    assert W.dtype == torch.float32 and W.dim() == 2 and W.stride(1) == 1
    assert n_reset is None or (n_reset.dtype == torch.int64 and n_reset.numel() == 1)
    C, D = W.shape
    n = state.idx.numel()
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_osci_sparse_workspace_bytes(C, D, gs_mode, n, 2), W.device)
    _check(_lib.nvfp4_osci_sparse_suppress(_ptr(W), W.stride(0), C, D, gs_mode, n, _ptr(state.idx), _ptr(state.D_M), _ptr(state.D_Q),
                                           float(tau), _ptr(n_reset), _ptr(ws), ws.numel(), _stream_ptr()),
           "nvfp4_osci_sparse_suppress")


@dataclass
class LayerConfig:
    gs_mode: int = GS_TENSOR
    seed: int = 0
    rounding: tuple = (ROUND_RTN, ROUND_RTN, ROUND_SR, ROUND_SR, ROUND_SR, ROUND_SR)
    y_dtype: int = DT_BF16
    dx_dtype: int = DT_BF16
    dw_dtype: int = DT_F32
    outliers: np.ndarray | None = None  # sorted outlier channel indices (host)
    dev_status: torch.Tensor | None = None
    rht: bool = False  # random Hadamard transformation of both operands of the two backward products
    outlier_fp8: bool = False  # outlier channels on a per-tensor power-of-two scaled E4M3 grid instead of BF16
    w_block16: bool = False  # weights in 16x16 scale squares (comparison recipe): dX uses the forward codes transposed, no Q4
    # run the independent chains of a call (dX beside dW, the weight quantizer beside the activation quantizer) on a
    # second stream: the stream and its three events are created here, with torch, and handed to the library
    concurrent: bool = True
    # device index arrays, built by prepare()
    _outl: torch.Tensor | None = None
    _keep: torch.Tensor | None = None
    _map: torch.Tensor | None = None
    _D: int = -1
    _side: tuple | None = None

    def side(self, device):
        """(stream, fork, join, aux) of the second stream for `device`, created on first use; None when not concurrent."""
        if not self.concurrent:
            return None
        dev = torch.device(device)
        dev = torch.device("cuda", torch.cuda.current_device()) if dev.index is None else dev
        if self._side is None or self._side[0] != dev:
            with torch.cuda.device(dev):
                self._side = (dev, torch.cuda.Stream(device=dev), torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event())
                for ev in self._side[2:]:
                    ev.record(self._side[1])  # forces creation of the underlying CUDA events (torch makes them lazily)
        return self._side[1:]

    def prepare(self, D: int, device="cuda"):
        """Uploads the OutControl index arrays for hidden size D (index bookkeeping only)."""
        self.side(device)
        if self.outliers is None or len(self.outliers) == 0 or self._D == D:
            return
        outl = np.asarray(self.outliers, dtype=np.int64)
        mask = np.ones(D, dtype=bool)
        mask[outl] = False
        keep = np.nonzero(mask)[0]
        cmap = np.full(D, -1, dtype=np.int32)
        cmap[keep] = np.arange(len(keep), dtype=np.int32)
        self._outl = torch.from_numpy(outl.astype(np.int32)).to(device)
        self._keep = torch.from_numpy(keep.astype(np.int32)).to(device)
        self._map = torch.from_numpy(cmap).to(device)
        self._D = D

    @property
    def n_out(self) -> int:
        return 0 if self.outliers is None else len(self.outliers)

    def c(self) -> CLayerCfg:
        side = self._side[1:] if (self.concurrent and self._side is not None) else None
        sp = (side[0].cuda_stream, side[1].cuda_event, side[2].cuda_event, side[3].cuda_event) if side else (0, 0, 0, 0)
        return CLayerCfg(self.gs_mode, (c_i32 * 6)(*self.rounding), self.seed, self.y_dtype, self.dx_dtype, self.dw_dtype,
                         self.n_out, _ptr(self._outl), _ptr(self._keep), _ptr(self._map), _ptr(self.dev_status), int(self.rht),
                         int(self.outlier_fp8), int(self.w_block16), *sp)


@dataclass
class Saved:
    qx: Operand
    qw: Operand
    X: torch.Tensor
    W: torch.Tensor
    X_out: torch.Tensor | None = None  # [N_tok, Kh] bf16, OutControl only
    W_out: torch.Tensor | None = None  # [C, Kh] bf16

    def c(self) -> CSaved:
        return CSaved(self.qx.c(), self.qw.c(), _ptr(self.X), _ptr(self.W), self.X.stride(0), self.W.stride(0),
                      self.X.shape[0], self.X.shape[1], self.W.shape[0], _ptr(self.X_out), _ptr(self.W_out))


def alloc_saved(X: torch.Tensor, W: torch.Tensor, cfg: "LayerConfig") -> "Saved":
    """Device buffers of everything forward leaves for backward."""
    N_tok, D = X.shape
    C = W.shape[0]
    Dk = D - cfg.n_out
    Kh = _lib.nvfp4_outlier_pad(cfg.n_out)
    xo = torch.empty((N_tok, Kh), dtype=torch.bfloat16, device=X.device) if Kh else None
    wo = torch.empty((C, Kh), dtype=torch.bfloat16, device=X.device) if Kh else None
    return Saved(alloc_operand(N_tok, Dk, cfg.gs_mode, SF_TILED128x4, X.device), alloc_operand(C, Dk, cfg.gs_mode, SF_TILED128x4, X.device),
                 X, W, xo, wo)


def linear_workspace(op_kind: int, N_tok: int, D: int, C: int, cfg: LayerConfig, device="cuda") -> torch.Tensor:
    return _workspace(_lib.nvfp4_linear_workspace_bytes(op_kind, N_tok, D, C, cfg.n_out, cfg.gs_mode), device)


def nvfp4_linear_bwd_operand(op_kind: int, which: int, N_tok: int, D: int, C: int, cfg: LayerConfig, workspace: torch.Tensor) -> Operand:
    """View of backward operand Q3..Q6 (which = 3..6) inside the workspace of a backward call (no copy, nothing launched)."""
    co = COperand()
    _check(_lib.nvfp4_linear_bwd_operand(op_kind, which, N_tok, D, C, cfg.n_out, cfg.gs_mode, _ptr(workspace), workspace.numel(),
                                         ctypes.byref(co)), "nvfp4_linear_bwd_operand")
    base = workspace.data_ptr()

    def view(ptr, nbytes, dtype):
        off = ptr - base
        return workspace[off: off + nbytes].view(dtype)

    R, K = co.R, co.K
    return Operand(view(co.codes, _lib.nvfp4_operand_codes_bytes(R, K), torch.uint8),
                   view(co.sf, _lib.nvfp4_operand_sf_bytes(R, K, SF_TILED128x4), torch.uint8),
                   view(co.gscale, 4 * _lib.nvfp4_operand_gscale_count(R, K, cfg.gs_mode), torch.float32), R, K, cfg.gs_mode,
                   SF_TILED128x4)


def nvfp4_linear_fwd(X: torch.Tensor, W: torch.Tensor, cfg: LayerConfig, Y: torch.Tensor | None = None,
                     saved: Saved | None = None, workspace: torch.Tensor | None = None):
    N_tok, D = X.shape
    C = W.shape[0]
    cfg.prepare(D, X.device)
    Dk = D - cfg.n_out
    if saved is None:
        saved = alloc_saved(X, W, cfg)
    else:
        saved.X, saved.W = X, W
    if Y is None:
        Y = _matrix(N_tok, C, cfg.y_dtype, X.device)
    ws = workspace if workspace is not None else linear_workspace(OP_FWD, N_tok, D, C, cfg, X.device)
    cs, cc = saved.c(), cfg.c()
    _check(_lib.nvfp4_linear_fwd(_ptr(X), X.stride(0), _ptr(W), W.stride(0), N_tok, D, C, ctypes.byref(cc), _ptr(Y),
                                 Y.stride(0), ctypes.byref(cs), _ptr(ws), ws.numel(), _stream_ptr()), "nvfp4_linear_fwd")
    return Y, saved


def nvfp4_linear_bwd_dx(dY: torch.Tensor, saved: Saved, cfg: LayerConfig, dX: torch.Tensor | None = None,
                        workspace: torch.Tensor | None = None) -> torch.Tensor:
    N_tok, D = saved.X.shape
    C = saved.W.shape[0]
    if dX is None:
        dX = _matrix(N_tok, D, cfg.dx_dtype, dY.device)
    ws = workspace if workspace is not None else linear_workspace(OP_BWD_DX, N_tok, D, C, cfg, dY.device)
    cs, cc = saved.c(), cfg.c()
    _check(_lib.nvfp4_linear_bwd_dx(_ptr(dY), dY.stride(0), ctypes.byref(cs), ctypes.byref(cc), _ptr(dX), dX.stride(0),
                                    _ptr(ws), ws.numel(), _stream_ptr()), "nvfp4_linear_bwd_dx")
    return dX


def nvfp4_linear_bwd_dw(dY: torch.Tensor, saved: Saved, cfg: LayerConfig, dW: torch.Tensor | None = None,
                        workspace: torch.Tensor | None = None) -> torch.Tensor:
    N_tok, D = saved.X.shape
    C = saved.W.shape[0]
    if dW is None:
        dW = _matrix(C, D, cfg.dw_dtype, dY.device)
    ws = workspace if workspace is not None else linear_workspace(OP_BWD_DW, N_tok, D, C, cfg, dY.device)
    cs, cc = saved.c(), cfg.c()
    _check(_lib.nvfp4_linear_bwd_dw(_ptr(dY), dY.stride(0), ctypes.byref(cs), ctypes.byref(cc), _ptr(dW), dW.stride(0),
                                    _ptr(ws), ws.numel(), _stream_ptr()), "nvfp4_linear_bwd_dw")
    return dW


def nvfp4_linear_bwd(dY: torch.Tensor, saved: Saved, cfg: LayerConfig, dX: torch.Tensor | None = None, dW: torch.Tensor | None = None,
                     workspace: torch.Tensor | None = None):
    """Both backward products in one call (dX, dW); the per-tensor amax of dY is computed once where Q3 and Q5 share it."""
    N_tok, D = saved.X.shape
    C = saved.W.shape[0]
    cfg.prepare(D, dY.device)
    if dX is None:
        dX = _matrix(N_tok, D, cfg.dx_dtype, dY.device)
    if dW is None:
        dW = _matrix(C, D, cfg.dw_dtype, dY.device)
    ws = workspace if workspace is not None else linear_workspace(OP_BWD, N_tok, D, C, cfg, dY.device)
    cs, cc = saved.c(), cfg.c()
    _check(_lib.nvfp4_linear_bwd(_ptr(dY), dY.stride(0), ctypes.byref(cs), ctypes.byref(cc), _ptr(dX), dX.stride(0), _ptr(dW),
                                 dW.stride(0), _ptr(ws), ws.numel(), _stream_ptr()), "nvfp4_linear_bwd")
    return dX, dW


# ------------------------------------------------------------------------------------------------------------
# simulated FP6 x FP4 products (paper Sec. 5.4, "Precision Switching in Final Stage")
# ------------------------------------------------------------------------------------------------------------
@dataclass
class DenseOperand:
    """Device buffers of a dense simulation operand [R, K]: vals = P * S_block as BF16 [R, ld], one FP32 global scale."""

    vals: torch.Tensor  # bfloat16 [R, ld]
    gscale: torch.Tensor  # float32 [1]
    R: int
    K: int

    @property
    def ld(self) -> int:
        return _lib.nvfp4_dense_ld(self.K)

    def c(self) -> CDenseOperand:
        return CDenseOperand(_ptr(self.vals), _ptr(self.gscale), self.R, self.K, self.ld)


def alloc_dense(R: int, K: int, device="cuda", poison: bool = False) -> DenseOperand:
    vals = torch.full((R, _lib.nvfp4_dense_ld(K)), 7.0 if poison else 0.0, dtype=torch.bfloat16, device=device)
    return DenseOperand(vals, torch.zeros(1, dtype=torch.float32, device=device), R, K)


def nvfp4_fp6_quantize(src: torch.Tensor, rounding: int = ROUND_RTN, seed: int = 0, stream_id: int = 0,
                       out: DenseOperand | None = None, workspace: torch.Tensor | None = None) -> DenseOperand:
    assert src.dtype == torch.bfloat16 and src.dim() == 2 and src.stride(1) == 1
    rows, cols = src.shape
    if out is None:
        out = alloc_dense(rows, cols, src.device)
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_fp6_workspace_bytes(), src.device)
    co = out.c()
    _check(_lib.nvfp4_fp6_quantize(_ptr(src), rows, cols, src.stride(0), rounding, seed, stream_id, ctypes.byref(co), _ptr(ws),
                                   ws.numel(), _stream_ptr()), "nvfp4_fp6_quantize")
    return out


def nvfp4_fp6_requantize_t(inp: DenseOperand, rounding: int = ROUND_SR, seed: int = 0, stream_id: int = 0,
                           out: DenseOperand | None = None, workspace: torch.Tensor | None = None) -> DenseOperand:
    if out is None:
        out = alloc_dense(inp.K, inp.R, inp.vals.device)
    ws = workspace if workspace is not None else _workspace(_lib.nvfp4_fp6_workspace_bytes(), inp.vals.device)
    ci, co = inp.c(), out.c()
    _check(_lib.nvfp4_fp6_requantize_t(ctypes.byref(ci), rounding, seed, stream_id, ctypes.byref(co), _ptr(ws), ws.numel(),
                                       _stream_ptr()), "nvfp4_fp6_requantize_t")
    return out


def nvfp4_expand_operand(inp: Operand, out: DenseOperand | None = None) -> DenseOperand:
    if out is None:
        out = alloc_dense(inp.R, inp.K, inp.codes.device)
    ci, co = inp.c(), out.c()
    _check(_lib.nvfp4_expand_operand(ctypes.byref(ci), ctypes.byref(co), _stream_ptr()), "nvfp4_expand_operand")
    return out


def nvfp4_dense_gemm(A: DenseOperand, B: DenseOperand, c_dtype: int = DT_F32, out: torch.Tensor | None = None,
                     dev_status: torch.Tensor | None = None) -> torch.Tensor:
    if out is None:
        out = _matrix(A.R, B.R, c_dtype, A.vals.device)
    ca, cb = A.c(), B.c()
    _check(_lib.nvfp4_dense_gemm(ctypes.byref(ca), ctypes.byref(cb), _ptr(out), c_dtype, out.stride(0), _ptr(dev_status),
                                 _stream_ptr()), "nvfp4_dense_gemm")
    return out


def fp6_linear_fwd(X: torch.Tensor, W: torch.Tensor, c_dtype: int = DT_BF16):
    """Y = Q6_D(X) Q4_D(W^T): the calls of the simulated layer in order (sequencing only; every step is a library call).
    Returns (Y, saved = (dense X-hat operand, FP4 operand of W))."""
    qx6 = nvfp4_fp6_quantize(X, ROUND_RTN, 0, 1)
    qw = nvfp4_quantize(W, AXIS_ROW, ROUND_RTN, 0, 2, GS_TENSOR)
    Y = nvfp4_dense_gemm(qx6, nvfp4_expand_operand(qw), c_dtype)
    return Y, (qx6, qw)


def fp6_linear_bwd(dY: torch.Tensor, saved, seed: int = 0, dx_dtype: int = DT_BF16, dw_dtype: int = DT_F32):
    """dX = Q6_S(dY) Q4_S(W-hat), dW = Q4_S(dY^T) Q6_S(X-hat). Returns (dX, dW, the four backward operands)."""
    qx6, qw = saved
    q3 = nvfp4_fp6_quantize(dY, ROUND_SR, seed, 3)
    q4 = nvfp4_requantize_t(qw, ROUND_SR, seed, 4)
    dX = nvfp4_dense_gemm(q3, nvfp4_expand_operand(q4), dx_dtype)
    q5 = nvfp4_quantize(dY, AXIS_COL, ROUND_SR, seed, 5, GS_TENSOR)
    q6 = nvfp4_fp6_requantize_t(qx6, ROUND_SR, seed, 6)
    dW = nvfp4_dense_gemm(nvfp4_expand_operand(q5), q6, dw_dtype)
    return dX, dW, (q3, q4, q5, q6)
