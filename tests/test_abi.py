"""CPU-side checks of the boundary: the shared library loads, exports every symbol the header declares, its
host-only helpers agree with the documented layout, and bad arguments are refused before anything launches."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def binding():
    from paper_2510_27527_b200 import build

    build.build()
    from paper_2510_27527_b200 import binding as b

    return b


def _declared(header_name):
    header = open(os.path.join(ROOT, "include", header_name)).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    return set(re.findall(r"\b(nvfp4_[a-z0-9_]+)\s*\(", header))


def test_every_declared_symbol_is_exported(binding):
    declared = _declared("nvfp4.h")
    assert {"nvfp4_quantize", "nvfp4_linear_fwd", "nvfp4_linear_bwd_dx", "nvfp4_linear_bwd_dw", "nvfp4_gemm",
            "nvfp4_requantize_t", "nvfp4_gemm_ex", "nvfp4_quantize_static"} <= declared
    for name in declared:
        assert hasattr(binding.lib, name), name
    assert declared == set(binding.EXPORTS)
    # the measurement aids: the launch counter in the main library, the issue loop in a library of its own
    aids = _declared("nvfp4_measure.h")
    assert aids == set(binding.MEASURE_EXPORTS) == {"nvfp4_launch_count", "nvfp4_mma_issue_probe", "nvfp4_mma_issue_probe_n"}
    assert hasattr(binding.lib, "nvfp4_launch_count") and not hasattr(binding.lib, "nvfp4_mma_issue_probe")
    assert hasattr(binding.measure_lib(), "nvfp4_mma_issue_probe")
    # headers of the include directory are exactly these two
    assert sorted(os.listdir(os.path.join(ROOT, "include"))) == ["nvfp4.h", "nvfp4_measure.h"]


def test_size_helpers(binding):
    L = binding.lib
    assert L.nvfp4_padded_k(1) == 128 and L.nvfp4_padded_k(128) == 128 and L.nvfp4_padded_k(129) == 256
    assert L.nvfp4_operand_codes_bytes(3, 16) == 3 * 64
    assert L.nvfp4_operand_sf_bytes(3, 16, binding.SF_LINEAR) == 3 * 8
    assert L.nvfp4_operand_sf_bytes(3, 16, binding.SF_TILED128x4) == 128 * 16
    assert L.nvfp4_operand_sf_bytes(129, 300, binding.SF_TILED128x4) == 256 * 32
    assert L.nvfp4_operand_gscale_count(7, 300, binding.GS_TENSOR) == 1
    assert L.nvfp4_operand_gscale_count(7, 300, binding.GS_ROW) == 7
    assert L.nvfp4_operand_gscale_count(7, 300, binding.GS_BLOCK128) == 7 * 3
    assert L.nvfp4_status_string(0) == b"ok" and b"workspace" in L.nvfp4_status_string(5)
    assert L.nvfp4_linear_workspace_bytes(binding.OP_BWD_DX, 256, 512, 512, 0, 0) > 256 * 512 // 2


def test_bad_arguments_are_refused_on_the_host(binding):
    L, b = binding.lib, binding
    op = b.COperand(0x1000, 0x2000, 0x3000, 4, 32, 0, 0)
    ws = 0x4000
    q = lambda *a: L.nvfp4_quantize(*a)
    assert q(0, 4, 32, 32, 0, 0, 0, 0, 0, None, 0, ctypes.byref(op), ws, 256, None) == 1  # null source
    assert q(0x100, 4, 32, 32, 2, 0, 0, 0, 0, None, 0, ctypes.byref(op), ws, 256, None) == 4  # bad axis
    assert q(0x100, 4, 32, 32, 0, 7, 0, 0, 0, None, 0, ctypes.byref(op), ws, 256, None) == 4  # bad rounding
    assert q(0x100, -1, 32, 32, 0, 0, 0, 0, 0, None, 0, ctypes.byref(op), ws, 256, None) == 2  # negative size
    assert q(0x100, 5, 32, 32, 0, 0, 0, 0, 0, None, 0, ctypes.byref(op), ws, 256, None) == 2  # out shape mismatch
    assert q(0x104, 4, 32, 32, 0, 0, 0, 0, 0, None, 0, ctypes.byref(op), ws, 256, None) == 3  # misaligned source
    assert q(0x100, 4, 32, 36, 0, 0, 0, 0, 0, None, 0, ctypes.byref(op), ws, 256, None) == 3  # ld not multiple of 8
    assert q(0x100, 4, 32, 32, 0, 0, 0, 0, 0, None, 0, ctypes.byref(op), ws, 8, None) == 5  # workspace too small
    assert q(0x100, 4, 32, 32, 0, 0, 0, 0, 7, 0x6000, 32, ctypes.byref(op), ws, 256, None) == 4  # transformation + column list
    bad = b.COperand(0x1000, 0x2000, 0x3000, 4, 32, 9, 0)
    assert q(0x100, 4, 32, 32, 0, 0, 0, 0, 0, None, 0, ctypes.byref(bad), ws, 256, None) == 4  # bad gs_mode
    a = b.COperand(0x1000, 0x2000, 0x3000, 4, 32, 0, 1)
    c = b.COperand(0x1000, 0x2000, 0x3000, 4, 64, 0, 1)
    assert L.nvfp4_gemm(ctypes.byref(a), ctypes.byref(c), 0x5000, 1, 4, 0, None, None, 0, None) == 2  # K mismatch
    lin = b.COperand(0x1000, 0x2000, 0x3000, 4, 32, 0, 0)
    assert L.nvfp4_gemm(ctypes.byref(a), ctypes.byref(lin), 0x5000, 1, 4, 0, None, None, 0, None) == 4  # linear scales
    a2 = b.COperand(0x1000, 0x2000, 0x3000, 4, 32, 0, 1)
    bad_variant = b.CGemmOpts(7, 0, 0)
    assert L.nvfp4_gemm_ex(ctypes.byref(a), ctypes.byref(a2), 0x5000, 1, 4, 0, None, ctypes.byref(bad_variant), None, 0, None) == 4
    neg_limit = b.CGemmOpts(0, 0, -5)
    assert L.nvfp4_gemm_ex(ctypes.byref(a), ctypes.byref(a2), 0x5000, 1, 4, 0, None, ctypes.byref(neg_limit), None, 0, None) == 4
    g2 = b.COperand(0x1000, 0x2000, 0x3000, 4, 32, 2, 1)
    pair = b.CGemmOpts(b.GEMM_PAIR256, 0, 0)
    assert L.nvfp4_gemm_ex(ctypes.byref(g2), ctypes.byref(g2), 0x5000, 1, 4, 0, None, ctypes.byref(pair), None, 0, None) == 4
    # a side stream without its events is refused
    cfg = b.CLayerCfg(0, (ctypes.c_int32 * 6)(0, 0, 1, 1, 1, 1), 0, 0, 0, 1, 0, None, None, None, None, 0, 0, 0, 0x7000, None, None, None)
    sv = b.CSaved(a, a2, 0x100, 0x200, 32, 32, 4, 32, 4, None, None)
    assert L.nvfp4_linear_fwd(0x100, 32, 0x200, 32, 4, 32, 4, ctypes.byref(cfg), 0x300, 8, ctypes.byref(sv), 0x400, 1 << 20, None) == 1


def test_bad_arguments_of_the_calibration_and_oscireset_entry_points(binding):
    L = binding.lib
    f32 = ctypes.c_float
    assert L.nvfp4_outlier_accumulate(0, 64, 8, 64, 0x2000, 0x3000, 1 << 20, None) == 1  # null source
    assert L.nvfp4_outlier_accumulate(0x1000, 60, 8, 64, 0x2000, 0x3000, 1 << 20, None) == 3  # ld < D
    assert L.nvfp4_outlier_accumulate(0x1000, 64, 8, 64, 0x2000, 0x3000, 16, None) == 5  # workspace too small
    assert L.nvfp4_outlier_select(0x1000, 8, 9, 0x2000, 0x3000, 0x4000, None) == 2  # n_out > D
    assert L.nvfp4_outlier_select(0x1000, 8, 2, None, 0x3000, 0x4000, None) == 1  # missing output
    assert L.nvfp4_osci_update(0x1000, 16, 4, 16, 7, 1, 0x2000, 0x3000, 0x4000, 0x5000, 256, None) == 4  # bad gs_mode
    assert L.nvfp4_osci_update(0x1000, 8, 4, 16, 0, 1, 0x2000, 0x3000, 0x4000, 0x5000, 256, None) == 2  # ld < D
    assert L.nvfp4_osci_update(0x1004, 16, 4, 16, 0, 1, 0x2000, 0x3000, 0x4000, 0x5000, 256, None) == 3  # misaligned
    assert L.nvfp4_osci_suppress(0x1000, 16, 4, 16, 0, None, 0x4000, f32(8.0), None, 0x5000, 256, None) == 1
    big = 1 << 16
    assert L.nvfp4_osci_sparse_update(0x1000, big, big, big, 0, 0, 10, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000, 1 << 40,
                                      None) == 9  # C * D >= 2^31
    assert L.nvfp4_osci_sparse_update(0x1000, 16, 4, 16, 0, 0, 65, 0x2000, 0x3000, 0x4000, 0x5000, 0x6000, 0x7000, 1 << 20,
                                      None) == 2  # n_track > C * D
    assert L.nvfp4_osci_sparse_workspace_bytes(64, 64, 0, 100, 0) > 64 * 64 * 4
    assert L.nvfp4_osci_sparse_workspace_bytes(64, 64, 0, 100, 1) < 4096
    assert L.nvfp4_linear_workspace_bytes(binding.OP_BWD, 256, 512, 512, 0, 0) > L.nvfp4_linear_workspace_bytes(
        binding.OP_BWD_DX, 256, 512, 512, 0, 0)


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2510_27527_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+\S*oracle", text, flags=re.M), f
                assert "nvfp4_oracle" not in text and "libnvfp4_oracle" not in text, f
