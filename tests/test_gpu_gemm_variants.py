"""The GEMM kernel variants through nvfp4_gemm_ex, each against the oracle's FP64 product of the dequantized operands: the
CTA-pair kernels (256 x 256 and 256 x 192 tiles) on ragged shapes in both scale modes it supports, both output types, with and without
accumulation; guard bands around C for every kernel; and the bounded-wait path (a wait that runs out must end the kernel
with a status word, never hang)."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.gpu_util import bf16_ulp_close, check_sampled, rel_fro, upload_operand

pytestmark = pytest.mark.gpu

POISON = -7.0


def B():
    from paper_2510_27527_b200 import binding

    return binding


def quantized_pair(M, N, K, gs_mode, seed=1):
    x, _ = synth.activations(M, K, seed, n_outlier=4, factor=30.0)
    w = synth.weights(N, K, seed + 1)
    a = orc.quantize(x, orc.AXIS_ROW, orc.RTN, gs_mode)
    bb = orc.quantize(w, orc.AXIS_ROW, orc.SR, gs_mode, seed=4, stream_id=2)
    return a, bb


def guarded_c(M, N, dtype, extra_rows=3):
    """C [M, N] as a view of a larger poisoned buffer: at least 8 more columns to the right of every row (rows stay 16-byte
    aligned), extra_rows rows below."""
    ld = (N + 8 + 7) // 8 * 8
    full = torch.full((M + extra_rows, ld), POISON, dtype=dtype, device="cuda")
    return full, full[:M, :N]


def guard_intact(full, M, N):
    torch.cuda.synchronize()
    f = full.float()
    bad = torch.nonzero(f != POISON)
    bad = bad[(bad[:, 0] >= M) | (bad[:, 1] >= N)]
    assert bad.numel() == 0, f"{bad.shape[0]} elements outside C[{M}, {N}] were overwritten, first (row, column): {bad[:6].tolist()}"
    return True


@pytest.mark.parametrize("variant", [1, 2, 3])
@pytest.mark.parametrize("gs_mode", [0, 1])
@pytest.mark.parametrize("shape", [(300, 520, 3072), (256, 256, 512), (130, 700, 1280), (520, 330, 768)])
def test_variants_match_fp64_with_guard_bands(variant, gs_mode, shape):
    b = B()
    M, N, K = shape
    a, bb = quantized_pair(M, N, K, gs_mode)
    A64, B64 = orc.dequantize(a), orc.dequantize(bb)
    want = orc.gemm_tn(A64, B64)
    absdot = np.abs(A64) @ np.abs(B64).T
    da, db = upload_operand(a, b), upload_operand(bb, b)
    # FP32 output
    full, C = guarded_c(M, N, torch.float32)
    b.nvfp4_gemm_ex(da, db, b.DT_F32, out=C, variant=variant)
    assert guard_intact(full, M, N)
    got = C.cpu().numpy()
    assert rel_fro(got, want) <= 1e-5
    assert np.all(np.abs(got - want) <= 1e-3 * absdot + 1e-30)
    # accumulate into the existing FP32 C
    b.nvfp4_gemm_ex(da, db, b.DT_F32, out=C, accumulate=True, variant=variant)
    assert guard_intact(full, M, N)
    assert rel_fro(C.cpu().numpy(), 2.0 * want) <= 1e-5
    # BF16 output: one rounding of the FP32 result; then accumulation in BF16 storage
    full16, C16 = guarded_c(M, N, torch.bfloat16)
    b.nvfp4_gemm_ex(da, db, b.DT_BF16, out=C16, variant=variant)
    assert guard_intact(full16, M, N)
    first = C16.float().cpu().numpy().astype(np.float64)
    assert np.all(bf16_ulp_close(first, want, 1.0, 1e-5 * absdot))
    b.nvfp4_gemm_ex(da, db, b.DT_BF16, out=C16, accumulate=True, variant=variant)
    assert guard_intact(full16, M, N)
    assert np.all(bf16_ulp_close(C16.float().cpu().numpy(), first + want, 1.0, 1e-5 * absdot))


@pytest.mark.parametrize("shape", [(300, 520, 640), (128, 136, 256)])
def test_outer_block_kernel_guard_bands(shape):
    b = B()
    M, N, K = shape
    a, bb = quantized_pair(M, N, K, 2)
    want = orc.gemm_operands(a, bb)
    da, db = upload_operand(a, b), upload_operand(bb, b)
    for dt, tdt in ((b.DT_F32, torch.float32), (b.DT_BF16, torch.bfloat16)):
        full, C = guarded_c(M, N, tdt)
        b.nvfp4_gemm(da, db, dt, out=C)
        assert guard_intact(full, M, N)
        assert rel_fro(C.float().cpu().numpy(), want) <= (1e-5 if dt == b.DT_F32 else 4e-3)
        if dt == b.DT_F32:
            b.nvfp4_gemm(da, db, dt, out=C, accumulate=True)
            assert guard_intact(full, M, N)
            assert rel_fro(C.cpu().numpy(), 2.0 * want) <= 1e-5


@pytest.mark.parametrize("gs_mode", [0, 1])
def test_pair_kernel_is_what_large_ragged_products_run(gs_mode):
    """4000 x 2600 x 4096: 16 x 11 = 176 tiles of 256 x 256 (16 x 14 of 256 x 192), the shape class nvfp4_gemm sends to a
    CTA-pair kernel by itself; the last tile row and column are ragged (rows beyond M in the second CTA's half, columns
    beyond N)."""
    b = B()
    M, N, K = 4000, 2600, 4096
    a, bb = quantized_pair(M, N, K, gs_mode, seed=11)
    A64, B64 = orc.dequantize(a), orc.dequantize(bb)
    da, db = upload_operand(a, b), upload_operand(bb, b)
    rng = np.random.default_rng(5)
    full, C = guarded_c(M, N, torch.float32)
    b.nvfp4_gemm(da, db, b.DT_F32, out=C)
    assert guard_intact(full, M, N)
    check_sampled(C, A64, B64, rng, False, "auto 4000x2600x4096 f32")
    # the explicit variants give the same matrix up to FP32 summation order
    C2 = b.nvfp4_gemm_ex(da, db, b.DT_F32, variant=b.GEMM_PAIR256)
    C3 = b.nvfp4_gemm_ex(da, db, b.DT_F32, variant=b.GEMM_PAIR192)
    C1 = b.nvfp4_gemm_ex(da, db, b.DT_F32, variant=b.GEMM_TILE128)
    torch.cuda.synchronize()
    assert torch.equal(C2, C) or torch.equal(C3, C)  # one of the two pair kernels ran
    for other in (C1, C2, C3):
        assert float((other - C).norm() / C.norm()) <= 1e-6
    full16, C16 = guarded_c(M, N, torch.bfloat16)
    b.nvfp4_gemm(da, db, b.DT_BF16, out=C16)
    assert guard_intact(full16, M, N)
    check_sampled(C16, A64, B64, rng, True, "auto 4000x2600x4096 bf16")


@pytest.mark.parametrize("variant", [1, 2, 3])
def test_a_wait_that_runs_out_ends_the_kernel_with_a_status(variant):
    """The first operand stage is made to expect bytes that never arrive and the wait bound is shortened to about a
    millisecond: the kernel must return, report NVFP4_ERR_TIMEOUT through the status word, and leave the device usable:
    the same product right afterwards is correct."""
    b = B()
    M, N, K = {1: (128, 128, 512), 2: (256, 256, 512), 3: (256, 192, 512)}[variant]
    a, bb = quantized_pair(M, N, K, 0, seed=21)
    want = orc.gemm_operands(a, bb)
    da, db = upload_operand(a, b), upload_operand(bb, b)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    b.nvfp4_gemm_ex(da, db, b.DT_F32, dev_status=status, variant=variant, wait_limit_cycles=2_000_000, starve_first_stage=True)
    torch.cuda.synchronize()  # returns: every role gave up within its bound
    assert int(status.item()) == b.ERR_TIMEOUT
    status.zero_()
    C = b.nvfp4_gemm_ex(da, db, b.DT_F32, dev_status=status, variant=variant)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert rel_fro(C.cpu().numpy(), want) <= 1e-5
