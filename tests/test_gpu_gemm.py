"""GPU parity of the block-scaled FP4 GEMM (tcgen05) against the oracle's dequantize-then-FP64 product."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.gpu_util import bf16_ulp_close, rel_fro, upload_operand

pytestmark = pytest.mark.gpu


def B():
    from paper_2510_27527_b200 import binding

    return binding


def const_operand(R, K, code, sf_byte, gs_mode=0):
    codes = np.full((R, K // 2), code | (code << 4), dtype=np.uint8)
    sf = np.full((R, K // 16), sf_byte, dtype=np.uint8)
    gshape = {0: (1,), 1: (R,), 2: (R, (K + 127) // 128)}[gs_mode]
    return orc.Operand(codes, sf, np.ones(gshape, dtype=np.float32), R, K, gs_mode)


@pytest.mark.parametrize("which", ["A", "B"])
def test_scale_layout_one_hot_probe(which):
    """All codes 1.0, all scales 1.0 except one (row, k-block): exactly that row (or column) of C changes, by 16."""
    b = B()
    M, N, K = 256, 256, 512
    for (r, kb) in [(0, 0), (37, 5), (129, 17), (255, 31), (64, 16), (200, 3)]:
        a, bb = const_operand(M, K, 2, 0x38), const_operand(N, K, 2, 0x38)
        (a if which == "A" else bb).sf[r, kb] = 0x40  # 2.0
        C = b.nvfp4_gemm(upload_operand(a, b), upload_operand(bb, b), b.DT_F32)
        torch.cuda.synchronize()
        C = C.cpu().numpy()
        expect = np.full((M, N), float(K))
        if which == "A":
            expect[r, :] += 16
        else:
            expect[:, r] += 16
        assert np.array_equal(C, expect), (which, r, kb, np.argwhere(C != expect)[:4])


def test_code_layout_one_hot_probe():
    """One non-zero code per operand: C has a single non-zero entry where the k positions meet."""
    b = B()
    M, N, K = 128, 128, 256
    for (m, n, k) in [(0, 0, 0), (5, 77, 1), (127, 3, 255), (64, 64, 130), (33, 90, 63)]:
        a, bb = const_operand(M, K, 0, 0x38), const_operand(N, K, 0, 0x38)
        a.codes[m, k // 2] = 5 << (4 * (k & 1))  # 3.0
        bb.codes[n, k // 2] = 12 << (4 * (k & 1))  # -2.0
        C = b.nvfp4_gemm(upload_operand(a, b), upload_operand(bb, b), b.DT_F32).cpu().numpy()
        expect = np.zeros((M, N))
        expect[m, n] = -6.0
        assert np.array_equal(C, expect), (m, n, k)
        # shifting the k of one operand breaks the match
        bb.codes[:] = 0
        bb.codes[n, ((k + 1) % K) // 2] = 12 << (4 * ((k + 1) & 1))
        C = b.nvfp4_gemm(upload_operand(a, b), upload_operand(bb, b), b.DT_F32).cpu().numpy()
        assert not C.any()


@pytest.mark.parametrize("gs_mode", [0, 1, 2])
@pytest.mark.parametrize("shape", [(128, 128, 256), (256, 384, 1024), (130, 70, 144), (1, 8, 16), (300, 520, 640)])
def test_exact_on_integer_valued_operands(gs_mode, shape):
    """Power-of-two scales and small-integer codes: every partial sum is an integer below 2^24, so FP32
    accumulation is exact and the result must equal the FP64 product exactly."""
    b = B()
    M, N, K = shape
    rng = np.random.default_rng(M + N + K)

    def rnd_operand(R):
        K16 = (K + 15) // 16 * 16
        nib = rng.choice([0, 2, 4, 6, 10, 12, 14], size=(R, K16)).astype(np.uint8)  # 0, +-1, +-2, +-4
        nib[:, K:] = 0
        codes = (nib[:, 0::2] | (nib[:, 1::2] << 4)).astype(np.uint8)
        sf = rng.choice([0x30, 0x38, 0x40], size=(R, K16 // 16)).astype(np.uint8)  # 0.5, 1, 2
        gs = {0: np.array([0.25], dtype=np.float32), 1: rng.choice([0.5, 1.0, 4.0], size=R).astype(np.float32),
              2: rng.choice([0.5, 1.0, 4.0], size=(R, (K + 127) // 128)).astype(np.float32)}[gs_mode]
        return orc.Operand(codes, sf, gs, R, K, gs_mode)

    a, bb = rnd_operand(M), rnd_operand(N)
    want = orc.gemm_operands(a, bb)
    got = b.nvfp4_gemm(upload_operand(a, b), upload_operand(bb, b), b.DT_F32).cpu().numpy()
    assert np.array_equal(got.astype(np.float64), want)


@pytest.mark.parametrize("gs_mode", [0, 1, 2])
@pytest.mark.parametrize("shape", [(256, 512, 512), (384, 256, 2048), (200, 136, 400), (512, 1024, 4096)])
def test_random_operands_against_fp64(gs_mode, shape):
    b = B()
    M, N, K = shape
    x, _ = synth.activations(M, K, 1, n_outlier=4, factor=30.0)
    w = synth.weights(N, K, 2)
    a = orc.quantize(x, orc.AXIS_ROW, orc.RTN, gs_mode)
    bb = orc.quantize(w, orc.AXIS_ROW, orc.SR, gs_mode, seed=4, stream_id=2)
    A64, B64 = orc.dequantize(a), orc.dequantize(bb)
    want = orc.gemm_tn(A64, B64)
    got = b.nvfp4_gemm(upload_operand(a, b), upload_operand(bb, b), b.DT_F32).cpu().numpy()
    assert rel_fro(got, want) <= 1e-3  # the stated bar (normwise); actual error is FP32 accumulation noise
    assert rel_fro(got, want) <= 1e-5
    absdot = np.abs(A64) @ np.abs(B64).T
    assert np.all(np.abs(got - want) <= 1e-3 * absdot + 1e-30)
    # BF16 output: the FP32 result rounded once
    got16 = b.nvfp4_gemm(upload_operand(a, b), upload_operand(bb, b), b.DT_BF16).float().cpu().numpy()
    assert np.all(bf16_ulp_close(got16, want, 1.0, 1e-5 * absdot))
    # accumulate into an existing FP32 C
    C0 = torch.full((M, (N + 7) // 8 * 8), 3.0, device="cuda")[:, :N]
    b.nvfp4_gemm(upload_operand(a, b), upload_operand(bb, b), b.DT_F32, out=C0, accumulate=True)
    assert rel_fro(C0.cpu().numpy() - 3.0, want) <= 1e-4


def test_gemm_consumes_device_quantizer_output():
    """Quantize on the device (tiled scales), multiply on the device, compare with the oracle end to end."""
    b = B()
    from tests.gpu_util import to_dev_bf16

    M, N, K = 384, 640, 1024
    x, _ = synth.activations(M, K, 5, n_outlier=8, factor=30.0)
    w = synth.weights(N, K, 6)
    for gs_mode in (0, 1, 2):
        qa = b.nvfp4_quantize(to_dev_bf16(x), b.AXIS_ROW, b.ROUND_RTN, 0, 1, gs_mode)
        qb = b.nvfp4_quantize(to_dev_bf16(w), b.AXIS_ROW, b.ROUND_RTN, 0, 2, gs_mode)
        got = b.nvfp4_gemm(qa, qb, b.DT_F32).cpu().numpy()
        want = orc.gemm_operands(orc.quantize(x, gs_mode=gs_mode), orc.quantize(w, gs_mode=gs_mode))
        assert rel_fro(got, want) <= 1e-5


def test_block128_gemm_k_limit_is_reported():
    """The outer-block (BLOCK128) product keeps the tile's global scales in shared memory: K up to 16384."""
    b = B()
    a = b.alloc_operand(128, 16384 + 128, b.GS_BLOCK128)
    with pytest.raises(b.Nvfp4Error) as e:
        b.nvfp4_gemm(a, a, b.DT_F32)
    assert e.value.status == 9
    ok = b.alloc_operand(128, 16384, b.GS_BLOCK128)
    ok.gscale.fill_(1.0)
    C = b.nvfp4_gemm(ok, ok, b.DT_F32)
    torch.cuda.synchronize()
    assert not C.any()


def test_block128_scale_layout_one_hot_probe():
    """All codes and block scales 1.0; one outer-block scale of A (or B) doubled: exactly that row (column) of C
    grows by 128."""
    b = B()
    M, N, K = 256, 128, 640
    for which, (r, g) in (("A", (130, 3)), ("B", (77, 0)), ("A", (0, 4)), ("B", (127, 2))):
        a, bb = const_operand(M, K, 2, 0x38, 2), const_operand(N, K, 2, 0x38, 2)
        (a if which == "A" else bb).gscale[r, g] = 2.0
        C = b.nvfp4_gemm(upload_operand(a, b), upload_operand(bb, b), b.DT_F32).cpu().numpy()
        expect = np.full((M, N), float(K))
        if which == "A":
            expect[r, :] += 128
        else:
            expect[:, r] += 128
        assert np.array_equal(C, expect), (which, r, g)


def test_mma_issue_probe_runs_and_reports_its_work():
    """The measurement aid: a short issue loop completes (its single wait is bounded) and reports 148-ish SMs' worth of
    flops; the status word stays 0."""
    from paper_2510_27527_b200 import binding as b

    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    fl = b.nvfp4_mma_issue_probe(8, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert fl == sms * 8 * 4 * 2.0 * 128 * 256 * 64


@pytest.mark.parametrize("n", [32, 128, 256])
@pytest.mark.parametrize("loop_kind", [0, 1, 2, 3, 4])
def test_mma_issue_probe_loop_kinds_complete(n, loop_kind):
    """Every loop structure of the probe (plain, with scale copies, with commits, the two ring walks) drains with status 0,
    reports the flops of its instruction shape and a plausible cycle count: at least n / 2 cycles per 128 x n x 64 MMA for
    n >= 128 (the tensor pipe's rate), and not absurdly more."""
    from paper_2510_27527_b200 import binding as b

    iters = 64
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(2, dtype=torch.int64, device="cuda")
    fl = b.nvfp4_mma_issue_probe(iters, st, n, 0, 0, loop_kind == 4, cnt, loop_kind)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    assert fl == sms * iters * 4 * 2.0 * 128 * n * 64
    per_mma = int(cnt[1].item()) / (iters * 4)
    assert per_mma < 2000
    if n >= 128:
        assert per_mma >= 0.9 * n / 2
    assert int(cnt[0].item()) == 0  # no side warps


@pytest.mark.parametrize("side_kind", [0, 1, 2, 3])
def test_mma_issue_probe_side_warps_count_their_bytes(side_kind):
    from paper_2510_27527_b200 import binding as b

    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    cnt = torch.zeros(2, dtype=torch.int64, device="cuda")
    b.nvfp4_mma_issue_probe(256, st, 128, 3, side_kind, False, cnt, 1)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    moved = int(cnt[0].item())
    unit = {0: 4096, 1: 32 * 128 * 4, 2: 3 * 8192, 3: 3 * 8192}[side_kind]
    assert moved > 0 and moved % unit == 0


def test_mma_issue_probe_refuses_values_outside_its_ranges():
    from paper_2510_27527_b200 import binding as b

    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    for kw in (dict(n=64), dict(loop_kind=5), dict(side_warps=7), dict(side_kind=4)):
        with pytest.raises(b.Nvfp4Error):
            b.nvfp4_mma_issue_probe(8, st, **kw)
    with pytest.raises(b.Nvfp4Error):
        b.nvfp4_mma_issue_probe(0, st)
