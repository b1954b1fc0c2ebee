"""The workspace-free quantize entry point (for callers that cannot allocate device memory where they call from)
must give exactly what nvfp4_quantize gives. Collected last on purpose: it is an add-on, and a run that stops at the
first failure should already have gone through every other test."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.gpu_util import assert_operand_equal

pytestmark = pytest.mark.gpu


def same(a, b):
    torch.cuda.synchronize()
    return (torch.equal(a.codes, b.codes) and torch.equal(a.sf, b.sf)
            and np.array_equal(a.gscale.cpu().numpy().view(np.uint32), b.gscale.cpu().numpy().view(np.uint32)))


def test_static_scratch_quantize_matches_workspace_quantize_twice_in_a_row():
    from paper_2510_27527_b200 import binding as b

    assert b.lib.nvfp4_quantize_static_max_rows() == 65536
    x1, _ = synth.activations(300, 1000, 1, n_outlier=5, factor=40.0)
    x2 = synth.gradients(520, 272, 2, 1e-3) * np.float32(1e-3)  # much smaller amax: stale cells would show
    d1, d2 = b.upload_bf16(x1), b.upload_bf16(synth.round_to_bf16(x2))
    for mode in (b.GS_TENSOR, b.GS_ROW, b.GS_BLOCK128):
        for axis in (b.AXIS_ROW, b.AXIS_COL):
            for (d, rounding, seed) in ((d1, b.ROUND_RTN, 0), (d2, b.ROUND_SR, 77), (d1, b.ROUND_SR, 78)):
                ref = b.nvfp4_quantize(d, axis, rounding, seed, 3, mode)
                got = b.nvfp4_quantize_static(d, axis, rounding, seed, 3, mode)  # consecutive calls share the cells
                assert same(got, ref), (mode, axis, rounding)
    # and against the oracle itself, not only against the sibling entry point
    want = orc.quantize(x1, orc.AXIS_ROW, orc.SR, orc.GS_ROW, 78, 3)
    assert_operand_equal(b.nvfp4_quantize_static(d1, b.AXIS_ROW, b.ROUND_SR, 78, 3, b.GS_ROW), want, "static scratch, ROW mode, SR")


def test_static_scratch_capacity_is_enforced_before_any_launch():
    from paper_2510_27527_b200 import binding as b

    rows = 65536 + 128
    src = torch.zeros((rows, 16), dtype=torch.bfloat16, device="cuda")
    out = b.alloc_operand(rows, 16, b.GS_ROW)
    n0 = b.lib.nvfp4_launch_count()
    with pytest.raises(b.Nvfp4Error) as e:
        b.nvfp4_quantize_static(src, b.AXIS_ROW, b.ROUND_RTN, 0, 0, b.GS_ROW, out=out)
    assert e.value.status == 9 and b.lib.nvfp4_launch_count() == n0
    # the same shape is fine in the modes that need a single cell
    b.nvfp4_quantize_static(src, b.AXIS_ROW, b.ROUND_RTN, 0, 0, b.GS_TENSOR, out=b.alloc_operand(rows, 16, b.GS_TENSOR))
    torch.cuda.synchronize()
