"""GPU parity of the OsciReset kernels (Algorithms 1 and 2): statistics, snapshot and reset are float32 element
operations with a fixed order, so they are compared bit for bit with the oracle."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from oracle import oscireset as osc
from paper_2510_27527_b200 import synth

pytestmark = pytest.mark.gpu
MODES = [orc.GS_TENSOR, orc.GS_ROW, orc.GS_BLOCK128]


def B():
    from paper_2510_27527_b200 import binding

    return binding


def dev(W, pad=0):
    """Upload a float32 matrix, optionally into a wider buffer (leading dimension > columns)."""
    t = torch.from_numpy(np.ascontiguousarray(W)).cuda()
    if pad:
        buf = torch.full((W.shape[0], W.shape[1] + pad), 7.0, dtype=torch.float32, device="cuda")
        buf[:, : W.shape[1]] = t
        return buf[:, : W.shape[1]]
    return t


def bits(a):
    return np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)


@pytest.mark.parametrize("shape", [(1, 16), (5, 48), (48, 272), (130, 200), (64, 1024 + 36), (33, 130)])
@pytest.mark.parametrize("gs_mode", MODES)
def test_update_and_suppress_bit_exact(shape, gs_mode):
    b = B()
    C, D = shape
    traj, _ = synth.weight_trajectory(C, D, 5, seed=17 + D)
    st_ref = osc.Stats((C, D))
    state = b.alloc_osci_state(dev(traj[0]))
    for t, W in enumerate(traj):
        osc.update_stats(W, st_ref, t, gs_mode)
        b.nvfp4_osci_update(dev(W, pad=4 if t % 2 else 0), state, t, gs_mode)
        torch.cuda.synchronize()
        assert np.array_equal(bits(state.W_prev.cpu().numpy()), bits(st_ref.W_prev)), f"W_prev t={t}"
        assert np.array_equal(bits(state.D_M.cpu().numpy()), bits(st_ref.D_M)), f"D_M t={t}"
        bad = np.argwhere(bits(state.D_Q.cpu().numpy()) != bits(st_ref.D_Q))
        assert len(bad) == 0, f"D_Q t={t}: {len(bad)} differ, first {bad[:4].tolist()}"
    for tau in (8.0, 0.0):
        want, mask = osc.suppress(traj[-1], st_ref, tau, gs_mode)
        Wd = dev(traj[-1], pad=8)
        n = torch.zeros(1, dtype=torch.int64, device="cuda")
        b.nvfp4_osci_suppress(Wd, state, tau, gs_mode, n_reset=n)
        torch.cuda.synchronize()
        assert np.array_equal(bits(Wd.cpu().numpy()), bits(want)), f"suppress tau={tau}"
        assert int(n.item()) == int(mask.sum())


def test_padding_of_a_strided_weight_buffer_is_untouched():
    b = B()
    traj, _ = synth.weight_trajectory(16, 40, 2, seed=4)
    buf = torch.full((16, 48), 7.0, dtype=torch.float32, device="cuda")
    buf[:, :40] = torch.from_numpy(traj[2]).cuda()
    W = buf[:, :40]
    state = b.alloc_osci_state(W)
    b.nvfp4_osci_update(dev(traj[0]), state, 0)
    b.nvfp4_osci_update(dev(traj[1]), state, 1)
    b.nvfp4_osci_update(W, state, 2)
    b.nvfp4_osci_suppress(W, state, 0.0)
    torch.cuda.synchronize()
    assert torch.all(buf[:, 40:] == 7.0)


@pytest.mark.parametrize("gs_mode", MODES)
def test_reset_leaves_the_forward_weight_operand_unchanged(gs_mode):
    """The paper's claim about Algorithm 1, end to end on the device: quantizing the weights for the forward pass before
    and after the reset gives the same operand."""
    b = B()
    traj, _ = synth.weight_trajectory(128, 512, 6, seed=9)
    state = b.alloc_osci_state(dev(traj[0]))
    for t, W in enumerate(traj):
        b.nvfp4_osci_update(dev(W), state, t, gs_mode)
    W = dev(traj[-1])
    before = b.nvfp4_quantize(W.to(torch.bfloat16), b.AXIS_ROW, b.ROUND_RTN, 0, 2, gs_mode)
    n = torch.zeros(1, dtype=torch.int64, device="cuda")
    b.nvfp4_osci_suppress(W, state, 8.0, gs_mode, n_reset=n)
    after = b.nvfp4_quantize(W.to(torch.bfloat16), b.AXIS_ROW, b.ROUND_RTN, 0, 2, gs_mode)
    torch.cuda.synchronize()
    assert int(n.item()) > 0
    assert torch.equal(before.codes, after.codes) and torch.equal(before.sf, after.sf) and torch.equal(before.gscale, after.gscale)


@pytest.mark.parametrize("shape", [(1, 16), (5, 48), (48, 272), (130, 200), (64, 1024 + 36), (300, 520)])
@pytest.mark.parametrize("gs_mode", MODES)
def test_memory_efficient_statistics_bit_exact(shape, gs_mode):
    """Algorithm 3: tracked index set, snapshots and path lengths identical to the oracle's; the reset as well."""
    b = B()
    C, D = shape
    traj, _ = synth.weight_trajectory(C, D, 4, seed=5 + D)
    n_track = max(1, (C * D) // 12)
    ref = osc.SparseStats(n_track)
    state = b.alloc_osci_sparse_state(n_track)
    for t, W in enumerate(traj):
        osc.update_stats_sparse(W, ref, t, gs_mode)
        b.nvfp4_osci_sparse_update(dev(W, pad=4 if t % 2 else 0), state, t, gs_mode)
        torch.cuda.synchronize()
        got_idx = state.idx.cpu().numpy().astype(np.int64)
        if t == 0:
            bad = np.nonzero(got_idx != ref.idx)[0]
            assert len(bad) == 0, f"idx: {len(bad)} differ, first at {bad[:4].tolist()}: {got_idx[bad[:4]].tolist()} vs {ref.idx[bad[:4]].tolist()}"
        assert np.array_equal(bits(state.WM_prev.cpu().numpy()), bits(ref.WM_prev)), f"WM t={t}"
        assert np.array_equal(bits(state.WQ_prev.cpu().numpy()), bits(ref.WQ_prev)), f"WQ t={t}"
        assert np.array_equal(bits(state.D_M.cpu().numpy()), bits(ref.D_M)), f"D_M t={t}"
        assert np.array_equal(bits(state.D_Q.cpu().numpy()), bits(ref.D_Q)), f"D_Q t={t}"
    for tau in (8.0, 0.0):
        want, hit = osc.suppress_sparse(traj[-1], ref, tau, gs_mode)
        Wd = dev(traj[-1], pad=8)
        n = torch.zeros(1, dtype=torch.int64, device="cuda")
        b.nvfp4_osci_sparse_suppress(Wd, state, tau, gs_mode, n_reset=n)
        torch.cuda.synchronize()
        assert np.array_equal(bits(Wd.cpu().numpy()), bits(want)), f"sparse suppress tau={tau}"
        assert int(n.item()) == int(hit.sum())


def test_selection_with_massive_ties_and_extreme_counts():
    """Scores with very few distinct values (a matrix that is already on the grid scores 0 everywhere): the tie rule
    decides everything; also n_track = all elements."""
    b = B()
    C, D = 40, 64
    W = np.zeros((C, D), dtype=np.float32)
    W[:, 0] = 6.0  # every block: scale from 6, everything else exactly 0 -> all scores 0
    W[3, 5] = 0.7  # a single positive score
    for n_track in (1, 2, 100, C * D):
        ref = osc.SparseStats(n_track)
        osc.update_stats_sparse(W, ref, 0, orc.GS_TENSOR)
        state = b.alloc_osci_sparse_state(n_track)
        b.nvfp4_osci_sparse_update(dev(W), state, 0, b.GS_TENSOR)
        torch.cuda.synchronize()
        assert np.array_equal(state.idx.cpu().numpy().astype(np.int64), ref.idx), n_track
