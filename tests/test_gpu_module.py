"""The autograd wrapper: forward and both gradients of NVFP4Linear against the oracle, and the per-call seed."""
import numpy as np
import pytest
import torch

from oracle import nvfp4_oracle as orc
from paper_2510_27527_b200 import synth
from tests.gpu_util import bf16_ulp_close, to_dev_bf16

pytestmark = pytest.mark.gpu


def test_module_forward_backward_match_the_oracle():
    from paper_2510_27527_b200 import binding as b
    from paper_2510_27527_b200.module import NVFP4Linear, call_seed

    N_tok, D, C = 192, 256, 128
    X, W, dY, ch = synth.layer_inputs(3, N_tok, D, C, n_outlier=3, factor=30.0, grad_scale=1e-3)
    lin = NVFP4Linear(D, C, cfg=b.LayerConfig(gs_mode=b.GS_TENSOR, seed=40, outliers=ch, rht=True))
    with torch.no_grad():
        lin.weight.copy_(to_dev_bf16(W))
    for call in range(2):  # every call has its own key, derived from the base seed, the module instance and the call number
        x = to_dev_bf16(X).reshape(4, 48, D).requires_grad_(True)
        y = lin(x)
        y.backward(to_dev_bf16(dY).reshape(4, 48, C))
        torch.cuda.synchronize()
        ocfg = orc.LayerConfig(gs_mode=orc.GS_TENSOR, seed=call_seed(40, lin.layer_id, call), outliers=ch, rht=True)
        Yo, so = orc.linear_fwd(X, W, ocfg)
        dXo, dWo = orc.linear_bwd_dx(dY, so, ocfg), orc.linear_bwd_dw(dY, so, ocfg)
        assert np.all(bf16_ulp_close(y.detach().reshape(N_tok, C).float().cpu().numpy(), Yo, 1.0, 1e-4 * np.abs(Yo).mean()))
        assert np.all(bf16_ulp_close(x.grad.reshape(N_tok, D).float().cpu().numpy(), dXo, 1.0, 1e-4 * np.abs(dXo).mean()))
        assert np.all(bf16_ulp_close(lin.weight.grad.float().cpu().numpy(), dWo, 1.0, 1e-4 * np.abs(dWo).mean()))
        lin.weight.grad = None
