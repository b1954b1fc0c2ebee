"""torch.autograd wrapper around the C-ABI layer calls: `NVFP4Linear` is a drop-in `nn.Linear` (no bias inside the FP4
product; an optional bias is added in BF16) whose forward is `nvfp4_linear_fwd` and whose backward is `nvfp4_linear_bwd`
(paper Sec. 2.3: Y = Q1(X) Q2(W)^T, dX = Q3(dY) Q4(W-hat), dW = Q5(dY^T) Q6(X-hat)). Argument marshalling only: every step
of the path runs in the library's kernels. The stochastic-rounding key of a call is derived from the configuration's base
seed, the module instance and the call number, so that neither two steps of one layer nor two layers of a model built
from the same configuration share their draws.
"""
from __future__ import annotations

import dataclasses

import torch

from . import binding as B


_MASK64 = (1 << 64) - 1


def call_seed(base_seed: int, layer_id: int, call: int) -> int:
    """64-bit Philox key of one forward / backward call: a fixed mixing (splitmix64 finaliser) of the base seed, the module
    instance and the call number. Distinct (layer, call) pairs give distinct, unrelated keys; layers of equal shape would
    otherwise draw identical stochastic-rounding bits element for element."""
    z = (base_seed + 0x9E3779B97F4A7C15 * (layer_id + 1) + 0xD1B54A32D192ED03 * (call + 1)) & _MASK64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _MASK64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _MASK64
    return z ^ (z >> 31)


class _NVFP4LinearFn(torch.autograd.Function):
    @staticmethod
    def forward(ctx, x2d: torch.Tensor, weight: torch.Tensor, cfg: B.LayerConfig):
        y, saved = B.nvfp4_linear_fwd(x2d, weight, cfg)
        ctx.saved_ops, ctx.cfg = saved, cfg
        return y

    @staticmethod
    def backward(ctx, dy: torch.Tensor):
        dy = dy.contiguous()
        if dy.dtype != torch.bfloat16:
            dy = dy.to(torch.bfloat16)
        dx, dw = B.nvfp4_linear_bwd(dy, ctx.saved_ops, ctx.cfg)
        return dx, dw, None


class NVFP4Linear(torch.nn.Module):
    """y = x W^T (+ bias) with the NVFP4 forward and backward products. Inputs and weights are BF16 on a CUDA device."""

    _instances = 0  # every module takes the next id: its own stream of stochastic-rounding keys

    def __init__(self, in_features: int, out_features: int, bias: bool = False, cfg: B.LayerConfig | None = None, device="cuda"):
        super().__init__()
        self.in_features, self.out_features = in_features, out_features
        self.weight = torch.nn.Parameter(torch.empty(out_features, in_features, dtype=torch.bfloat16, device=device))
        torch.nn.init.normal_(self.weight, std=0.02)
        self.bias = torch.nn.Parameter(torch.zeros(out_features, dtype=torch.bfloat16, device=device)) if bias else None
        self.cfg = cfg if cfg is not None else B.LayerConfig()
        self._calls = 0
        self.layer_id = NVFP4Linear._instances
        NVFP4Linear._instances += 1

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        lead = x.shape[:-1]
        x2d = x.reshape(-1, self.in_features)
        if x2d.dtype != torch.bfloat16:
            x2d = x2d.to(torch.bfloat16)
        x2d = x2d.contiguous()
        # a fresh configuration per call: same options and index arrays, this layer's key of this call
        cfg = dataclasses.replace(self.cfg, seed=call_seed(self.cfg.seed, self.layer_id, self._calls), y_dtype=B.DT_BF16, dx_dtype=B.DT_BF16, dw_dtype=B.DT_BF16)
        self._calls += 1
        y = _NVFP4LinearFn.apply(x2d, self.weight, cfg)
        if self.bias is not None:
            y = y + self.bias
        return y.reshape(*lead, self.out_features)
