"""torch.autograd wrapper around the C-ABI layer calls: `NVFP4Linear` is a drop-in `nn.Linear` (no bias inside the FP4
product; an optional bias is added in BF16) whose forward is `nvfp4_linear_fwd` and whose backward is `nvfp4_linear_bwd`
(paper Sec. 2.3: Y = Q1(X) Q2(W)^T, dX = Q3(dY) Q4(W-hat), dW = Q5(dY^T) Q6(X-hat)). Argument marshalling only: every step
of the path runs in the library's kernels. The stochastic-rounding seed advances with every forward call, so that the
backward of step t draws from its own Philox key.
"""
from __future__ import annotations

import dataclasses

import torch

from . import binding as B


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

    def __init__(self, in_features: int, out_features: int, bias: bool = False, cfg: B.LayerConfig | None = None, device="cuda"):
        super().__init__()
        self.in_features, self.out_features = in_features, out_features
        self.weight = torch.nn.Parameter(torch.empty(out_features, in_features, dtype=torch.bfloat16, device=device))
        torch.nn.init.normal_(self.weight, std=0.02)
        self.bias = torch.nn.Parameter(torch.zeros(out_features, dtype=torch.bfloat16, device=device)) if bias else None
        self.cfg = cfg if cfg is not None else B.LayerConfig()
        self._calls = 0

    def forward(self, x: torch.Tensor) -> torch.Tensor:
        lead = x.shape[:-1]
        x2d = x.reshape(-1, self.in_features)
        if x2d.dtype != torch.bfloat16:
            x2d = x2d.to(torch.bfloat16)
        x2d = x2d.contiguous()
        # a fresh configuration per call: same options and index arrays, the next seed
        cfg = dataclasses.replace(self.cfg, seed=self.cfg.seed + self._calls, y_dtype=B.DT_BF16, dx_dtype=B.DT_BF16, dw_dtype=B.DT_BF16)
        self._calls += 1
        y = _NVFP4LinearFn.apply(x2d, self.weight, cfg)
        if self.bias is not None:
            y = y + self.bias
        return y.reshape(*lead, self.out_features)
