"""Thin PyTorch harness over the HDQT GEMM calls: an autograd function for a linear layer whose three
matrix products (forward, dX, dW) all run through the library, plus the synthetic MLP workload.

Everything that is not a matmul (bias, ReLU, loss, SGD) stays in fp32 torch ops, as in the paper
(Section 3: only matmul inputs and accumulators are quantized).
"""
from __future__ import annotations

from typing import Optional

import torch

from . import hdqt

# Philox stream tags: 8*layer + 2*gemm_kind + operand, so that no two stochastic roundings of one step
# share a counter; the step index goes into the seed.
_KIND = {"fwd": 0, "dgrad": 1, "wgrad": 2}


_WORKSPACES = {}


def _workspace(desc, M: int, N: int, K: int, device):
    """One cached workspace per GEMM shape and device (all calls are ordered on the current stream)."""
    key = (M, N, K, desc.had_block, str(device))
    ws = _WORKSPACES.get(key)
    if ws is None:
        ws = _WORKSPACES[key] = hdqt.Workspace(desc, M, N, K, device)
    return ws


def _desc(kind: str, layer_id: int, seed: int, **over):
    base = 8 * layer_id + 2 * _KIND[kind]
    return hdqt.default_desc(kind, seed=seed, tag_a=base, tag_b=base + 1, **over)


class HdqtLinearFunction(torch.autograd.Function):
    """y = x @ w with w stored [D, C]; forward, dX and dW are HDQT GEMMs."""

    @staticmethod
    def forward(ctx, x, w, layer_id: int, seed: int, over: dict):
        x = x.contiguous()
        w = w.contiguous()
        d = _desc("fwd", layer_id, seed, **over)
        y, _ = hdqt.gemm_fwd(x, w, desc=d, workspace=_workspace(d, x.shape[0], w.shape[1], x.shape[1], x.device))
        ctx.save_for_backward(x, w)
        ctx.meta = (layer_id, seed, over)
        return y

    @staticmethod
    def backward(ctx, g):
        x, w = ctx.saved_tensors
        layer_id, seed, over = ctx.meta
        g = g.contiguous()
        dx = dw = None
        if ctx.needs_input_grad[0]:
            d = _desc("dgrad", layer_id, seed, **over)
            dx, _ = hdqt.gemm_dgrad(g, w, desc=d, workspace=_workspace(d, g.shape[0], w.shape[0], g.shape[1], g.device))
        if ctx.needs_input_grad[1]:
            d = _desc("wgrad", layer_id, seed, **over)
            dw, _ = hdqt.gemm_wgrad(x, g, desc=d, workspace=_workspace(d, x.shape[1], g.shape[1], x.shape[0], x.device))
        return dx, dw, None, None, None


class HdqtLinear(torch.nn.Module):
    """Linear layer (weight [D, C], the paper's W in R^{DxC}) with HDQT matmuls."""

    def __init__(self, in_features: int, out_features: int, layer_id: int = 0, bias: bool = True, **over):
        super().__init__()
        self.weight = torch.nn.Parameter(torch.empty(in_features, out_features))
        torch.nn.init.kaiming_uniform_(self.weight.t(), a=5 ** 0.5)
        self.bias = torch.nn.Parameter(torch.zeros(out_features)) if bias else None
        self.layer_id = layer_id
        self.over = over
        self.step = 0          # advanced by the training loop; feeds the Philox seed

    def forward(self, x):
        y = HdqtLinearFunction.apply(x, self.weight, self.layer_id, self.step, self.over)
        return y if self.bias is None else y + self.bias


class Mlp(torch.nn.Module):
    """1152 -> 512 -> 256 -> 12 with ReLU (the synthetic sensor-window workload); quantized=False gives
    the fp32 torch model of the same shape and initialisation for comparison."""

    def __init__(self, sizes=(1152, 512, 256, 12), quantized: bool = True, **over):
        super().__init__()
        self.quantized = quantized
        self.layers = torch.nn.ModuleList(
            [HdqtLinear(a, b, layer_id=i, **over) for i, (a, b) in enumerate(zip(sizes[:-1], sizes[1:]))])

    def set_step(self, step: int):
        for l in self.layers:
            l.step = step

    def forward(self, x):
        for i, l in enumerate(self.layers):
            x = l(x) if self.quantized else x @ l.weight + l.bias
            if i + 1 < len(self.layers):
                x = torch.relu(x)
        return x


def sensor_window_batch(batch: int, features: int, classes: int, seed: int, device):
    """Synthetic stand-in for flattened 9-channel x 128-sample windows: features ~ N(mu_class, 1) with
    class means mu ~ N(0, 0.5^2)."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    means = torch.randn(classes, features, generator=g, device=device) * 0.5
    labels = torch.randint(0, classes, (batch,), generator=g, device=device)
    x = means[labels] + torch.randn(batch, features, generator=g, device=device)
    return x, labels


def train_step(model: Mlp, opt: torch.optim.Optimizer, x, labels, step: int):
    model.set_step(step)
    opt.zero_grad(set_to_none=True)
    loss = torch.nn.functional.cross_entropy(model(x), labels)
    loss.backward()
    opt.step()
    return loss
