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


# Delayed scaling (optional, `delayed=True` in the layer overrides): every (layer, product, operand) keeps two
# history buffers of partial calibration maxima; a step quantizes with the maxima its predecessor left and leaves
# its own (the library's quantize pass produces them for free), so that only a layer's first step runs the
# calibration pass.
_HISTORY = {}


def _history(layer_id: int, kind: str, device):
    key = (layer_id, kind, str(device))
    h = _HISTORY.get(key)
    if h is None:
        h = _HISTORY[key] = {"bufs": [[torch.zeros(hdqt.AMAX_HISTORY_WORDS, dtype=torch.int32, device=device)
                                       for _ in range(2)] for _ in range(2)], "calls": 0}
    return h


def reset_delayed_scaling():
    """Forget every carried maximum (call when tensor shapes or roles change, e.g. between unrelated models)."""
    _HISTORY.clear()


def _desc(kind: str, layer_id: int, seed: int, device=None, **over):
    base = 8 * layer_id + 2 * _KIND[kind]
    over = dict(over)
    if over.pop("delayed", False) and device is not None:
        h = _history(layer_id, kind, device)
        cur, prev = h["bufs"][h["calls"] & 1], h["bufs"][(h["calls"] + 1) & 1]
        over["amax_hist_out_a"], over["amax_hist_out_b"] = cur[0], cur[1]
        if h["calls"] > 0:
            over["amax_hist_in_a"], over["amax_hist_in_b"] = prev[0], prev[1]
        h["calls"] += 1
    return hdqt.default_desc(kind, seed=seed, tag_a=base, tag_b=base + 1, **over)


class HdqtLinearFunction(torch.autograd.Function):
    """y = act(x @ w + b) with w stored [D, C]; forward, dX and dW are HDQT GEMMs.  Bias and ReLU (both optional)
    are applied inside the forward GEMM's dequantising epilogue."""

    @staticmethod
    def forward(ctx, x, w, bias, relu: bool, layer_id: int, seed: int, over: dict):
        x = x.contiguous()
        w = w.contiguous()
        extra = dict(over)
        if bias is not None:
            extra["bias"] = bias.contiguous()
        if relu:
            extra["flags"] = int(extra.get("flags", 0)) | hdqt.FLAG_RELU
        d = _desc("fwd", layer_id, seed, x.device, **extra)
        y, _ = hdqt.gemm_fwd(x, w, desc=d, workspace=_workspace(d, x.shape[0], w.shape[1], x.shape[1], x.device))
        ctx.save_for_backward(x, w, y if relu else None)
        ctx.meta = (layer_id, seed, over, bias is not None)
        return y

    @staticmethod
    def backward(ctx, g):
        x, w, y = ctx.saved_tensors
        layer_id, seed, over, has_bias = ctx.meta
        g = g.contiguous()
        if y is not None:
            g = g * (y > 0)
        dx = dw = db = None
        if ctx.needs_input_grad[0]:
            d = _desc("dgrad", layer_id, seed, g.device, **over)
            dx, _ = hdqt.gemm_dgrad(g, w, desc=d, workspace=_workspace(d, g.shape[0], w.shape[0], g.shape[1], g.device))
        if ctx.needs_input_grad[1]:
            d = _desc("wgrad", layer_id, seed, g.device, **over)
            dw, _ = hdqt.gemm_wgrad(x, g, desc=d, workspace=_workspace(d, x.shape[1], g.shape[1], x.shape[0], x.device))
        if has_bias and ctx.needs_input_grad[2]:
            db = g.sum(0)
        return dx, dw, db, None, None, None, None


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

    def forward(self, x, relu: bool = False):
        return HdqtLinearFunction.apply(x, self.weight, self.bias, relu, self.layer_id, self.step, self.over)


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
            last = i + 1 == len(self.layers)
            if self.quantized:
                x = l(x, relu=not last)          # bias and ReLU inside the forward GEMM's epilogue
            else:
                x = x @ l.weight + l.bias
                if not last:
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


class GraphedTrainStep:
    """One training step (forward, loss, backward, optimiser step) of a fixed-shape model recorded into CUDA
    graphs and replayed: the library calls never synchronise the host and allocate nothing per call, so a whole
    step is one graph launch instead of several hundred kernel launches with their host-side cost.

    The Philox seed of a recorded call is fixed, so the stochastic roundings of successive replays are told apart
    on the device: every quantized layer gets `philox_offset` = a device counter that the graph itself increments
    once per step (step k rounds with (seed, offset) = (base_step, k)).  Two graphs are recorded and replayed
    alternately, because delayed scaling ping-pongs between two history buffers per tensor.

    `forward(x)` maps the static input batch to logits; `warmup` eager steps run first (they are real training
    steps: optimiser state and workspaces must exist before the recording)."""

    def __init__(self, model: torch.nn.Module, opt: torch.optim.Optimizer, x: torch.Tensor, labels: torch.Tensor,
                 forward=None, base_step: int = 0, warmup: int = 3):
        self.model, self.opt = model, opt
        self.forward = forward if forward is not None else model
        dev = x.device
        self.counter = torch.zeros(1, dtype=torch.int32, device=dev)
        for m in model.modules():
            if isinstance(m, (HdqtLinear, HdqtConv2d)):
                m.over = dict(m.over, philox_offset=self.counter)
                m.step = base_step
        self.x, self.labels = x.clone(), labels.clone()
        self.steps = 0
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream(dev))
        with torch.cuda.stream(side):
            for _ in range(warmup):
                self._body()
        torch.cuda.current_stream(dev).wait_stream(side)
        self.graphs, self.losses = [], []
        for _ in range(2):
            g = torch.cuda.CUDAGraph()
            opt.zero_grad(set_to_none=True)
            with torch.cuda.graph(g, pool=self.graphs[0].pool() if self.graphs else None):
                loss = self._body()
            self.graphs.append(g)
            self.losses.append(loss)
        self.steps = warmup

    def _body(self):
        self.opt.zero_grad(set_to_none=True)
        loss = torch.nn.functional.cross_entropy(self.forward(self.x), self.labels)
        loss.backward()
        self.opt.step()
        self.counter += 1
        return loss

    def __call__(self, x: torch.Tensor, labels: torch.Tensor) -> torch.Tensor:
        """Copies the batch into the static buffers and replays one step; returns the (static) loss tensor."""
        self.x.copy_(x, non_blocking=True)
        self.labels.copy_(labels, non_blocking=True)
        i = self.steps & 1
        self.graphs[i].replay()
        self.steps += 1
        return self.losses[i]


# ---- convolution as an im2col GEMM -------------------------------------------------------------------
# The transform and the quantizer act along the contraction dimension of the matmul a convolution lowers to
# (paper Section 3: Z = X W for every layer): rows = output positions (batch x Ho x Wo), contraction =
# Cin x kh x kw, columns = output channels.

# Layout: activations are handled as NHWC (the channels-last storage of a [B, C, H, W] tensor), and the
# contraction index runs over (kh, kw, cin) with cin fastest, so that every 32-wide Hadamard block / accumulator
# tile of a layer with cin % 32 == 0 is 32 consecutive channels of one input pixel.

def _nhwc(x):
    """[B, C, H, W] (any strides) -> contiguous [B, H, W, C] (no copy for channels-last tensors)."""
    return x.permute(0, 2, 3, 1).contiguous()


def _im2col(x, kernel, stride, padding):
    """x [B, Cin, H, W] -> (X_col [B*Ho*Wo, kh*kw*Cin] contiguous, Ho, Wo): one strided copy per kernel tap."""
    B, C, H, W = x.shape
    Ho = (H + 2 * padding - kernel) // stride + 1
    Wo = (W + 2 * padding - kernel) // stride + 1
    xn = _nhwc(x)
    if kernel == 1 and padding == 0:
        return xn[:, ::stride, ::stride, :].reshape(B * Ho * Wo, C), Ho, Wo
    if padding:
        xn = torch.nn.functional.pad(xn, (0, 0, padding, padding, padding, padding))
    cols = torch.empty((B, Ho, Wo, kernel * kernel, C), dtype=x.dtype, device=x.device)
    for kh in range(kernel):
        for kw in range(kernel):
            cols[:, :, :, kh * kernel + kw, :] = xn[:, kh:kh + (Ho - 1) * stride + 1:stride,
                                                    kw:kw + (Wo - 1) * stride + 1:stride, :]
    return cols.view(B * Ho * Wo, kernel * kernel * C), Ho, Wo


def _col2im(dcols, xshape, kernel, stride, padding, Ho, Wo):
    """Adjoint of _im2col: dX_col [B*Ho*Wo, kh*kw*Cin] -> dX as a channels-last [B, Cin, H, W] tensor."""
    B, C, H, W = xshape
    d = dcols.view(B, Ho, Wo, kernel * kernel, C)
    if kernel == 1 and padding == 0:
        if stride == 1:
            return d.view(B, H, W, C).permute(0, 3, 1, 2)
        dx = torch.zeros((B, H, W, C), dtype=dcols.dtype, device=dcols.device)
        dx[:, ::stride, ::stride, :] = d[:, :, :, 0, :]
        return dx.permute(0, 3, 1, 2)
    dx = torch.zeros((B, H + 2 * padding, W + 2 * padding, C), dtype=dcols.dtype, device=dcols.device)
    for kh in range(kernel):
        for kw in range(kernel):
            dx[:, kh:kh + (Ho - 1) * stride + 1:stride, kw:kw + (Wo - 1) * stride + 1:stride, :] += d[:, :, :, kh * kernel + kw, :]
    return dx[:, padding:padding + H, padding:padding + W, :].permute(0, 3, 1, 2)


def _weight_matrix(w):
    """[Cout, Cin, kh, kw] -> [Cout, kh*kw*Cin] in the contraction order of _im2col (the "[C, D]" weight layout)."""
    return w.permute(0, 2, 3, 1).reshape(w.shape[0], -1)


class HdqtConv2dFunction(torch.autograd.Function):
    """y = conv2d(x, w) (no bias) with the forward, dX and dW products as HDQT GEMMs on the patch (im2col)
    matrix.  With cin % 32 == 0 the forward and dW products gather the patches straight from the NHWC
    activation inside the library's transform/quantize kernels (no patch matrix is materialised); other layers
    (the 3-channel stem) build the matrix with torch copies.  dX of a stride-1 layer (cout % 32 == 0) is the
    convolution of G with the rotated kernel through the same implicit path (contraction over kh x kw x cout);
    strided and 1x1 layers take the dgrad GEMM on the patch matrix followed by its scatter-add."""

    @staticmethod
    def forward(ctx, x, w, stride: int, padding: int, layer_id: int, seed: int, over: dict, implicit: bool):
        B, Cin, H, W = x.shape
        Cout, _, kh, kw = w.shape
        d = _desc("fwd", layer_id, seed, x.device, **over)
        implicit = implicit and Cin % 32 == 0 and d.had_block == 32
        wk = w.permute(0, 2, 3, 1).contiguous()                   # [Cout, kh, kw, Cin]
        wm = wk.view(Cout, kh * kw * Cin)
        if implicit:
            xn = _nhwc(x)
            Ho, Wo = hdqt.conv2d_out_size(H, W, kh, stride, padding)
            y4, _ = hdqt.conv2d_fwd(xn, wk, stride, padding, desc=d,
                                    workspace=_workspace(d, B * Ho * Wo, Cout, kh * kw * Cin, x.device))
            ctx.save_for_backward(xn, wm)
        else:
            xc, Ho, Wo = _im2col(x, kh, stride, padding)
            y2d, _ = hdqt.gemm_fwd(xc, wm, desc=d, w_is_cd=True,
                                   workspace=_workspace(d, xc.shape[0], Cout, xc.shape[1], x.device))
            y4 = y2d.view(B, Ho, Wo, Cout)
            ctx.save_for_backward(xc, wm)
        ctx.meta = (layer_id, seed, over, (B, Cin, H, W), (Cout, Cin, kh, kw), stride, padding, Ho, Wo, implicit)
        # [B, Ho, Wo, Cout] is the channels-last storage of [B, Cout, Ho, Wo]: no copy
        return y4.permute(0, 3, 1, 2)

    @staticmethod
    def backward(ctx, g):
        xs, wm = ctx.saved_tensors
        layer_id, seed, over, xshape, wshape, stride, padding, Ho, Wo, implicit = ctx.meta
        B = xshape[0]
        Cout, Cin, kh, kw = wshape
        gn = _nhwc(g)                                             # [B, Ho, Wo, Cout]
        g2d = gn.view(B * Ho * Wo, Cout)
        dx = dw = None
        if ctx.needs_input_grad[0]:
            d = _desc("dgrad", layer_id, seed, g.device, **over)
            if implicit and stride == 1 and kh > 1 and Cout % 32 == 0:
                # the input gradient of a stride-1 convolution is a convolution of G with the rotated kernel
                dxn, _ = hdqt.conv2d_dgrad(gn, wm.view(Cout, kh, kw, Cin), padding, desc=d,
                                           workspace=_workspace(d, B * xshape[2] * xshape[3], Cin, kh * kw * Cout, g.device))
                dx = dxn.permute(0, 3, 1, 2)
            else:
                dxc, _ = hdqt.gemm_dgrad(g2d, wm, desc=d, w_is_cd=True,
                                         workspace=_workspace(d, g2d.shape[0], wm.shape[1], Cout, g.device))
                dx = _col2im(dxc, xshape, kh, stride, padding, Ho, Wo)
        if ctx.needs_input_grad[1]:
            d = _desc("wgrad", layer_id, seed, g.device, **over)
            if implicit:
                dwk, _ = hdqt.conv2d_wgrad(xs, gn, kh, stride, padding, desc=d,
                                           workspace=_workspace(d, Cout, wm.shape[1], g2d.shape[0], g.device))
            else:
                dwm, _ = hdqt.gemm_wgrad(xs, g2d, desc=d, w_is_cd=True,
                                         workspace=_workspace(d, Cout, wm.shape[1], xs.shape[0], g.device))
                dwk = dwm.view(Cout, kh, kw, Cin)
            dw = dwk.permute(0, 3, 1, 2)
        return dx, dw, None, None, None, None, None, None


class HdqtConv2d(torch.nn.Module):
    """3x3 / 1x1 convolution without bias; quantized=False runs torch's fp32 convolution on the same weights."""

    def __init__(self, cin: int, cout: int, kernel: int, stride: int = 1, padding: int = 0, layer_id: int = 0,
                 quantized: bool = True, implicit: bool = True, **over):
        super().__init__()
        self.implicit = implicit     # False: always materialise the patch matrix
        self.weight = torch.nn.Parameter(torch.empty(cout, cin, kernel, kernel))
        torch.nn.init.kaiming_normal_(self.weight, mode="fan_out", nonlinearity="relu")
        self.stride, self.padding, self.layer_id, self.quantized, self.over = stride, padding, layer_id, quantized, over
        self.step = 0

    def forward(self, x):
        if not self.quantized:
            return torch.nn.functional.conv2d(x, self.weight, None, self.stride, self.padding)
        return HdqtConv2dFunction.apply(x, self.weight, self.stride, self.padding, self.layer_id, self.step, self.over,
                                        self.implicit)


class _BasicBlock(torch.nn.Module):
    def __init__(self, cin, cout, stride, ids, quantized, over):
        super().__init__()
        self.conv1 = HdqtConv2d(cin, cout, 3, stride, 1, next(ids), quantized, **over)
        self.bn1 = torch.nn.BatchNorm2d(cout)
        self.conv2 = HdqtConv2d(cout, cout, 3, 1, 1, next(ids), quantized, **over)
        self.bn2 = torch.nn.BatchNorm2d(cout)
        self.shortcut = None
        if stride != 1 or cin != cout:
            self.shortcut = HdqtConv2d(cin, cout, 1, stride, 0, next(ids), quantized, **over)
            self.bn_sc = torch.nn.BatchNorm2d(cout)

    def forward(self, x):
        y = torch.relu(self.bn1(self.conv1(x)))
        y = self.bn2(self.conv2(y))
        sc = x if self.shortcut is None else self.bn_sc(self.shortcut(x))
        return torch.relu(y + sc)


class ResNet18Width(torch.nn.Module):
    """ResNet-18-width network for 32x32x3 inputs (3x3 stem, four stages of two basic blocks with 64/128/256/512
    channels, global average pool, linear head).  Every convolution and the head go through the HDQT GEMMs;
    batch norm, ReLU, pooling, loss and the optimiser stay in fp32 torch ops.  `num_outputs` is the size of the
    head; `forward(x, n_seen)` uses only the first n_seen output neurons (a head that grows with the classes seen)."""

    def __init__(self, num_outputs: int = 100, quantized: bool = True, widths=(64, 128, 256, 512), **over):
        super().__init__()
        ids = iter(range(1000))
        self.quantized = quantized
        self.stem = HdqtConv2d(3, widths[0], 3, 1, 1, next(ids), quantized, **over)
        self.bn = torch.nn.BatchNorm2d(widths[0])
        blocks, cin = [], widths[0]
        for i, w in enumerate(widths):
            for j in range(2):
                blocks.append(_BasicBlock(cin, w, 2 if (i > 0 and j == 0) else 1, ids, quantized, over))
                cin = w
        self.blocks = torch.nn.ModuleList(blocks)
        self.head = HdqtLinear(cin, num_outputs, layer_id=next(ids), **over)

    def set_step(self, step: int):
        for m in self.modules():
            if isinstance(m, (HdqtConv2d, HdqtLinear)):
                m.step = step

    def forward(self, x, n_seen: Optional[int] = None):
        y = torch.relu(self.bn(self.stem(x)))
        for b in self.blocks:
            y = b(y)
        y = y.mean(dim=(2, 3))
        head = self.head
        n = head.weight.shape[1] if n_seen is None else n_seen
        w = head.weight if n == head.weight.shape[1] else head.weight[:, :n].contiguous()
        if self.quantized:
            return HdqtLinearFunction.apply(y.contiguous(), w, head.bias[:n], False, head.layer_id, head.step, head.over)
        return y @ w + head.bias[:n]


def class_patterns(classes: int, seed: int, device, size: int = 32, waves: int = 4):
    """One low-frequency pattern per class: a sum of a few 2-D cosines with class-specific frequencies, phases
    and colour weights, scaled to [0, 1].  Returns [classes, 3, size, size]."""
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    fx = torch.randint(0, 4, (classes, waves), generator=g, device=device).float()
    fy = torch.randint(0, 4, (classes, waves), generator=g, device=device).float()
    ph = torch.rand(classes, waves, generator=g, device=device) * 6.2831853
    amp = torch.randn(classes, 3, waves, generator=g, device=device)
    t = torch.arange(size, device=device).float() / size
    arg = 6.2831853 * (fx[:, :, None, None] * t[None, None, :, None] + fy[:, :, None, None] * t[None, None, None, :]) \
        + ph[:, :, None, None]                                                  # [classes, waves, size, size]
    pat = torch.einsum("ckw,cwxy->ckxy", amp, torch.cos(arg))
    lo = pat.amin(dim=(1, 2, 3), keepdim=True)
    hi = pat.amax(dim=(1, 2, 3), keepdim=True)
    return (pat - lo) / (hi - lo + 1e-6)


def synthetic_images(labels: torch.Tensor, patterns: torch.Tensor, seed: int, blend: float = 0.5):
    """Stand-in for 32x32x3 natural images: pixels ~ U[0,1] blended with the label's low-frequency pattern."""
    g = torch.Generator(device=labels.device)
    g.manual_seed(seed)
    noise = torch.rand((labels.numel(),) + tuple(patterns.shape[1:]), generator=g, device=labels.device)
    return (1.0 - blend) * noise + blend * patterns[labels]


def cnn_train_step(model: ResNet18Width, opt, x, labels, step: int, n_seen: Optional[int] = None):
    model.set_step(step)
    opt.zero_grad(set_to_none=True)
    loss = torch.nn.functional.cross_entropy(model(x, n_seen), labels)
    loss.backward()
    opt.step()
    return loss


def class_incremental_run(quantized: bool, device, tasks: int = 5, classes_per_task: int = 20,
                          steps_per_task: int = 1000, batch: int = 128, memory: int = 2000, seed: int = 0,
                          lr: float = 0.05, test_per_class: int = 20, blend: float = 0.2, log=None,
                          graphed: bool = False, **over):
    """Plain-replay class-incremental training of the ResNet-18-width model on synthetic classes (paper
    Section 4: tasks arrive one after the other, a bounded memory of exemplars is replayed, the head grows with
    the classes seen; appendix: SGD lr 0.05, momentum 0.9, weight decay 2e-4, memory 2000).  Each batch mixes
    new-task samples and replayed exemplars 1:1.  `blend` is the weight of the class pattern in an image (the rest
    is uniform noise): small enough that the task is not solved trivially.  Returns a dict with the final accuracy over all classes seen,
    the accuracy after each task and the number of steps taken.  graphed=True replays each task's training step from
    CUDA graphs (recorded anew per task, because the head grows)."""
    n_classes = tasks * classes_per_task
    patterns = class_patterns(n_classes, seed, device)
    torch.manual_seed(seed)
    model = ResNet18Width(n_classes, quantized=quantized, **over).to(device)
    opt = torch.optim.SGD(model.parameters(), lr=lr, momentum=0.9, weight_decay=2e-4)
    g = torch.Generator(device=device)
    g.manual_seed(seed + 1)
    mem_x = mem_y = None
    step = 0
    acc_after = []
    test_y = torch.arange(n_classes, device=device).repeat_interleave(test_per_class)
    test_x = synthetic_images(test_y, patterns, seed=seed + 777, blend=blend)
    for task in range(tasks):
        lo, hi = task * classes_per_task, (task + 1) * classes_per_task
        n_new = batch if mem_x is None else batch // 2
        model.train()
        stepper = None
        for _ in range(steps_per_task):
            y = torch.randint(lo, hi, (n_new,), generator=g, device=device)
            x = synthetic_images(y, patterns, seed=seed + 1000 + step, blend=blend)
            if mem_x is not None:
                idx = torch.randint(0, mem_x.shape[0], (batch - n_new,), generator=g, device=device)
                x = torch.cat([x, mem_x[idx]])
                y = torch.cat([y, mem_y[idx]])
            if not graphed:
                loss = cnn_train_step(model, opt, x, y, step, n_seen=hi)
                step += 1
            elif stepper is None:
                # (its three warm-up steps train on this first batch and count as steps of the task)
                stepper = GraphedTrainStep(model, opt, x, y, forward=lambda inp, n=hi: model(inp, n),
                                           base_step=(task + 1) * 1000003)
                loss = stepper.losses[0]
                step += 3
            else:
                loss = stepper(x, y)
                step += 1
        del stepper
        # exemplar memory: equal quota per class seen so far, random selection
        quota = memory // hi
        keep_x, keep_y = [], []
        if mem_x is not None:
            for c in range(lo):
                sel = (mem_y == c).nonzero().flatten()[:quota]
                keep_x.append(mem_x[sel]); keep_y.append(mem_y[sel])
        new_y = torch.arange(lo, hi, device=device).repeat_interleave(quota)
        keep_x.append(synthetic_images(new_y, patterns, seed=seed + 5000 + task, blend=blend)); keep_y.append(new_y)
        mem_x, mem_y = torch.cat(keep_x), torch.cat(keep_y)
        # accuracy over every class seen so far
        model.eval()
        with torch.no_grad():
            m = test_y < hi
            pred = []
            for i in range(0, int(m.sum()), 500):
                model.set_step(10 ** 6 + i)
                pred.append(model(test_x[m][i:i + 500], hi).argmax(1))
            acc = float((torch.cat(pred) == test_y[m]).float().mean())
        acc_after.append(acc)
        if log:
            log(f"task {task}: loss {loss.item():.3f} accuracy over {hi} classes {acc:.3f}")
    return {"final_accuracy": acc_after[-1], "accuracy_after_task": acc_after, "steps": step}
