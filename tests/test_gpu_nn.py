"""The autograd wrapper routes forward, dX and dW through the library with the documented seeds/tags, and a
short run on the synthetic MLP workload learns (training-level accuracy is reported, not gated)."""
import numpy as np
import pytest
import torch

from oracle import hdqt_oracle as O

pytestmark = pytest.mark.gpu


def test_linear_layer_gradients_match_the_oracle_gemms():
    from paper_2310_03675_b200 import nn as hnn
    torch.manual_seed(0)
    layer = hnn.HdqtLinear(96, 40, layer_id=2, bias=False).cuda()
    layer.step = 5
    x = torch.randn(64, 96, device="cuda", requires_grad=True)
    y = layer(x)
    g = torch.randn(64, 40, device="cuda") * 1e-3
    y.backward(g)
    X, W, G = x.detach().cpu().numpy(), layer.weight.detach().cpu().numpy(), g.cpu().numpy()
    base = 8 * 2
    want_y = O.gemm_fwd(X, W, O.fwd_desc(seed=5, tag_a=base, tag_b=base + 1))["out"]
    want_dx = O.gemm_dgrad(G, W, O.dgrad_desc(seed=5, tag_a=base + 2, tag_b=base + 3))["out"]
    want_dw = O.gemm_wgrad(X, G, O.wgrad_desc(seed=5, tag_a=base + 4, tag_b=base + 5))["out"]
    assert np.array_equal(y.detach().cpu().numpy(), want_y)
    assert np.array_equal(x.grad.cpu().numpy(), want_dx)
    assert np.array_equal(layer.weight.grad.cpu().numpy(), want_dw)


def test_mlp_learns_the_synthetic_task():
    from paper_2310_03675_b200 import nn as hnn
    torch.manual_seed(1)
    model = hnn.Mlp().cuda()
    opt = torch.optim.SGD(model.parameters(), lr=0.01, momentum=0.9)
    x, labels = hnn.sensor_window_batch(256, 1152, 12, seed=3, device="cuda")
    first = last = None
    for step in range(40):
        loss = hnn.train_step(model, opt, x, labels, step)
        first = loss.item() if first is None else first
        last = loss.item()
    assert np.isfinite(last) and last < 0.5 * first


def test_delayed_scaling_in_the_linear_layer_matches_the_oracle_with_carried_maxima():
    """Second step of a layer with delayed scaling: every operand is quantized with the maximum its counterpart had
    one step earlier (the first step measures)."""
    from paper_2310_03675_b200 import nn as hnn
    hnn.reset_delayed_scaling()
    torch.manual_seed(0)
    layer = hnn.HdqtLinear(96, 40, layer_id=5, bias=False, delayed=True).cuda()
    xs = [torch.randn(64, 96, device="cuda") * s for s in (1.0, 1.5)]
    gs = [torch.randn(64, 40, device="cuda") * s for s in (1e-3, 6e-4)]
    outs = []
    for step in range(2):
        layer.step = step
        x = xs[step].clone().requires_grad_(True)
        layer.weight.grad = None
        y = layer(x)
        y.backward(gs[step])
        outs.append((y.detach().cpu().numpy(), x.grad.cpu().numpy(), layer.weight.grad.cpu().numpy()))
    W = layer.weight.detach().cpu().numpy()
    X0, X1, G0, G1 = (t.cpu().numpy() for t in (xs[0], xs[1], gs[0], gs[1]))

    def amax_h(v):
        return np.float32(np.abs(O.fwht_blockdiag(O.pad_contraction(np.ascontiguousarray(v), 32), 32)).max())

    def product(a_view, b_view, a_prev, b_prev, desc):
        Aq, sa, _ = O.quantize_hadamard(np.ascontiguousarray(a_view), 32, 4, desc.clip_a, desc.round_a, 1, desc.tag_a,
                                        amax=amax_h(a_prev))
        Bq, sb, _ = O.quantize_hadamard(np.ascontiguousarray(b_view), 32, 4, desc.clip_b, desc.round_b, 1, desc.tag_b,
                                        amax=amax_h(b_prev))
        return O.gemm_i8_tiled(Aq, Bq, sa, sb)[0]

    base = 8 * 5
    want_y = product(X1, W.T, X0, W.T, O.fwd_desc(tag_a=base, tag_b=base + 1))
    want_dx = product(G1, W, G0, W, O.dgrad_desc(tag_a=base + 2, tag_b=base + 3))
    want_dw = product(X1.T, G1.T, X0.T, G0.T, O.wgrad_desc(tag_a=base + 4, tag_b=base + 5))
    y1, dx1, dw1 = outs[1]
    assert np.array_equal(y1, want_y) and np.array_equal(dx1, want_dx) and np.array_equal(dw1, want_dw)
    # and the first step was an ordinary measured-maximum step
    first = O.gemm_fwd(X0, W, O.fwd_desc(seed=0, tag_a=base, tag_b=base + 1))["out"]
    assert np.array_equal(outs[0][0], first)
    hnn.reset_delayed_scaling()
