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
