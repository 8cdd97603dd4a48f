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


def test_graphed_step_equals_eager_steps():
    """A training step replayed from a CUDA graph, with the random stream advanced by the device-side Philox word,
    gives the same losses bit for bit as eager steps that pass the same (seed, offset) pairs."""
    from paper_2310_03675_b200 import nn as hnn
    dev = torch.device("cuda")
    sizes = (96, 64, 12)

    def make():
        torch.manual_seed(0)
        m = hnn.Mlp(sizes).to(dev)
        return m, torch.optim.SGD(m.parameters(), lr=0.05, momentum=0.9)

    batches = [hnn.sensor_window_batch(64, sizes[0], sizes[-1], seed=i, device=dev) for i in range(9)]
    # eager: every layer reads the step from a device word that the loop advances
    m1, o1 = make()
    word = torch.zeros(1, dtype=torch.int32, device=dev)
    for l in m1.layers:
        l.over = dict(l.over, philox_offset=word)
    eager = []
    for x, y in batches:
        eager.append(float(hnn.train_step(m1, o1, x, y, step=0).detach()))
        word += 1
    # graphed: three eager warm-up steps inside the constructor, then replays
    m2, o2 = make()
    stepper = None
    graphed = []
    for i, (x, y) in enumerate(batches):
        if i < 3:
            continue
        if stepper is None:
            # the constructor's warm-up steps train on its example batch: feed it the first three batches in turn
            stepper = _warm_graphed(hnn, m2, o2, batches[:3])
            graphed = list(stepper.warm_losses)
        graphed.append(float(stepper(x, y).detach()))
    assert graphed == eager
    assert len(set(eager)) == len(eager)


def _warm_graphed(hnn, model, opt, first):
    """GraphedTrainStep whose warm-up steps run on the given batches (one each)."""
    it = iter(first)
    losses = []

    class Stepper(hnn.GraphedTrainStep):
        def _body(self):
            if len(losses) < len(first):
                x, y = next(it)
                self.x.copy_(x); self.labels.copy_(y)
            loss = super()._body()
            if len(losses) < len(first):
                losses.append(float(loss.detach()))
            return loss

    s = Stepper(model, opt, first[0][0], first[0][1], warmup=len(first))
    s.warm_losses = losses
    return s
