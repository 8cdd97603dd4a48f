"""The convolution layer as an im2col GEMM: forward, dX and dW of every distinct convolution shape of the
ResNet-18-width model (batch 128, 32x32 inputs) bit for bit against the CPU oracle run on the same im2col
matrices; a short training run of the whole model; the class-incremental loop end to end on a tiny budget.
Training-level accuracy is reported, not gated."""
import numpy as np
import pytest
import torch

from oracle import hdqt_oracle as O

pytestmark = pytest.mark.gpu

# (Cin, Cout, kernel, stride, padding, input size): stem, the four stages' 3x3 convolutions (first of a stage
# with stride 2), and the 1x1 shortcuts
CONV_SHAPES = [
    (3, 64, 3, 1, 1, 32),        # stem: K = 27 -> 32
    (64, 64, 3, 1, 1, 32),       # stage 1: K = 576, 131072 rows (wgrad contraction of 131072 = 4096 tiles)
    (64, 128, 3, 2, 1, 32),      # stage 2 entry
    (64, 128, 1, 2, 0, 32),      # stage 2 shortcut: K = 64
    (128, 128, 3, 1, 1, 16),     # stage 2: K = 1152
    (128, 256, 3, 2, 1, 16),     # stage 3 entry
    (128, 256, 1, 2, 0, 16),     # stage 3 shortcut: K = 128
    (256, 256, 3, 1, 1, 8),      # stage 3: K = 2304
    (256, 512, 3, 2, 1, 8),      # stage 4 entry
    (256, 512, 1, 2, 0, 8),      # stage 4 shortcut: K = 256
    (512, 512, 3, 1, 1, 4),      # stage 4: K = 4608
]


@pytest.mark.parametrize("cin,cout,k,stride,pad,size", CONV_SHAPES)
def test_conv_layer_matches_oracle_on_the_im2col_matrices(cin, cout, k, stride, pad, size):
    from paper_2310_03675_b200 import nn as hnn
    B = 128
    torch.manual_seed(cin * 7 + cout + k)
    layer = hnn.HdqtConv2d(cin, cout, k, stride, pad, layer_id=3).cuda()
    layer.step = 11
    x = torch.relu(torch.randn(B, cin, size, size, device="cuda")).requires_grad_(True)     # post-ReLU activations
    y = layer(x)
    g = (torch.distributions.StudentT(3.0).sample(y.shape).cuda() * 1e-3).contiguous(memory_format=torch.channels_last)
    y.backward(g)
    torch.cuda.synchronize()
    # the same matrices on the host (contraction order (kh, kw, cin), as the layer lays them out)
    xc, Ho, Wo = hnn._im2col(x.detach(), k, stride, pad)
    Xc = xc.cpu().numpy()                                              # [B*Ho*Wo, k*k*Cin]
    Wm = hnn._weight_matrix(layer.weight.detach()).cpu().numpy()       # [Cout, K]
    G2 = g.permute(0, 2, 3, 1).reshape(B * Ho * Wo, cout).cpu().numpy()
    if k == 3 and stride == 1 and cin >= 64:
        # the im2col matrix really is the convolution's patch matrix: row (b, ho, wo), tap (1, 2), channel 5
        b_, ho_, wo_ = 3, 1, 2
        assert Xc[(b_ * Ho + ho_) * Wo + wo_, (1 * 3 + 2) * cin + 5] == x[b_, 5, ho_ + 1 - pad, wo_ + 2 - pad].item()
    base = 8 * 3
    want_y = O.gemm_fwd(Xc, Wm.T, O.fwd_desc(seed=11, tag_a=base, tag_b=base + 1))
    want_dx = O.gemm_dgrad(G2, Wm.T, O.dgrad_desc(seed=11, tag_a=base + 2, tag_b=base + 3))
    want_dw = O.gemm_wgrad(Xc, G2, O.wgrad_desc(seed=11, tag_a=base + 4, tag_b=base + 5))
    got_y = y.detach().permute(0, 2, 3, 1).reshape(B * Ho * Wo, cout).cpu().numpy()
    assert np.array_equal(got_y, want_y["out"])
    # dW comes back in the weight's layout: as a [Cout, K] matrix it is the transposed oracle result
    assert np.array_equal(hnn._weight_matrix(layer.weight.grad).cpu().numpy(), want_dw["out"].T)
    conv_dgrad = cin % 32 == 0 and stride == 1 and k > 1          # dX as a convolution of G with the rotated kernel
    if conv_dgrad:
        # patch matrix of G (padding k-1-pad) times the rotated kernel [Cin, (kh, kw, cout)], dgrad roles
        gc, H2, W2 = hnn._im2col(g, k, 1, k - 1 - pad)
        assert (H2, W2) == (size, size)
        w_rot = layer.weight.detach().permute(0, 2, 3, 1).flip(1, 2).permute(3, 1, 2, 0).reshape(cin, -1)
        want = O.hdqt_gemm(gc.cpu().numpy(), w_rot.cpu().numpy(), O.dgrad_desc(seed=11, tag_a=base + 2, tag_b=base + 3))
        got_dx = x.grad.permute(0, 2, 3, 1).reshape(B * size * size, cin).cpu().numpy()
        assert np.array_equal(got_dx, want["out"])
    else:
        # dX: the column-matrix gradient is scattered back by the layer's own adjoint of im2col (torch adds,
        # fp32); scatter the oracle's column gradient with the same routine
        dxc = torch.from_numpy(want_dx["out"]).cuda()
        want_dx_img = hnn._col2im(dxc, x.shape, k, stride, pad, Ho, Wo)
        assert torch.equal(x.grad, want_dx_img)
    # the same layer with the patch matrix materialised (no implicit gather) gives identical results (dX of a
    # stride-1 layer: a different but equally valid arrangement of the same product, equal up to rounding noise)
    if cin % 32 == 0:
        twin = hnn.HdqtConv2d(cin, cout, k, stride, pad, layer_id=3, implicit=False).cuda()
        twin.load_state_dict(layer.state_dict())
        twin.step = 11
        x2 = x.detach().clone().requires_grad_(True)
        y2 = twin(x2)
        y2.backward(g)
        assert torch.equal(y2, y) and torch.equal(twin.weight.grad, layer.weight.grad)
        dxc = torch.from_numpy(want_dx["out"]).cuda()
        assert torch.equal(x2.grad, hnn._col2im(dxc, x.shape, k, stride, pad, Ho, Wo))
        if conv_dgrad:
            true_dx = torch.autograd.grad(torch.nn.functional.conv2d(x2, layer.weight.detach(), None, stride, pad), x2, g)[0]
            err_conv = (x.grad - true_dx).norm() / true_dx.norm()
            err_cols = (x2.grad - true_dx).norm() / true_dx.norm()
            # heavy-tailed gradients with one scale per tensor: most codes are zero and the rounding noise is as
            # large as the signal in both arrangements; what is checked is that they lose the same amount
            assert abs(err_conv - err_cols) < 0.05 * err_cols, (float(err_conv), float(err_cols))
        else:
            assert torch.equal(x2.grad, x.grad)
    # and the layer agrees with torch's fp32 convolution up to quantisation noise (layout / adjoint sanity)
    ref = torch.nn.functional.conv2d(x.detach(), layer.weight.detach(), None, stride, pad)
    rel = (y.detach() - ref).norm() / ref.norm()
    assert rel < 0.5


def test_conv_gemm_intermediates_at_the_longest_contraction():
    """Stage-1 weight gradient: contraction over 131072 output positions (4096 accumulator tiles, the 16-bit lane
    sums widen 16 times): codes of both operands and the integer sums against the oracle."""
    from paper_2310_03675_b200 import hdqt
    rows, K, C = 131072, 576, 64
    g = torch.Generator(device="cuda"); g.manual_seed(5)
    X = torch.relu(torch.randn(rows, K, generator=g, device="cuda"))
    G = torch.randn(rows, C, generator=g, device="cuda") * 1e-3
    desc = hdqt.default_desc("wgrad", seed=2)
    status = hdqt.new_status("cuda")
    out, ws = hdqt.gemm_wgrad(X, G, desc=desc, w_is_cd=True, dev_status=status)
    hdqt.check_device_status(status)
    want = O.gemm_wgrad(X.cpu().numpy(), G.cpu().numpy(), O.wgrad_desc(seed=2, tag_a=desc.tag_a, tag_b=desc.tag_b))
    # [C, D] layout: the GEMM's A operand is G^T (descriptor operand b), its B operand X^T
    assert np.array_equal(ws.codes_a().cpu().numpy(), want["Bq"])
    assert np.array_equal(ws.codes_b().cpu().numpy(), want["Aq"])
    _, S, _ = hdqt.gemm_i8_tiled(ws.codes_a(), ws.codes_b(), ws.scalar("step_a"), ws.scalar("step_b"), want_S=True)
    assert np.array_equal(S.cpu().numpy().astype(np.int64), want["S"].T)
    assert np.array_equal(out.cpu().numpy(), want["out"].T)


def test_resnet18_width_step_runs_and_learns():
    from paper_2310_03675_b200 import nn as hnn
    dev = torch.device("cuda")
    patterns = hnn.class_patterns(100, seed=1, device=dev)
    torch.manual_seed(0)
    model = hnn.ResNet18Width(100).to(dev)
    opt = torch.optim.SGD(model.parameters(), lr=0.05, momentum=0.9, weight_decay=2e-4)
    g = torch.Generator(device=dev); g.manual_seed(3)
    labels = torch.randint(0, 100, (128,), generator=g, device=dev)
    x = hnn.synthetic_images(labels, patterns, seed=4)
    assert x.shape == (128, 3, 32, 32) and 0.0 <= float(x.min()) and float(x.max()) <= 1.0
    losses = [hnn.cnn_train_step(model, opt, x, labels, step).item() for step in range(12)]
    # 4-bit operands learn more slowly than fp32 (paper Section 4.1: lower final accuracy): only progress is required
    assert np.isfinite(losses).all() and losses[-1] < losses[0] - 0.2
    # the fp32 twin has the same parameters and shapes (what the accuracy comparison of the incremental run uses)
    twin = hnn.ResNet18Width(100, quantized=False).to(dev)
    assert [p.shape for p in twin.parameters()] == [p.shape for p in model.parameters()]


@pytest.mark.parametrize("extra", [{}, {"graphed": True, "delayed": True}])
def test_class_incremental_loop_end_to_end_on_a_small_budget(extra):
    """Two tasks of five classes, a few steps each: head growth, replay mixing, exemplar quota and evaluation run
    through the quantized path (eager, and replayed from CUDA graphs recorded per task with delayed scaling); the
    accuracies are only required to be well-formed."""
    from paper_2310_03675_b200 import nn as hnn
    hnn.reset_delayed_scaling()
    res = hnn.class_incremental_run(True, torch.device("cuda"), tasks=2, classes_per_task=5, steps_per_task=6,
                                    batch=32, memory=40, seed=0, test_per_class=4, **extra)
    hnn.reset_delayed_scaling()
    assert res["steps"] == (16 if extra else 12) and len(res["accuracy_after_task"]) == 2
    assert all(0.0 <= a <= 1.0 for a in res["accuracy_after_task"])


def _patch_matrix_by_loops(x, kh, kw, stride, pad):
    """Plain-loop patch matrix of an NHWC array (written independently of the harness): row (b, ho, wo), column
    (i, j, c) with c fastest, zeros outside the image."""
    B, H, W, C = x.shape
    Ho, Wo = (H + 2 * pad - kh) // stride + 1, (W + 2 * pad - kw) // stride + 1
    out = np.zeros((B * Ho * Wo, kh * kw * C), dtype=np.float32)
    for b in range(B):
        for ho in range(Ho):
            for wo in range(Wo):
                r = (b * Ho + ho) * Wo + wo
                for i in range(kh):
                    for j in range(kw):
                        hi, wi = ho * stride + i - pad, wo * stride + j - pad
                        if 0 <= hi < H and 0 <= wi < W:
                            out[r, (i * kw + j) * C:(i * kw + j + 1) * C] = x[b, hi, wi]
    return out, Ho, Wo


@pytest.mark.parametrize("B,H,W,C,kh,kw,stride,pad,cout", [(3, 10, 7, 32, 3, 2, 2, 1, 24), (2, 5, 9, 64, 1, 3, 1, 0, 40),
                                                           (5, 6, 6, 96, 3, 3, 1, 2, 130), (2, 8, 8, 32, 3, 3, 2, 0, 16)])
def test_implicit_convolution_entry_points_on_odd_geometries(B, H, W, C, kh, kw, stride, pad, cout):
    """hdqt_conv2d_fwd / hdqt_conv2d_wgrad through the binding on non-square images and kernels, strides, wide
    padding and ragged row counts, against the oracle on a patch matrix built by plain loops."""
    from paper_2310_03675_b200 import hdqt
    rng = np.random.default_rng(B * 100 + H)
    x = np.maximum(rng.standard_normal((B, H, W, C)), 0).astype(np.float32)
    if stride == 2 and pad == 0:
        # the last row and column are in no patch here: the largest value of the tensor sits there and must not
        # enter the calibration (the library calibrates on the tensor itself only when the patches cover it)
        x[:, H - 1, :, :] *= 40.0
    w = (rng.standard_normal((cout, kh, kw, C)) * 0.05).astype(np.float32)
    Xc, Ho, Wo = _patch_matrix_by_loops(x, kh, kw, stride, pad)
    g = (rng.standard_t(3, size=(B, Ho, Wo, cout)) * 1e-3).astype(np.float32)
    Wm = w.reshape(cout, -1)
    status = hdqt.new_status("cuda")
    xd, wd, gd = (torch.from_numpy(t).cuda() for t in (x, w, g))
    y, ws = hdqt.conv2d_fwd(xd, wd, stride, pad, desc=hdqt.default_desc("fwd", seed=4), dev_status=status)
    want = O.gemm_fwd(Xc, Wm.T, O.fwd_desc(seed=4, tag_a=0, tag_b=1))
    assert np.array_equal(ws.codes_a().cpu().numpy(), want["Aq"])
    assert np.array_equal(y.cpu().numpy().reshape(-1, cout), want["out"])
    dw, ws = hdqt.conv2d_wgrad(xd, gd, (kh, kw), stride, pad, desc=hdqt.default_desc("wgrad", seed=4), dev_status=status)
    hdqt.check_device_status(status)
    want = O.gemm_wgrad(Xc, g.reshape(-1, cout), O.wgrad_desc(seed=4, tag_a=4, tag_b=5))
    assert np.array_equal(ws.codes_b().cpu().numpy(), want["Aq"])      # [C, D] layout: operands trade places
    assert np.array_equal(dw.cpu().numpy().reshape(cout, -1), want["out"].T)
    # channels not a multiple of 32 are refused on the host
    bad = torch.zeros((1, 4, 4, 24), device="cuda")
    with pytest.raises(hdqt.HdqtError) as err:
        hdqt.conv2d_fwd(bad, torch.zeros((8, 3, 3, 24), device="cuda"), 1, 1)
    assert err.value.status == 2
