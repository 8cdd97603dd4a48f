"""Host-side checks of the harness' convolution lowering (plain torch on CPU tensors, no kernel launch)."""
import pytest
import torch

from paper_2310_03675_b200 import nn as hnn


@pytest.mark.parametrize("k,stride,pad", [(3, 1, 1), (3, 2, 1), (1, 2, 0), (1, 1, 0), (3, 1, 0)])
def test_patch_matrix_reproduces_the_convolution_and_col2im_is_its_adjoint(k, stride, pad):
    torch.manual_seed(k * 10 + stride)
    x = torch.randn(2, 5, 8, 7, dtype=torch.float64)
    w = torch.randn(4, 5, k, k, dtype=torch.float64)
    xc, Ho, Wo = hnn._im2col(x, k, stride, pad)
    y = (xc @ hnn._weight_matrix(w).t()).view(2, Ho, Wo, 4).permute(0, 3, 1, 2)
    ref = torch.nn.functional.conv2d(x, w, None, stride, pad)
    assert torch.allclose(y, ref, atol=1e-12)
    # <im2col(x), g> == <x, col2im(g)> for any g: col2im is the adjoint, i.e. the data gradient's scatter-add
    g = torch.randn_like(xc)
    back = hnn._col2im(g, x.shape, k, stride, pad, Ho, Wo)
    assert abs(float((xc * g).sum()) - float((x * back).sum())) < 1e-9 * float(g.abs().sum())


@pytest.mark.parametrize("k,pad", [(3, 1), (3, 0), (5, 2), (3, 2)])
def test_data_gradient_of_a_stride_1_convolution_is_a_convolution_with_the_rotated_kernel(k, pad):
    """The identity behind the implicit data-gradient path: dX = conv(G, W rotated by 180 degrees with the channel
    roles exchanged, padding k-1-p), contraction over (kh, kw, cout)."""
    torch.manual_seed(k + pad)
    x = torch.randn(2, 6, 9, 8, dtype=torch.float64, requires_grad=True)
    w = torch.randn(5, 6, k, k, dtype=torch.float64)
    y = torch.nn.functional.conv2d(x, w, None, 1, pad)
    g = torch.randn_like(y)
    (dx,) = torch.autograd.grad(y, x, g)
    # the same layout transformations as hdqt.conv2d_dgrad: W[Cout,kh,kw,Cin] -> [Cin,kh,kw,Cout], taps flipped
    wk = w.permute(0, 2, 3, 1)
    w_rot = wk.flip(1, 2).permute(3, 1, 2, 0).contiguous()
    gc, H2, W2 = hnn._im2col(g, k, 1, k - 1 - pad)
    assert (H2, W2) == (x.shape[2], x.shape[3])
    dx2 = (gc @ w_rot.reshape(w_rot.shape[0], -1).t()).view(2, H2, W2, 6).permute(0, 3, 1, 2)
    assert torch.allclose(dx2, dx, atol=1e-11)


def test_synthetic_image_recipe_is_seeded_and_bounded():
    dev = torch.device("cpu")
    pat = hnn.class_patterns(7, seed=3, device=dev)
    assert pat.shape == (7, 3, 32, 32) and float(pat.min()) >= 0.0 and float(pat.max()) <= 1.0
    labels = torch.tensor([0, 3, 6, 3])
    a = hnn.synthetic_images(labels, pat, seed=11, blend=0.2)
    b = hnn.synthetic_images(labels, pat, seed=11, blend=0.2)
    assert torch.equal(a, b) and not torch.equal(a, hnn.synthetic_images(labels, pat, seed=12, blend=0.2))
    assert float(a.min()) >= 0.0 and float(a.max()) <= 1.0
    # two images of one class share the class pattern: their difference is pure noise of weight 0.8
    assert float((a[1] - a[3]).abs().max()) <= 0.8 + 1e-6
