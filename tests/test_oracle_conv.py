"""Pins of the convolution oracle (oracle/conv_oracle.py) against things other than itself: the
definition as nested Python loops, the unfolded-input matrix product, torch's conv2d and autograd in
fp64, finite differences, special filters, the stride-2 / stride-1 relation, adjointness; and planted
mistakes (a transposed filter, a shifted tap, sum-for-mean) that at least one pin must catch."""
import numpy as np
import pytest
import torch

from oracle import conv_oracle as co
from paper_1705_09056_b200 import workloads as wl

SHAPES = [  # B, C, O, H, W, stride
    (2, 3, 4, 5, 6, 1),
    (1, 2, 3, 6, 6, 2),
    (2, 1, 2, 7, 5, 2),      # odd sizes: the last stride-2 window hangs over the border
    (1, 3, 2, 1, 1, 1),      # a single pixel: only the centre tap sees data
    (1, 1, 1, 2, 2, 2),
]


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


@pytest.mark.parametrize("B,C,O,H,W,stride", SHAPES)
@pytest.mark.parametrize("relu", [False, True])
def test_forward_equals_the_definition_written_as_nested_loops(B, C, O, H, W, stride, relu):
    x, w, b = _rand((B, C, H, W), 1), _rand((O, C, 3, 3), 2), _rand((O,), 3)
    y, pre = co.conv3x3_forward(x, w, b, stride, relu)
    ref = co.conv3x3_forward_loops(x, w, b, stride, relu)
    assert y.shape == (B, O, co.out_size(H, stride), co.out_size(W, stride))
    assert np.allclose(y, ref, rtol=0, atol=1e-12)
    if relu:
        assert np.all(y >= 0) and np.allclose(y, np.maximum(pre, 0))


def _unfold(x, stride):
    """im2col written out here, independently: rows (b, i, j), columns (c, kh, kw)."""
    B, C, H, W = x.shape
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    M = np.zeros((B * Ho * Wo, C * 9))
    for b in range(B):
        for i in range(Ho):
            for j in range(Wo):
                for c in range(C):
                    for kh in range(3):
                        for kw in range(3):
                            r, q = stride * i + kh - 1, stride * j + kw - 1
                            if 0 <= r < H and 0 <= q < W:
                                M[(b * Ho + i) * Wo + j, (c * 3 + kh) * 3 + kw] = x[b, c, r, q]
    return M, Ho, Wo


@pytest.mark.parametrize("B,C,O,H,W,stride", SHAPES)
def test_convolution_is_a_matrix_product_on_the_unfolded_input(B, C, O, H, W, stride):
    x, w = _rand((B, C, H, W), 4), _rand((O, C, 3, 3), 5)
    M, Ho, Wo = _unfold(x, stride)
    ref = (M @ w.reshape(O, C * 9).T).reshape(B, Ho, Wo, O).transpose(0, 3, 1, 2)
    y, _ = co.conv3x3_forward(x, w, None, stride)
    assert np.allclose(y, ref, rtol=0, atol=1e-12)
    # and the weight gradient is the transposed product: dW = dY^T M
    dy = _rand(y.shape, 6)
    dw, db = co.conv3x3_weight_grad(dy, x, stride)
    ref_dw = (dy.transpose(0, 2, 3, 1).reshape(-1, O).T @ M).reshape(O, C, 3, 3)
    assert np.allclose(dw, ref_dw, rtol=0, atol=1e-12)
    assert np.allclose(db, dy.sum(axis=(0, 2, 3)))


@pytest.mark.parametrize("B,C,O,H,W,stride", SHAPES + [(3, 16, 32, 32, 32, 2), (2, 3, 16, 32, 32, 1)])
def test_forward_and_both_gradients_match_torch_in_fp64(B, C, O, H, W, stride):
    x, w, b = _rand((B, C, H, W), 7), _rand((O, C, 3, 3), 8), _rand((O,), 9)
    tx, tw, tb = (torch.tensor(v, dtype=torch.float64, requires_grad=True) for v in (x, w, b))
    ty = torch.relu(torch.nn.functional.conv2d(tx, tw, tb, stride=stride, padding=1))
    y, pre = co.conv3x3_forward(x, w, b, stride, relu=True)
    assert np.allclose(y, ty.detach().numpy(), rtol=1e-12, atol=1e-12)
    r = _rand(y.shape, 10)
    (ty * torch.tensor(r)).sum().backward()
    d = co.relu_backward(r, pre)
    dw, db = co.conv3x3_weight_grad(d, x, stride)
    dx = co.conv3x3_input_grad(d, w, (H, W), stride)
    assert np.allclose(dw, tw.grad.numpy(), rtol=1e-11, atol=1e-11)
    assert np.allclose(db, tb.grad.numpy(), rtol=1e-11, atol=1e-11)
    assert np.allclose(dx, tx.grad.numpy(), rtol=1e-11, atol=1e-11)


@pytest.mark.parametrize("stride", [1, 2])
def test_gradients_match_central_differences(stride):
    B, C, O, H, W = 2, 2, 3, 5, 4
    x, w, b = _rand((B, C, H, W), 11), _rand((O, C, 3, 3), 12), _rand((O,), 13)
    r = _rand((B, O, co.out_size(H, stride), co.out_size(W, stride)), 14)

    def loss(x_, w_, b_):
        return float(np.sum(co.conv3x3_forward(x_, w_, b_, stride)[0] * r))

    dw, db = co.conv3x3_weight_grad(r, x, stride)
    dx = co.conv3x3_input_grad(r, w, (H, W), stride)
    eps = 1e-6
    rng = np.random.default_rng(15)
    for _ in range(12):
        i = tuple(rng.integers(0, s) for s in w.shape)
        wp, wm = w.copy(), w.copy()
        wp[i] += eps; wm[i] -= eps
        assert abs((loss(x, wp, b) - loss(x, wm, b)) / (2 * eps) - dw[i]) <= 1e-6 * max(1.0, abs(dw[i]))
        j = tuple(rng.integers(0, s) for s in x.shape)
        xp, xm = x.copy(), x.copy()
        xp[j] += eps; xm[j] -= eps
        assert abs((loss(xp, w, b) - loss(xm, w, b)) / (2 * eps) - dx[j]) <= 1e-6 * max(1.0, abs(dx[j]))
    for o in range(O):
        bp, bm = b.copy(), b.copy()
        bp[o] += eps; bm[o] -= eps
        assert abs((loss(x, w, bp) - loss(x, w, bm)) / (2 * eps) - db[o]) <= 1e-6 * max(1.0, abs(db[o]))


def test_special_filters_centre_tap_mixes_channels_and_an_off_centre_tap_shifts():
    B, C, O, H, W = 2, 3, 2, 4, 5
    x = _rand((B, C, H, W), 16)
    mix = _rand((O, C), 17)
    w = np.zeros((O, C, 3, 3))
    w[:, :, 1, 1] = mix
    y, _ = co.conv3x3_forward(x, w, None, 1)
    assert np.allclose(y, np.einsum("oc,bchw->bohw", mix, x))
    # tap (kh, kw) = (0, 2) reads x[i - 1, j + 1]: the image moved down one row and left one column, zeros at the border
    w = np.zeros((1, 1, 3, 3)); w[0, 0, 0, 2] = 1.0
    y, _ = co.conv3x3_forward(x[:, :1], w, None, 1)
    ref = np.zeros((B, 1, H, W))
    ref[:, :, 1:, :W - 1] = x[:, :1, :H - 1, 1:]
    assert np.array_equal(y, ref)


def test_stride_two_is_stride_one_sampled_at_even_positions_and_adjointness():
    x, w, b = _rand((2, 3, 9, 8), 18), _rand((4, 3, 3, 3), 19), _rand((4,), 20)
    y1, _ = co.conv3x3_forward(x, w, b, 1)
    y2, _ = co.conv3x3_forward(x, w, b, 2)
    assert np.array_equal(y2, y1[:, :, ::2, ::2])
    for stride in (1, 2):
        y, _ = co.conv3x3_forward(x, w, None, stride)
        dy = _rand(y.shape, 21)
        assert abs(np.sum(dy * y) - np.sum(co.conv3x3_input_grad(dy, w, (9, 8), stride) * x)) <= 1e-10 * abs(np.sum(dy * y))


def test_planted_mistakes_are_caught():
    """A correlation written as a true convolution (flipped filter), a tap shifted by one, and a padded border
    that wraps around: each differs from the nested-loop definition on a generic input."""
    x, w, b = _rand((1, 2, 5, 5), 22), _rand((2, 2, 3, 3), 23), _rand((2,), 24)
    ref = co.conv3x3_forward_loops(x, w, b, 1, False)
    flipped, _ = co.conv3x3_forward(x, w[:, :, ::-1, ::-1], b, 1)
    assert not np.allclose(flipped, ref, atol=1e-6)
    transposed, _ = co.conv3x3_forward(x, w.transpose(0, 1, 3, 2), b, 1)
    assert not np.allclose(transposed, ref, atol=1e-6)
    wrapped = sum(np.einsum("oc,bchw->bohw", w[:, :, kh, kw], np.roll(x, (1 - kh, 1 - kw), axis=(2, 3)))
                  for kh in range(3) for kw in range(3)) + b[None, :, None, None]
    assert np.allclose(wrapped[:, :, 1:-1, 1:-1], ref[:, :, 1:-1, 1:-1])       # equal in the interior ...
    assert not np.allclose(wrapped, ref, atol=1e-6)                            # ... but not at the border


def test_cifar_shaped_workload_and_layer_stack():
    """The synthetic stand-in for the paper's CIFAR-10 residual networks: 32x32x3 inputs, widths 16/32/64,
    stride 2 where the width doubles; He-initialised filters in one parameter row per node."""
    w = wl.conv_workload(n=3, batch=4, seed=5)
    assert w.plan == ((3, 16, 1), (16, 16, 1), (16, 32, 2), (32, 32, 1), (32, 64, 2), (64, 64, 1))
    assert w.inputs.shape == (3, 4, 3, 32, 32) and w.inputs.dtype == torch.float32
    assert w.params.shape == (3, wl.conv_param_count(w.plan))
    assert wl.conv_param_count(w.plan) == sum(o * c * 9 + o for c, o, _ in w.plan)
    again = wl.conv_workload(n=3, batch=4, seed=5)
    assert torch.equal(again.inputs, w.inputs) and torch.equal(again.params, w.params)
    assert not torch.equal(w.params[0], w.params[1])            # every node has its own filters
    acts = co.layers_forward(w.inputs[0].numpy(), w.params[0].numpy(), w.plan)
    assert [a.shape for a in acts] == [(4, 3, 32, 32), (4, 16, 32, 32), (4, 16, 32, 32), (4, 32, 16, 16),
                                       (4, 32, 16, 16), (4, 64, 8, 8), (4, 64, 8, 8)]
    # He initialisation keeps the activations' scale through the ReLU layers
    for a in acts[1:]:
        assert 0.2 < float(np.sqrt(np.mean(a.astype(np.float64) ** 2))) < 5.0
