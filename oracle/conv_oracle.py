"""CPU oracle for the convolution layer family.  TEST INFRASTRUCTURE ONLY.

The paper's image workloads are residual networks on CIFAR-10 (Section 5.1 "Datasets and models":
ResNet-20; Section 5.3: a 32-layer residual network), i.e. stacks of 3x3 convolutions on 32x32x3 inputs
with channel widths 16 / 32 / 64 and a stride-2 convolution where the width doubles.  The paper prints
no formula for them; a 3x3 convolution with zero padding 1 and stride s is, by its textbook definition,

    y[b, o, i, j] = bias[o] + sum_{c, kh, kw} w[o, c, kh, kw] * x[b, c, s*i + kh - 1, s*j + kw - 1]

with x read as zero outside the image, optionally followed by ReLU (ReLU'(0) = 0 as in the MLP oracle).
The functions below are that definition and its two adjoints, written as plain loops over the nine
kernel taps in fp64, one rounding to fp32 where a caller stores the result.  They share no code with the
CUDA library and neither imports the other.

Pins (tests/test_oracle_conv.py): a seven-fold nested pure-Python loop on tiny shapes; the identity
"convolution = matrix product on the unfolded (im2col) input"; torch.nn.functional.conv2d and
torch.autograd in fp64 (library routines); central finite differences of a scalar loss; special filters
(a centre tap is a 1x1 channel mix, an off-centre tap is a shift with a zero border); stride 2 equals
stride 1 sampled at the even positions; <dy, conv(x)> = <conv_input_grad(dy), x> (adjointness).
"""
from __future__ import annotations

import numpy as np


def out_size(h: int, stride: int) -> int:
    """Output height/width of a 3x3 convolution with padding 1: floor((h + 2 - 3) / stride) + 1."""
    return (h - 1) // stride + 1


def conv3x3_forward(x, w, bias=None, stride=1, relu=False):
    """y = conv(x, w) + bias (then ReLU): x [B][C][H][W], w [O][C][3][3], bias [O] -> y [B][O][H'][W'], fp64.
    Returns (y, pre) with pre the value before the ReLU (equal to y when relu is False)."""
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    B, C, H, W = x.shape
    O = w.shape[0]
    assert w.shape == (O, C, 3, 3) and stride in (1, 2)
    Ho, Wo = out_size(H, stride), out_size(W, stride)
    xp = np.zeros((B, C, H + 2, W + 2))
    xp[:, :, 1:H + 1, 1:W + 1] = x
    pre = np.zeros((B, O, Ho, Wo))
    for kh in range(3):
        for kw in range(3):
            # the input pixel under tap (kh, kw) of every output position: rows s*i + kh, columns s*j + kw of xp
            patch = xp[:, :, kh:kh + stride * (Ho - 1) + 1:stride, kw:kw + stride * (Wo - 1) + 1:stride]
            pre += np.einsum("oc,bchw->bohw", w[:, :, kh, kw], patch)
    if bias is not None:
        pre += np.asarray(bias, dtype=np.float64)[None, :, None, None]
    return (np.maximum(pre, 0.0) if relu else pre), pre


def relu_backward(dy, pre):
    """dy * [pre > 0] (ReLU'(0) = 0)."""
    return np.asarray(dy, dtype=np.float64) * (np.asarray(pre) > 0.0)


def conv3x3_input_grad(dy, w, in_hw, stride=1):
    """dx[b, c, h, w'] = sum_{o, kh, kw} w[o, c, kh, kw] dy[b, o, i, j] over the (i, j) with
    s*i + kh - 1 = h and s*j + kw - 1 = w': the adjoint of conv3x3_forward in x.  dy is the gradient at the
    convolution's output (after relu_backward when the layer has a ReLU)."""
    dy = np.asarray(dy, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    B, O, Ho, Wo = dy.shape
    C = w.shape[1]
    H, W = in_hw
    assert (Ho, Wo) == (out_size(H, stride), out_size(W, stride))
    dxp = np.zeros((B, C, H + 2, W + 2))
    for kh in range(3):
        for kw in range(3):
            dxp[:, :, kh:kh + stride * (Ho - 1) + 1:stride, kw:kw + stride * (Wo - 1) + 1:stride] += \
                np.einsum("oc,bohw->bchw", w[:, :, kh, kw], dy)
    return dxp[:, :, 1:H + 1, 1:W + 1]


def conv3x3_weight_grad(dy, x, stride=1):
    """(dw, dbias): dw[o, c, kh, kw] = sum_{b, i, j} dy[b, o, i, j] x[b, c, s*i + kh - 1, s*j + kw - 1],
    dbias[o] = sum_{b, i, j} dy[b, o, i, j]: the adjoint in w and bias (a SUM over the minibatch; the caller
    divides by B where the loss is a mean)."""
    dy = np.asarray(dy, dtype=np.float64)
    x = np.asarray(x, dtype=np.float64)
    B, O, Ho, Wo = dy.shape
    _, C, H, W = x.shape
    xp = np.zeros((B, C, H + 2, W + 2))
    xp[:, :, 1:H + 1, 1:W + 1] = x
    dw = np.zeros((O, C, 3, 3))
    for kh in range(3):
        for kw in range(3):
            patch = xp[:, :, kh:kh + stride * (Ho - 1) + 1:stride, kw:kw + stride * (Wo - 1) + 1:stride]
            dw[:, :, kh, kw] = np.einsum("bohw,bchw->oc", dy, patch)
    return dw, dy.sum(axis=(0, 2, 3))


def conv3x3_forward_loops(x, w, bias, stride, relu):
    """The definition as seven nested pure-Python loops (tiny shapes only): the brute-force pin."""
    B, C, H, W = x.shape
    O = w.shape[0]
    Ho, Wo = out_size(H, stride), out_size(W, stride)
    y = np.zeros((B, O, Ho, Wo))
    for b in range(B):
        for o in range(O):
            for i in range(Ho):
                for j in range(Wo):
                    acc = float(bias[o]) if bias is not None else 0.0
                    for c in range(C):
                        for kh in range(3):
                            for kw in range(3):
                                r, q = stride * i + kh - 1, stride * j + kw - 1
                                if 0 <= r < H and 0 <= q < W:
                                    acc += float(w[o, c, kh, kw]) * float(x[b, c, r, q])
                    y[b, o, i, j] = max(acc, 0.0) if relu else acc
    return y


def layers_forward(x, params, plan):
    """A stack of 3x3 convolutions, each followed by ReLU, as a chain of conv3x3_forward calls.
    plan: [(C_in, C_out, stride)]; params: one fp32 row [w_1 (O x C x 3 x 3 row-major) | b_1 | w_2 | b_2 ...].
    Every stored activation is rounded to fp32 (it is what the next layer reads).  Returns the list of
    activations [x, y_1, y_2, ...] as fp32 arrays."""
    acts = [np.asarray(x, dtype=np.float32)]
    off = 0
    for (cin, cout, stride) in plan:
        wsz = cout * cin * 9
        w = np.asarray(params[off: off + wsz]).reshape(cout, cin, 3, 3)
        b = np.asarray(params[off + wsz: off + wsz + cout])
        off += wsz + cout
        y, _ = conv3x3_forward(acts[-1], w, b, stride, relu=True)
        acts.append(y.astype(np.float32))
    assert off == len(params)
    return acts
