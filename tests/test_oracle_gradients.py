"""Pins for the oracle's per-node minibatch gradients (Algorithm 1, step 3, footnote a)."""
import numpy as np
import pytest
import torch

from oracle import dpsgd_oracle as orc


def _fd(loss, x, eps=1e-6):
    g = np.zeros_like(x, dtype=np.float64)
    for t in range(x.size):
        xp, xm = x.astype(np.float64).copy(), x.astype(np.float64).copy()
        xp[t] += eps
        xm[t] -= eps
        g[t] = (loss(xp) - loss(xm)) / (2 * eps)
    return g


def _data(rng, m, d):
    return rng.standard_normal((m, d)).astype(np.float32)


def test_lsq_gradient_matches_finite_differences():
    rng = np.random.default_rng(0)
    A, y = _data(rng, 20, 5), rng.standard_normal(20).astype(np.float32)
    x = rng.standard_normal(5).astype(np.float32)
    idx = np.array([3, 3, 7, 19, 0, 11], dtype=np.int32)      # repeats allowed
    g = orc.grad_lsq(x, A, y, idx)
    assert np.allclose(g, _fd(lambda v: orc.loss_lsq(v, A, y, idx), x), rtol=1e-7, atol=1e-8)


def test_lsq_gradient_single_sample_textbook():
    A = np.array([[1.0, 2.0, -1.0]], dtype=np.float32)
    y = np.array([0.5], dtype=np.float32)
    x = np.array([0.25, -0.5, 2.0], dtype=np.float32)
    r = (0.25 - 1.0 - 2.0) - 0.5
    assert np.allclose(orc.grad_lsq(x, A, y, np.array([0])), r * A[0].astype(np.float64))


def test_logistic_gradient_matches_finite_differences():
    rng = np.random.default_rng(1)
    A = _data(rng, 30, 6)
    y = np.where(rng.standard_normal(30) >= 0, 1.0, -1.0).astype(np.float32)
    x = (0.3 * rng.standard_normal(7)).astype(np.float32)
    idx = rng.integers(0, 30, 9).astype(np.int32)
    for lam in (0.0, 1e-4, 0.5):
        g = orc.grad_logistic(x, A, y, idx, lam)
        fd = _fd(lambda v: orc.loss_logistic(v, A, y, idx, lam), x)
        assert np.allclose(g, fd, rtol=1e-6, atol=1e-8)


def test_logistic_single_sample_reduces_to_textbook():
    """lambda = 0, B = 1: gradient = -y sigma(-y z) [a, 1]."""
    A = np.array([[0.5, -1.5, 2.0]], dtype=np.float32)
    x = np.array([0.1, 0.2, -0.3, 0.05], dtype=np.float32)
    for yv in (1.0, -1.0):
        y = np.array([yv], dtype=np.float32)
        z = float(A[0].astype(np.float64) @ x[:3].astype(np.float64) + np.float64(x[3]))
        sig = 1.0 / (1.0 + np.exp(yv * z))
        expect = -yv * sig * np.array([0.5, -1.5, 2.0, 1.0])
        assert np.allclose(orc.grad_logistic(x, A, y, np.array([0]), 0.0), expect, rtol=1e-12)


def test_logistic_penalty_skips_bias():
    rng = np.random.default_rng(2)
    A = _data(rng, 8, 4)
    y = np.ones(8, dtype=np.float32)
    x = rng.standard_normal(5).astype(np.float32)
    idx = np.arange(8)
    d = orc.grad_logistic(x, A, y, idx, 0.7) - orc.grad_logistic(x, A, y, idx, 0.0)
    assert np.allclose(d[:-1], 0.7 * x[:-1].astype(np.float64)) and d[-1] == 0.0


@pytest.mark.parametrize("dims", [(4, 6, 3), (5, 7, 6, 4)])
def test_mlp_gradient_matches_finite_differences(dims):
    rng = np.random.default_rng(3)
    N = sum(dims[l + 1] * dims[l] + dims[l + 1] for l in range(len(dims) - 1))
    A = _data(rng, 12, dims[0])
    labels = rng.integers(0, dims[-1], 12).astype(np.int32)
    x = (0.5 * rng.standard_normal(N)).astype(np.float32)
    idx = np.array([0, 5, 5, 11, 2], dtype=np.int32)
    g = orc.grad_mlp(x, dims, A, labels, idx)
    fd = _fd(lambda v: orc.loss_mlp(v, dims, A, labels, idx), x, eps=1e-6)
    assert np.allclose(g, fd, rtol=2e-6, atol=2e-8)


@pytest.mark.parametrize("dims", [(8, 16, 5), (6, 9, 8, 3)])
def test_mlp_gradient_matches_torch_autograd(dims):
    """Library pin: the same network built from torch.nn.functional ops in fp64."""
    rng = np.random.default_rng(4)
    N = sum(dims[l + 1] * dims[l] + dims[l + 1] for l in range(len(dims) - 1))
    A = _data(rng, 40, dims[0])
    labels = rng.integers(0, dims[-1], 40).astype(np.int32)
    x = (0.4 * rng.standard_normal(N)).astype(np.float32)
    idx = rng.integers(0, 40, 16).astype(np.int32)
    xt = torch.tensor(x, dtype=torch.float64, requires_grad=True)
    h = torch.tensor(A[idx], dtype=torch.float64)
    off = 0
    for l in range(len(dims) - 1):
        o, i = dims[l + 1], dims[l]
        Wl = xt[off: off + o * i].reshape(o, i); off += o * i
        bl = xt[off: off + o]; off += o
        h = torch.nn.functional.linear(h, Wl, bl)
        if l + 2 < len(dims):
            h = torch.relu(h)
    loss = torch.nn.functional.cross_entropy(h, torch.tensor(labels[idx], dtype=torch.long))
    loss.backward()
    assert abs(float(loss.detach()) - orc.loss_mlp(x, dims, A, labels, idx)) < 1e-12
    assert np.allclose(orc.grad_mlp(x, dims, A, labels, idx), xt.grad.numpy(), rtol=1e-10, atol=1e-13)


def test_gradients_use_each_nodes_own_row_and_data():
    """dF(X_k; xi_k): row i is the gradient at x_{k,i} on node i's data and indices."""
    rng = np.random.default_rng(5)
    n, m, d, B = 3, 10, 4, 6
    A = rng.standard_normal((n, m, d)).astype(np.float32)
    y = rng.standard_normal((n, m)).astype(np.float32)
    X = rng.standard_normal((n, d)).astype(np.float32)
    idx = rng.integers(0, m, (n, B)).astype(np.int32)
    G = orc.gradients(X, orc.MODEL_LSQ, (d,), A, y, idx)
    assert G.dtype == np.float32
    for i in range(n):
        assert np.array_equal(G[i], orc.grad_lsq(X[i], A[i], y[i], idx[i]).astype(np.float32))


def test_mlp_near_zero_gates_and_flip():
    """A unit whose pre-activation is exactly zero is reported; flipping its gate changes only
    what that unit back-propagates (ReLU'(0) = 0 by default, 1 when flipped)."""
    dims = (3, 2, 2)
    x = np.array([1.0, -1.0, 0.0, 0.5, 0.5, 0.5, 0.0, -1.5,      # W1 (2x3), b1
                  1.0, 2.0, -1.0, 0.5, 0.0, 0.0], dtype=np.float32)  # W2 (2x2), b2
    A = np.array([[1.0, 1.0, 7.0], [1.0, 2.0, 0.0]], dtype=np.float32)   # sample 0: z = (0, 3); sample 1: z = (-1, 0)
    labels = np.array([0, 1], dtype=np.int32)
    idx = np.array([0, 1])
    ties = orc.mlp_near_zero_gates(x, dims, A, idx, 1e-6)
    assert ties == [(0, 0, 0), (0, 1, 1)]
    assert orc.mlp_near_zero_gates(x, dims, A, np.array([0]), 1e-6) == [(0, 0, 0)]
    g0 = orc.grad_mlp(x, dims, A, labels, idx)
    g1 = orc.grad_mlp(x, dims, A, labels, idx, flip=[(0, 0, 0)])
    assert np.all(g0[0:3] == 0)          # row 0 of W1: sample 0 gated off (z = 0), sample 1 off (z < 0)
    assert np.any(g1[0:3] != 0)          # flipped: sample 0 now back-propagates through unit 0
    assert np.array_equal(g0[8:], g1[8:])  # the output layer's gradient does not depend on the gate
    assert np.array_equal(g0[3:6], g1[3:6])
