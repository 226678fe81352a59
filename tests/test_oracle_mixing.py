"""Pins for the oracle's gossip step, consensus distance and whole iteration.

Each test checks the oracle against something the paper or the mathematics fixes:
Section 3 (definition of W, global form), Theorem 3 (ring), Assumption 1-2 and Lemma 5
(spectral contraction), the proof of Theorem 1 (average preservation), Eq. 10 / Eq. 13
(consensus quantity), Section 2 / Table 1 (centralized PSGD as minibatch SGD).
"""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(rng, *shape):
    return rng.standard_normal(shape).astype(np.float32)


# ---- topologies handed to both sides ------------------------------------------------------

def test_ring_builder_matches_theorem3_matrix():
    rows = []
    with open(os.path.join(GOLDEN, "ring_w_theorem3.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                rows.append([float(Fraction(t)) for t in line.split()])
    golden = np.array(rows)
    W = wl.csr_to_dense(6, *wl.ring(6))
    assert np.allclose(W, golden.astype(np.float32).astype(np.float64), rtol=0, atol=0)


@pytest.mark.parametrize("name,n", [("ring", 1), ("ring", 2), ("ring", 3), ("ring", 8), ("ring", 112),
                                    ("torus", 4), ("torus", 64), ("dense", 5), ("dense", 64),
                                    ("ring+antipode", 16)])
def test_topologies_are_symmetric_doubly_stochastic(name, n):
    rp, col, val = wl.topology(name, n)
    W = wl.csr_to_dense(n, rp, col, val)
    assert np.array_equal(W, W.T)
    assert np.all(W >= 0) and np.all(W <= 1)
    assert np.allclose(W.sum(axis=1), 1.0, atol=1e-6)
    for i in range(n):
        c = col[rp[i]:rp[i + 1]]
        assert np.all(np.diff(c) > 0)


def test_small_rings_sum_duplicates():
    assert np.allclose(wl.csr_to_dense(2, *wl.ring(2)), [[1 / 3, 2 / 3], [2 / 3, 1 / 3]], atol=1e-7)
    assert np.allclose(wl.csr_to_dense(3, *wl.ring(3)), np.full((3, 3), 1 / 3), atol=1e-7)
    assert np.allclose(wl.csr_to_dense(1, *wl.ring(1)), [[1.0]], atol=1e-7)


def test_torus_neighbours():
    W = wl.csr_to_dense(64, *wl.torus2d(8, 8))
    i = 3 * 8 + 7
    nz = set(np.nonzero(W[i])[0])
    assert nz == {i, 2 * 8 + 7, 4 * 8 + 7, 3 * 8 + 6, 3 * 8 + 0}
    assert np.allclose(W[i][list(nz)], 0.2, atol=1e-7)


# ---- spectral quantities ------------------------------------------------------------------

@pytest.mark.parametrize("n", [3, 8, 16, 32, 64, 112])
def test_rho_of_ring_matches_closed_form_spectrum(n):
    """A circulant ring with weights 1/3 has eigenvalues (1 + 2 cos(2 pi j / n)) / 3."""
    ev = (1 + 2 * np.cos(2 * np.pi * np.arange(n) / n)) / 3
    second = np.sort(np.abs(ev))[-2]
    W = wl.csr_to_dense(n, *wl.ring(n))
    assert abs(orc.spectral_rho(W) - second ** 2) < 1e-7


def test_rho_of_torus_and_dense():
    # 8x8 torus: eigenvalues (1 + 2cos a + 2cos b)/5; the largest non-principal one in
    # magnitude is (3 + 2 cos(pi/4))/5
    W = wl.csr_to_dense(64, *wl.torus2d(8, 8))
    assert abs(np.sqrt(orc.spectral_rho(W)) - (3 + 2 * np.cos(np.pi / 4)) / 5) < 1e-6
    assert orc.spectral_rho(wl.csr_to_dense(7, *wl.dense_uniform(7))) < 1e-12


# ---- mixing -------------------------------------------------------------------------------

@pytest.mark.parametrize("n,N,seed", [(2, 3, 0), (3, 7, 1), (4, 5, 2), (5, 7, 3), (5, 1, 4)])
def test_mix_update_equals_brute_force_dense_product(n, N, seed):
    rng = np.random.default_rng(seed)
    rp, col, val = wl.random_symmetric_doubly_stochastic(n, seed)
    W = wl.csr_to_dense(n, rp, col, val)
    X, G = _rand(rng, n, N), _rand(rng, n, N)
    gamma = np.float32(0.37)
    brute = np.zeros((n, N))
    for i in range(n):
        for c in range(N):
            s = 0.0
            for j in range(n):
                s += W[i, j] * float(X[j, c])
            brute[i, c] = s - float(gamma) * float(G[i, c])
    got = orc.mix_update(X, G, rp, col, val, gamma)
    assert got.dtype == np.float32
    assert np.array_equal(got, brute.astype(np.float32))
    # footnote c order: W (X - gamma G)
    swapped = (W @ (X.astype(np.float64) - float(gamma) * G.astype(np.float64)))
    got_s = orc.mix_update_swapped(X, G, rp, col, val, gamma)
    assert np.allclose(got_s, swapped, rtol=2e-7, atol=1e-7)
    assert not np.allclose(got_s, got, atol=1e-3)


def test_mix_update_identity_and_zero_step():
    rng = np.random.default_rng(5)
    n, N = 6, 9
    X, G = _rand(rng, n, N), _rand(rng, n, N)
    # W = I: plain SGD on every row, one rounding
    out = orc.mix_update(X, G, *wl.identity(n), 0.25)
    assert np.array_equal(out, (X.astype(np.float64) - 0.25 * G.astype(np.float64)).astype(np.float32))
    # gamma = 0: pure mixing, independent of G
    rp, col, val = wl.ring(n)
    a = orc.mix_update(X, G, rp, col, val, 0.0)
    b = orc.mix_update(X, 0 * G, rp, col, val, 0.0)
    assert np.array_equal(a, b)
    third = np.float64(np.float32(1.0) / np.float32(3.0))
    assert np.allclose(a[2], third * (X[1].astype(np.float64) + X[2] + X[3]), rtol=1e-7)
    assert np.allclose(a[0], third * (X[5].astype(np.float64) + X[0] + X[1]), rtol=1e-7)


@pytest.mark.parametrize("name,n", [("ring", 8), ("torus", 16), ("dense", 6), ("ring+antipode", 8)])
def test_mixing_preserves_the_node_average(name, n):
    """X_k W 1/n = X_k 1/n (proof of Theorem 1): with gradients the average moves by
    -gamma * mean gradient only."""
    rng = np.random.default_rng(6)
    rp, col, val = wl.topology(name, n)
    X, G = _rand(rng, n, 33), _rand(rng, n, 33)
    gamma = 0.1
    out = orc.mix_update(X, G, rp, col, val, gamma)
    expect = orc.node_average(X) - np.float64(np.float32(gamma)) * orc.node_average(G)
    assert np.allclose(orc.node_average(out), expect, atol=n * 2.0 ** -23)


@pytest.mark.parametrize("name,n", [("ring", 8), ("ring", 16), ("torus", 16), ("ring+antipode", 12)])
def test_zero_gradient_contracts_by_sqrt_rho(name, n):
    """Assumption 1-2 / Lemma 5: ||X_{k+1} - 1 xbar^T||_F <= sqrt(rho) ||X_k - 1 xbar^T||_F."""
    rng = np.random.default_rng(7)
    rp, col, val = wl.topology(name, n)
    sqrt_rho = np.sqrt(orc.spectral_rho(wl.csr_to_dense(n, rp, col, val)))
    assert sqrt_rho < 1
    X = _rand(rng, n, 50)
    Z = np.zeros_like(X)
    d = np.sqrt(orc.consensus_dist(X))
    for _ in range(25):
        X = orc.mix_update(X, Z, rp, col, val, 0.3)
        d_new = np.sqrt(orc.consensus_dist(X))
        assert d_new <= sqrt_rho * d * (1 + 1e-5) + 1e-6
        d = d_new


def test_worst_case_contraction_is_attained_on_the_ring():
    """Start on the eigenvector of lambda_2: the distance shrinks by exactly sqrt(rho)."""
    n = 16
    rp, col, val = wl.ring(n)
    lam2 = (1 + 2 * np.cos(2 * np.pi / n)) / 3
    v = np.cos(2 * np.pi * np.arange(n) / n)
    X = np.outer(v, np.ones(4)).astype(np.float32)
    d0 = np.sqrt(orc.consensus_dist(X))
    X1 = orc.mix_update(X, np.zeros_like(X), rp, col, val, 1.0)
    assert abs(np.sqrt(orc.consensus_dist(X1)) / d0 - lam2) < 1e-6


def test_dense_w_zero_gradient_reaches_consensus_in_one_step():
    rng = np.random.default_rng(8)
    n = 8
    X = _rand(rng, n, 21)
    out = orc.mix_update(X, np.zeros_like(X), *wl.dense_uniform(n), 0.5)
    assert orc.consensus_dist(out) < 1e-12
    assert np.allclose(out[3], orc.node_average(X), atol=1e-6)


# ---- consensus distance -------------------------------------------------------------------

def test_consensus_distance_identities():
    rng = np.random.default_rng(9)
    n, N = 7, 13
    X = _rand(rng, n, N)
    xbar = X.astype(np.float64).sum(axis=0) / n
    alt = float(np.sum(X.astype(np.float64) ** 2) - n * np.sum(xbar ** 2))   # ||X||_F^2 - n||xbar||^2
    assert abs(orc.consensus_dist(X) - alt) < 1e-9
    per_node = [float(np.sum((xbar - X[i]) ** 2)) for i in range(n)]          # Q_{k,i}, Eq. 10
    assert abs(orc.consensus_dist(X) - sum(per_node)) < 1e-10
    same = np.tile(X[0], (n, 1))
    assert orc.consensus_dist(same) == 0.0                                    # x_{0,i} = x_0
    Y = np.zeros((2, 1), dtype=np.float32)
    Y[0, 0], Y[1, 0] = 1.0, -1.0
    assert orc.consensus_dist(Y) == 2.0


# ---- whole iteration ----------------------------------------------------------------------

def _full_batch_lsq(n=4, m=12, d=5, seed=10):
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((n, m, d)).astype(np.float32)
    y = rng.standard_normal((n, m)).astype(np.float32)
    return A, y


def test_least_squares_dense_swapped_follows_gradient_descent_closed_form():
    """Full local batches, W = 11^T/n, footnote-c order: every row is gradient descent on the
    quadratic f, so x_k = (I - (I - gamma H)^k) x*, H = mean a a^T, x* = H^{-1} mean(y a)."""
    n, m, d = 4, 12, 5
    A, y = _full_batch_lsq(n, m, d)
    A64, y64 = A.astype(np.float64).reshape(-1, d), y.astype(np.float64).reshape(-1)
    H = A64.T @ A64 / (n * m)
    x_star = np.linalg.solve(H, A64.T @ y64 / (n * m))
    gamma = np.float32(0.2)
    rp, col, val = wl.dense_uniform(n)
    X = np.zeros((n, d), dtype=np.float32)
    full = np.tile(np.arange(m, dtype=np.int32), (n, 1))
    K = 40
    for _ in range(K):
        G = orc.gradients(X, orc.MODEL_LSQ, (d,), A, y, full)
        X = orc.mix_update_swapped(X, G, rp, col, val, gamma)
    Mk = np.linalg.matrix_power(np.eye(d) - float(gamma) * H, K)
    expect = (np.eye(d) - Mk) @ x_star
    for i in range(n):
        assert np.allclose(X[i], expect, rtol=0, atol=5e-6)
    # and it converges to the least-squares solution
    for _ in range(400):
        G = orc.gradients(X, orc.MODEL_LSQ, (d,), A, y, full)
        X = orc.mix_update_swapped(X, G, rp, col, val, gamma)
    assert np.allclose(X[0], x_star, atol=1e-5)


def test_ring_least_squares_average_follows_the_closed_form_too():
    """With full batches and a quadratic objective, sum_i grad f_i(x_i) is linear in X, but the
    local Hessians differ, so only the *fixed point* is checked on the ring: the average
    reaches the neighbourhood of x* (the consensus error is O(gamma))."""
    n, m, d = 6, 40, 4
    A, y = _full_batch_lsq(n, m, d, seed=12)
    A64, y64 = A.astype(np.float64).reshape(-1, d), y.astype(np.float64).reshape(-1)
    x_star = np.linalg.lstsq(A64, y64, rcond=None)[0]
    rp, col, val = wl.ring(n)
    X = np.zeros((n, d), dtype=np.float32)
    full = np.tile(np.arange(m, dtype=np.int32), (n, 1))
    for _ in range(3000):
        X = orc.mix_update(X, orc.gradients(X, orc.MODEL_LSQ, (d,), A, y, full), rp, col, val, 0.01)
    assert np.linalg.norm(orc.node_average(X) - x_star) < 0.02 * max(1.0, np.linalg.norm(x_star))


def test_config1_stochastic_run_converges_to_planted_solution():
    """n = 8 ring, 64 parameters, minibatch 16, gamma 0.05, 200 iterations from zero:
    the node average lands near w* (noise 0.1, transient (1-gamma)^200 ~ 3.5e-5)."""
    w = wl.config(0)
    A, y = w.A.numpy(), w.y.numpy()
    rp, col, val = w.csr()
    o = orc.Oracle(w.n, w.N, rp, col, val, w.gamma, seed=1234, model=orc.MODEL_LSQ, dims=w.dims,
                   batch=w.batch, A=A, y=y)
    d0 = np.linalg.norm(w.extra["w_star"].numpy())
    for k in range(w.iterations):
        o.step(k)
    err = np.linalg.norm(orc.node_average(o.X) - w.extra["w_star"].numpy().astype(np.float64))
    assert err < 0.08 * d0
    assert o.consensus_dist() < 0.5


def _logistic_setup(n=5, m=30, d=6, B=4, seed=13):
    rng = np.random.default_rng(seed)
    A = rng.standard_normal((n, m, d)).astype(np.float32)
    y = np.where(rng.standard_normal((n, m)) >= 0, 1.0, -1.0).astype(np.float32)
    return A, y


def test_dense_w_swapped_order_is_centralized_minibatch_sgd():
    """Footnote c with W = 11^T/n: every row equals the C-PSGD iterate, every step."""
    n, m, d, B = 5, 30, 6, 4
    A, y = _logistic_setup(n, m, d, B)
    rp, col, val = wl.dense_uniform(n)
    seed, gamma, lam = 99, 0.3, 1e-2
    o = orc.Oracle(n, d + 1, rp, col, val, gamma, seed, orc.MODEL_LOGISTIC, (d,), B, lam, A, y,
                   swapped=True)
    x = np.zeros(d + 1, dtype=np.float32)
    for k in range(30):
        idx = orc.sample_indices(seed, k, n, B, m)
        grads = [orc.grad_logistic(x, A[i], y[i], idx[i], lam).astype(np.float32) for i in range(n)]
        x = orc.cpsgd_step(x, grads, gamma)
        o.step(k)
        for i in range(n):
            assert np.allclose(o.X[i], x, rtol=0, atol=3e-6)
        assert o.consensus_dist() < 1e-10


def test_dense_w_default_order_average_and_consensus_closed_forms():
    """Algorithm 1 order with W = 11^T/n: xbar_{k+1} = xbar_k - gamma mean_i g_i(x_{k,i}) and
    sum_i ||x_{k+1,i} - xbar_{k+1}||^2 = gamma^2 sum_i ||g_i - gbar||^2; the first step from
    a shared x_0 is exactly one C-PSGD step on the average."""
    n, m, d, B = 5, 30, 6, 4
    A, y = _logistic_setup(n, m, d, B, seed=14)
    rp, col, val = wl.dense_uniform(n)
    seed, gamma, lam = 7, 0.3, 0.0
    o = orc.Oracle(n, d + 1, rp, col, val, gamma, seed, orc.MODEL_LOGISTIC, (d,), B, lam, A, y)
    x0 = np.zeros(d + 1, dtype=np.float32)
    for k in range(10):
        xbar = orc.node_average(o.X)
        G = o.grad(k)
        if k == 0:
            c1 = orc.cpsgd_step(x0, G, gamma)
        o.mix_update(G)
        g64 = G.astype(np.float64)
        gam = np.float64(np.float32(gamma))
        assert np.allclose(orc.node_average(o.X), xbar - gam * g64.mean(axis=0), atol=2e-7)
        expect_c = gam ** 2 * np.sum((g64 - g64.mean(axis=0)) ** 2)
        assert abs(o.consensus_dist() - expect_c) <= 1e-5 * expect_c + 1e-12
        if k == 0:
            assert np.allclose(orc.node_average(o.X), c1, atol=2e-7)


def test_oracle_step_is_grad_then_mix_with_pre_mix_gradient():
    """The gradient in the update is taken at x_{k,i}, not at the mixed point."""
    n, m, d, B = 4, 16, 3, 2
    rng = np.random.default_rng(15)
    A = rng.standard_normal((n, m, d)).astype(np.float32)
    y = rng.standard_normal((n, m)).astype(np.float32)
    rp, col, val = wl.ring(n)
    o = orc.Oracle(n, d, rp, col, val, 0.1, 5, orc.MODEL_LSQ, (d,), B, 0.0, A, y)
    o.set_x(rng.standard_normal((n, d)))
    X0 = o.X.copy()
    idx = orc.sample_indices(5, 3, n, B, m)
    G = orc.gradients(X0, orc.MODEL_LSQ, (d,), A, y, idx)
    expect = orc.mix_update(X0, G, rp, col, val, 0.1)
    assert np.array_equal(o.step(3), expect)


# ---- momentum (Section 5.3: learning rate 0.1, momentum 0.9) ---------------------------------

def test_momentum_zero_beta_is_the_plain_step():
    rng = np.random.default_rng(20)
    n, N = 6, 11
    rp, col, val = wl.ring(n)
    X, V, G = _rand(rng, n, N), _rand(rng, n, N), _rand(rng, n, N)
    Xn, Vn = orc.mix_update_momentum(X, V, G, rp, col, val, 0.2, 0.0)
    assert np.array_equal(Vn, G)
    assert np.array_equal(Xn, orc.mix_update(X, G, rp, col, val, 0.2))


def test_momentum_constant_gradient_closed_form():
    """W = I and a constant gradient g: v_k = g (1 - beta^k)/(1 - beta) and
    x_k = x_0 - gamma g (k - beta (1 - beta^k)/(1 - beta)) / (1 - beta)."""
    n, N, K = 3, 5, 30
    rng = np.random.default_rng(21)
    X0, g = _rand(rng, n, N), _rand(rng, n, N)
    beta, gamma = 0.5, 0.25            # exact in fp32
    X, V = X0.copy(), np.zeros_like(X0)
    for _ in range(K):
        X, V = orc.mix_update_momentum(X, V, g, *wl.identity(n), gamma, beta)
    g64 = g.astype(np.float64)
    v_K = g64 * (1 - beta ** K) / (1 - beta)
    x_K = X0 - gamma * g64 * (K - beta * (1 - beta ** K) / (1 - beta)) / (1 - beta)
    assert np.allclose(V, v_K, rtol=1e-6)
    assert np.allclose(X, x_K, rtol=0, atol=2e-5)


def test_momentum_matches_brute_force_and_both_orders():
    rng = np.random.default_rng(22)
    n, N = 4, 6
    rp, col, val = wl.random_symmetric_doubly_stochastic(n, 5)
    W = wl.csr_to_dense(n, rp, col, val)
    X, V, G = _rand(rng, n, N), _rand(rng, n, N), _rand(rng, n, N)
    gamma, beta = np.float32(0.1), np.float32(0.9)
    Vb = float(beta) * V.astype(np.float64) + G
    Xn, Vn = orc.mix_update_momentum(X, V, G, rp, col, val, gamma, beta)
    assert np.allclose(Vn, Vb, rtol=1e-7)
    assert np.allclose(Xn, W @ X.astype(np.float64) - float(gamma) * Vn.astype(np.float64), rtol=1e-6, atol=1e-7)
    Xs, _ = orc.mix_update_momentum(X, V, G, rp, col, val, gamma, beta, swapped=True)
    assert np.allclose(Xs, W @ (X.astype(np.float64) - float(gamma) * Vn.astype(np.float64)), rtol=1e-6, atol=1e-7)
