"""GPU parity for nodes of different speed (Section 5.3, last paragraph): per-node minibatch sizes
and local steps that only some nodes take."""
import numpy as np
import pytest
import torch

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import binding, workloads as wl
from gpu_util import GpuRun, row_rel_err, TOL_STEP

pytestmark = pytest.mark.gpu


def _attach(run, w, precision=0):
    run.ctx.set_model(w.model, w.dims, w.l2_lambda, w.batch, precision)
    run.A = w.A.cuda()
    run.y = w.y.cuda()
    run.ctx.set_data(run.A, run.y)


def _ragged_reference(w, X, idx, sizes):
    """Oracle gradients with node i averaging over its first sizes[i] draws."""
    return orc.gradients(X, w.model, w.dims, w.A.numpy(), w.y.numpy(),
                         [idx[i, :sizes[i]] for i in range(w.n)], w.l2_lambda)


@pytest.mark.parametrize("d", [52, 1028])     # narrow rows: two kernels; wide rows: the kernel that keeps them in registers
@pytest.mark.parametrize("model", [binding.MODEL_LSQ, binding.MODEL_LOGISTIC])
def test_per_node_minibatch_sizes_linear(model, d):
    n, m, B = 6, 96, 16
    sizes = [1, 16, 7, 8, 9, 3]
    w = (wl.lsq_workload(n=n, d=d, m=m, batch=B, seed=4) if model == binding.MODEL_LSQ
         else wl.logistic_workload(n=n, d=d, m=m, batch=B, l2_lambda=1e-3, seed=4))
    rng = np.random.default_rng(2)
    X = (0.3 * rng.standard_normal((n, w.N))).astype(np.float32)
    seed = 21
    run = GpuRun(n, w.N, w.csr(), w.gamma, seed=seed, X=X)
    _attach(run, w)
    run.ctx.set_node_batches(sizes)
    for k in (0, 3):
        idx = orc.sample_indices(seed, k, n, B, m)
        assert np.array_equal(run.ctx.sample(k).cpu().numpy(), idx)     # all B draws still reported
        run.ctx.current()[:, :w.N] = torch.from_numpy(X).cuda()
        run.ctx.grad(k)
        G_ref = _ragged_reference(w, X, idx, sizes)
        assert row_rel_err(run.g(), G_ref) <= 2e-5
        run.ctx.mix_update()
        assert row_rel_err(run.x(), orc.mix_update(X, G_ref, *w.csr(), w.gamma)) <= TOL_STEP
    # every size equal to B is the plain gradient, bit for bit; NULL restores it too
    run.ctx.current()[:, :w.N] = torch.from_numpy(X).cuda()
    run.ctx.set_node_batches([B] * n)
    run.ctx.grad(5)
    full = run.g().copy()
    run.ctx.set_node_batches(None)
    run.ctx.grad(5)
    assert np.array_equal(run.g(), full)
    assert row_rel_err(full, _ragged_reference(w, X, orc.sample_indices(seed, 5, n, B, m), [B] * n)) <= 2e-5
    run.check_pads()
    run.close()


@pytest.mark.parametrize("precision", [0, 2])
def test_per_node_minibatch_sizes_mlp(precision):
    n, dims, m, B = 4, (64, 96, 10), 80, 16
    sizes = [16, 1, 5, 12]
    w = wl.mlp_workload(n=n, dims=dims, m=m, batch=B, gamma=0.05, seed=13)
    rng = np.random.default_rng(5)
    X = (np.tile(w.x0.numpy(), (n, 1)) + 0.02 * rng.standard_normal((n, w.N))).astype(np.float32)
    seed = 9
    run = GpuRun(n, w.N, w.csr(), w.gamma, seed=seed, X=X)
    _attach(run, w, precision)
    run.ctx.set_node_batches(sizes)
    for k in (0, 4):
        idx = orc.sample_indices(seed, k, n, B, m)
        for i in range(n):       # no hidden unit sits on the ReLU kink, so the gradient is unique
            assert orc.mlp_near_zero_gates(X[i], dims, w.A.numpy()[i], idx[i, :sizes[i]], 4e-6) == []
        run.ctx.current()[:, :w.N] = torch.from_numpy(X).cuda()
        run.ctx.grad(k)
        G_ref = _ragged_reference(w, X, idx, sizes)
        assert row_rel_err(run.g(), G_ref) <= 5e-5
        run.ctx.mix_update()
        assert row_rel_err(run.x(), orc.mix_update(X, G_ref, *w.csr(), w.gamma)) <= TOL_STEP
    run.check_pads()
    run.close()


def test_node_batch_sizes_are_validated():
    w = wl.lsq_workload(n=4, d=8, m=16, batch=4, seed=1)
    run = GpuRun(w.n, w.N, w.csr(), w.gamma, seed=1, X=np.zeros((w.n, w.N), np.float32))
    with pytest.raises(binding.DpsgdError) as e:
        run.ctx.set_node_batches([1, 2, 3, 4])            # no model yet
    assert e.value.status == binding.ERR_STATE
    _attach(run, w)
    for bad in ([0, 1, 1, 1], [1, 1, 5, 1], [-3, 1, 1, 1]):
        with pytest.raises(binding.DpsgdError) as e:
            run.ctx.set_node_batches(bad)
        assert e.value.status == binding.ERR_ARG
    run.ctx.set_node_batches([4, 3, 2, 1])
    run.ctx.step(0)
    # a new model drops the sizes: they were checked against the old batch
    run.ctx.set_model(w.model, w.dims, 0.0, 2, 0)
    run.ctx.set_data(run.A, run.y)
    run.ctx.grad(1)
    idx = orc.sample_indices(1, 1, w.n, 2, 16)
    G_ref = orc.gradients(run.x(), w.model, w.dims, w.A.numpy(), w.y.numpy(), idx)
    assert row_rel_err(run.g(), G_ref) <= 2e-5
    run.close()


@pytest.mark.parametrize("beta", [0.0, 0.9])
def test_local_steps_of_some_nodes_only(beta):
    """Faster nodes run extra minibatches between exchanges; the others keep their row (and their
    momentum buffer) until the next gossip step."""
    w = wl.logistic_workload(n=6, d=40, m=64, batch=8, gamma=0.2, l2_lambda=1e-3, seed=33)
    A, y = w.A.numpy(), w.y.numpy()
    csr, ident = w.csr(), wl.identity(w.n)
    seed = 8
    rng = np.random.default_rng(0)
    X0 = (0.1 * rng.standard_normal((w.n, w.N))).astype(np.float32)
    run = GpuRun(w.n, w.N, csr, w.gamma, seed=seed, X=X0)
    _attach(run, w)
    V = torch.zeros_like(run.X0)
    if beta > 0.0:
        run.ctx.set_momentum(beta, V)
    o = orc.Oracle(w.n, w.N, *csr, w.gamma, seed, w.model, w.dims, w.batch, w.l2_lambda, A, y)
    o.set_x(X0)
    Vr = np.zeros_like(X0)
    fast = [[1, 0, 1, 0, 0, 1], [0, 0, 1, 0, 0, 0]]
    for k in range(12):
        G = o.grad(k)
        if k % 3 == 2:
            run.ctx.step(k)
            o.X, Vr = orc.mix_update_momentum(o.X, Vr, G, *csr, w.gamma, beta)
        else:
            active = np.array(fast[k % 3], dtype=bool)
            run.ctx.local_step_nodes(k, active)
            Xn, Vn = orc.mix_update_momentum(o.X, Vr, G, *ident, w.gamma, beta)
            o.X = np.where(active[:, None], Xn, o.X)
            Vr = np.where(active[:, None], Vn, Vr)
        assert row_rel_err(run.x(), o.X) <= 1e-5, k
    if beta > 0.0:
        assert row_rel_err(V[:, :w.N].cpu().numpy(), Vr) <= 1e-5
    if beta == 0.0:      # all nodes active is the plain local step, bit for bit
        a = run.x().copy()
        run.ctx.local_step_nodes(50, [1] * w.n)
        b = run.x().copy()
        run.ctx.current()[:, :w.N] = torch.from_numpy(a).cuda()
        run.ctx.local_step(50)
        assert np.array_equal(run.x(), b)
    run.check_pads()
    run.close()
