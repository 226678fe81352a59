"""GPU parity: Philox minibatch sampler (bit-exact) and the linear-model gradients / whole steps."""
import numpy as np
import pytest
import torch

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import binding, workloads as wl
from gpu_util import GpuRun, row_rel_err, TOL_STEP, TOL_TRAJ, TOL_AVG

pytestmark = pytest.mark.gpu


def _attach(run, w, A, y, precision=0):
    run.ctx.set_model(w.model, w.dims, w.l2_lambda, w.batch, precision)
    run.A = torch.from_numpy(A).cuda()
    run.y = torch.from_numpy(y).cuda()
    run.ctx.set_data(run.A, run.y)


@pytest.mark.parametrize("n,B,m", [(8, 16, 1024), (16, 128, 65536), (32, 32, 1875), (112, 64, 4096),
                                   (3, 1, 1), (5, 7, 2 ** 31 - 1), (2, 4096, 77)])
def test_sampled_indices_are_bit_exact(n, B, m):
    seed = 0x9E3779B97F4A7C15
    ctx = binding.Dpsgd(n, 4, *wl.ring(n), gamma=0.1, seed=seed)
    ctx.set_model(binding.MODEL_LSQ, [4], 0.0, B)
    # only m matters to the sampler; a one-element stand-in keeps the test small
    A = torch.zeros((n, 1, 4), device="cuda")
    y = torch.zeros((n, 1), device="cuda")
    ctx._check(ctx._lib.dpsgd_set_data(ctx._h, A.data_ptr(), y.data_ptr(), m, 4))
    ctx._data_keep = [A, y]
    for k in (0, 1, 2, 999, 2 ** 32 - 1, 2 ** 32, (7 << 32) | 5, 2 ** 64 - 1):
        got = ctx.sample(k).cpu().numpy()
        assert np.array_equal(got, orc.sample_indices(seed, k, n, B, m)), k
    ctx.close()


def test_sampled_indices_bit_exact_over_a_whole_run_of_config1():
    w = wl.config(0)
    seed = 20170525
    ctx = binding.Dpsgd(w.n, w.N, *w.csr(), gamma=w.gamma, seed=seed)
    ctx.set_model(w.model, w.dims, 0.0, w.batch)
    A, y = w.A.cuda(), w.y.cuda()
    ctx.set_data(A, y)
    for k in range(w.iterations):
        assert np.array_equal(ctx.sample(k).cpu().numpy(),
                              orc.sample_indices(seed, k, w.n, w.batch, w.m_per_node))
    ctx.close()


LIN_CASES = [
    # model, n, d, m, B
    (binding.MODEL_LSQ, 8, 64, 1024, 16),          # config 1
    (binding.MODEL_LSQ, 3, 37, 50, 5),             # ragged d (scalar path)
    (binding.MODEL_LSQ, 2, 1, 9, 3),
    (binding.MODEL_LSQ, 5, 300, 200, 33),
    (binding.MODEL_LOGISTIC, 16, 4096, 512, 128),  # config 2 with a shortened local dataset
    (binding.MODEL_LOGISTIC, 4, 130, 64, 7),       # ragged d
    (binding.MODEL_LOGISTIC, 6, 260, 300, 128),
    (binding.MODEL_LOGISTIC, 1, 8, 10, 1),
    # rows of 4 KB and more stay in registers between the forward and the backward part
    (binding.MODEL_LSQ, 3, 1024, 40, 6),           # N == ld: no column beyond the parameters
    (binding.MODEL_LOGISTIC, 3, 2052, 50, 9),      # ragged against the 256 x 16-byte columns and the groups of four draws
    (binding.MODEL_LSQ, 2, 4096, 20, 1),
]


def _linear_workload(model, n, d, m, B, seed=0):
    if model == binding.MODEL_LSQ:
        return wl.lsq_workload(n=n, d=d, m=m, batch=B, seed=seed + 1)
    return wl.logistic_workload(n=n, d=d, m=m, batch=B, seed=seed + 2)


@pytest.mark.parametrize("model,n,d,m,B", LIN_CASES)
def test_linear_gradients_and_step_match_oracle(model, n, d, m, B):
    w = _linear_workload(model, n, d, m, B)
    A, y = w.A.numpy(), w.y.numpy()
    rng = np.random.default_rng(d)
    X = (0.3 * rng.standard_normal((n, w.N))).astype(np.float32)
    csr = w.csr()
    seed = 77
    run = GpuRun(n, w.N, csr, w.gamma, seed=seed, X=X)
    _attach(run, w, A, y)
    o = orc.Oracle(n, w.N, *csr, w.gamma, seed, w.model, w.dims, B, w.l2_lambda, A, y)
    for k in (0, 5):
        o.set_x(X)
        run.ctx.current()[:, :w.N] = torch.from_numpy(X).cuda()
        G_ref = o.grad(k)
        run.ctx.grad(k)
        assert row_rel_err(run.g(), G_ref) <= 2e-5
        assert float(run.G[:, w.N:].abs().max() if run.ld > w.N else 0.0) == 0.0
        X_ref = o.mix_update(G_ref)
        run.ctx.mix_update()
        assert row_rel_err(run.x(), X_ref) <= TOL_STEP
        run.check_pads()
    # dpsgd_step = grad + mix_update
    o.set_x(X)
    run.ctx.current()[:, :w.N] = torch.from_numpy(X).cuda()
    run.ctx.step(9)
    assert row_rel_err(run.x(), o.step(9)) <= TOL_STEP
    run.close()


@pytest.mark.parametrize("cfg,T", [(0, 200), (1, 60)])
def test_linear_trajectories(cfg, T):
    """Free-running trajectories of configs 1 and 2 (config 2 with 2048 local samples)."""
    w = wl.config(cfg) if cfg == 0 else wl.config(cfg, m=2048)
    A, y = w.A.numpy(), w.y.numpy()
    csr = w.csr()
    seed = 1234
    X0 = np.tile(w.x0.numpy(), (w.n, 1))
    run = GpuRun(w.n, w.N, csr, w.gamma, seed=seed, X=X0)
    _attach(run, w, A, y)
    o = orc.Oracle(w.n, w.N, *csr, w.gamma, seed, w.model, w.dims, w.batch, w.l2_lambda, A, y)
    o.set_x(X0)
    for k in range(T):
        run.ctx.step(k)
        o.step(k)
    got = run.x()
    assert row_rel_err(got, o.X) <= TOL_TRAJ
    avg_ref = orc.node_average(o.X)
    assert np.linalg.norm(got.astype(np.float64).mean(axis=0) - avg_ref) <= TOL_AVG * np.linalg.norm(avg_ref)
    c_ref = o.consensus_dist()
    assert abs(run.ctx.consensus_dist() - c_ref) <= 1e-2 * c_ref + 1e-12
    run.check_pads()
    run.close()


def test_gradient_calls_need_model_and_data():
    n = 4
    run = GpuRun(n, 8, wl.ring(n), 0.1)
    with pytest.raises(binding.DpsgdError) as e:
        run.ctx.grad(0)
    assert e.value.status == binding.ERR_STATE
    with pytest.raises(binding.DpsgdError) as e:
        run.ctx.set_model(binding.MODEL_LSQ, [9], 0.0, 4)      # N mismatch
    assert e.value.status == binding.ERR_ARG
    run.ctx.set_model(binding.MODEL_LSQ, [8], 0.0, 4)
    with pytest.raises(binding.DpsgdError) as e:
        run.ctx.step(0)
    assert e.value.status == binding.ERR_STATE
    run.close()


def test_checkpoint_resume_is_bit_identical():
    """The sampler is a pure function of (seed, k, node, draw): 40 steps equal 20 + restart + 20."""
    w = wl.lsq_workload(n=6, d=32, m=128, batch=8)
    A, y = w.A.numpy(), w.y.numpy()
    csr = w.csr()
    X0 = np.zeros((w.n, w.N), dtype=np.float32)
    a = GpuRun(w.n, w.N, csr, w.gamma, seed=5, X=X0)
    _attach(a, w, A, y)
    for k in range(40):
        a.ctx.step(k)
    b = GpuRun(w.n, w.N, csr, w.gamma, seed=5, X=X0)
    _attach(b, w, A, y)
    for k in range(20):
        b.ctx.step(k)
    saved = b.x()
    b.close()
    c = GpuRun(w.n, w.N, csr, w.gamma, seed=5, X=saved)
    _attach(c, w, A, y)
    for k in range(20, 40):
        c.ctx.step(k)
    assert np.array_equal(a.x(), c.x())
    a.close(); c.close()


def test_local_steps_between_exchanges_match_oracle():
    """tau = 3: two iterations without communication (the gossip step with W = I), then one with the
    ring, repeated; every step uses its own k for the sampler."""
    w = wl.logistic_workload(n=6, d=40, m=64, batch=8, gamma=0.2, l2_lambda=1e-3, seed=33)
    A, y = w.A.numpy(), w.y.numpy()
    csr = w.csr()
    seed = 8
    run = GpuRun(w.n, w.N, csr, w.gamma, seed=seed, X=np.zeros((w.n, w.N), np.float32))
    _attach(run, w, A, y)
    o = orc.Oracle(w.n, w.N, *csr, w.gamma, seed, w.model, w.dims, w.batch, w.l2_lambda, A, y)
    ident = wl.identity(w.n)
    for k in range(18):
        G = o.grad(k)
        if k % 3 == 2:
            run.ctx.step(k)
            o.mix_update(G)
        else:
            run.ctx.local_step(k)
            o.X = orc.mix_update(o.X, G, *ident, w.gamma)
    assert row_rel_err(run.x(), o.X) <= 1e-5
    run.check_pads()
    run.close()


def test_run_equals_repeated_steps():
    w = wl.lsq_workload(n=6, d=32, m=128, batch=8)
    A, y = w.A.numpy(), w.y.numpy()
    X0 = np.zeros((w.n, w.N), dtype=np.float32)
    a = GpuRun(w.n, w.N, w.csr(), w.gamma, seed=5, X=X0)
    _attach(a, w, A, y)
    for k in range(3, 63):
        a.ctx.step(k)
    b = GpuRun(w.n, w.N, w.csr(), w.gamma, seed=5, X=X0)
    _attach(b, w, A, y)
    b.ctx.run(3, 60)
    assert np.array_equal(a.x(), b.x())
    a.close(); b.close()


@pytest.mark.parametrize("model", [binding.MODEL_LSQ, binding.MODEL_LOGISTIC])
def test_graph_replayed_run_is_bit_identical_to_steps(model):
    """dpsgd_run replays a captured chain of 16 iterations for small problems (runs of at least 32); short
    and odd counts, several calls in a row and a change of gamma in between must all equal plain stepping."""
    w = _linear_workload(model, 8, 64, 256, 16)
    A, y = w.A.numpy(), w.y.numpy()
    X0 = np.zeros((w.n, w.N), dtype=np.float32)
    a = GpuRun(w.n, w.N, w.csr(), w.gamma, seed=5, X=X0)
    _attach(a, w, A, y)
    b = GpuRun(w.n, w.N, w.csr(), w.gamma, seed=5, X=X0)
    _attach(b, w, A, y)
    k = 0
    for count, gamma in ((9, w.gamma), (40, w.gamma), (3, w.gamma), (71, 0.5 * w.gamma), (33, 0.5 * w.gamma),
                         (32, w.gamma)):
        a.ctx.set_gamma(gamma); b.ctx.set_gamma(gamma)
        for t in range(count):
            a.ctx.step(k + t)
        b.ctx.run(k, count)
        k += count
        assert np.array_equal(a.x(), b.x()), (count, gamma)
    o = orc.Oracle(w.n, w.N, *w.csr(), w.gamma, 5, w.model, w.dims, w.batch, w.l2_lambda, A, y)
    for t in range(53):
        o.step(t)
    c = GpuRun(w.n, w.N, w.csr(), w.gamma, seed=5, X=X0)
    _attach(c, w, A, y)
    c.ctx.run(0, 53)
    assert row_rel_err(c.x(), o.X) <= TOL_TRAJ
    a.close(); b.close(); c.close()


@pytest.mark.parametrize("model,n,d,m,B,batches", [
    (binding.MODEL_LSQ, 8, 64, 1024, 16, None),           # config 1
    (binding.MODEL_LOGISTIC, 6, 260, 300, 24, None),      # rows of more than one 32-lane pass, bias column
    (binding.MODEL_LSQ, 5, 300, 200, 27, None),           # minibatch not a multiple of the eight slices
    (binding.MODEL_LOGISTIC, 4, 128, 64, 16, [16, 1, 9, 4]),   # per-node minibatch sizes
    (binding.MODEL_LSQ, 3, 4, 20, 3, None),
])
def test_one_launch_step_is_bit_identical_to_the_three_launches(model, n, d, m, B, batches):
    """Small linear models: dpsgd_step runs sample, gradient and gossip step as ONE kernel (a CTA per
    node).  X, G and the indices must equal those of the separate launches bit for bit, and the step takes
    one launch."""
    w = _linear_workload(model, n, d, m, B)
    A, y = w.A.numpy(), w.y.numpy()
    rng = np.random.default_rng(d)
    X = (0.3 * rng.standard_normal((n, w.N))).astype(np.float32)
    runs = []
    for mode in (0, 1):
        run = GpuRun(n, w.N, w.csr(), w.gamma, seed=11, X=X)
        _attach(run, w, A, y)
        if batches:
            run.ctx.set_node_batches(batches)
        run.ctx.set_fused_step(mode)
        runs.append(run)
    for k in range(5):
        before = [r.ctx.launch_count() for r in runs]
        for r in runs:
            r.G.fill_(7.0)
            r.ctx.step(k)
        assert runs[0].ctx.launch_count() - before[0] == 3
        assert runs[1].ctx.launch_count() - before[1] == 1
        assert np.array_equal(runs[0].g(), runs[1].g()), k
        assert np.array_equal(runs[0].x(), runs[1].x()), k
        assert torch.equal(runs[0].G, runs[1].G)                      # padding columns too
    o = orc.Oracle(n, w.N, *w.csr(), w.gamma, 11, w.model, w.dims, B, w.l2_lambda, A, y)
    if not batches:
        o.set_x(X)
        for k in range(5):
            o.step(k)
        assert row_rel_err(runs[1].x(), o.X) <= 5 * TOL_STEP
    for r in runs:
        r.check_pads()
        r.close()
