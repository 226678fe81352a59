"""GPU parity: the MLP iteration whose gossip step runs inside the weight-gradient kernels
(dpsgd_set_fused_step).  Algorithm 1 steps 3-5: X_next = W X - gamma dF(X; xi) (Section 3)."""
import numpy as np
import pytest
import torch

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import binding, workloads as wl
from gpu_util import GpuRun, row_rel_err, mlp_oracle_grad_matching_gates, TOL_STEP, TOL_TRAJ, TOL_AVG

pytestmark = pytest.mark.gpu


def _setup(w, seed, X, precision=0):
    A, y = w.A.numpy(), w.y.numpy()
    csr = w.csr()
    run = GpuRun(w.n, w.N, csr, w.gamma, seed=seed, X=X)
    run.ctx.set_model(w.model, w.dims, 0.0, w.batch, precision)
    run.A, run.y = torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda()
    run.ctx.set_data(run.A, run.y)
    o = orc.Oracle(w.n, w.N, *csr, w.gamma, seed, w.model, w.dims, w.batch, 0.0, A, y)
    o.set_x(X)
    return run, o


def _perturbed(w, seed):
    rng = np.random.default_rng(seed)
    return (np.tile(w.x0.numpy(), (w.n, 1)) + 0.02 * rng.standard_normal((w.n, w.N))).astype(np.float32)


FUSED_CASES = [
    (7, "ring", (260, 200, 10), 40, 12),              # ranges of several nodes per CTA, ragged tiles both ways
    # n, topology, dims, m, B
    (5, "ring", (784, 1024, 10), 64, 32),             # the 784-1024-10 network
    (4, "ring", (132, 200, 70, 10), 50, 16),          # widths that are no multiples of the 128 x 64 tiles
    (3, "ring", (1024, 2048, 2048, 10), 80, 64),      # the large network, three nodes
    (9, "torus", (64, 96, 80, 10), 40, 24),           # five entries per row of W
    (8, "ring+antipode", (256, 128, 20), 40, 8),      # four entries per row; a wide classifier layer
    (6, "dense", (128, 64, 10), 40, 8),               # six entries per row, taken from the CSR arrays
    (4, "ring", (20, 33, 7), 40, 5),                  # one small ragged block
    (4, "ring", (18, 33, 7), 40, 5),                  # rows of 18 floats: the fused kernel cannot take them, plain path
    (2, "ring", (64, 48, 12), 30, 4),                 # two nodes: coinciding neighbours summed in W
    (5, "ring", (64, 33, 36, 24, 10), 40, 8),         # third block starts at an odd column: left to the two stages
    (12, "dense", (128, 96, 10), 40, 8),              # W = 11^T/n with more entries per row than the kernels gather: column mean
]


@pytest.mark.parametrize("mode", [2, 3])      # 2: ring W on the kernel with the X window on chip; 3: the gathering kernel
@pytest.mark.parametrize("n,topology,dims,m,B", FUSED_CASES)
def test_fused_step_matches_oracle_and_two_stage_path(n, topology, dims, m, B, mode):
    if mode == 3 and topology != "ring":
        pytest.skip("same kernel as mode 2 for this W")
    w = wl.mlp_workload(n=n, dims=dims, m=m, batch=B, gamma=0.05, seed=21, topology=topology)
    X = _perturbed(w, 3)
    run, o = _setup(w, seed=5, X=X)
    for k in (0, 3):
        # reference: the oracle's step from X (ReLU ties resolved against the two-stage GPU gradient)
        o.set_x(X)
        run.ctx.current()[:, :w.N] = torch.from_numpy(X).cuda()
        run.ctx.set_fused_step(0)
        run.ctx.grad(k)
        G_ref, _ = mlp_oracle_grad_matching_gates(orc, o, k, run.g())
        X_ref = o.mix_update(G_ref)
        run.ctx.mix_update()
        X_two_stage = run.x().copy()
        # the fused iteration from the same X, with G poisoned: weight blocks must not be read from it
        run.ctx.current()[:, :w.N] = torch.from_numpy(X).cuda()
        run.G.fill_(float("nan"))
        run.ctx.set_fused_step(mode)
        run.ctx.step(k)
        got = run.x()
        assert np.isfinite(got).all()
        assert row_rel_err(got, X_ref) <= TOL_STEP
        assert row_rel_err(got, X_two_stage) <= 2e-6
        run.G.zero_()
        run.check_pads()
    run.close()


def test_fused_step_really_skips_the_gradient_blocks():
    """After a fused step the weight blocks of G are untouched, the bias blocks are written."""
    dims = (128, 256, 10)
    w = wl.mlp_workload(n=4, dims=dims, m=40, batch=16, gamma=0.05, seed=22)
    run, o = _setup(w, seed=1, X=_perturbed(w, 4))
    run.G.fill_(7.0)
    before = run.ctx.launch_count()
    run.ctx.set_fused_step(2)
    run.ctx.step(0)
    fused_launches = run.ctx.launch_count() - before
    g = run.g()
    w1 = dims[1] * dims[0]
    assert np.all(g[:, :w1] == 7.0)                       # hidden layer's weights: never written
    assert not np.any(g[:, w1:w1 + dims[1]] == 7.0)       # its biases: written, then mixed from G
    run.ctx.set_fused_step(0)
    before = run.ctx.launch_count()
    run.ctx.step(1)
    assert not np.any(run.g()[:, :w1] == 7.0)
    assert run.ctx.launch_count() - before == fused_launches      # the small mixing kernel replaces the large one
    run.close()


def test_fused_mode_one_leaves_small_blocks_to_the_two_stage_path():
    """Mode 1 fuses only where it is faster (blocks beyond L2): on a small network it is the plain iteration."""
    w = wl.mlp_workload(n=4, dims=(64, 96, 10), m=40, batch=8, gamma=0.05, seed=14)
    X = _perturbed(w, 6)
    outs = []
    for mode in (0, 1):
        run, _ = _setup(w, seed=2, X=X)
        run.G.fill_(7.0)
        run.ctx.set_fused_step(mode)
        run.ctx.step(0)
        assert not np.any(run.g()[:, :64 * 96] == 7.0)
        outs.append(run.x().copy())
        run.close()
    assert np.array_equal(outs[0], outs[1])
    run, _ = _setup(w, seed=2, X=X)
    with pytest.raises(binding.DpsgdError) as e:
        run.ctx.set_fused_step(4)
    assert e.value.status == binding.ERR_ARG
    run.close()


def test_fused_trajectory_matches_oracle():
    """784-1024-10 on a ring of 8 nodes, 40 free-running fused steps."""
    w = wl.mlp_workload(n=8, dims=(784, 1024, 10), m=256, batch=32, gamma=0.05, seed=5)
    X = np.tile(w.x0.numpy(), (w.n, 1))
    run, o = _setup(w, seed=9, X=X)
    run.ctx.set_fused_step(2)
    for k in range(40):
        run.ctx.step(k)
        o.step(k)
    got = run.x()
    assert row_rel_err(got, o.X) <= TOL_TRAJ
    avg_ref = orc.node_average(o.X)
    assert np.linalg.norm(got.astype(np.float64).mean(axis=0) - avg_ref) <= TOL_AVG * np.linalg.norm(avg_ref)
    c_ref = o.consensus_dist()
    assert abs(run.ctx.consensus_dist() - c_ref) <= 2e-2 * c_ref
    run.check_pads()
    run.close()


def test_fused_step_with_per_node_minibatch_sizes():
    n, dims, m, B = 4, (64, 96, 10), 80, 16
    sizes = [16, 1, 5, 12]
    w = wl.mlp_workload(n=n, dims=dims, m=m, batch=B, gamma=0.05, seed=13)
    X = _perturbed(w, 5)
    run, _ = _setup(w, seed=9, X=X)
    run.ctx.set_node_batches(sizes)
    idx = orc.sample_indices(9, 2, n, B, m)
    A, y = w.A.numpy(), w.y.numpy()
    G_ref = np.stack([orc.grad_mlp(X[i], dims, A[i], y[i], idx[i, :sizes[i]]) for i in range(n)]).astype(np.float32)
    for i in range(n):
        assert orc.mlp_near_zero_gates(X[i], dims, A[i], idx[i, :sizes[i]], 4e-6) == []
    run.ctx.set_fused_step(2)
    run.ctx.step(2)
    assert row_rel_err(run.x(), orc.mix_update(X, G_ref, *w.csr(), w.gamma)) <= TOL_STEP
    run.close()


@pytest.mark.parametrize("variant", ["swapped", "momentum", "fp32"])
def test_fused_request_falls_back_where_it_does_not_apply(variant):
    """Footnote c's order, momentum and the fp32 FMA kernels keep the two-stage iteration: asking for
    the fused one changes nothing there."""
    w = wl.mlp_workload(n=4, dims=(64, 96, 10), m=40, batch=8, gamma=0.05, seed=14)
    X = _perturbed(w, 6)
    outs = []
    for fused in (False, True):
        run, _ = _setup(w, seed=2, X=X, precision=2 if variant == "fp32" else 0)
        if variant == "swapped":
            run.ctx.set_order(True)
        if variant == "momentum":
            V = torch.zeros_like(run.X0)
            run.ctx.set_momentum(0.9, V)
        run.ctx.set_fused_step(2 if fused else 0)
        for k in range(3):
            run.ctx.step(k)
        outs.append(run.x().copy())
        run.close()
    assert np.array_equal(outs[0], outs[1])


def test_step_consensus_with_the_fused_iteration():
    """dpsgd_step_consensus in fused mode: the new X and its consensus distance (Theorem 4's
    sum_i ||xbar - x_i||^2) equal the two-stage iteration's."""
    w = wl.mlp_workload(n=6, dims=(128, 192, 10), m=60, batch=16, gamma=0.05, seed=31)
    X = _perturbed(w, 8)
    res = []
    for mode in (0, 2):
        run, o = _setup(w, seed=4, X=X)
        run.ctx.set_fused_step(mode)
        log = torch.zeros(3, dtype=torch.float64, device="cuda")
        for k in range(3):
            run.ctx.step_consensus(k, log[k:k + 1])
            if mode == 0:
                o.step(k)
        torch.cuda.synchronize()
        res.append((run.x().copy(), log.cpu().numpy()))
        if mode == 0:
            assert abs(res[0][1][2] - o.consensus_dist()) <= 1e-3 * o.consensus_dist()
        run.close()
    assert row_rel_err(res[1][0], res[0][0]) <= 1e-5
    assert np.all(np.abs(res[1][1] - res[0][1]) <= 1e-4 * res[0][1])
