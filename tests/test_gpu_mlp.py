"""GPU parity: MLP minibatch gradients (ReLU, softmax cross-entropy) and whole D-PSGD steps."""
import numpy as np
import pytest
import torch

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import binding, workloads as wl
from gpu_util import GpuRun, row_rel_err, mlp_oracle_grad_matching_gates, TOL_STEP, TOL_TRAJ, TOL_AVG

pytestmark = pytest.mark.gpu

# row-wise relative error of the gradient against the fp64 oracle, by arithmetic of the products:
# tensor cores (three TF32 MMAs on split operands, ~2^-20 per product) and exact fp32 FMA
TOL_G = {0: 5e-5, 2: 2e-5}


def _setup(w, seed, precision=0, X=None):
    A, y = w.A.numpy(), w.y.numpy()
    csr = w.csr()
    if X is None:
        X = np.tile(w.x0.numpy(), (w.n, 1))
    run = GpuRun(w.n, w.N, csr, w.gamma, seed=seed, X=X)
    run.ctx.set_model(w.model, w.dims, 0.0, w.batch, precision)
    run.A, run.y = torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda()
    run.ctx.set_data(run.A, run.y)
    o = orc.Oracle(w.n, w.N, *csr, w.gamma, seed, w.model, w.dims, w.batch, 0.0, A, y)
    o.set_x(X)
    return run, o


MLP_CASES = [
    # n, dims, m, B
    (3, (20, 33, 7), 40, 5),                 # ragged everything
    (4, (784, 1024, 10), 64, 32),            # the 784-1024-10 network, few nodes
    (2, (64, 96, 80, 10), 50, 16),           # three weight layers
    (5, (16, 10), 30, 8),                    # a single layer (softmax regression)
    (2, (1024, 2048, 2048, 10), 96, 64),     # the large network, two nodes
    (3, (130, 70, 3), 33, 1),                # minibatch of one
    (2, (128, 256, 128, 64, 10), 40, 24),    # four weight layers
    # more row blocks than persistent CTAs: the blocks left over after the full rounds are cut by k-blocks
    (80, (40, 512, 256, 10), 24, 8),         # fewer left-over k-blocks than CTAs (some CTAs get none)
    (100, (96, 640, 10), 24, 8),             # ranges of two k-blocks that cross row blocks of three
]


@pytest.mark.parametrize("precision", [0, 2])     # tensor cores (3 x TF32) and the fp32 FMA kernel
@pytest.mark.parametrize("n,dims,m,B", MLP_CASES)
def test_mlp_gradient_and_step_match_oracle(n, dims, m, B, precision):
    w = wl.mlp_workload(n=n, dims=dims, m=m, batch=B, gamma=0.05, seed=11)
    rng = np.random.default_rng(1)
    # perturb the shared initial point per node so that rows differ; biases non-zero
    X = (np.tile(w.x0.numpy(), (n, 1)) + 0.02 * rng.standard_normal((n, w.N))).astype(np.float32)
    run, o = _setup(w, seed=3, precision=precision, X=X)
    for k in (0, 7):
        o.set_x(X)
        run.ctx.current()[:, :w.N] = torch.from_numpy(X).cuda()
        assert np.array_equal(run.ctx.sample(k).cpu().numpy(), o.sample(k))
        run.ctx.grad(k)
        G_ref, _ = mlp_oracle_grad_matching_gates(orc, o, k, run.g())
        assert row_rel_err(run.g(), G_ref) <= TOL_G[precision]
        if run.ld > w.N:
            assert float(run.G[:, w.N:].abs().max()) == 0.0
        # per-layer check so that a wrong block cannot hide behind a large one
        off = 0
        for l in range(len(dims) - 1):
            for size in (dims[l + 1] * dims[l], dims[l + 1]):
                blk_ref, blk = G_ref[:, off:off + size], run.g()[:, off:off + size]
                scale = np.linalg.norm(blk_ref.astype(np.float64), axis=1).max()
                assert np.abs(blk.astype(np.float64) - blk_ref).max() <= TOL_G[precision] * max(scale, 1e-12), (l, size)
                off += size
        X_ref = o.mix_update(G_ref)
        run.ctx.mix_update()
        assert row_rel_err(run.x(), X_ref) <= TOL_STEP
        run.check_pads()
    run.close()


def test_mlp_trajectory_config3_shape_short():
    """784-1024-10 on a ring of 8 nodes, 40 free-running steps."""
    w = wl.mlp_workload(n=8, dims=(784, 1024, 10), m=256, batch=32, gamma=0.05, seed=5)
    run, o = _setup(w, seed=9)
    for k in range(40):
        run.ctx.step(k)
        o.step(k)
    got = run.x()
    assert row_rel_err(got, o.X) <= TOL_TRAJ
    avg_ref = orc.node_average(o.X)
    assert np.linalg.norm(got.astype(np.float64).mean(axis=0) - avg_ref) <= TOL_AVG * np.linalg.norm(avg_ref)
    c_ref = o.consensus_dist()
    assert abs(run.ctx.consensus_dist() - c_ref) <= 2e-2 * c_ref
    run.close()


def test_mlp_dense_w_side_by_side_with_ring():
    """D-PSGD on a ring next to the dense averaging matrix (the C-PSGD baseline), consensus
    distance per step: with W = 11^T/n it equals gamma^2 sum_i ||g_i - gbar||^2 every step."""
    n, dims, B = 6, (32, 48, 5), 8
    w = wl.mlp_workload(n=n, dims=dims, m=64, batch=B, gamma=0.1, seed=6)
    wd = wl.mlp_workload(n=n, dims=dims, m=64, batch=B, gamma=0.1, seed=6, topology="dense")
    ring, o_ring = _setup(w, seed=2)
    dense, o_dense = _setup(wd, seed=2)
    for k in range(15):
        ring.ctx.step(k); o_ring.step(k)
        dense.ctx.grad(k)
        g = dense.g().astype(np.float64)
        dense.ctx.mix_update()
        o_dense.step(k)
        expect = np.float64(np.float32(0.1)) ** 2 * np.sum((g - g.mean(axis=0)) ** 2)
        c = dense.ctx.consensus_dist()
        assert abs(c - expect) <= 1e-3 * expect
        assert abs(c - o_dense.consensus_dist()) <= 1e-3 * expect
        assert abs(ring.ctx.consensus_dist() - o_ring.consensus_dist()) <= 1e-3 * o_ring.consensus_dist()
    ring.close(); dense.close()


def test_mlp_single_tf32_pass_is_close_but_looser():
    """mlp_precision = 1: one TF32 MMA per product (10-bit mantissas): about 1e-3 on G."""
    w = wl.mlp_workload(n=3, dims=(256, 512, 10), m=64, batch=32, gamma=0.05, seed=12)
    run, o = _setup(w, seed=4, precision=1)
    run.ctx.grad(0)
    G_ref = o.grad(0)
    err = row_rel_err(run.g(), G_ref)
    assert 1e-6 < err <= 5e-3
    run.close()


def test_mlp_large_batch_uses_fma_kernel():
    """Minibatches above 128 do not fit one accumulator tile and take the fp32 FMA path."""
    w = wl.mlp_workload(n=2, dims=(64, 48, 6), m=300, batch=160, gamma=0.05, seed=13)
    run, o = _setup(w, seed=5)
    run.ctx.grad(0)
    G_ref, _ = mlp_oracle_grad_matching_gates(orc, o, 0, run.g())
    assert row_rel_err(run.g(), G_ref) <= TOL_G[2]
    run.close()
