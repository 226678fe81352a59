"""GPU parity for footnote c of Algorithm 1 (update locally, then average) and for the gossip
step that returns the consensus distance of the new X from the same pass."""
import numpy as np
import pytest
import torch

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import binding, workloads as wl
from gpu_util import GpuRun, row_rel_err, TOL_STEP, TOL_TRAJ

pytestmark = pytest.mark.gpu


def _rand(rng, n, N):
    return rng.standard_normal((n, N)).astype(np.float32)


@pytest.mark.parametrize("topo,n,N", [("ring", 8, 3001), ("ring", 64, 50021), ("ring", 3, 7), ("dense", 8, 999),
                                      ("dense", 112, 10000), ("torus", 16, 1234), ("torus", 64, 30011),
                                      ("ring+antipode", 8, 515), ("ring", 2, 100), ("dense", 1, 40)])
def test_swapped_order_matches_oracle_on_every_kernel(topo, n, N):
    rng = np.random.default_rng(n + N)
    csr = wl.topology(topo, n)
    X, G = _rand(rng, n, N), _rand(rng, n, N)
    ref = orc.mix_update_swapped(X, G, *csr, 0.3)
    plain = orc.mix_update(X, G, *csr, 0.3)
    tried = 0
    for kind in (-1, binding.MIX_RING, binding.MIX_UNIFORM_DENSE, binding.MIX_TILED_CSR, binding.MIX_GATHER_CSR):
        run = GpuRun(n, N, csr, 0.3, X=X)
        run.set_g(G)
        try:
            run.ctx.mix_kind(kind)
        except binding.DpsgdError:
            run.close()
            continue
        run.ctx.set_order(True)
        run.ctx.mix_update()
        assert row_rel_err(run.x(), ref) <= TOL_STEP, kind
        run.check_pads()
        run.ctx.set_order(False)                     # and back to the printed order
        run.ctx.current()[:, :N] = torch.from_numpy(X).cuda()
        run.ctx.mix_update()
        assert row_rel_err(run.x(), plain) <= TOL_STEP, kind
        run.close()
        tried += 1
    assert tried >= 2


def test_dense_w_swapped_order_is_centralized_sgd_on_the_gpu():
    """Footnote c with W = 1 1^T / n: every row equals the C-PSGD iterate at every step, so the
    consensus distance is exactly zero (Section 2: minibatch SGD with n gradients per step)."""
    w = wl.logistic_workload(n=6, d=40, m=64, batch=8, gamma=0.3, l2_lambda=1e-3, topology="dense", seed=21)
    A, y = w.A.numpy(), w.y.numpy()
    seed = 99
    run = GpuRun(w.n, w.N, w.csr(), w.gamma, seed=seed, X=np.zeros((w.n, w.N), np.float32))
    run.ctx.set_model(w.model, w.dims, w.l2_lambda, w.batch)
    run.A, run.y = torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda()
    run.ctx.set_data(run.A, run.y)
    run.ctx.set_order(True)
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    x = np.zeros(w.N, dtype=np.float32)
    for k in range(25):
        idx = orc.sample_indices(seed, k, w.n, w.batch, w.m_per_node)
        grads = [orc.grad_logistic(x, A[i], y[i], idx[i], w.l2_lambda).astype(np.float32) for i in range(w.n)]
        x = orc.cpsgd_step(x, grads, w.gamma)
        run.ctx.step_consensus(k, out)
        got = run.x()
        assert float(out.item()) == 0.0
        for i in range(w.n):
            assert np.allclose(got[i], x, rtol=0, atol=5e-6)
    run.close()


TILED = binding.MIX_TILED_CSR


@pytest.mark.parametrize("topo,n,N,swapped,kind", [
    ("ring", 16, 4097, False, -1), ("ring", 112, 20011, False, -1), ("ring", 8, 333, True, -1),
    ("dense", 64, 30000, False, -1), ("dense", 5, 77, False, -1), ("torus", 16, 2500, False, -1),
    ("torus", 16, 2500, True, -1), ("ring", 3, 5, False, -1),
    # any sparse W on the tile-staging kernel: the statistics come out of the gossip pass itself
    ("torus", 64, 40007, False, -1),            # beyond the small-problem switch: tiles of 64 columns, ragged tail
    ("torus", 64, 40007, True, -1),
    ("torus", 16, 2500, False, TILED), ("torus", 16, 2500, True, TILED),      # tiles of 128 columns
    ("torus", 100, 3001, False, TILED),         # one CTA per SM, 64-column tiles
    ("torus", 9, 1000, False, TILED), ("ring+antipode", 8, 70001, True, TILED),
    ("ring", 200, 777, False, TILED),           # 200 rows per tile: one stage fills most of the shared memory
])
def test_fused_consensus_matches_oracle(topo, n, N, swapped, kind):
    rng = np.random.default_rng(N)
    csr = wl.topology(topo, n)
    X = (2.0 + 0.05 * rng.standard_normal((n, N))).astype(np.float32)     # small spread on an offset
    G = _rand(rng, n, N)
    run = GpuRun(n, N, csr, 0.1, X=X)
    run.set_g(G)
    run.ctx.set_order(swapped)
    if kind >= 0:
        run.ctx.mix_kind(kind)
    out = torch.full((1,), -1.0, dtype=torch.float64, device="cuda")
    before = run.ctx.launch_count()
    run.ctx.mix_update_consensus(out)
    if kind == TILED or (topo == "torus" and n * N * 4 > 8 << 20):
        assert run.ctx.launch_count() - before == 2            # gossip kernel + the fixed-order sum of its partials
    ref = (orc.mix_update_swapped if swapped else orc.mix_update)(X, G, *csr, 0.1)
    assert row_rel_err(run.x(), ref) <= TOL_STEP
    c_ref = orc.consensus_dist(ref)
    c_fused = float(out.item())
    assert abs(c_fused - c_ref) <= 1e-5 * c_ref + 1e-9
    assert abs(run.ctx.consensus_dist() - c_fused) <= 1e-9 * c_ref + 1e-12     # the separate pass agrees
    run.check_pads()
    run.close()


def test_step_consensus_trajectory_on_a_small_mlp():
    """Ring and dense side by side with the consensus distance of every step, as in the 112-node
    configuration; the per-step values follow the oracle."""
    for topo in ("ring", "dense"):
        w = wl.mlp_workload(n=6, dims=(32, 48, 5), m=64, batch=16, gamma=0.1, seed=6, topology=topo)
        A, y = w.A.numpy(), w.y.numpy()
        X0 = np.tile(w.x0.numpy(), (w.n, 1))
        run = GpuRun(w.n, w.N, w.csr(), w.gamma, seed=2, X=X0)
        run.ctx.set_model(w.model, w.dims, 0.0, w.batch, 0)
        run.A, run.y = torch.from_numpy(A).cuda(), torch.from_numpy(y).cuda()
        run.ctx.set_data(run.A, run.y)
        o = orc.Oracle(w.n, w.N, *w.csr(), w.gamma, 2, w.model, w.dims, w.batch, 0.0, A, y)
        o.set_x(X0)
        log = torch.zeros(20, dtype=torch.float64, device="cuda")
        ref = []
        for k in range(20):
            run.ctx.step_consensus(k, log[k:k + 1])
            o.step(k)
            ref.append(o.consensus_dist())
        got = log.cpu().numpy()
        assert np.allclose(got, ref, rtol=5e-3, atol=1e-12)
        assert row_rel_err(run.x(), o.X) <= TOL_TRAJ
        run.close()


@pytest.mark.parametrize("topo,n,N,swapped", [("ring", 8, 3001, False), ("ring", 64, 20011, True),
                                              ("dense", 8, 999, False), ("torus", 16, 1234, False),
                                              ("torus", 16, 1234, True), ("ring+antipode", 8, 515, False)])
def test_momentum_steps_match_oracle(topo, n, N, swapped):
    """v <- beta v + g per node, then the gossip step with v (Section 5.3: momentum 0.9)."""
    rng = np.random.default_rng(N + 1)
    csr = wl.topology(topo, n)
    X = _rand(rng, n, N)
    gamma, beta = 0.1, 0.9
    run = GpuRun(n, N, csr, gamma, X=X)
    V = torch.zeros_like(run.X0)
    run.ctx.set_momentum(beta, V)
    run.ctx.set_order(swapped)
    Xr, Vr = X.copy(), np.zeros_like(X)
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    for k in range(6):
        G = _rand(rng, n, N)
        run.set_g(G)
        if k % 2 == 0:
            run.ctx.mix_update()
        else:
            run.ctx.mix_update_consensus(out)
        Xr, Vr = orc.mix_update_momentum(Xr, Vr, G, *csr, gamma, beta, swapped=swapped)
        if k % 2 == 1:
            c_ref = orc.consensus_dist(Xr)
            assert abs(float(out.item()) - c_ref) <= 1e-4 * c_ref + 1e-9
    assert row_rel_err(run.x(), Xr) <= 1e-5
    assert row_rel_err(V[:, :N].cpu().numpy(), Vr) <= 1e-5
    assert float(V[:, N:].abs().max()) == 0.0 if run.ld > N else True
    run.check_pads()
    # switching momentum off restores the plain step
    run.ctx.set_momentum(0.0, None)
    G = _rand(rng, n, N)
    run.set_g(G)
    run.ctx.mix_update()
    f = orc.mix_update_swapped if swapped else orc.mix_update
    assert row_rel_err(run.x(), f(Xr, G, *csr, gamma)) <= TOL_STEP
    run.close()


@pytest.mark.parametrize("swapped", [False, True])
@pytest.mark.parametrize("topo,kind,n,N", [("ring", 0, 3, 40), ("ring", 0, 5, 1031), ("ring", 0, 6, 77),
                                           ("ring", 0, 9, 4100), ("ring", 0, 64, 2051),
                                           ("dense", 1, 1, 40), ("dense", 1, 2, 77), ("dense", 1, 5, 1031),
                                           ("dense", 1, 9, 4100), ("dense", 1, 64, 2051)])
def test_momentum_inside_the_gossip_pass(topo, kind, n, N, swapped):
    """With the streaming kernel chosen (not the small-problem one), ring and uniform W update the
    momentum buffers in the same pass as the gossip step; results as with separate passes."""
    rng = np.random.default_rng(31 * n + N)
    csr = wl.topology(topo, n)
    X = _rand(rng, n, N)
    gamma, beta = 0.05, 0.9
    run = GpuRun(n, N, csr, gamma, X=X)
    run.ctx.mix_kind(kind)
    V0 = _rand(rng, n, N)
    V = torch.zeros_like(run.X0)
    V[:, :N] = torch.from_numpy(V0).cuda()
    run.ctx.set_momentum(beta, V)
    run.ctx.set_order(swapped)
    Xr, Vr = X.copy(), V0.copy()
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    for k in range(4):
        G = _rand(rng, n, N)
        run.set_g(G)
        if k % 2 == 0:
            run.ctx.mix_update()
        else:
            run.ctx.mix_update_consensus(out)
            torch.cuda.synchronize()
        Xr, Vr = orc.mix_update_momentum(Xr, Vr, G, *csr, gamma, beta, swapped=swapped)
        assert row_rel_err(run.x(), Xr) <= 1e-5
        assert row_rel_err(V[:, :N].cpu().numpy(), Vr) <= 1e-5
        if k % 2 == 1:
            c_ref = orc.consensus_dist(Xr)
            assert abs(float(out.item()) - c_ref) <= 1e-4 * c_ref + 1e-9
    run.check_pads()
    run.close()
