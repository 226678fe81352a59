"""GPU parity: fused gossip step, consensus distance and node average against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import binding, workloads as wl
from gpu_util import GpuRun, row_rel_err, TOL_STEP, TOL_TRAJ, TOL_AVG

pytestmark = pytest.mark.gpu


def _rand(rng, n, N):
    return rng.standard_normal((n, N)).astype(np.float32)


CASES = [
    # topology, n, N  (ragged N, N < one vector, several CTAs, the configs' shapes)
    ("ring", 3, 1), ("ring", 4, 5), ("ring", 5, 4097), ("ring", 8, 64), ("ring", 16, 4097),
    ("ring", 64, 100003), ("ring", 112, 33000), ("ring", 7, 1030), ("ring", 6, 262144 + 17),
    ("torus", 64, 50021), ("torus", 16, 777), ("torus", 4, 9),
    ("dense", 64, 70001), ("dense", 5, 13), ("dense", 1, 100), ("dense", 112, 20000), ("dense", 3, 40),
    ("ring+antipode", 16, 5000), ("identity", 6, 1000), ("ring", 2, 77), ("ring", 1, 33),
]


@pytest.mark.parametrize("topo,n,N", CASES)
def test_one_step_matches_oracle(topo, n, N):
    rng = np.random.default_rng(n * 1000 + N)
    csr = wl.topology(topo, n)
    X, G = _rand(rng, n, N), _rand(rng, n, N)
    gamma = 0.05
    run = GpuRun(n, N, csr, gamma, X=X)
    run.set_g(G)
    run.ctx.mix_update()
    ref = orc.mix_update(X, G, *csr, gamma)
    assert row_rel_err(run.x(), ref) <= TOL_STEP
    # elementwise: fp32 FMA chain vs fp64 with one rounding differs by a few ulp of the terms
    scale = np.abs(wl.csr_to_dense(n, *csr)) @ np.abs(X).astype(np.float64) + gamma * np.abs(G)
    deg = int(np.max(np.diff(csr[0])))
    assert np.all(np.abs(run.x().astype(np.float64) - ref) <= (deg + 4) * 6e-8 * scale + 1e-30)
    run.check_pads()
    run.close()


@pytest.mark.parametrize("topo,n,N", [("ring", 8, 3001), ("torus", 16, 1234), ("dense", 8, 999),
                                      ("ring+antipode", 8, 515)])
def test_every_applicable_kernel_agrees_with_oracle(topo, n, N):
    rng = np.random.default_rng(17)
    csr = wl.topology(topo, n)
    X, G = _rand(rng, n, N), _rand(rng, n, N)
    ref = orc.mix_update(X, G, *csr, 0.3)
    tried = 0
    for kind in (binding.MIX_RING, binding.MIX_UNIFORM_DENSE, binding.MIX_TILED_CSR, binding.MIX_GATHER_CSR):
        run = GpuRun(n, N, csr, 0.3, X=X)
        run.set_g(G)
        try:
            run.ctx.mix_kind(kind)
        except binding.DpsgdError as e:
            assert e.status == binding.ERR_UNSUPPORTED
            run.close()
            continue
        run.ctx.mix_update()
        assert row_rel_err(run.x(), ref) <= TOL_STEP, binding.MIX_NAMES[kind]
        run.check_pads()
        run.close()
        tried += 1
    assert tried >= 1


def test_kernel_selection_follows_structure_of_w():
    for topo, n, want in (("ring", 8, binding.MIX_RING), ("dense", 8, binding.MIX_UNIFORM_DENSE),
                          ("ring", 64, binding.MIX_RING), ("dense", 64, binding.MIX_UNIFORM_DENSE)):
        ctx = binding.Dpsgd(n, 64, *wl.topology(topo, n), gamma=0.1)
        assert ctx.mix_kind() == want
        ctx.close()
    ctx = binding.Dpsgd(64, 64, *wl.topology("torus", 64), gamma=0.1)
    assert ctx.mix_kind() in (binding.MIX_TILED_CSR, binding.MIX_GATHER_CSR)
    with pytest.raises(binding.DpsgdError):
        ctx.mix_kind(binding.MIX_RING)
    ctx.close()


@pytest.mark.parametrize("topo,n", [("ring", 8), ("torus", 16), ("dense", 8), ("ring", 64)])
def test_trajectory_and_average_over_many_steps(topo, n):
    """Free-running: 50 steps with fresh gradients each step, GPU and oracle never re-synchronised."""
    N, T, gamma = 2051, 50, 0.01
    rng = np.random.default_rng(3)
    csr = wl.topology(topo, n)
    X = _rand(rng, n, N)
    run = GpuRun(n, N, csr, gamma, X=X)
    ref = X.copy()
    for k in range(T):
        G = _rand(rng, n, N)
        run.set_g(G)
        run.ctx.mix_update()
        ref = orc.mix_update(ref, G, *csr, gamma)
    got = run.x()
    assert row_rel_err(got, ref) <= TOL_TRAJ
    avg_ref = orc.node_average(ref)
    avg_got = got.astype(np.float64).mean(axis=0)
    assert np.linalg.norm(avg_got - avg_ref) / np.linalg.norm(avg_ref) <= TOL_AVG
    run.check_pads()
    run.close()


@pytest.mark.parametrize("topo,n", [("ring", 16), ("torus", 16), ("dense", 6)])
def test_gpu_mixing_preserves_average_and_contracts(topo, n):
    """The invariants of the proof of Theorem 1 and of Lemma 5 hold for the kernels too."""
    N = 3000
    rng = np.random.default_rng(4)
    csr = wl.topology(topo, n)
    sqrt_rho = np.sqrt(orc.spectral_rho(wl.csr_to_dense(n, *csr)))
    X = _rand(rng, n, N)
    run = GpuRun(n, N, csr, 0.5, X=X)          # G stays zero
    mean0 = X.astype(np.float64).mean(axis=0)
    d = np.sqrt(run.ctx.consensus_dist())
    for _ in range(10):
        run.ctx.mix_update()
        d_new = np.sqrt(run.ctx.consensus_dist())
        assert d_new <= sqrt_rho * d * (1 + 1e-4) + 1e-4
        d = d_new
    assert np.max(np.abs(run.x().astype(np.float64).mean(axis=0) - mean0)) <= 10 * n * 2.0 ** -23
    run.close()


@pytest.mark.parametrize("n,N", [(1, 5), (2, 3), (8, 64), (16, 4097), (64, 30011), (112, 5000)])
def test_consensus_distance_and_average_match_oracle(n, N):
    rng = np.random.default_rng(n + N)
    X = (5.0 + 0.01 * rng.standard_normal((n, N))).astype(np.float32)   # small spread on a large offset
    run = GpuRun(n, N, wl.ring(n), 0.1, X=X)
    ref = orc.consensus_dist(X)
    got = run.ctx.consensus_dist()
    assert abs(got - ref) <= 1e-5 * ref + 1e-12
    xbar = run.ctx.average()[:N].cpu().numpy()
    assert np.allclose(xbar, orc.node_average(X), rtol=1e-6, atol=1e-7)
    # identical rows (x_{0,i} = x_0): exactly zero
    same = np.tile(X[0], (n, 1))
    run2 = GpuRun(n, N, wl.ring(n), 0.1, X=same)
    assert run2.ctx.consensus_dist() == 0.0
    run.close(); run2.close()


def test_dense_w_zero_gradient_gives_consensus_in_one_step():
    rng = np.random.default_rng(5)
    n, N = 16, 5003
    X = _rand(rng, n, N)
    run = GpuRun(n, N, wl.dense_uniform(n), 0.2, X=X)
    run.ctx.mix_update()
    assert run.ctx.consensus_dist() <= 1e-9 * N
    assert np.allclose(run.x()[3], orc.node_average(X), atol=1e-6)
    run.close()


def test_two_runs_are_bit_identical_and_gamma_can_change():
    rng = np.random.default_rng(6)
    n, N = 16, 9001
    csr = wl.torus2d(4, 4)
    X, G = _rand(rng, n, N), _rand(rng, n, N)
    outs = []
    for _ in range(2):
        run = GpuRun(n, N, csr, 0.1, X=X)
        run.set_g(G)
        for _k in range(5):
            run.ctx.mix_update()
        outs.append((run.x(), run.ctx.consensus_dist()))
        run.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][1] == outs[1][1]
    run = GpuRun(n, N, csr, 0.1, X=X)
    run.set_g(G)
    run.ctx.set_gamma(0.7)
    run.ctx.mix_update()
    assert row_rel_err(run.x(), orc.mix_update(X, G, *csr, 0.7)) <= TOL_STEP
    run.close()


def test_host_gradient_entry_point_matches_device_path():
    rng = np.random.default_rng(7)
    n, N = 8, 4099
    csr = wl.ring(n)
    X, G = _rand(rng, n, N), _rand(rng, n, N)
    run = GpuRun(n, N, csr, 0.05, X=X)
    Gh = torch.from_numpy(G).pin_memory()
    c = run.ctx.mix_update_host(Gh)
    ref = orc.mix_update(X, G, *csr, 0.05)
    assert row_rel_err(run.x(), ref) <= TOL_STEP
    assert abs(c - orc.consensus_dist(ref)) <= 1e-5 * orc.consensus_dist(ref)
    run.check_pads()
    run.close()


def test_bind_argument_checks():
    n, N = 4, 100
    ctx = binding.Dpsgd(n, N, *wl.ring(n), gamma=0.1)
    with pytest.raises(binding.DpsgdError) as e:
        ctx.mix_update()
    assert e.value.status == binding.ERR_STATE
    buf = torch.zeros(3 * n * 128 + 64, device="cuda")
    p = buf.data_ptr()
    with pytest.raises(binding.DpsgdError) as e:
        ctx.bind_raw(p, p + 4 * n * 128, p + 8 * n * 128, 96)      # ld < N
    assert e.value.status == binding.ERR_ARG
    with pytest.raises(binding.DpsgdError) as e:
        ctx.bind_raw(p, p + 4 * n * 128, p + 8 * n * 128, 104)     # ld not a multiple of 32
    assert e.value.status == binding.ERR_ALIGN
    with pytest.raises(binding.DpsgdError) as e:
        ctx.bind_raw(p + 4, p + 4 * n * 128, p + 8 * n * 128, 128)  # misaligned
    assert e.value.status == binding.ERR_ALIGN
    with pytest.raises(binding.DpsgdError) as e:
        ctx.bind_raw(p, p + 4 * 128, p + 8 * n * 128, 128)          # overlap
    assert e.value.status == binding.ERR_ARG
    with pytest.raises(binding.DpsgdError) as e:
        ctx.bind_raw(p, 0, p + 8 * n * 128, 128)
    assert e.value.status == binding.ERR_ARG
    ctx.bind_raw(p, p + 4 * n * 128, p + 8 * n * 128, 128)
    ctx.mix_update()
    torch.cuda.synchronize()
    ctx.close()


def test_full_size_stress_shape_on_column_slices():
    """n = 64 x N = 25,000,000 (the bandwidth configuration), in the launch shape the benchmark
    times.  The step is separable per column, so the oracle checks column slices: the first
    columns, the last ones including the ragged tail, and three random blocks."""
    n, N = 64, 25_000_000
    free, _ = torch.cuda.mem_get_info()
    if free < 22 * 2 ** 30:
        pytest.skip("needs 20 GB of device memory")
    ld = wl.padded_ld(N)
    X0 = wl.stress_matrix(n, ld, N, 11, "cuda")
    G = wl.stress_matrix(n, ld, N, 12, "cuda")
    X1 = torch.zeros_like(X0)
    width = 50_000
    rng = np.random.default_rng(8)
    starts = [0, N - width] + [int(s) for s in rng.integers(width, N - 2 * width, 3)]
    for topo in ("ring", "torus", "dense"):
        csr = wl.topology(topo, n)
        ctx = binding.Dpsgd(n, N, *csr, gamma=0.01)
        ctx.bind(X0, X1, G)
        ctx.mix_update()
        out = ctx.current()
        assert out.data_ptr() == X1.data_ptr()
        for s in starts:
            xs = X0[:, s:s + width].cpu().numpy()
            gs = G[:, s:s + width].cpu().numpy()
            ref = orc.mix_update(xs, gs, *csr, 0.01)
            assert row_rel_err(out[:, s:s + width].cpu().numpy(), ref) <= TOL_STEP, (topo, s)
        # property that holds at any size: the node average moves by -gamma * mean gradient
        avg = ctx.average()[:N].double()
        expect = X0[:, :N].double().mean(dim=0) - 0.01 * G[:, :N].double().mean(dim=0)
        assert float((avg - expect).abs().max()) <= 1e-5
        ctx.close()
