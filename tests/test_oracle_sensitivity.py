"""How far two runs of the ORACLE drift apart when one of them starts a rounding error away: the yardstick
for the free-running trajectory tolerances (rows 1e-3, node average 1e-4 after T iterations).

Algorithm 1 on the convex models contracts a perturbation; on a ReLU network it does not: the stochastic
gradient is piecewise linear in x, a perturbation moves pre-activations across zero, every such flip changes
the gradient by a finite amount, and the runs separate at a steady rate.  The test shows both with the oracle
alone (fp64 on both sides, same indices), so the effect belongs to the problem, not to an implementation."""
import numpy as np

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import workloads as wl


def _twin_separation(w, seed, T, eps):
    A, y = w.A.numpy(), w.y.numpy()
    runs = []
    for _ in range(2):
        o = orc.Oracle(w.n, w.N, *w.csr(), w.gamma, seed, w.model, w.dims, w.batch, w.l2_lambda, A, y)
        o.set_x(np.tile(w.x0.numpy(), (w.n, 1)))
        runs.append(o)
    rng = np.random.default_rng(0)
    base = runs[1].X.astype(np.float64)
    # the second run starts eps away (relative, every element; an absolute eps where the start is zero)
    runs[1].X = (base * (1.0 + eps * rng.standard_normal(base.shape)) + eps * (base == 0) * rng.standard_normal(base.shape)
                 ).astype(np.float32)

    def sep():
        a, b = runs[0].X.astype(np.float64), runs[1].X.astype(np.float64)
        return float(np.linalg.norm(a.mean(0) - b.mean(0)) / max(np.linalg.norm(a.mean(0)), 1e-30))

    first = None
    for k in range(T):
        for o in runs:
            o.step(k)
        if k == 0:
            first = sep()
    return first, sep()


def test_relu_network_separates_two_oracle_runs_far_beyond_the_initial_difference():
    """A network of the 112-node configuration's depth (reduced widths), ring of 4, minibatch 64, gamma 0.02,
    300 iterations: two oracle runs 1e-6 apart at the start end about 1e-4 apart on the node average (the
    trajectory tolerance itself), two orders of magnitude more than they started."""
    w = wl.mlp_workload(n=4, dims=(128, 256, 256, 10), m=512, batch=64, gamma=0.02, seed=170509060)
    first, last = _twin_separation(w, 20254, 300, 1e-6)
    assert first <= 2e-6
    assert last >= 2e-5 and last >= 20 * first, (first, last)


def test_least_squares_contracts_the_same_perturbation():
    """The convex control: on least squares the same experiment ends closer than it started."""
    w = wl.lsq_workload(n=8, d=64, m=256, batch=16)
    first, last = _twin_separation(w, 7, 200, 1e-6)
    assert last <= first, (first, last)
