"""The pins must bite: plant one plausible mistake at a time in the ORACLE (CPU only) and
check that at least one pin test fails."""
import numpy as np
import pytest

from oracle import dpsgd_oracle as orc
import test_oracle_gradients as tg
import test_oracle_mixing as tm
import test_oracle_sampler as ts


def _fails(test, *args):
    try:
        test(*args)
    except AssertionError:
        return True
    return False


def test_swapped_philox_multipliers_are_caught(monkeypatch):
    monkeypatch.setattr(orc, "_PHILOX_M0", np.uint64(0xCD9E8D57))
    monkeypatch.setattr(orc, "_PHILOX_M1", np.uint64(0xD2511F53))
    assert _fails(ts.test_philox_matches_curand_host_generator)


def test_nine_round_philox_is_caught(monkeypatch):
    real = orc.philox_round
    calls = {"n": 0}

    def skipping(c, k):
        calls["n"] += 1
        return c if calls["n"] % 10 == 0 else real(c, k)
    monkeypatch.setattr(orc, "philox_round", skipping)
    assert _fails(ts.test_philox_matches_curand_host_generator)


def test_wrong_update_sign_is_caught(monkeypatch):
    real = orc.mix_update
    monkeypatch.setattr(orc, "mix_update",
                        lambda X, G, rp, c, v, g: real(X, -G, rp, c, v, g))
    assert _fails(tm.test_mix_update_equals_brute_force_dense_product, 3, 7, 1)
    assert _fails(tm.test_mixing_preserves_the_node_average, "ring", 8)


def test_dropped_neighbour_is_caught(monkeypatch):
    real = orc.mix_update

    def lossy(X, G, rp, col, val, g):
        val = np.array(val, copy=True)
        val[int(rp[1]) - 1] = 0           # forget the last neighbour of node 0
        return real(X, G, rp, col, val, g)
    monkeypatch.setattr(orc, "mix_update", lossy)
    assert _fails(tm.test_mixing_preserves_the_node_average, "ring", 8)
    assert _fails(tm.test_mix_update_equals_brute_force_dense_product, 4, 5, 2)


def test_gradient_at_mixed_point_is_caught(monkeypatch):
    """Taking the gradient after mixing instead of at x_{k,i} changes the step."""
    def wrong_step(self, k):
        Z = np.zeros_like(self.X)
        mixed = orc.mix_update(self.X, Z, self.row_ptr, self.col, self.val, 0.0)
        G = orc.gradients(mixed, self.model, self.dims, self.A, self.y, self.sample(k), self.lam)
        self.X = (mixed.astype(np.float64) - np.float64(np.float32(self.gamma)) * G).astype(np.float32)
        return self.X
    monkeypatch.setattr(orc.Oracle, "step", wrong_step)
    assert _fails(tm.test_oracle_step_is_grad_then_mix_with_pre_mix_gradient)


def test_logistic_mistakes_are_caught(monkeypatch):
    real = orc.grad_logistic
    monkeypatch.setattr(orc, "grad_logistic", lambda *a: -real(*a))
    assert _fails(tg.test_logistic_gradient_matches_finite_differences)
    monkeypatch.setattr(orc, "grad_logistic",
                        lambda x, A, y, idx, lam: real(x, A, y, idx, lam) + lam * np.r_[0 * x[:-1], x[-1]])
    assert _fails(tg.test_logistic_penalty_skips_bias)


def test_mlp_sum_instead_of_mean_is_caught(monkeypatch):
    real = orc.grad_mlp
    monkeypatch.setattr(orc, "grad_mlp", lambda x, d, A, l, idx: real(x, d, A, l, idx) * len(idx))
    assert _fails(tg.test_mlp_gradient_matches_torch_autograd, (8, 16, 5))
    assert _fails(tg.test_mlp_gradient_matches_finite_differences, (4, 6, 3))


def test_mlp_transposed_weight_view_is_caught(monkeypatch):
    real = orc._mlp_views

    def transposed(x, dims):
        Ws, bs = real(x, dims)
        return [W.reshape(W.shape[1], W.shape[0]).T for W in Ws], bs
    monkeypatch.setattr(orc, "_mlp_views", transposed)
    assert _fails(tg.test_mlp_gradient_matches_torch_autograd, (8, 16, 5))


def test_consensus_mean_instead_of_sum_is_caught(monkeypatch):
    real = orc.consensus_dist
    monkeypatch.setattr(orc, "consensus_dist", lambda X: real(X) / X.shape[0])
    assert _fails(tm.test_consensus_distance_identities)
