"""The give-up path of the bounded device-side waits, driven without faulting anything: a self-test CTA
waits on a barrier at which nothing arrives, gives up after a few thousand polls, raises the status
word and returns.  The next synchronising call must report DPSGD_ERR_TIMEOUT exactly once, and the
context must work as before afterwards."""
import numpy as np
import pytest
import torch

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import binding, workloads as wl
from gpu_util import GpuRun, row_rel_err, TOL_STEP

pytestmark = pytest.mark.gpu


def _run(n=6, N=5000, seed=3):
    rng = np.random.default_rng(seed)
    X = rng.standard_normal((n, N)).astype(np.float32)
    G = rng.standard_normal((n, N)).astype(np.float32)
    run = GpuRun(n, N, wl.ring(n), 0.1, X=X)
    run.set_g(G)
    return run, X, G


@pytest.mark.parametrize("collector", ["sync", "consensus_dist", "set_model", "set_node_batches"])
def test_wait_that_runs_out_is_reported_once_by_the_next_synchronising_call(collector):
    run, X, G = _run()
    ctx = run.ctx
    ctx.sync()                                   # nothing pending
    ctx.selftest_wait(2048)
    ctx.mix_update()                             # asynchronous calls cannot see the word
    with pytest.raises(binding.DpsgdError) as e:
        if collector == "sync":
            ctx.sync()
        elif collector == "consensus_dist":
            ctx.consensus_dist()
        elif collector == "set_model":
            ctx.set_model(binding.MODEL_LSQ, [5000], 0.0, 4)
        else:
            ctx.set_model(binding.MODEL_LSQ, [5000], 0.0, 4)     # collects and clears ...
    assert e.value.status == binding.ERR_TIMEOUT
    if collector == "set_node_batches":
        ctx.set_model(binding.MODEL_LSQ, [5000], 0.0, 4)         # ... so this one succeeds
        ctx.selftest_wait(64)
        with pytest.raises(binding.DpsgdError) as e2:
            ctx.set_node_batches([4] * 6)
        assert e2.value.status == binding.ERR_TIMEOUT
    ctx.sync()                                   # reported once: the word was cleared
    # the step enqueued behind the self-test ran normally, and so does the next one
    ref = orc.mix_update(X, G, *wl.ring(6), 0.1)
    assert row_rel_err(run.x(), ref) <= TOL_STEP
    ctx.mix_update()
    assert row_rel_err(run.x(), orc.mix_update(ref, G, *wl.ring(6), 0.1)) <= TOL_STEP
    assert abs(ctx.consensus_dist() - orc.consensus_dist(run.x())) <= 1e-5 * orc.consensus_dist(run.x())
    run.check_pads()
    run.close()


def test_destroy_reports_a_pending_timeout_and_argument_limits():
    run, _, _ = _run()
    lib = binding.load_library()
    with pytest.raises(binding.DpsgdError) as e:
        run.ctx.selftest_wait(0)
    assert e.value.status == binding.ERR_ARG
    with pytest.raises(binding.DpsgdError) as e:
        run.ctx.selftest_wait((1 << 20) + 1)
    assert e.value.status == binding.ERR_ARG
    run.ctx.selftest_wait(1)
    h = run.ctx._h
    run.ctx._h = type(h)()                        # hand the handle to the raw call below
    assert lib.dpsgd_destroy(h) == binding.ERR_TIMEOUT
    assert lib.dpsgd_sync(None) == binding.ERR_ARG
    torch.cuda.synchronize()
