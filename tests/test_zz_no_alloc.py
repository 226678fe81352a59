"""The allocation-free consensus distance (dpsgd_consensus_dist_noalloc) against the context's
dpsgd_consensus_dist.

Collected last on purpose: a run that stops at the first failure has then already run every other
test.  The entry point serves callers that cannot let the library allocate (all device memory
pre-reserved by the caller, no context at hand); its scratch is one array inside the library
that every call shares, so the test calls it twice in a row on different inputs, the second
smaller than the first, to show that what the first call left behind is never read.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import dpsgd_oracle as orc
from paper_1705_09056_b200 import binding, workloads as wl

pytestmark = pytest.mark.gpu


def _matrix(n, N, seed, spread):
    ld = wl.padded_ld(N)
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    X = torch.zeros((n, ld), device="cuda")
    X[:, :N] = 3.0 + spread * torch.randn((n, N), generator=g, device="cuda")
    return X


def _with_context(X, N):
    n, ld = X.shape
    ctx = binding.Dpsgd(n, N, *wl.ring(n), gamma=0.1)
    ctx.bind(X, torch.zeros_like(X), torch.zeros_like(X))
    v = ctx.consensus_dist()
    ctx.close()
    return v


def test_noalloc_consensus_matches_context_entry_point_twice_in_a_row():
    cases = [(64, 300_007, 1, 0.5), (16, 4097, 2, 0.01)]      # large first, then small
    mats = [(_matrix(n, N, seed, spread), N) for n, N, seed, spread in cases]
    want = [_with_context(X, N) for X, N in mats]
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    got = []
    for X, N in mats:                                          # two calls back to back
        binding.consensus_dist_noalloc(X, N, out)
        got.append(float(out.item()))
    for g, w_ in zip(got, want):
        assert abs(g - w_) <= 1e-5 * w_ + 1e-12                # the tolerance of the other consensus tests
        assert g == w_                                         # same kernels, same order: bit-identical
    for (X, N), g in zip(mats, got):                           # and the definition itself (Eq. 10), on the CPU
        ref = orc.consensus_dist(X[:, :N].cpu().numpy())
        assert abs(g - ref) <= 1e-5 * ref
    # and again in the opposite order, reusing the same output cell
    binding.consensus_dist_noalloc(mats[1][0], mats[1][1], out)
    assert float(out.item()) == want[1]
    binding.consensus_dist_noalloc(mats[0][0], mats[0][1], out)
    assert float(out.item()) == want[0]


def test_noalloc_consensus_rejects_oversized_and_malformed_input():
    lib = binding.load_library()
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    X = torch.zeros((2, 64), device="cuda")
    too_wide = binding.NOALLOC_MAX_LD + 32
    st = lib.dpsgd_consensus_dist_noalloc(X.data_ptr(), 2, too_wide, too_wide, 0, out.data_ptr())
    assert st == binding.ERR_UNSUPPORTED
    assert b"exceeds" in lib.dpsgd_last_error(None)
    assert lib.dpsgd_consensus_dist_noalloc(None, 2, 64, 64, 0, out.data_ptr()) == binding.ERR_ARG
    assert lib.dpsgd_consensus_dist_noalloc(X.data_ptr(), 2, 64, 48, 0, out.data_ptr()) == binding.ERR_ARG
    assert lib.dpsgd_consensus_dist_noalloc(X.data_ptr(), 2, 40, 40, 0, out.data_ptr()) == binding.ERR_ALIGN
    assert lib.dpsgd_consensus_dist_noalloc(X.data_ptr() + 4, 2, 32, 32, 0, out.data_ptr()) == binding.ERR_ALIGN
    torch.cuda.synchronize()
