"""Host-side checks that need no GPU: the C-ABI library loads, exports every symbol the header
declares, and rejects invalid arguments before touching CUDA."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_1705_09056_b200 import binding, workloads as wl

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1705_09056_b200 import build
    build.build()
    return binding.load_library()


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            names |= set(re.findall(r"DPSGD_API\s+[\w\s\*]+?\b(dpsgd_\w+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported_and_bound(lib):
    declared = _declared()
    assert len(declared) >= 17
    for name in declared:
        assert hasattr(lib, name), name
    assert declared == set(binding.SIGNATURES), declared ^ set(binding.SIGNATURES)


def _create(lib, n, N, rp, col, val, gamma=0.1, seed=1):
    h = ctypes.c_void_p()
    rp, col, val = (np.ascontiguousarray(rp, np.int32), np.ascontiguousarray(col, np.int32),
                    np.ascontiguousarray(val, np.float32))
    st = lib.dpsgd_create(ctypes.byref(h), n, N, rp.ctypes.data, col.ctypes.data, val.ctypes.data,
                          gamma, seed)
    return st, h, lib.dpsgd_last_error(None).decode()


def test_create_rejects_bad_sizes_and_null_pointers(lib):
    rp, col, val = wl.ring(4)
    assert _create(lib, 0, 8, rp, col, val)[0] == binding.ERR_ARG
    assert _create(lib, 70000, 8, rp, col, val)[0] == binding.ERR_ARG
    assert _create(lib, 4, 0, rp, col, val)[0] == binding.ERR_ARG
    h = ctypes.c_void_p()
    assert lib.dpsgd_create(ctypes.byref(h), 4, 8, None, None, None, 0.1, 0) == binding.ERR_ARG
    assert lib.dpsgd_create(None, 4, 8, rp.ctypes.data, col.ctypes.data, val.ctypes.data, 0.1, 0) == binding.ERR_ARG
    assert _create(lib, 4, 8, rp, col, val, gamma=float("nan"))[0] == binding.ERR_ARG


def test_create_rejects_matrices_that_are_not_symmetric_doubly_stochastic(lib):
    """Section 3: W_ij in [0,1], W_ij = W_ji, rows sum to one."""
    n = 4
    rp, col, val = wl.ring(n)
    cases = {}
    v = val.copy(); v[0] = 0.5
    cases["row sum"] = (rp, col, v)
    # asymmetric but row-stochastic: directed cycle
    cases["asymmetric"] = (np.arange(n + 1), (np.arange(n) + 1) % n, np.ones(n))
    v = val.copy(); v[0], v[1] = -0.1, v[1] + v[0] + 0.1
    cases["negative"] = (rp, col, v)
    c = col.copy(); c[1] = 9
    cases["column range"] = (rp, c, val)
    c = col.copy(); c[0], c[1] = col[1], col[0]
    cases["unsorted"] = (rp, c, val)
    r = rp.copy(); r[0] = 1
    cases["row_ptr start"] = (r, col, val)
    # symmetric values but mismatched mirror entry
    W = wl.csr_to_dense(n, rp, col, val).astype(np.float32)
    W[0, 1] += 0.01; W[0, 0] -= 0.01
    cases["mirror"] = wl.dense_to_csr(W.astype(np.float64))
    for name, (a, b, c_) in cases.items():
        st, h, msg = _create(lib, n, 8, a, b, c_)
        assert st == binding.ERR_W_INVALID, (name, st, msg)
        assert h.value is None and msg


def test_null_context_is_an_argument_error(lib):
    out = ctypes.c_double()
    assert lib.dpsgd_mix_update(None) == binding.ERR_ARG
    assert lib.dpsgd_step(None, 0) == binding.ERR_ARG
    assert lib.dpsgd_grad(None, 0) == binding.ERR_ARG
    assert lib.dpsgd_consensus_dist(None, ctypes.byref(out)) == binding.ERR_ARG
    assert lib.dpsgd_destroy(None) == binding.ERR_ARG
    assert lib.dpsgd_set_gamma(None, 0.1) == binding.ERR_ARG


def test_no_cpu_fallback_without_a_device(lib):
    """A valid W on a machine without CUDA must fail loudly, not compute on the CPU."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    st, h, msg = _create(lib, 4, 8, *wl.ring(4))
    assert st == binding.ERR_CUDA and h.value is None and msg
    with pytest.raises(binding.DpsgdError):
        binding.Dpsgd(4, 8, *wl.ring(4), gamma=0.1)


def test_missing_library_raises(tmp_path):
    with pytest.raises(binding.DpsgdError):
        binding.load_library(str(tmp_path / "libdpsgd.so"))
