"""Thin ctypes binding of libdpsgd.so: argument marshalling only.

Every step of the D-PSGD iteration (Algorithm 1 of arXiv 1705.09056) runs inside the CUDA
library; torch is used here for device memory and the current stream.  There is no CPU
fallback: if the library is missing or a call fails, a DpsgdError is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdpsgd.so")

OK, ERR_ARG, ERR_W_INVALID, ERR_ALIGN, ERR_STATE, ERR_UNSUPPORTED, ERR_CUDA, ERR_TIMEOUT = range(8)
STATUS_NAMES = ["OK", "ERR_ARG", "ERR_W_INVALID", "ERR_ALIGN", "ERR_STATE", "ERR_UNSUPPORTED",
                "ERR_CUDA", "ERR_TIMEOUT"]
MODEL_LSQ, MODEL_LOGISTIC, MODEL_MLP = 0, 1, 2
MIX_RING, MIX_UNIFORM_DENSE, MIX_TILED_CSR, MIX_GATHER_CSR = 0, 1, 2, 3
MIX_NAMES = {0: "ring", 1: "uniform_dense", 2: "tiled_csr", 3: "gather_csr"}

_vp, _i32, _i64, _u64, _f32 = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint64,
                               ctypes.c_float)

# name -> argument types (all return int32 status except dpsgd_last_error)
SIGNATURES = {
    "dpsgd_create": [ctypes.POINTER(_vp), _i32, _i64, _vp, _vp, _vp, _f32, _u64],
    "dpsgd_destroy": [_vp],
    "dpsgd_bind": [_vp, _vp, _vp, _vp, _i64, _vp],
    "dpsgd_set_model": [_vp, _i32, _vp, _i32, _f32, _i32, _i32],
    "dpsgd_set_data": [_vp, _vp, _vp, _i64, _i32],
    "dpsgd_sample": [_vp, _u64, _vp],
    "dpsgd_grad": [_vp, _u64],
    "dpsgd_mix_update": [_vp],
    "dpsgd_step": [_vp, _u64],
    "dpsgd_run": [_vp, _u64, _i64],
    "dpsgd_local_step": [_vp, _u64],
    "dpsgd_local_step_nodes": [_vp, _u64, _vp],
    "dpsgd_set_node_batches": [_vp, _vp],
    "dpsgd_set_order": [_vp, _i32],
    "dpsgd_set_fused_step": [_vp, _i32],
    "dpsgd_set_momentum": [_vp, _f32, _vp],
    "dpsgd_mix_update_consensus": [_vp, _vp],
    "dpsgd_step_consensus": [_vp, _u64, _vp],
    "dpsgd_consensus_dist": [_vp, ctypes.POINTER(ctypes.c_double)],
    "dpsgd_sync": [_vp],
    "dpsgd_selftest_wait": [_vp, ctypes.c_uint32],
    "dpsgd_average": [_vp, _vp],
    "dpsgd_conv3x3_forward": [_vp, _vp, _i32, _i32, _i32, _i32, _i32, _i32, _i64, _i64, _i32, _vp],
    "dpsgd_conv3x3_backward": [_vp, _vp, _vp, _vp, _i32, _i32, _i32, _i32, _i32, _i32, _i64, _i64, _i32, _vp],
    "dpsgd_mix_update_host": [_vp, _vp, _i64, ctypes.POINTER(ctypes.c_double)],
    "dpsgd_consensus_dist_noalloc": [_vp, _i32, _i64, _i64, _vp, _vp],
    "dpsgd_current": [_vp, ctypes.POINTER(_vp)],
    "dpsgd_set_gamma": [_vp, _f32],
    "dpsgd_mix_kind": [_vp, _i32, ctypes.POINTER(_i32)],
    "dpsgd_launch_count": [_vp, ctypes.POINTER(_i64)],
    "dpsgd_last_error": [_vp],
}

_lib = None


class DpsgdError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES[status] if 0 <= status < 8 else status}: {message}")
        self.status = status


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Loads libdpsgd.so (built in-tree by `python -m paper_1705_09056_b200.build`)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or LIB_PATH
    if not os.path.exists(p):
        raise DpsgdError(ERR_STATE, f"{p} not found: build it with paper_1705_09056_b200/build.py "
                                    "(there is no CPU fallback)")
    lib = ctypes.CDLL(p)
    for name, argtypes in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.argtypes = argtypes
        fn.restype = ctypes.c_char_p if name == "dpsgd_last_error" else ctypes.c_int32
    if path is None:
        _lib = lib
    return lib


def _ptr(t) -> int:
    if t is None:
        return 0
    if isinstance(t, torch.Tensor):
        return t.data_ptr()
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return int(t)


NOALLOC_MAX_LD = 67108864


def consensus_dist_noalloc(X: torch.Tensor, N: int, out: torch.Tensor, stream=None) -> torch.Tensor:
    """sum_i ||xbar - x_i||^2 of the rows of X (n x ld, columns [N, ld) zero) into the one-element
    float64 CUDA tensor `out`, without any allocation inside the library: for callers that own
    all device memory themselves or have no context.  Asynchronous on the stream; see
    dpsgd_consensus_dist_noalloc in include/dpsgd.h for the size limit and the shared scratch."""
    lib = load_library()
    assert X.is_cuda and X.dtype == torch.float32 and X.is_contiguous() and X.dim() == 2
    assert out.is_cuda and out.dtype == torch.float64 and out.numel() == 1
    s = stream if stream is not None else torch.cuda.current_stream(X.device)
    with torch.cuda.device(X.device):
        st = lib.dpsgd_consensus_dist_noalloc(_ptr(X), X.shape[0], N, X.shape[1], s.cuda_stream, _ptr(out))
    if st != OK:
        raise DpsgdError(st, lib.dpsgd_last_error(None).decode())
    return out


class Dpsgd:
    """One D-PSGD context: n nodes with N parameters each, mixing matrix W (host CSR)."""

    def __init__(self, n: int, N: int, row_ptr, col_idx, val, gamma: float, seed: int = 0):
        self._lib = load_library()
        self._h = _vp()
        rp = np.ascontiguousarray(row_ptr, dtype=np.int32)
        ci = np.ascontiguousarray(col_idx, dtype=np.int32)
        va = np.ascontiguousarray(val, dtype=np.float32)
        st = self._lib.dpsgd_create(ctypes.byref(self._h), n, N, rp.ctypes.data, ci.ctypes.data,
                                    va.ctypes.data, gamma, seed)
        if st != OK:
            msg = self._lib.dpsgd_last_error(None).decode()
            self._h = _vp()
            raise DpsgdError(st, msg)
        self.n, self.N, self.gamma, self.seed = n, N, gamma, seed
        self._keep = []       # tensors bound to the context stay referenced here
        self._data_keep = []

    # -- plumbing --------------------------------------------------------------------------
    def _check(self, st: int):
        if st != OK:
            raise DpsgdError(st, self._lib.dpsgd_last_error(self._h).decode())

    def close(self):
        if getattr(self, "_h", None) is not None and self._h.value:
            self._lib.dpsgd_destroy(self._h)
            self._h = _vp()
        self._keep, self._data_keep = [], []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C ABI, one method per entry point --------------------------------------------
    def bind(self, X0: torch.Tensor, X1: torch.Tensor, G: torch.Tensor, stream=None):
        for t in (X0, X1, G):
            assert t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.dim() == 2
            assert t.shape == X0.shape
        s = stream if stream is not None else torch.cuda.current_stream(X0.device)
        self._check(self._lib.dpsgd_bind(self._h, _ptr(X0), _ptr(X1), _ptr(G), X0.shape[1],
                                         s.cuda_stream))
        self._keep = [X0, X1, G, s]
        self.ld = X0.shape[1]

    def bind_raw(self, X0: int, X1: int, G: int, ld: int, stream: int = 0):
        """Binds raw addresses (for argument-checking tests)."""
        self._check(self._lib.dpsgd_bind(self._h, X0, X1, G, ld, stream))

    def set_model(self, kind: int, dims: Sequence[int], l2_lambda: float = 0.0, batch: int = 1,
                  mlp_precision: int = 0):
        d = np.ascontiguousarray(dims, dtype=np.int32)
        self._check(self._lib.dpsgd_set_model(self._h, kind, d.ctypes.data, len(d), l2_lambda, batch,
                                              mlp_precision))
        self.batch = batch

    def set_data(self, A: torch.Tensor, y: torch.Tensor):
        assert A.is_cuda and A.dtype == torch.float32 and A.is_contiguous() and A.dim() == 3
        assert y.is_cuda and y.is_contiguous() and y.dtype in (torch.float32, torch.int32)
        assert y.shape == A.shape[:2] and A.shape[0] == self.n
        self._check(self._lib.dpsgd_set_data(self._h, _ptr(A), _ptr(y), A.shape[1], A.shape[2]))
        self._data_keep = [A, y]

    def sample(self, k: int, idx: Optional[torch.Tensor] = None) -> torch.Tensor:
        if idx is None:
            idx = torch.empty((self.n, self.batch), dtype=torch.int32, device=self._data_keep[0].device)
        self._check(self._lib.dpsgd_sample(self._h, k, _ptr(idx)))
        return idx

    def grad(self, k: int):
        self._check(self._lib.dpsgd_grad(self._h, k))

    def mix_update(self):
        self._check(self._lib.dpsgd_mix_update(self._h))

    def step(self, k: int):
        self._check(self._lib.dpsgd_step(self._h, k))

    def local_step(self, k: int):
        """Gradient step without communication (several minibatches between exchanges)."""
        self._check(self._lib.dpsgd_local_step(self._h, k))

    def local_step_nodes(self, k: int, active):
        """The local step for the nodes with a non-zero entry of `active` (length n) only."""
        arr = (ctypes.c_int32 * self.n)(*[1 if a else 0 for a in active])
        self._check(self._lib.dpsgd_local_step_nodes(self._h, k, arr))

    def set_node_batches(self, sizes):
        """Per-node minibatch sizes B_i <= batch (length n), or None for the common size."""
        if sizes is None:
            self._check(self._lib.dpsgd_set_node_batches(self._h, None))
            return
        arr = (ctypes.c_int32 * self.n)(*[int(b) for b in sizes])
        self._check(self._lib.dpsgd_set_node_batches(self._h, arr))

    def set_order(self, update_then_mix: bool):
        """Footnote c of Algorithm 1: apply the local gradient first, then average."""
        self._check(self._lib.dpsgd_set_order(self._h, 1 if update_then_mix else 0))

    def set_fused_step(self, mode: int):
        """MLP: let step() apply the gossip step inside the weight-gradient kernels (those blocks of G
        are then not written).  0 off, 1 where it is faster, 2 wherever the kernel applies."""
        self._check(self._lib.dpsgd_set_fused_step(self._h, int(mode)))

    def set_momentum(self, beta: float, V: Optional[torch.Tensor]):
        """Heavy-ball momentum (Section 5.3): V is an n x ld fp32 CUDA tensor, zero at the start; None = off."""
        if V is not None:
            assert V.is_cuda and V.dtype == torch.float32 and V.is_contiguous() and V.shape == self._keep[0].shape
        self._check(self._lib.dpsgd_set_momentum(self._h, beta, _ptr(V)))
        self._momentum_keep = V

    def mix_update_consensus(self, out: torch.Tensor):
        """Gossip step that also writes the new consensus distance into `out` (one float64 on the device)."""
        assert out.is_cuda and out.dtype == torch.float64 and out.numel() >= 1
        self._check(self._lib.dpsgd_mix_update_consensus(self._h, _ptr(out)))

    def step_consensus(self, k: int, out: torch.Tensor):
        assert out.is_cuda and out.dtype == torch.float64 and out.numel() >= 1
        self._check(self._lib.dpsgd_step_consensus(self._h, k, _ptr(out)))

    def run(self, k_first: int, iterations: int):
        """Iterations k_first .. k_first + iterations - 1 of Algorithm 1, enqueued by one call."""
        self._check(self._lib.dpsgd_run(self._h, k_first, iterations))

    def consensus_dist(self) -> float:
        out = ctypes.c_double()
        self._check(self._lib.dpsgd_consensus_dist(self._h, ctypes.byref(out)))
        return out.value

    def sync(self):
        """Waits for the bound stream; raises ERR_TIMEOUT if a kernel's bounded wait ran out meanwhile."""
        self._check(self._lib.dpsgd_sync(self._h))

    def selftest_wait(self, max_polls: int = 4096):
        """Enqueues the self-test CTA whose wait runs out (see dpsgd_selftest_wait)."""
        self._check(self._lib.dpsgd_selftest_wait(self._h, max_polls))

    def conv3x3_forward(self, x: torch.Tensor, c_out: int, stride: int, w_off: int, b_off: int, relu: bool = True,
                        out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """3x3 convolution (padding 1) of x [n][B][C][H][W] with every node's own filters, read from the
        current X at columns w_off (filters) and b_off (biases)."""
        assert x.is_cuda and x.dtype == torch.float32 and x.is_contiguous() and x.dim() == 5 and x.shape[0] == self.n
        _, B, C, H, W = x.shape
        ho, wo = (H - 1) // stride + 1, (W - 1) // stride + 1
        if out is None:
            out = torch.empty((self.n, B, c_out, ho, wo), dtype=torch.float32, device=x.device)
        assert out.is_cuda and out.is_contiguous() and tuple(out.shape) == (self.n, B, c_out, ho, wo)
        self._check(self._lib.dpsgd_conv3x3_forward(self._h, _ptr(x), B, C, H, W, c_out, stride, w_off, b_off,
                                                    1 if relu else 0, _ptr(out)))
        return out

    def conv3x3_backward(self, x: torch.Tensor, y: Optional[torch.Tensor], dy: torch.Tensor, stride: int, w_off: int,
                         b_off: int, relu: bool = True, want_dx: bool = True) -> Optional[torch.Tensor]:
        """Backward of conv3x3_forward: filter and bias gradients (sums over the minibatch) into the bound G at
        columns w_off / b_off; returns the gradient at the layer's input (None when want_dx is False)."""
        assert x.is_cuda and x.is_contiguous() and dy.is_cuda and dy.is_contiguous() and x.dim() == 5 and dy.dim() == 5
        _, B, C, H, W = x.shape
        c_out = dy.shape[2]
        dx = torch.empty_like(x) if want_dx else None
        self._check(self._lib.dpsgd_conv3x3_backward(self._h, _ptr(x), _ptr(y), _ptr(dy), B, C, H, W, c_out, stride,
                                                     w_off, b_off, 1 if relu else 0, _ptr(dx)))
        return dx

    def average(self, xbar: Optional[torch.Tensor] = None) -> torch.Tensor:
        if xbar is None:
            xbar = torch.empty(self.ld, dtype=torch.float32, device=self._keep[0].device)
        self._check(self._lib.dpsgd_average(self._h, _ptr(xbar)))
        return xbar

    def mix_update_host(self, G_host, ld_host: Optional[int] = None) -> float:
        out = ctypes.c_double()
        if ld_host is None:
            ld_host = G_host.shape[1]
        self._check(self._lib.dpsgd_mix_update_host(self._h, _ptr(G_host), ld_host, ctypes.byref(out)))
        return out.value

    def current(self) -> torch.Tensor:
        p = _vp()
        self._check(self._lib.dpsgd_current(self._h, ctypes.byref(p)))
        for t in self._keep[:2]:
            if t.data_ptr() == p.value:
                return t
        raise DpsgdError(ERR_STATE, "current buffer is not one of the bound tensors")

    def set_gamma(self, gamma: float):
        self._check(self._lib.dpsgd_set_gamma(self._h, gamma))
        self.gamma = gamma

    def mix_kind(self, force: int = -1) -> int:
        out = _i32()
        self._check(self._lib.dpsgd_mix_kind(self._h, force, ctypes.byref(out)))
        return out.value

    def launch_count(self) -> int:
        out = _i64()
        self._check(self._lib.dpsgd_launch_count(self._h, ctypes.byref(out)))
        return out.value
