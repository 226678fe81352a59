"""Seeded synthetic inputs for D-PSGD runs: mixing matrices, datasets, initial points.

This module only *produces inputs* (topologies as CSR, design matrices, labels, initial
parameter rows).  It contains none of the method's arithmetic (no sampling of minibatches,
no gradients, no mixing), so the same bytes can be handed both to the CUDA library and to
an independent checker.

Topologies follow Section 3 of the paper (W symmetric, doubly stochastic, W_ij in [0,1]);
the ring is the matrix printed in Theorem 3.  The 2-D torus and the dense 11^T/n matrix are
not in the paper: the torus is a degree-4 graph with weight 1/5 on self and neighbours, and
the dense matrix is the averaging step of centralized PSGD (Section 2 / Table 1).

Datasets are stand-ins for the paper's CIFAR-10 / NLC workloads (Section 5): Gaussian
designs with a planted linear model or a random "teacher" network that assigns labels.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np
import torch

MODEL_LSQ = 0
MODEL_LOGISTIC = 1
MODEL_MLP = 2


# --------------------------------------------------------------------------------------
# Mixing matrices (CSR, fp32 values, sorted unique columns per row)
# --------------------------------------------------------------------------------------

def _csr_from_rows(rows: List[Dict[int, float]]) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    row_ptr = np.zeros(len(rows) + 1, dtype=np.int32)
    cols: List[int] = []
    vals: List[float] = []
    for i, r in enumerate(rows):
        for j in sorted(r):
            cols.append(j)
            vals.append(r[j])
        row_ptr[i + 1] = len(cols)
    return row_ptr, np.asarray(cols, dtype=np.int32), np.asarray(vals, dtype=np.float32)


def ring(n: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Ring of Theorem 3: W_ii = W_{i,i-1} = W_{i,i+1} = 1/3 (indices mod n).

    For n < 3 the two neighbours coincide (or are the node itself); coinciding entries are
    summed so that rows still add up to one.
    """
    rows: List[Dict[int, float]] = []
    for i in range(n):
        r: Dict[int, float] = {}
        for j in ((i - 1) % n, i, (i + 1) % n):
            r[j] = r.get(j, 0.0) + 1.0 / 3.0
        rows.append(r)
    return _csr_from_rows(rows)


def torus2d(rows_: int, cols_: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """rows_ x cols_ torus, node id = r*cols_ + c, weight 1/5 on self and the 4 neighbours."""
    out: List[Dict[int, float]] = []
    for r in range(rows_):
        for c in range(cols_):
            d: Dict[int, float] = {}
            for (rr, cc) in ((r, c), ((r - 1) % rows_, c), ((r + 1) % rows_, c),
                             (r, (c - 1) % cols_), (r, (c + 1) % cols_)):
                j = rr * cols_ + cc
                d[j] = d.get(j, 0.0) + 1.0 / 5.0
            out.append(d)
    return _csr_from_rows(out)


def dense_uniform(n: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """W = 1 1^T / n stored as CSR with n*n entries (the C-PSGD averaging step)."""
    row_ptr = (np.arange(n + 1, dtype=np.int64) * n).astype(np.int32)
    col = np.tile(np.arange(n, dtype=np.int32), n)
    val = np.full(n * n, np.float32(1.0) / np.float32(n), dtype=np.float32)
    return row_ptr, col, val


def ring_with_antipode(n: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Ring plus one link to the farthest node (Section 5.3, 16 machines); weights 1/4. n even, n >= 6."""
    assert n % 2 == 0 and n >= 6
    rows: List[Dict[int, float]] = []
    for i in range(n):
        r: Dict[int, float] = {}
        for j in ((i - 1) % n, i, (i + 1) % n, (i + n // 2) % n):
            r[j] = r.get(j, 0.0) + 0.25
        rows.append(r)
    return _csr_from_rows(rows)


def identity(n: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    return (np.arange(n + 1, dtype=np.int32), np.arange(n, dtype=np.int32),
            np.ones(n, dtype=np.float32))


def random_symmetric_doubly_stochastic(n: int, seed: int, terms: int = 4
                                       ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Convex combination of symmetrised permutation matrices (P + P^T)/2 and the identity.

    Weights are multiples of 1/64 so that every entry and every row sum is exact in fp32.
    """
    rng = np.random.default_rng(seed)
    parts = rng.multinomial(64, np.ones(terms + 1) / (terms + 1))
    W = np.zeros((n, n), dtype=np.float64)
    W += parts[0] / 64.0 * np.eye(n)
    for t in range(terms):
        p = rng.permutation(n)
        P = np.zeros((n, n))
        P[np.arange(n), p] = 1.0
        W += parts[t + 1] / 64.0 * 0.5 * (P + P.T)
    return dense_to_csr(W)


def dense_to_csr(W: np.ndarray) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    n = W.shape[0]
    rows = [{int(j): float(W[i, j]) for j in range(n) if W[i, j] != 0.0} for i in range(n)]
    return _csr_from_rows(rows)


def csr_to_dense(n: int, row_ptr, col, val) -> np.ndarray:
    W = np.zeros((n, n), dtype=np.float64)
    for i in range(n):
        for p in range(int(row_ptr[i]), int(row_ptr[i + 1])):
            W[i, int(col[p])] += float(val[p])
    return W


def topology(name: str, n: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    if name == "ring":
        return ring(n)
    if name == "dense":
        return dense_uniform(n)
    if name == "torus":
        s = int(round(math.sqrt(n)))
        assert s * s == n, "torus needs a square node count"
        return torus2d(s, s)
    if name == "ring+antipode":
        return ring_with_antipode(n)
    if name == "identity":
        return identity(n)
    raise ValueError(name)


# --------------------------------------------------------------------------------------
# Model shapes
# --------------------------------------------------------------------------------------

def mlp_param_count(dims: Sequence[int]) -> int:
    """Row layout [W_1 (out x in, row-major) | b_1 | W_2 | b_2 | ...]."""
    return sum(dims[l + 1] * dims[l] + dims[l + 1] for l in range(len(dims) - 1))


def padded_ld(N: int) -> int:
    """Leading dimension of the stacked matrices: N rounded up to 32 floats (128 bytes)."""
    return (N + 31) // 32 * 32


# --------------------------------------------------------------------------------------
# Workloads
# --------------------------------------------------------------------------------------

@dataclass
class Workload:
    """Everything one D-PSGD run needs, as torch tensors on one device (fp32 / int32)."""
    name: str
    n: int
    N: int
    topology: str
    gamma: float
    iterations: int
    model: Optional[int] = None          # MODEL_* or None when gradients are supplied
    dims: Tuple[int, ...] = ()           # lsq/logistic: (d,), mlp: layer widths
    batch: int = 0
    l2_lambda: float = 0.0
    m_per_node: int = 0
    A: Optional[torch.Tensor] = None     # [n][m][d] fp32
    y: Optional[torch.Tensor] = None     # [n][m] fp32 targets/labels(+-1) or int32 classes
    x0: Optional[torch.Tensor] = None    # [N] fp32, shared by all nodes (Algorithm 1 input)
    extra: Dict[str, object] = field(default_factory=dict)

    @property
    def ld(self) -> int:
        return padded_ld(self.N)

    def csr(self):
        return topology(self.topology, self.n)


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _randn(shape, g: torch.Generator, device) -> torch.Tensor:
    return torch.randn(shape, generator=g, device=device, dtype=torch.float32)


def _he_init_row(dims: Sequence[int], g: torch.Generator, device) -> torch.Tensor:
    parts = []
    for l in range(len(dims) - 1):
        fan_in, fan_out = dims[l], dims[l + 1]
        parts.append((_randn((fan_out, fan_in), g, device) * math.sqrt(2.0 / fan_in)).reshape(-1))
        parts.append(torch.zeros(fan_out, device=device, dtype=torch.float32))
    return torch.cat(parts)


def _teacher_labels(inputs: torch.Tensor, dims: Sequence[int], g: torch.Generator, device,
                    chunk: int = 8192) -> torch.Tensor:
    """Classes assigned by a fixed random network of the same widths (argmax of its logits)."""
    Ws = [_randn((dims[l + 1], dims[l]), g, device) * math.sqrt(2.0 / dims[l])
          for l in range(len(dims) - 1)]
    flat = inputs.reshape(-1, dims[0])
    out = torch.empty(flat.shape[0], dtype=torch.int32, device=device)
    for s in range(0, flat.shape[0], chunk):
        h = flat[s:s + chunk].double()
        for l, Wl in enumerate(Ws):
            h = h @ Wl.double().T
            if l + 1 < len(Ws):
                h = torch.relu(h)
        out[s:s + chunk] = torch.argmax(h, dim=1).to(torch.int32)
    return out.reshape(inputs.shape[:-1])


def lsq_workload(n=8, d=64, m=1024, batch=16, gamma=0.05, iterations=200, noise=0.1,
                 topology="ring", seed=170509056, device="cpu") -> Workload:
    """Least squares with a planted w*: y = a.w* + noise*N(0,1); all nodes start at 0."""
    g = _gen(device, seed)
    w_star = _randn((d,), g, device)
    A = _randn((n, m, d), g, device)
    y = (A.double() @ w_star.double()).float() + noise * _randn((n, m), g, device)
    return Workload("lsq", n, d, topology, gamma, iterations, MODEL_LSQ, (d,), batch, 0.0, m,
                    A.contiguous(), y.contiguous(), torch.zeros(d, device=device),
                    {"w_star": w_star})


def logistic_workload(n=16, d=4096, m=65536, batch=128, gamma=0.1, iterations=1000,
                      l2_lambda=1e-4, noise=0.5, topology="ring", seed=170509057,
                      device="cpu") -> Workload:
    """L2-regularised logistic regression, labels +-1 = sign(a.w* + noise*N(0,1)) (+1 at 0).

    Samples are i.i.d. from one distribution on every node (a shared, shuffled database).
    Parameters are [w (d) | bias]; nodes start at 0.
    """
    g = _gen(device, seed)
    w_star = _randn((d,), g, device)
    A = torch.empty((n, m, d), device=device, dtype=torch.float32)
    y = torch.empty((n, m), device=device, dtype=torch.float32)
    for i in range(n):                       # node by node keeps the temporaries small
        A[i] = _randn((m, d), g, device)
        z = A[i] @ w_star + noise * _randn((m,), g, device)
        y[i] = torch.where(z >= 0, 1.0, -1.0)
    return Workload("logistic", n, d + 1, topology, gamma, iterations, MODEL_LOGISTIC, (d,),
                    batch, l2_lambda, m, A, y, torch.zeros(d + 1, device=device),
                    {"w_star": w_star})


def mlp_workload(n=32, dims=(784, 1024, 10), m=1875, batch=32, gamma=0.05, iterations=500,
                 topology="ring", seed=170509058, device="cpu") -> Workload:
    """MLP (ReLU, softmax cross-entropy); N(0,1) inputs; labels from a random teacher network;
    He-initialised parameter row shared by all nodes."""
    g = _gen(device, seed)
    A = _randn((n, m, dims[0]), g, device)
    y = _teacher_labels(A, dims, g, device)
    x0 = _he_init_row(dims, g, device)
    return Workload("mlp", n, mlp_param_count(dims), topology, gamma, iterations, MODEL_MLP,
                    tuple(dims), batch, 0.0, m, A.contiguous(), y.contiguous(), x0)


def stress_workload(n=64, N=25_000_000, gamma=0.01, iterations=50, topology="ring",
                    seed=170509059, device="cpu") -> Workload:
    """Mix+update bandwidth stress: gradients are supplied by the caller each step."""
    w = Workload("stress", n, N, topology, gamma, iterations)
    w.extra["seed"] = seed
    return w


def stress_matrix(n: int, ld: int, N: int, seed: int, device) -> torch.Tensor:
    """n x ld fp32 N(0,1) matrix whose padding columns [N, ld) are zero."""
    g = _gen(device, seed)
    M = torch.empty((n, ld), device=device, dtype=torch.float32)
    for i in range(n):
        M[i].normal_(generator=g)
    if ld > N:
        M[:, N:] = 0
    return M


# --------------------------------------------------------------------------------------
# Convolution layer family (stand-in for the paper's CIFAR-10 residual networks, Sections 5.1 / 5.3)
# --------------------------------------------------------------------------------------

# (C_in, C_out, stride) of the 3x3 convolutions: 32x32x3 inputs, widths 16 / 32 / 64, a stride-2 layer
# where the width doubles (one layer of each kind a 20- or 32-layer residual network is built from).
CIFAR_PLAN = ((3, 16, 1), (16, 16, 1), (16, 32, 2), (32, 32, 1), (32, 64, 2), (64, 64, 1))


def conv_param_count(plan) -> int:
    """Row layout [w_1 (C_out x C_in x 3 x 3, row-major) | b_1 | w_2 | b_2 | ...]."""
    return sum(o * c * 9 + o for c, o, _ in plan)


@dataclass
class ConvWorkload:
    """Per-node image minibatches and per-node filter banks (fp32 torch tensors on one device)."""
    n: int
    batch: int
    plan: Tuple[Tuple[int, int, int], ...]
    inputs: torch.Tensor       # [n][B][3][32][32], N(0,1)
    params: torch.Tensor       # [n][conv_param_count(plan)], He-scaled filters, small non-zero biases


def conv_workload(n=8, batch=32, plan=CIFAR_PLAN, hw=32, seed=170509061, device="cpu") -> ConvWorkload:
    """CIFAR-shaped synthetic inputs (3 x hw x hw, N(0,1)) and, per node, its own He-initialised filters
    (the nodes' models differ between synchronisations, so every node convolves with its own weights)."""
    g = _gen(device, seed)
    inputs = _randn((n, batch, plan[0][0], hw, hw), g, device)
    rows = []
    for _ in range(n):
        parts = []
        for (cin, cout, _) in plan:
            parts.append((_randn((cout, cin, 3, 3), g, device) * math.sqrt(2.0 / (cin * 9))).reshape(-1))
            parts.append(0.05 * _randn((cout,), g, device))
        rows.append(torch.cat(parts))
    return ConvWorkload(n, batch, tuple(tuple(p) for p in plan), inputs.contiguous(), torch.stack(rows).contiguous())


def config(idx: int, device="cpu", **over) -> Workload:
    """The five benchmark configurations (0-based)."""
    if idx == 0:
        return lsq_workload(device=device, **over)
    if idx == 1:
        return logistic_workload(device=device, **over)
    if idx == 2:
        return mlp_workload(device=device, **over)
    if idx == 3:
        return stress_workload(device=device, **over)
    if idx == 4:
        kw = dict(n=112, dims=(1024, 2048, 2048, 10), m=4096, batch=64, gamma=0.02,
                  iterations=300, seed=170509060)
        kw.update(over)
        return mlp_workload(device=device, **kw)
    raise ValueError(idx)


def stack_rows(x0: torch.Tensor, n: int, ld: int) -> torch.Tensor:
    """n identical copies of x0 as an n x ld matrix with zero padding (x_{0,i} = x_0)."""
    X = torch.zeros((n, ld), device=x0.device, dtype=torch.float32)
    X[:, : x0.numel()] = x0
    return X
