"""CPU oracle for D-PSGD (Lian et al., arXiv 1705.09056).  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 restatement of what the hot path computes, written from the paper so
that it can be checked against it by eye.  It shares no code with the CUDA library and
neither imports the other.  Only tests, the smoke check and the benchmark's CPU-baseline
leg may call it; the product path never does.

State is held the way the CUDA side holds it: the n local models x_{k,i} are the rows of an
n x N fp32 matrix (the paper's X_k in R^{N x n}, transposed; W is symmetric so
X_k W  <->  W X_k^T).  Arithmetic is fp64 on the fp32 state, with one rounding to fp32 per
stored value.

Pins (see tests/test_oracle_*.py):
  philox4x32_10 ......... bijectivity of the round, cuRAND host generator (library routine)
  sample_indices ........ range, chi-square uniformity, distinct (k, i) streams
  grad_* ................ central finite differences of the fp64 losses; torch.autograd (MLP);
                          textbook one-sample logistic formula
  mix_update ............ brute-force dense W @ X, mean preservation, sqrt(rho) contraction,
                          W = I, gamma = 0, closed-form ring spectrum
  consensus_dist ........ ||X||_F^2 - n ||xbar||^2 identity, zero at identical rows
  momentum .............. beta = 0 reduces to mix_update; constant-gradient closed form
  step / run ............ least-squares gradient descent closed form; dense-W reduction to
                          centralized minibatch SGD
  MLP trajectories ...... parity unpinned beyond the per-step pins above (non-convex, no
                          closed form)
"""
from __future__ import annotations

import numpy as np

MODEL_LSQ = 0
MODEL_LOGISTIC = 1
MODEL_MLP = 2

# ------------------------------------------------------------------------------------------
# Algorithm 1 step 2: every node draws xi_{k,i} from its own local data.
# The paper fixes no generator; this implementation uses the counter-based Philox4x32-10 of Salmon,
# Moraes, Dror and Shaw (SC'11), keyed by the run seed, with the counter holding
# (draw block, node, iteration).
# ------------------------------------------------------------------------------------------

_PHILOX_M0 = np.uint64(0xD2511F53)
_PHILOX_M1 = np.uint64(0xCD9E8D57)
_PHILOX_W0 = np.uint64(0x9E3779B9)   # golden ratio
_PHILOX_W1 = np.uint64(0xBB67AE85)   # sqrt(3) - 1
_MASK32 = np.uint64(0xFFFFFFFF)
_SH32 = np.uint64(32)


def philox_round(c, k):
    """One Philox4x32 round on counters c (4 arrays of uint64 holding 32-bit words)."""
    p0 = _PHILOX_M0 * c[0]
    p1 = _PHILOX_M1 * c[2]
    hi0, lo0 = p0 >> _SH32, p0 & _MASK32
    hi1, lo1 = p1 >> _SH32, p1 & _MASK32
    return [hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0]


def philox4x32_10(c0, c1, c2, c3, k0, k1):
    """Philox4x32 with 10 rounds.  All arguments broadcastable integer arrays of 32-bit
    words; returns four uint32 arrays."""
    c = [np.asarray(v, dtype=np.uint64) & _MASK32 for v in np.broadcast_arrays(c0, c1, c2, c3)]
    k = [np.asarray(k0, dtype=np.uint64) & _MASK32, np.asarray(k1, dtype=np.uint64) & _MASK32]
    for r in range(10):
        if r > 0:
            k = [(k[0] + _PHILOX_W0) & _MASK32, (k[1] + _PHILOX_W1) & _MASK32]
        c = philox_round(c, k)
    return [v.astype(np.uint32) for v in c]


def sample_indices(seed: int, k: int, n: int, B: int, m: int) -> np.ndarray:
    """Minibatch indices of every node for iteration k: int32 [n][B], i.i.d. uniform on
    [0, m) with replacement (Algorithm 1 step 2 with the minibatch of footnote a).

    Draw b of node i uses word (b mod 4) of philox(counter = (b div 4, i, k_lo, k_hi),
    key = (seed_lo, seed_hi)) and maps the 32-bit word u to floor(u * m / 2^32).
    """
    assert 0 < m < 2 ** 31
    blocks = np.arange((B + 3) // 4, dtype=np.uint64)[None, :]
    node = np.arange(n, dtype=np.uint64)[:, None]
    words = philox4x32_10(blocks, node, k & 0xFFFFFFFF, (k >> 32) & 0xFFFFFFFF,
                          seed & 0xFFFFFFFF, (seed >> 32) & 0xFFFFFFFF)
    # [n][block][word] flattened: draw b sits at position 4*(b div 4) + (b mod 4)
    u = np.stack(words, axis=-1).reshape(n, -1)[:, :B].astype(np.uint64)
    return ((u * np.uint64(m)) >> _SH32).astype(np.int32)


# ------------------------------------------------------------------------------------------
# Algorithm 1 step 3: the local stochastic gradient at the node's own x_{k,i} (minibatch mean,
# footnote a).  One node at a time; x is that node's fp32 parameter row.
# ------------------------------------------------------------------------------------------

def loss_lsq(x, A, y, idx):
    """(1/B) sum_b 1/2 (a_b . x - y_b)^2 in fp64."""
    a = A[idx].astype(np.float64)
    r = a @ np.asarray(x, dtype=np.float64) - y[idx].astype(np.float64)
    return 0.5 * np.mean(r * r)


def grad_lsq(x, A, y, idx):
    a = A[idx].astype(np.float64)
    r = a @ np.asarray(x, dtype=np.float64) - y[idx].astype(np.float64)
    return (r @ a) / len(idx)


def loss_logistic(x, A, y, idx, lam):
    """(1/B) sum_b log(1 + exp(-y_b (a_b . w + bias))) + lam/2 |w|^2, x = [w | bias]."""
    x = np.asarray(x, dtype=np.float64)
    w, bias = x[:-1], x[-1]
    z = A[idx].astype(np.float64) @ w + bias
    yy = y[idx].astype(np.float64)
    return np.mean(np.logaddexp(0.0, -yy * z)) + 0.5 * lam * np.dot(w, w)


def grad_logistic(x, A, y, idx, lam):
    x = np.asarray(x, dtype=np.float64)
    w, bias = x[:-1], x[-1]
    a = A[idx].astype(np.float64)
    yy = y[idx].astype(np.float64)
    z = a @ w + bias
    s = 1.0 / (1.0 + np.exp(yy * z))          # sigma(-y z)
    coef = -yy * s / len(idx)
    g = np.empty_like(x)
    g[:-1] = coef @ a + lam * w               # no penalty on the bias
    g[-1] = np.sum(coef)
    return g


def _mlp_views(x, dims):
    off = 0
    Ws, bs = [], []
    for l in range(len(dims) - 1):
        o, i = dims[l + 1], dims[l]
        Ws.append(x[off: off + o * i].reshape(o, i)); off += o * i
        bs.append(x[off: off + o]); off += o
    assert off == x.shape[0]
    return Ws, bs


def _mlp_forward(x, dims, A, idx):
    Ws, bs = _mlp_views(np.asarray(x, dtype=np.float64), dims)
    h = [A[idx].astype(np.float64)]
    pre = []
    for l in range(len(Ws)):
        z = h[-1] @ Ws[l].T + bs[l]
        pre.append(z)
        h.append(np.maximum(z, 0.0) if l + 1 < len(Ws) else z)
    return Ws, h, pre


def loss_mlp(x, dims, A, labels, idx):
    """Mean softmax cross-entropy of a ReLU MLP; x = [W_1 | b_1 | W_2 | b_2 | ...]."""
    _, h, _ = _mlp_forward(x, dims, A, idx)
    z = h[-1] - np.max(h[-1], axis=1, keepdims=True)
    logp = z - np.log(np.sum(np.exp(z), axis=1, keepdims=True))
    return -np.mean(logp[np.arange(len(idx)), labels[idx]])


def mlp_near_zero_gates(x, dims, A, idx, rel):
    """Hidden units whose pre-activation z is so close to 0 that fp32 rounding may put it on the
    other side: |z| <= rel * (|h_{l-1}| |W_l|^T + |b_l|).  Returns [(layer l, sample b, unit)] with
    l the 0-based index of the weight layer producing the unit.  For such a unit ReLU'(z) = 0 and
    ReLU'(z) = 1 are both results a correct fp32 implementation can reach."""
    Ws, h, pre = _mlp_forward(x, dims, A, idx)
    _, bs = _mlp_views(np.asarray(x, dtype=np.float64), dims)
    out = []
    for l in range(len(Ws) - 1):
        bound = np.abs(h[l]) @ np.abs(Ws[l]).T + np.abs(bs[l])
        for b, u in np.argwhere(np.abs(pre[l]) <= rel * bound):
            out.append((l, int(b), int(u)))
    return out


def grad_mlp(x, dims, A, labels, idx, flip=()):
    """Minibatch-mean gradient by back-propagation, ReLU'(0) = 0.  `flip` lists (layer, sample,
    unit) gates from mlp_near_zero_gates whose ReLU' decision is inverted (test use only)."""
    B = len(idx)
    Ws, h, pre = _mlp_forward(x, dims, A, idx)
    gates = [p > 0.0 for p in pre[:-1]]
    for (l, b, u) in flip:
        gates[l][b, u] = ~gates[l][b, u]
    z = h[-1] - np.max(h[-1], axis=1, keepdims=True)
    p = np.exp(z)
    p /= np.sum(p, axis=1, keepdims=True)
    delta = p
    delta[np.arange(B), labels[idx]] -= 1.0
    delta /= B
    parts = [None] * len(Ws)
    for l in range(len(Ws) - 1, -1, -1):
        parts[l] = (delta.T @ h[l], np.sum(delta, axis=0))
        if l > 0:
            delta = (delta @ Ws[l]) * gates[l - 1]
    return np.concatenate([np.concatenate([gw.reshape(-1), gb]) for gw, gb in parts])


def gradients(X, model, dims, A, y, idx, lam=0.0):
    """All n local gradients at the nodes' own rows: fp32 [n][N] (the paper's dF(X_k; xi_k))."""
    n = X.shape[0]
    G = np.empty(X.shape, dtype=np.float32)
    for i in range(n):
        if model == MODEL_LSQ:
            g = grad_lsq(X[i], A[i], y[i], idx[i])
        elif model == MODEL_LOGISTIC:
            g = grad_logistic(X[i], A[i], y[i], idx[i], lam)
        elif model == MODEL_MLP:
            g = grad_mlp(X[i], dims, A[i], y[i], idx[i])
        else:
            raise ValueError(model)
        G[i] = g.astype(np.float32)
    return G


# ------------------------------------------------------------------------------------------
# Algorithm 1 steps 4-5 / the global form X_{k+1} = X_k W - gamma dF(X_k; xi_k).
# ------------------------------------------------------------------------------------------

def mix_update(X, G, row_ptr, col, val, gamma):
    """x_{k+1,i} = sum_j W_ij x_{k,j} - gamma g_i for every node; W in CSR with fp32 values.

    fp64 accumulation in CSR order, one rounding to fp32."""
    n = X.shape[0]
    g64 = np.float64(np.float32(gamma))
    out = np.empty_like(X, dtype=np.float32)
    for i in range(n):
        acc = np.zeros(X.shape[1], dtype=np.float64)
        for p in range(int(row_ptr[i]), int(row_ptr[i + 1])):
            acc += np.float64(val[p]) * X[int(col[p])].astype(np.float64)
        acc -= g64 * G[i].astype(np.float64)
        out[i] = acc.astype(np.float32)
    return out


def mix_update_swapped(X, G, row_ptr, col, val, gamma):
    """Footnote c of Algorithm 1: update locally first, then average:
    x_{k+1,i} = sum_j W_ij (x_{k,j} - gamma g_j)."""
    n = X.shape[0]
    g64 = np.float64(np.float32(gamma))
    out = np.empty_like(X, dtype=np.float32)
    for i in range(n):
        acc = np.zeros(X.shape[1], dtype=np.float64)
        for p in range(int(row_ptr[i]), int(row_ptr[i + 1])):
            j = int(col[p])
            acc += np.float64(val[p]) * (X[j].astype(np.float64) - g64 * G[j].astype(np.float64))
        out[i] = acc.astype(np.float32)
    return out


def momentum_buffer(V, G, beta):
    """Heavy-ball momentum of the Torch runs of Section 5.3 (learning rate 0.1, momentum 0.9), kept
    per node: v_{k+1,i} = beta v_{k,i} + g_i.  fp64 arithmetic, one rounding to fp32."""
    b64 = np.float64(np.float32(beta))
    return (b64 * V.astype(np.float64) + G.astype(np.float64)).astype(np.float32)


def mix_update_momentum(X, V, G, row_ptr, col, val, gamma, beta, swapped=False):
    """D-PSGD iteration with the momentum buffer in place of the raw gradient:
    V' = beta V + G, then X' = W X - gamma V' (or W (X - gamma V') in footnote c's order).
    Returns (X', V')."""
    Vn = momentum_buffer(V, G, beta)
    f = mix_update_swapped if swapped else mix_update
    return f(X, Vn, row_ptr, col, val, gamma), Vn


def node_average(X):
    """Output of Algorithm 1: (1/n) sum_i x_{K,i}, fp64."""
    return np.mean(X.astype(np.float64), axis=0)


def consensus_dist(X):
    """sum_i || xbar - x_i ||^2 = sum_i Q_{k,i} (Eq. 10); M_k of Eq. 13 is this over n."""
    X64 = X.astype(np.float64)
    d = X64 - np.mean(X64, axis=0, keepdims=True)
    return float(np.sum(d * d))


def spectral_rho(W):
    """rho = (max(|lambda_2|, |lambda_n|))^2 of Assumption 1-2, from a symmetric eigen-solve."""
    ev = np.sort(np.abs(np.linalg.eigvalsh(np.asarray(W, dtype=np.float64))))
    return float(ev[-2] ** 2) if len(ev) > 1 else 0.0


def cpsgd_step(x, grads, gamma):
    """Centralized PSGD: one model, the n nodes' gradients averaged (minibatch SGD with n
    gradients per step, Section 2 / Table 1)."""
    g64 = np.float64(np.float32(gamma))
    return (np.asarray(x, dtype=np.float64)
            - g64 * np.mean(np.asarray(grads, dtype=np.float64), axis=0)).astype(np.float32)


# ------------------------------------------------------------------------------------------
# Whole iteration
# ------------------------------------------------------------------------------------------

class Oracle:
    """Algorithm 1 run for all n nodes at once on the CPU."""

    def __init__(self, n, N, row_ptr, col, val, gamma, seed, model=None, dims=(), batch=0,
                 lam=0.0, A=None, y=None, swapped=False):
        self.n, self.N = n, N
        self.row_ptr, self.col, self.val = (np.asarray(row_ptr), np.asarray(col),
                                            np.asarray(val, dtype=np.float32))
        self.gamma, self.seed = gamma, seed
        self.model, self.dims, self.batch, self.lam = model, tuple(dims), batch, lam
        self.A, self.y = A, y
        self.swapped = swapped
        self.X = np.zeros((n, N), dtype=np.float32)

    def set_x(self, X):
        self.X = np.array(X, dtype=np.float32).reshape(self.n, self.N)

    def sample(self, k):
        return sample_indices(self.seed, k, self.n, self.batch, self.A.shape[1])

    def grad(self, k):
        return gradients(self.X, self.model, self.dims, self.A, self.y, self.sample(k), self.lam)

    def mix_update(self, G):
        f = mix_update_swapped if self.swapped else mix_update
        self.X = f(self.X, G, self.row_ptr, self.col, self.val, self.gamma)
        return self.X

    def step(self, k):
        return self.mix_update(self.grad(k))

    def consensus_dist(self):
        return consensus_dist(self.X)
