"""Helpers shared by the GPU parity tests: build a context from numpy inputs, compare rows."""
import numpy as np
import torch

from paper_1705_09056_b200 import binding, workloads as wl

TOL_STEP = 1e-5        # per-step relative tolerance in fp32 (row-wise 2-norm)
TOL_TRAJ = 1e-3        # free-running trajectory after T steps
TOL_AVG = 1e-4         # node average


def row_rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    """max_i ||got_i - ref_i||_2 / max(||ref_i||_2, tiny)."""
    got64, ref64 = got.astype(np.float64), ref.astype(np.float64)
    num = np.linalg.norm(got64 - ref64, axis=1)
    den = np.maximum(np.linalg.norm(ref64, axis=1), 1e-30)
    return float(np.max(num / den))


class GpuRun:
    """Device buffers + context for one run; X/G given as numpy n x N (no padding)."""

    def __init__(self, n, N, csr, gamma, seed=0, X=None, canary=True):
        self.n, self.N, self.ld = n, N, wl.padded_ld(N)
        dev = torch.device("cuda:0")
        # one allocation with canary pads between and after the three matrices
        pad = 64
        rows = self.n * self.ld
        self.flat = torch.full((3 * (rows + pad) + pad,), 12345.0, dtype=torch.float32, device=dev)
        base = pad
        self.bufs = []
        for t in range(3):
            self.bufs.append(self.flat[base: base + rows].view(self.n, self.ld))
            base += rows + pad
        for b in self.bufs:
            b.zero_()
        self.X0, self.X1, self.G = self.bufs
        if X is not None:
            self.X0[:, :N] = torch.from_numpy(np.ascontiguousarray(X, dtype=np.float32)).to(dev)
        self.ctx = binding.Dpsgd(n, N, *csr, gamma=gamma, seed=seed)
        self.ctx.bind(self.X0, self.X1, self.G)

    def set_g(self, G):
        self.G[:, :self.N] = torch.from_numpy(np.ascontiguousarray(G, dtype=np.float32)).to(self.G.device)

    def x(self) -> np.ndarray:
        return self.ctx.current()[:, :self.N].cpu().numpy()

    def g(self) -> np.ndarray:
        return self.G[:, :self.N].cpu().numpy()

    def check_pads(self):
        """Canaries around the buffers untouched, padding columns still zero."""
        torch.cuda.synchronize()
        mask = torch.ones_like(self.flat, dtype=torch.bool)
        for b in self.bufs:
            off = (b.data_ptr() - self.flat.data_ptr()) // 4
            mask[off: off + b.numel()] = False
        assert bool(torch.all(self.flat[mask] == 12345.0)), "write outside the bound buffers"
        if self.ld > self.N:
            assert float(self.ctx.current()[:, self.N:].abs().max()) == 0.0, "padding of X not zero"

    def close(self):
        self.ctx.close()


GATE_REL = 4e-6   # pre-activations within this (relative to the sum of |terms|) may round either way in fp32


def mlp_oracle_grad_matching_gates(orc, o, k, G_gpu):
    """The oracle's MLP gradients for iteration k.  A hidden unit whose fp64 pre-activation is
    within fp32 rounding of zero has two valid ReLU' decisions; for those units (and only
    those) the decision that brings the oracle closer to the GPU result is taken, one unit at a
    time.  Everything else is the oracle's own fp64 arithmetic."""
    idx = o.sample(k)
    G = np.empty((o.n, o.N), dtype=np.float32)
    flips = 0
    for i in range(o.n):
        args = (o.X[i], o.dims, o.A[i], o.y[i], idx[i])
        ties = orc.mlp_near_zero_gates(o.X[i], o.dims, o.A[i], idx[i], GATE_REL)
        assert len(ties) <= 64, "too many near-zero pre-activations for a meaningful comparison"
        chosen = []
        best = orc.grad_mlp(*args).astype(np.float32)
        best_err = np.linalg.norm(best.astype(np.float64) - G_gpu[i])
        for t in ties:
            cand = orc.grad_mlp(*args, flip=chosen + [t]).astype(np.float32)
            err = np.linalg.norm(cand.astype(np.float64) - G_gpu[i])
            if err < best_err:
                best, best_err, chosen = cand, err, chosen + [t]
        flips += len(chosen)
        G[i] = best
    return G, flips
