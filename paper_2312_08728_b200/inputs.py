"""Seeded synthetic inputs for buffered mini-batch gradient descent (BMGD).

This module only draws data.  It holds none of the method's arithmetic (no
shuffle, no gradient, no update) so that the CUDA path and the CPU oracle can
both be fed from it without sharing anything else.

The designs follow the simulation section of the paper (Section 4.1): Gaussian
predictors with an AR(rho) covariance, a fixed coefficient vector, Gaussian noise
for the linear model and Bernoulli-logit labels for the logistic model.  The
softmax workload (class mean plus unit noise, uniform labels) is the C-class
extension of the same recipe.  The paper's image datasets are not used; these
draws stand in for them.

Vocabulary (paper, Section 2.2): N rows in the whole sample, K buffers of N0 rows,
mini-batches of n rows, T rounds ("buffer epochs") per buffer, E passes over the
whole sample ("iterations"), Rc replicate chains, C classes.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional, Tuple

import torch

LOSS_LINEAR = 0
LOSS_LOGISTIC = 1
LOSS_SOFTMAX = 2

DTYPE_F64 = 0
DTYPE_F32 = 1
DTYPE_BF16 = 2  # bf16 rows, fp32 parameters

_TORCH_X = {DTYPE_F64: torch.float64, DTYPE_F32: torch.float32, DTYPE_BF16: torch.bfloat16}
_TORCH_THETA = {DTYPE_F64: torch.float64, DTYPE_F32: torch.float32, DTYPE_BF16: torch.float32}


@dataclasses.dataclass(frozen=True)
class Workload:
    """One BMGD job: data shape, buffering and optimisation schedule."""

    name: str
    loss: int
    dtype: int
    N: int          # rows in the whole sample
    p: int          # predictors per row
    K: int          # buffers per pass over the sample
    n: int          # mini-batch size
    T: int          # rounds per buffer
    lr: float       # learning rate alpha
    epochs: int     # passes over the whole sample
    Rc: int = 1     # replicate chains sharing the buffer
    C: int = 1      # classes (softmax only)
    rho: float = 0.0
    seed: int = 0
    design: str = ""  # "unit-signal": theta* drawn standard normal and scaled so that var(x.theta*) = 1

    @property
    def N0(self) -> int:
        return -(-self.N // self.K)

    @property
    def M(self) -> int:
        return -(-self.N0 // self.n)

    @property
    def x_dtype(self) -> torch.dtype:
        return _TORCH_X[self.dtype]

    @property
    def theta_dtype(self) -> torch.dtype:
        return _TORCH_THETA[self.dtype]

    @property
    def x_itemsize(self) -> int:
        return {DTYPE_F64: 8, DTYPE_F32: 4, DTYPE_BF16: 2}[self.dtype]

    @property
    def y_itemsize(self) -> int:
        return 4 if self.loss == LOSS_SOFTMAX else {DTYPE_F64: 8, DTYPE_F32: 4, DTYPE_BF16: 4}[self.dtype]

    @property
    def row_bytes(self) -> int:
        """Bytes of one sample as stored: the row of X plus its response."""
        return self.p * self.x_itemsize + self.y_itemsize

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


# The five synthetic jobs.  cfg1 is small enough for the oracle to finish in
# seconds; cfg2 is the replicate-chain job; cfg3 the large logistic job; cfg4 the
# image-shaped softmax job; cfg5 the host-streaming stress (T is swept by callers).
WORKLOADS = {
    "cfg1": Workload("cfg1", LOSS_LINEAR, DTYPE_F64, N=10_000, p=10, K=5, n=100, T=5, lr=0.05,
                     epochs=2, rho=0.5, seed=0),
    "cfg2": Workload("cfg2", LOSS_LINEAR, DTYPE_F32, N=1_000_000, p=100, K=10, n=1_000, T=10, lr=0.01,
                     epochs=3, Rc=64, rho=0.5, seed=0),
    "cfg3": Workload("cfg3", LOSS_LOGISTIC, DTYPE_F32, N=10_000_000, p=200, K=10, n=4_096, T=5, lr=0.5,
                     epochs=2, rho=0.0, seed=0),
    "cfg4": Workload("cfg4", LOSS_SOFTMAX, DTYPE_BF16, N=200_000, p=3_072, K=10, n=256, T=4, lr=0.1,
                     epochs=2, C=10, seed=0),
    "cfg5": Workload("cfg5", LOSS_LINEAR, DTYPE_F32, N=50_000_000, p=64, K=20, n=2_048, T=5, lr=0.01,
                     epochs=1, rho=0.5, seed=0),
    # The shape of the paper's own linear simulation (Section 4.1): N = 100,000, p = 500, Sigma = 0.8^|i-j|, unit signal
    # variance, buffers of 10,000, mini-batches of 1,000, T = 5 with alpha T = 0.01, 100 passes, 100 replicates.  Here the
    # replicates are chains over one data set with their own shuffles; the paper redraws the data for each.
    "sim41": Workload("sim41", LOSS_LINEAR, DTYPE_F32, N=100_000, p=500, K=10, n=1_000, T=5, lr=0.002,
                      epochs=100, Rc=100, rho=0.8, seed=41, design="unit-signal"),
}


def _simulation_grid():
    """The rest of the paper's linear simulation (Section 4.1), same data design as `sim41`.

    First experiment: buffers of 10,000, mini-batches of 1,000, T in {1, 5, 10} at a fixed product alpha T (0.01 here;
    T = 1 is plain MGD).  Second experiment: T = 5, n in {250, 500, 1000}, K in {2, 5} buffers, 30 passes, with the
    constant rate alpha = 0.005 (`a`) or alpha = 1/(T K M) (`b`), M = N0 / n mini-batches per buffer."""
    base = WORKLOADS["sim41"]
    out = {}
    for T in (1, 10):
        out[f"sim41-T{T}"] = dataclasses.replace(base, name=f"sim41-T{T}", T=T, lr=0.01 / T)
    for K in (2, 5):
        for n in (250, 500, 1000):
            M = (base.N // K) // n
            out[f"sim41-K{K}-n{n}-a"] = dataclasses.replace(base, name=f"sim41-K{K}-n{n}-a", K=K, n=n, T=5, lr=0.005, epochs=30)
            out[f"sim41-K{K}-n{n}-b"] = dataclasses.replace(base, name=f"sim41-K{K}-n{n}-b", K=K, n=n, T=5,
                                                            lr=1.0 / (5 * K * M), epochs=30)
    return out


WORKLOADS.update(_simulation_grid())


def buffer_seed(base_seed: int, epoch: int, k: int, K: int) -> int:
    """64-bit shuffle seed handed to the call that processes buffer k of pass `epoch`."""
    return (int(base_seed) + epoch * K + k) & 0xFFFFFFFFFFFFFFFF


def _gen(seed: int, stream: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((int(seed) * 1_000_003 + stream * 7_919 + 12_345) & 0x7FFFFFFFFFFFFFFF)
    return g


def _ar_rows(rows: int, p: int, rho: float, g: torch.Generator) -> torch.Tensor:
    """rows x p standard normal draws with covariance rho^|j-k| (fp64)."""
    z = torch.randn(rows, p, generator=g, dtype=torch.float64)
    if rho != 0.0:
        s = math.sqrt(1.0 - rho * rho)
        for j in range(1, p):
            z[:, j] = rho * z[:, j - 1] + s * z[:, j]
    return z


def theta_star(w: Workload) -> torch.Tensor:
    """True coefficients of the generating model, fp64; [p] or [p, C]."""
    if w.design == "unit-signal":
        # the paper's simulation design (Section 4.1): theta* ~ N(0, I), then scaled so that theta*' Sigma theta* = 1
        z = torch.randn(w.p, generator=_gen(w.seed, 1), dtype=torch.float64)
        idx = torch.arange(w.p, dtype=torch.float64)
        sigma = w.rho ** (idx[:, None] - idx[None, :]).abs() if w.rho != 0.0 else torch.eye(w.p, dtype=torch.float64)
        return z / torch.sqrt(z @ sigma @ z)
    if w.loss == LOSS_LINEAR:
        return torch.ones(w.p, dtype=torch.float64)
    if w.loss == LOSS_LOGISTIC:
        return torch.randn(w.p, generator=_gen(w.seed, 1), dtype=torch.float64) / math.sqrt(w.p)
    # softmax: class means play the role of the signal; there is no "true W"
    return torch.zeros(w.p, w.C, dtype=torch.float64)


def class_means(w: Workload) -> torch.Tensor:
    return 0.1 * torch.randn(w.C, w.p, generator=_gen(w.seed, 2), dtype=torch.float64)


def make_rows(w: Workload, start: int, rows: int) -> Tuple[torch.Tensor, torch.Tensor]:
    """Draw rows [start, start+rows) of the sample.

    Returns (X, y): X is [rows, p] in the workload's storage dtype; y is [rows] in
    the parameter dtype for linear/logistic and int32 class labels for softmax.
    The draw depends only on (w.seed, start, rows), so callers that always ask
    for the same blocks get the same data.
    """
    g = _gen(w.seed, 1000 + start)
    if w.loss == LOSS_SOFTMAX:
        labels = torch.randint(0, w.C, (rows,), generator=g, dtype=torch.int64)
        mu = class_means(w)
        x = torch.randn(rows, w.p, generator=g, dtype=torch.float32)
        x += mu[labels].to(torch.float32)
        return x.to(w.x_dtype).contiguous(), labels.to(torch.int32).contiguous()
    if rows * w.p > 50_000_000:
        # large draws: fp32 noise is enough, and half the memory
        x = torch.randn(rows, w.p, generator=g, dtype=torch.float32)
        if w.rho != 0.0:
            s = math.sqrt(1.0 - w.rho * w.rho)
            for j in range(1, w.p):
                x[:, j] = w.rho * x[:, j - 1] + s * x[:, j]
        x = x.to(w.x_dtype)
    else:
        x = _ar_rows(rows, w.p, w.rho, g).to(w.x_dtype)
    ts = theta_star(w)
    # the response is computed from the stored (rounded) predictors
    eta = x.to(torch.float64) @ ts
    if w.loss == LOSS_LINEAR:
        y = eta + torch.randn(rows, generator=g, dtype=torch.float64)
    else:
        y = (torch.rand(rows, generator=g, dtype=torch.float64) < torch.sigmoid(eta)).to(torch.float64)
    return x.contiguous(), y.to(w.theta_dtype).contiguous()


def make_buffer(w: Workload, k: int, rows: Optional[int] = None) -> Tuple[torch.Tensor, torch.Tensor]:
    """Buffer k of the fixed contiguous partition: rows [k*N0, min((k+1)*N0, N))."""
    start = k * w.N0
    cnt = min(w.N0, w.N - start) if rows is None else rows
    return make_rows(w, start, cnt)


def make_dataset(w: Workload) -> Tuple[torch.Tensor, torch.Tensor]:
    """All K buffers concatenated: X [N, p], y [N]."""
    xs, ys = zip(*(make_buffer(w, k) for k in range(w.K)))
    return torch.cat(xs), torch.cat(ys)
