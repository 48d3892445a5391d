"""Seeded synthetic workloads for the CADA hot path.

This module only manufactures *inputs* (feature matrices, labels, initial iterates and
hyper-parameter records).  It contains none of the method's arithmetic: no gradients, no
upload rule, no optimiser and no minibatch sampler.  Both the CUDA library's tests and the
CPU oracle's tests draw their inputs from here so that the two sides see identical bytes.

The five workloads mirror the shapes of the paper's experiments (Section 4 and the
"Simulation details" of the supplement), whose public datasets are not shipped:

  C1  22 features + bias, M=10 uniform workers           (shape of the ijcnn1 test)
  C2  54 features, M=20 heterogeneous workers             (shape of the covtype test)
  C3  784 sparse non-negative features -> 10 classes      (shape of the MNIST regression test)
  C4  784-200-10 ReLU network on the C3 inputs, bf16      (stands in for the small CNN test)
  C5  4,096 dense features, M=256 workers                 (bandwidth stress; not in the paper)

Everything is deterministic in ``data_seed = 201215469 + 1000 * config_number``.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Tuple

import numpy as np

MODEL_LOGISTIC = 0
MODEL_SOFTMAX = 1
MODEL_MLP2 = 2

RULE_CADA1 = 1
RULE_CADA2 = 2

BASE_SEED = 201215469


@dataclasses.dataclass
class Workload:
    """One synthetic problem instance: shapes, hyper-parameters and seeds."""

    name: str
    config: int
    model: int
    M: int                      # workers
    n_samples: int              # rows held by each worker
    n_features: int
    batch: int                  # minibatch rows per worker per iteration
    iters: int                  # iterations of a full run
    n_classes: int = 1
    n_hidden: int = 0
    has_bias: int = 0
    alpha: float = 0.01
    beta1: float = 0.9
    beta2: float = 0.99
    eps: float = 1e-8
    c: float = 0.6
    d_max: int = 10
    D: int = 100
    lam: float = 0.0            # L2 coefficient, loss += lam/2 * ||theta||^2
    x_bf16: bool = False        # features stored as bfloat16 (C4)
    ldx: int = 0                # row pitch in elements (0 -> derived: n_features rounded up to 16 bytes)
    flip: float = 0.0           # label-flip probability (binary models)

    def __post_init__(self):
        if self.ldx == 0:
            per16 = 8 if self.x_bf16 else 4
            self.ldx = (self.n_features + per16 - 1) // per16 * per16

    @property
    def p(self) -> int:
        """Dimension of theta implied by the model shape."""
        f, c, h, b = self.n_features, self.n_classes, self.n_hidden, self.has_bias
        if self.model == MODEL_LOGISTIC:
            return f + b
        if self.model == MODEL_SOFTMAX:
            return f * c + b * c
        return f * h + h + h * c + c

    @property
    def data_seed(self) -> int:
        return BASE_SEED + 1000 * self.config

    @property
    def sample_seed(self) -> int:
        return self.data_seed + 1

    def scaled(self, **kw) -> "Workload":
        """A copy with some fields replaced (used for reduced-size test cases)."""
        w = dataclasses.replace(self, **kw)
        if "n_features" in kw and "ldx" not in kw:
            w.ldx = 0
            w.__post_init__()
        return w


def workload(name: str) -> Workload:
    """The five benchmark workloads by name ("C1".."C5"), plus "C5S", a 1 GB cut of C5."""
    name = name.upper()
    if name == "C1":
        return Workload("C1", 1, MODEL_LOGISTIC, M=10, n_samples=5000, n_features=22, has_bias=1,
                        batch=32, iters=200, lam=1e-4, c=0.6, d_max=10, D=100, flip=0.10)
    if name == "C2":
        return Workload("C2", 2, MODEL_LOGISTIC, M=20, n_samples=29000, n_features=54, has_bias=0,
                        batch=100, iters=1000, c=0.6, d_max=10, D=50, flip=0.05)
    if name == "C3":
        return Workload("C3", 3, MODEL_SOFTMAX, M=20, n_samples=3000, n_features=784, n_classes=10,
                        has_bias=1, batch=64, iters=2000, c=0.6, d_max=10, D=100)
    if name == "C4":
        return Workload("C4", 4, MODEL_MLP2, M=10, n_samples=6000, n_features=784, n_classes=10,
                        n_hidden=200, has_bias=1, batch=128, iters=2000, alpha=0.001, c=0.6,
                        d_max=10, D=50, x_bf16=True)
    if name == "C5":
        return Workload("C5", 5, MODEL_LOGISTIC, M=256, n_samples=8192, n_features=4096, has_bias=0,
                        batch=512, iters=500, c=0.6, d_max=10, D=100, flip=0.10)
    if name == "C5S":
        # C5 cut down to 1 GB of X (still far larger than L2): the case profiler captures run on
        return Workload("C5S", 5, MODEL_LOGISTIC, M=32, n_samples=2048, n_features=4096, has_bias=0,
                        batch=512, iters=20, c=0.6, d_max=10, D=100, flip=0.10)
    raise KeyError(name)


# ----------------------------------------------------------------------------------------------
# helpers
# ----------------------------------------------------------------------------------------------

def bf16_representable(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bfloat16 (ties to even) and return them as fp32.

    Pure bit manipulation on the stored inputs; used only to make C4's features exactly
    representable in the 16-bit storage format.
    """
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def _pad_rows(X: np.ndarray, ldx: int) -> np.ndarray:
    n, f = X.shape
    if ldx == f:
        return np.ascontiguousarray(X)
    out = np.zeros((n, ldx), dtype=X.dtype)
    out[:, :f] = X
    return out


def _binary_labels(rng, X, theta_star, bias, flip):
    z = X.astype(np.float64) @ theta_star + bias
    y = np.where(z >= 0.0, 1.0, -1.0)
    flips = rng.random(X.shape[0]) < flip
    y[flips] = -y[flips]
    return y.astype(np.float32)


def _sparse_uniform(rng, n, f):
    """Entries are 0 with probability 0.8, otherwise U[0,1)."""
    x = rng.random((n, f), dtype=np.float32)
    keep = rng.random((n, f), dtype=np.float32) < 0.2
    return np.where(keep, x, np.float32(0.0))


def _label_skewed_worker(rng, n, f, w_star, n_classes, favoured):
    """Rows whose planted argmax label follows the worker's skewed class distribution."""
    # class drawn per sample: favoured pair with prob 0.8 (split evenly), else uniform over the rest
    others = [c for c in range(n_classes) if c not in favoured]
    pick_fav = rng.random(n) < 0.8
    want = np.where(pick_fav, rng.choice(favoured, size=n), rng.choice(others, size=n))
    X = np.empty((n, f), dtype=np.float32)
    y = np.empty(n, dtype=np.int32)
    need = {c: list(np.nonzero(want == c)[0]) for c in range(n_classes)}
    remaining = n
    rounds = 0
    while remaining > 0:
        rounds += 1
        if rounds > 400:
            raise RuntimeError("label-skew rejection sampling did not finish")
        cand = _sparse_uniform(rng, 4096, f)
        lab = np.argmax(cand.astype(np.float64) @ w_star, axis=1)
        for c in range(n_classes):
            slots = need[c]
            if not slots:
                continue
            rows = np.nonzero(lab == c)[0][: len(slots)]
            for r in rows:
                s = slots.pop()
                X[s] = cand[r]
                y[s] = c
                remaining -= 1
    return X, y


# ----------------------------------------------------------------------------------------------
# host generators (C1-C4 and any reduced-size case)
# ----------------------------------------------------------------------------------------------

def make_host_data(w: Workload) -> Tuple[List[np.ndarray], List[np.ndarray], np.ndarray]:
    """Per-worker feature matrices [n_samples x ldx] (fp32; bf16-representable when x_bf16),
    per-worker labels (fp32 +-1 for the binary model, int32 class otherwise) and theta0 (fp32)."""
    rng = np.random.default_rng(w.data_seed)
    f, n = w.n_features, w.n_samples
    Xs, ys = [], []
    if w.model == MODEL_LOGISTIC:
        theta_star = rng.standard_normal(f + 1)
        scale = 1.0 if f < 1024 else 1.0 / math.sqrt(f)
        theta_star[:f] *= scale
        bias = theta_star[f] if w.has_bias else 0.0
        heterogeneous = (w.config == 2)
        n_bin = int(round(0.3 * f)) if heterogeneous else 0
        bin_cols = rng.permutation(f)[:n_bin]
        for m in range(w.M):
            X = rng.standard_normal((n, f), dtype=np.float32)
            if heterogeneous:
                mu = (0.5 * rng.standard_normal(f)).astype(np.float32)
                X += mu[None, :]
                X[:, bin_cols] = (X[:, bin_cols] > 0).astype(np.float32)
            y = _binary_labels(rng, X, theta_star[:f], bias, w.flip)
            Xs.append(_pad_rows(X, w.ldx))
            ys.append(y)
        theta0 = np.zeros(w.p, dtype=np.float32)
    else:
        w_star = rng.standard_normal((f, w.n_classes))
        for m in range(w.M):
            favoured = [(2 * m) % w.n_classes, (2 * m + 1) % w.n_classes]
            X, y = _label_skewed_worker(rng, n, f, w_star, w.n_classes, favoured)
            if w.x_bf16:
                X = bf16_representable(X)
            Xs.append(_pad_rows(X, w.ldx))
            ys.append(y)
        if w.model == MODEL_SOFTMAX:
            theta0 = np.zeros(w.p, dtype=np.float32)
        else:
            h, c = w.n_hidden, w.n_classes
            w1 = rng.standard_normal((f, h)) / math.sqrt(f)
            w2 = rng.standard_normal((h, c)) / math.sqrt(h)
            theta0 = np.concatenate([w1.ravel(), np.zeros(h), w2.ravel(), np.zeros(c)]).astype(np.float32)
    return Xs, ys, theta0


def random_theta(w: Workload, scale: float, seed_offset: int = 7) -> np.ndarray:
    """A seeded non-trivial iterate (tests use it so that gradients are not those at zero)."""
    rng = np.random.default_rng(w.data_seed + seed_offset)
    return (scale * rng.standard_normal(w.p)).astype(np.float32)


# ----------------------------------------------------------------------------------------------
# device generator (C5 and other cases too large to build on the host)
# ----------------------------------------------------------------------------------------------

def make_device_logistic(w: Workload, device="cuda"):
    """Dense N(0,1) binary-logistic data generated directly in device memory.

    Returns (X, y, theta0): X is one [M, n_samples, ldx] fp32 tensor (worker m's matrix is X[m]),
    y is [M, n_samples] fp32 +-1.  Labels are sign(x . theta*) with ``flip`` of them negated.
    """
    import torch

    assert w.model == MODEL_LOGISTIC and not w.has_bias and w.ldx == w.n_features
    g = torch.Generator(device=device)
    g.manual_seed(w.data_seed)
    f = w.n_features
    theta_star = torch.randn(f, generator=g, device=device, dtype=torch.float32) / math.sqrt(f)
    X = torch.empty((w.M, w.n_samples, f), device=device, dtype=torch.float32)
    y = torch.empty((w.M, w.n_samples), device=device, dtype=torch.float32)
    for m in range(w.M):
        X[m].normal_(generator=g)
        z = X[m] @ theta_star
        ym = torch.where(z >= 0, 1.0, -1.0)
        flips = torch.rand(w.n_samples, generator=g, device=device) < w.flip
        y[m] = torch.where(flips, -ym, ym)
    theta0 = torch.zeros(w.p, device=device, dtype=torch.float32)
    return X, y, theta0
