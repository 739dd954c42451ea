"""Seeded synthetic inputs for the LAQ hot path.

Every workload is produced on the host with numpy from a fixed seed (generated in fp64, stored as
fp32) and handed, as plain arrays, both to the CUDA library and to whatever checks it.  This module
holds input preparation only: shapes, value distributions, labels, the initial iterate and the
step size.  None of the method's arithmetic (quantizer, trigger, aggregation, model gradients)
lives here.

The five workloads take the SHAPES of the problems the paper experiments on (Sec. 5 and the
supplement's "Simulation details": MNIST-shaped 784-feature 10-class data split over M = 10
workers, a 22-feature and a 54-feature binary problem, a 784-200-10 ReLU network) and a large
synthetic gradient stream; no record of any public dataset is used or reproduced.
"""
from dataclasses import dataclass, field
from typing import List, Optional
import numpy as np

MODEL_LOGREG_BIN, MODEL_SOFTMAX, MODEL_MLP2, MODEL_SYNTH, MODEL_EXTERNAL = 0, 1, 2, 3, 4


@dataclass
class Workload:
    name: str
    model: int
    M: int
    p: int
    N: List[int]
    n_features: int = 0
    n_classes: int = 0
    n_hidden: int = 0
    alpha: float = 0.02
    lam: float = 0.0
    b: int = 4
    D: int = 10
    xi: Optional[np.ndarray] = None
    tbar: int = 100
    iters: int = 200
    seed: int = 0
    synth_sigma: float = 0.1
    synth_eta0: float = 0.05
    bf16_ops: int = 0
    X: List[np.ndarray] = field(default_factory=list)   # per worker, [N_m, F] fp32
    y: List[np.ndarray] = field(default_factory=list)   # per worker, [N_m] int32
    theta0: Optional[np.ndarray] = None                 # [p] fp32 (None = zeros)
    L_smooth: Optional[float] = None                    # smoothness bound used for alpha (if any)

    def __post_init__(self):
        if self.xi is None:
            self.xi = np.full(self.D, 0.8 / self.D, dtype=np.float32)
        self.xi = np.asarray(self.xi, dtype=np.float32)
        self.alpha = float(np.float32(self.alpha))
        self.lam = float(np.float32(self.lam))


def lambda_max_gram(X64, iters=1000):
    """Largest eigenvalue of X^T X by power iteration in fp64 (start = ones, fixed iteration count)."""
    G = X64.T @ X64
    v = np.ones(G.shape[0])
    v /= np.linalg.norm(v)
    lam = 0.0
    for _ in range(iters):
        w = G @ v
        lam = float(v @ w)
        nw = np.linalg.norm(w)
        if nw == 0.0:
            break
        v = w / nw
    return lam


def _split(X, y, M, n_per):
    Xs = [np.ascontiguousarray(X[m * n_per:(m + 1) * n_per], dtype=np.float32) for m in range(M)]
    ys = [np.ascontiguousarray(y[m * n_per:(m + 1) * n_per], dtype=np.int32) for m in range(M)]
    return Xs, ys


def _sigmoid(z):
    return 0.5 * (1.0 + np.tanh(0.5 * z))


def c0(seed=0, M=10, n_per=500, F=22, iters=200):
    """Small binary l2-regularised logistic regression: N(0,1) features, Bernoulli(sigma(x.theta*)) labels."""
    rng = np.random.default_rng(seed)
    theta_star = rng.standard_normal(F)
    X = rng.standard_normal((M * n_per, F)).astype(np.float32)
    X64 = X.astype(np.float64)
    y = (rng.random(M * n_per) < _sigmoid(X64 @ theta_star)).astype(np.int32)
    lam = 1e-3
    L = lambda_max_gram(X64) / (4.0 * M * n_per) + lam
    Xs, ys = _split(X, y, M, n_per)
    return Workload("c0_logreg22", MODEL_LOGREG_BIN, M, F, [n_per] * M, n_features=F, alpha=1.0 / L,
                    lam=lam, b=4, D=10, tbar=100, iters=iters, seed=seed, X=Xs, y=ys, L_smooth=L)


def _mnist_shaped(rng, n, F=784, C=10, density=0.19, score_std=2.0):
    """Sparse-support features in (0,1], labels = argmax of planted linear scores plus Gumbel noise."""
    mask = rng.random((n, F)) < density
    vals = 1.0 - rng.random((n, F))          # uniform on (0, 1]
    X = np.where(mask, vals, 0.0).astype(np.float32)
    # a planted score of the given standard deviation: E[x^2] = density / 3 per feature
    Theta = rng.standard_normal((C, F)) * (score_std / np.sqrt(density * F / 3.0))
    scores = X.astype(np.float64) @ Theta.T
    gumbel = -np.log(-np.log(rng.random((n, C))))
    y = np.argmax(scores + gumbel, axis=1).astype(np.int32)
    return X, y


def c1(seed=1, M=10, n_per=6000, F=784, C=10, iters=500):
    """10-class softmax regression on MNIST-shaped inputs (about 19 % nonzeros, uniform on the support)."""
    rng = np.random.default_rng(seed)
    X, y = _mnist_shaped(rng, M * n_per, F, C)
    lam = 0.01
    L = lambda_max_gram(X.astype(np.float64)) / (2.0 * M * n_per) + lam
    Xs, ys = _split(X, y, M, n_per)
    return Workload("c1_softmax784x10", MODEL_SOFTMAX, M, C * F, [n_per] * M, n_features=F, n_classes=C,
                    alpha=1.0 / L, lam=lam, b=4, D=10, tbar=100, iters=iters, seed=seed, X=Xs, y=ys,
                    L_smooth=L)


def c2(seed=2, M=10, n_per=58101, iters=1000, theta0_scale=0.0):
    """Binary logistic regression, 54 features: 10 Gaussian columns, a 4-way and a 40-way one-hot group.
    theta0_scale > 0 starts from a small random iterate instead of zero (at theta = 0 every residual is
    +-1/2, so the gradient of a rarely active one-hot column can cancel to exactly zero)."""
    rng = np.random.default_rng(seed)
    n = M * n_per
    F = 54
    X = np.zeros((n, F), dtype=np.float32)
    X[:, :10] = rng.standard_normal((n, 10)).astype(np.float32)
    for start, width in ((10, 4), (14, 40)):
        prob = 0.93 ** np.arange(width)      # skewed, but every worker still sees every category at reduced size
        prob /= prob.sum()
        cat = rng.choice(width, size=n, p=prob)
        X[np.arange(n), start + cat] = 1.0
    theta_star = rng.standard_normal(F)
    X64 = X.astype(np.float64)
    y = (rng.random(n) < _sigmoid(X64 @ theta_star)).astype(np.int32)
    lam = 0.01
    L = lambda_max_gram(X64) / (4.0 * n) + lam
    Xs, ys = _split(X, y, M, n_per)
    theta0 = (theta0_scale * rng.standard_normal(F)).astype(np.float32) if theta0_scale > 0 else None
    return Workload("c2_logreg54", MODEL_LOGREG_BIN, M, F, [n_per] * M, n_features=F, alpha=1.0 / L,
                    lam=lam, b=8, D=10, tbar=100, iters=iters, seed=seed, X=Xs, y=ys, L_smooth=L, theta0=theta0)


def c3(seed=3, M=10, n_per=6000, F=784, H=200, C=10, iters=1000, bf16_ops=1):
    """One-hidden-layer ReLU network F-H-C on MNIST-shaped inputs; He-normal weights, zero biases."""
    rng = np.random.default_rng(seed)
    X, y = _mnist_shaped(rng, M * n_per, F, C)
    p = H * F + H + C * H + C
    theta0 = np.zeros(p)
    theta0[:H * F] = rng.standard_normal(H * F) * np.sqrt(2.0 / F)
    o = H * F + H
    theta0[o:o + C * H] = rng.standard_normal(C * H) * np.sqrt(2.0 / H)
    Xs, ys = _split(X, y, M, n_per)
    return Workload("c3_mlp784_200_10", MODEL_MLP2, M, p, [n_per] * M, n_features=F, n_classes=C,
                    n_hidden=H, alpha=0.02, lam=0.01, b=8, D=10, tbar=100, iters=iters, seed=seed,
                    X=Xs, y=ys, theta0=theta0.astype(np.float32), bf16_ops=bf16_ops)


def c4(seed=4, M=64, p=25_600_000, b=8, iters=200, sigma=0.1, eta0=0.05, xi_scale=1.0):
    """Large-p throughput workload: M gradient vectors of p coordinates, regenerated every iteration
    inside the library from (seed, worker, coordinate, iteration); no data shard."""
    D = 10
    xi = np.full(D, 0.8 / D * xi_scale, dtype=np.float32)
    return Workload("c4_synth_M%d_p%d_b%d" % (M, p, b), MODEL_SYNTH, M, p, [0] * M, alpha=0.02, b=b,
                    D=D, xi=xi, tbar=100, iters=iters, seed=seed, synth_sigma=sigma, synth_eta0=eta0)
