"""Pins for the oracle's model gradients (supplement, "Simulation details") and the synthetic stream."""
import numpy as np
import pytest
from scipy.special import expit, logsumexp

import oracle


def _data(rng, n, F, C=None):
    X = rng.standard_normal((n, F)).astype(np.float32)
    y = rng.integers(0, 2 if C is None else C, size=n).astype(np.int32)
    return X, y


def _fd(loss_fn, theta, idx, h=1e-6):
    out = []
    for i in idx:
        e = np.zeros_like(theta)
        e[i] = h
        out.append((loss_fn(theta + e) - loss_fn(theta - e)) / (2 * h))
    return np.array(out)


def test_logreg_closed_forms_at_zero():
    rng = np.random.default_rng(0)
    X, y = _data(rng, 300, 7)
    loss, g = oracle.grad_logreg_bin(X, y, np.zeros(7), 1.0 / 300, 1.0, 0.0)
    assert loss == pytest.approx(np.log(2.0), rel=1e-14)                     # softplus(0) = log 2
    np.testing.assert_allclose(g, ((0.5 - y)[:, None] * X).sum(0) / 300, rtol=1e-13, atol=1e-15)


def test_logreg_against_library_loss_and_finite_differences():
    rng = np.random.default_rng(1)
    n, F, lam, N, share = 200, 9, 0.03, 500, 0.4
    X, y = _data(rng, n, F)
    theta = rng.standard_normal(F)

    def lib_loss(th):          # library routines only: logaddexp for softplus
        z = X.astype(np.float64) @ th
        return (np.logaddexp(0.0, z) - y * z).sum() / N + share * 0.5 * lam * th @ th

    loss, g = oracle.grad_logreg_bin(X, y, theta, 1.0 / N, share, lam)
    assert loss == pytest.approx(lib_loss(theta), rel=1e-13)
    np.testing.assert_allclose(g, _fd(lib_loss, theta, range(F)), rtol=1e-6, atol=1e-9)
    # and against the textbook gradient (sigma(z) - y) x
    z = X.astype(np.float64) @ theta
    np.testing.assert_allclose(g, ((expit(z) - y)[:, None] * X).sum(0) / N + share * lam * theta, rtol=1e-12)


def test_softmax_closed_forms_and_library():
    rng = np.random.default_rng(2)
    n, F, C, lam, N, share = 150, 11, 5, 0.01, 400, 0.375
    X, y = _data(rng, n, F, C)
    loss0, _ = oracle.grad_softmax(X, y, np.zeros(C * F), C, 1.0 / n, 1.0, 0.0)
    assert loss0 == pytest.approx(np.log(C), rel=1e-14)
    theta = 0.3 * rng.standard_normal(C * F)

    def lib_loss(th):
        Z = X.astype(np.float64) @ th.reshape(C, F).T
        return (logsumexp(Z, axis=1) - Z[np.arange(n), y]).sum() / N + share * 0.5 * lam * th @ th

    loss, g = oracle.grad_softmax(X, y, theta, C, 1.0 / N, share, lam)
    assert loss == pytest.approx(lib_loss(theta), rel=1e-13)
    np.testing.assert_allclose(g, _fd(lib_loss, theta, range(C * F)), rtol=2e-6, atol=1e-9)


def test_softmax_two_classes_reduces_to_binary_logistic():
    rng = np.random.default_rng(3)
    n, F = 120, 6
    X, y = _data(rng, n, F)
    w = rng.standard_normal(F)
    theta2 = np.concatenate([np.zeros(F), w])       # class-1 score minus class-0 score = x.w
    l2, g2 = oracle.grad_softmax(X, y, theta2, 2, 1.0 / n, 1.0, 0.0)
    l1, g1 = oracle.grad_logreg_bin(X, y, w, 1.0 / n, 1.0, 0.0)
    assert l2 == pytest.approx(l1, rel=1e-13)
    np.testing.assert_allclose(g2[F:], g1, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(g2[:F], -g1, rtol=1e-12, atol=1e-15)


def test_worker_gradients_sum_to_the_gradient_of_the_pooled_problem():
    rng = np.random.default_rng(4)
    M, n, F, C, lam = 4, 50, 8, 3, 0.02
    X, y = _data(rng, M * n, F, C)
    theta = rng.standard_normal(C * F)
    N = M * n
    tot_l, tot_g = 0.0, np.zeros(C * F)
    for m in range(M):
        l, g = oracle.grad_softmax(X[m * n:(m + 1) * n], y[m * n:(m + 1) * n], theta, C, 1.0 / N, n / N, lam)
        tot_l += l
        tot_g += g
    l_all, g_all = oracle.grad_softmax(X, y, theta, C, 1.0 / N, 1.0, lam)
    assert tot_l == pytest.approx(l_all, rel=1e-13)
    np.testing.assert_allclose(tot_g, g_all, rtol=1e-12, atol=1e-15)


def _mlp_lib_loss(X, y, th, F, H, C, N, share, lam, cast=None):
    cast = cast or (lambda a: a)
    W1, b1 = th[:H * F].reshape(H, F), th[H * F:H * F + H]
    o = H * F + H
    W2, b2 = th[o:o + C * H].reshape(C, H), th[o + C * H:]
    Hid = np.maximum(cast(X.astype(np.float64)) @ cast(W1).T + b1, 0.0)
    Z = Hid @ W2.T + b2
    n = X.shape[0]
    return (logsumexp(Z, axis=1) - Z[np.arange(n), y]).sum() / N + share * 0.5 * lam * th @ th


def test_mlp_gradient_by_finite_differences():
    rng = np.random.default_rng(5)
    n, F, H, C, lam, N, share = 40, 12, 7, 4, 0.01, 100, 0.4
    X, y = _data(rng, n, F, C)
    p = H * F + H + C * H + C
    theta = 0.5 * rng.standard_normal(p)
    loss, g = oracle.grad_mlp2(X, y, theta, H, C, 1.0 / N, share, lam, bf16_ops=0)
    f = lambda th: _mlp_lib_loss(X, y, th, F, H, C, N, share, lam)
    assert loss == pytest.approx(f(theta), rel=1e-13)
    np.testing.assert_allclose(g, _fd(f, theta, range(p), h=1e-6), rtol=5e-6, atol=2e-9)


def test_mlp_bf16_operand_rounding_against_torch_casts():
    """With bf16 operands, the hidden layer sees bf16(X) and bf16(W1); the W1 gradient is
    bf16(dH)^T bf16(X); everything else is unrounded.  Rebuilt here with torch's bf16 casts."""
    import torch
    rng = np.random.default_rng(6)
    n, F, H, C, lam, N, share = 30, 10, 6, 3, 0.01, 60, 0.5
    X, y = _data(rng, n, F, C)
    p = H * F + H + C * H + C
    theta = (0.5 * rng.standard_normal(p)).astype(np.float32).astype(np.float64)
    bf = lambda a: torch.from_numpy(np.asarray(a, np.float32)).to(torch.bfloat16).to(torch.float64).numpy()
    loss, g = oracle.grad_mlp2(X, y, theta, H, C, 1.0 / N, share, lam, bf16_ops=1)
    assert loss == pytest.approx(_mlp_lib_loss(X, y, theta, F, H, C, N, share, lam, cast=bf), rel=1e-13)
    W1, b1 = theta[:H * F].reshape(H, F), theta[H * F:H * F + H]
    o = H * F + H
    W2, b2 = theta[o:o + C * H].reshape(C, H), theta[o + C * H:]
    Xr = bf(X)
    Hid = np.maximum(Xr @ bf(W1).T + b1, 0.0)
    Z = Hid @ W2.T + b2
    P = np.exp(Z - logsumexp(Z, axis=1, keepdims=True))
    P[np.arange(n), y] -= 1.0
    dH = (P @ W2) * (Hid > 0)
    gW1 = bf(dH).T @ Xr
    ref = np.concatenate([gW1.ravel(), dH.sum(0), (P.T @ Hid).ravel(), P.sum(0)]) / N + share * lam * theta
    np.testing.assert_allclose(g, ref, rtol=1e-11, atol=1e-14)


def test_synthetic_stream_statistics_and_determinism():
    M, p, sigma, eta0 = 8, 200_000, 0.1, 0.05
    g1 = oracle.synth_gradient(4, 2, M, p, 1, sigma, eta0)
    assert np.array_equal(g1, oracle.synth_gradient(4, 2, M, p, 1, sigma, eta0))
    assert not np.array_equal(g1, oracle.synth_gradient(5, 2, M, p, 1, sigma, eta0))
    assert not np.array_equal(g1, oracle.synth_gradient(4, 3, M, p, 1, sigma, eta0))
    g0 = oracle.synth_gradient(4, 2, M, p, 0, sigma, eta0).astype(np.float64)     # k = 0: no drift term
    assert abs(g0.mean()) < 4 * sigma / np.sqrt(p)
    assert g0.std() == pytest.approx(sigma, rel=0.01)
    assert np.abs(g0).max() <= sigma * 510 / np.sqrt(21845.0) * (1 + 1e-6)
    # drift: g^k - g^0 = k eta_m sigma w with w uncorrelated with z and of unit variance
    k, eta_m = 40, eta0 * 3 / M
    w = (oracle.synth_gradient(4, 2, M, p, k, sigma, eta0).astype(np.float64) - g0) / (k * eta_m)
    assert w.std() == pytest.approx(sigma, rel=0.01)
    assert abs(np.corrcoef(w, g0)[0, 1]) < 0.01


def test_synthetic_stream_follows_its_written_definition():
    """Bit-for-bit against the definition evaluated with numpy integer/fp32 operations."""
    def fmix(x):
        x = np.uint32(x)
        x ^= x >> np.uint32(16); x = np.uint32(x * np.uint32(0x85ebca6b))
        x ^= x >> np.uint32(13); x = np.uint32(x * np.uint32(0xc2b2ae35))
        x ^= x >> np.uint32(16)
        return x
    seed, m, M, p, k, sigma, eta0 = (7 << 32) | 12345, 5, 16, 1003, 9, 0.1, 0.05
    nv = (p + 3) // 4
    with np.errstate(over="ignore"):
        key = fmix(np.uint32(seed & 0xffffffff) ^ fmix(np.uint32(seed >> 32) + np.uint32(0x9e3779b9) * np.uint32(m + 1)))
        h0 = fmix(np.arange(nv, dtype=np.uint32) ^ key)
        h1 = np.uint32(h0 * np.uint32(0x9e3779b1))
        h1 ^= h1 >> np.uint32(15)
    z = np.zeros((nv, 4), np.int32)
    for j, h in enumerate((h0, h1)):
        b = [((h >> np.uint32(s)) & np.uint32(255)).astype(np.int32) for s in (0, 8, 16, 24)]
        z[:, 2 * j] = b[0] + b[1] + b[2] + b[3] - 510
        z[:, 2 * j + 1] = b[0] - b[1] + b[2] - b[3]
    cz = np.float32(np.float64(np.float32(sigma)) / np.sqrt(21845.0))
    drift = np.float32(k) * np.float32(np.float64(np.float32(eta0)) * (m + 1) / M)
    partner = z[:, [2, 3, 0, 1]]
    # small integers times an fp32 factor plus a small integer: exact in fp64, so one rounding = fma
    a = (np.float64(drift) * partner.astype(np.float64) + z.astype(np.float64)).astype(np.float32)
    ref = (a * cz).reshape(-1)[:p]
    np.testing.assert_array_equal(oracle.synth_gradient(seed, m, M, p, k, sigma, eta0), ref)


def test_synthetic_stream_coordinates_are_uncorrelated():
    g = oracle.synth_gradient(11, 0, 4, 400_000, 0, 1.0, 0.0).astype(np.float64).reshape(-1, 4)
    c = np.corrcoef(g.T)
    assert np.max(np.abs(c - np.eye(4))) < 0.01            # within a group of four
    flat = g.reshape(-1)
    for lag in (1, 2, 3, 4, 5, 8, 64):
        assert abs(np.corrcoef(flat[:-lag], flat[lag:])[0, 1]) < 0.01
    assert np.allclose(g.std(0), 1.0, rtol=0.01) and np.all(np.abs(g.mean(0)) < 0.01)
