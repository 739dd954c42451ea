"""Convergence diagnostics (Lyapunov function of Sec. 3): the library's vectorised arithmetic against the oracle's
term-by-term sum on the CPU, and on the GPU's own trace against the oracle's run."""
import numpy as np
import pytest

import oracle
from paper_1909_07588_b200 import diagnostics


def test_lyapunov_matches_the_term_by_term_sum():
    rng = np.random.default_rng(3)
    for D in (1, 2, 5, 10):
        n = 40
        loss = np.sort(rng.random(n))[::-1] + 1.0
        d2 = rng.random(n)
        xi = rng.random(D) * 0.1
        got = diagnostics.lyapunov(loss, d2, xi, 0.37, 0.9)
        np.testing.assert_allclose(got, oracle.lyapunov(loss, d2, xi, 0.37, 0.9), rtol=1e-13)
    np.testing.assert_allclose(diagnostics.lyapunov_weights([0.25, 0.5], 0.5), [1.5, 1.0])
    np.testing.assert_allclose(diagnostics.quantization_error_bound([[7.0, 14.0]], 3), [[1.0, 4.0]])
    assert diagnostics.linear_rate(0.5 ** np.arange(30)) == pytest.approx(0.5, rel=1e-9)


@pytest.mark.gpu
def test_lyapunov_of_a_gpu_run_follows_the_oracle_and_decays():
    """C0 with the lemma's parameters (xi_d = 1/(16 D), alpha = 1/(8 L)): the Lyapunov function of the CUDA path's
    run equals that of the fp64 oracle's run to the trajectory tolerance while both are well above fp32 rounding,
    and it decays at a linear rate (Theorem 1)."""
    from paper_1909_07588_b200 import laq, workloads
    w = workloads.c0(iters=300)
    w.alpha = np.float32(w.alpha / 8.0)                       # the workload's alpha is 1/L
    w.xi = np.full(w.D, 1.0 / (16 * w.D), np.float32)
    n = w.iters
    ctx = laq.from_workload(w, trace_capacity=n)
    tr = ctx.step(n, trace=True)
    ctx.close()
    o = oracle.OracleLaq(64, oracle.MODEL_LOGREG_BIN, w.M, w.p, N=w.N, n_features=w.n_features, alpha=w.alpha,
                         lam=w.lam, b=w.b, D=w.D, xi=w.xi, tbar=w.tbar)
    for m in range(w.M):
        o.set_shard(m, w.X[m], w.y[m])
    ol, od = [], []
    for _ in range(n):
        st = o.step()
        ol.append(st["loss"])
        od.append(st["dtheta2"])
    # f*: Newton's method on the pooled problem in fp64 (strongly convex through the regulariser)
    X = np.concatenate(w.X).astype(np.float64)
    y = np.concatenate(w.y).astype(np.float64)
    th = np.zeros(w.p)
    for _ in range(30):
        z = X @ th
        s = 1.0 / (1.0 + np.exp(-z))
        g = X.T @ (s - y) / len(y) + w.lam * th
        Hm = (X * (s * (1 - s))[:, None]).T @ X / len(y) + w.lam * np.eye(w.p)
        th -= np.linalg.solve(Hm, g)
    z = X @ th
    f_star = np.mean(np.logaddexp(0.0, z) - y * z) + 0.5 * w.lam * th @ th
    v_gpu = diagnostics.lyapunov(tr["loss"], tr["dtheta2"], w.xi, w.alpha, f_star)
    v_ref = oracle.lyapunov(ol, od, w.xi, w.alpha, f_star)
    assert np.all(v_ref > 0)
    big = v_ref > 1e-3 * v_ref[0]
    assert big.sum() >= 20
    # V subtracts f* from a loss whose per-sample terms are fp32: an absolute 1e-6 f* rides on the relative band
    np.testing.assert_allclose(v_gpu[big], v_ref[big], rtol=1e-4, atol=1e-6 * f_star)
    sigma = diagnostics.linear_rate(v_gpu, 5, int(big.sum()), floor=0.0)
    assert 0.0 < sigma < 1.0
    assert v_gpu[big.sum() - 1] < 0.05 * v_gpu[0]
    eb = diagnostics.quantization_error_bound(tr["R"], w.b).max(axis=1)
    assert eb[n - 1] < eb[0]
