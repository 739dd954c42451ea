"""Pins for the oracle's trigger (Eq. (7a)/(7b)) and whole iteration (Eq. (4), Algorithm 2)."""
import numpy as np
import pytest

import oracle
from paper_1909_07588_b200 import workloads


def test_trigger_hand_numbers():
    # D = 2, xi = (1/2, 1/4), differences (4, 8) newest first, alpha = 1/2, M = 2:
    # sum_d xi_d diff_d = 4, alpha^2 M^2 = 1, rhs = 4 + 3 (1 + 2) = 13
    for n_dq, want in ((12.5, True), (13.0, True), (13.5, False)):
        skip, rhs = oracle.trigger(n_dq, 1.0, 2.0, [4.0, 8.0], [0.5, 0.25], 0.5, 2, clock=0, tbar=5)
        assert rhs == 13.0 and skip is want
    # (7b): the clock overrides a satisfied (7a)
    assert oracle.trigger(0.0, 1.0, 2.0, [4.0, 8.0], [0.5, 0.25], 0.5, 2, clock=5, tbar=5)[0] is True
    assert oracle.trigger(0.0, 1.0, 2.0, [4.0, 8.0], [0.5, 0.25], 0.5, 2, clock=6, tbar=5)[0] is False
    # the order of the history matters: weights pair with differences newest first
    _, rhs2 = oracle.trigger(0.0, 0.0, 0.0, [8.0, 4.0], [0.5, 0.25], 0.5, 2, clock=0, tbar=5)
    assert rhs2 == 5.0
    # 1/(alpha^2 M^2) scaling
    _, rhs3 = oracle.trigger(0.0, 0.0, 0.0, [4.0, 8.0], [0.5, 0.25], 0.25, 4, clock=0, tbar=5)
    assert rhs3 == 4.0


def _quadratic_problem(rng, M, p, Lm):
    """f_m = (L_m / 2) ||theta - c_m||^2 : gradient L_m (theta - c_m), smoothness constant L_m."""
    c = rng.standard_normal((M, p))
    Lm = np.asarray(Lm, dtype=np.float64)
    grad = lambda th: Lm[:, None] * (th[None, :] - c)
    return c, grad


def _run_given(o, grad, iters, theta0):
    """Drive the oracle with externally computed gradients; returns per-iteration skip masks."""
    skips = []
    theta = np.array(theta0, dtype=np.float64)
    for _ in range(iters):
        st = o.step_given(grad(theta))
        skips.append(st["skip"].copy())
        theta = o.state(big=False)["theta"]
    return np.array(skips)


@pytest.mark.parametrize("precision", [64, 32])
def test_server_aggregate_equals_sum_of_stored_quantized_gradients(precision):
    """Eq. (4) plus the server recovery imply grad^k = sum_m Q_m(theta_hat_m^k) at every k."""
    rng = np.random.default_rng(0)
    M, p = 5, 37
    _, grad = _quadratic_problem(rng, M, p, rng.uniform(0.2, 2.0, M))
    o = oracle.OracleLaq(precision, oracle.MODEL_GIVEN, M, p, alpha=0.05, b=3, D=4, tbar=6)
    theta = np.zeros(p)
    some_skip = False
    for k in range(60):
        st = o.step_given(grad(theta))
        s = o.state()
        theta = s["theta"]
        some_skip |= bool(st["skip"].any())
        tol = 1e-12 if precision == 64 else 2e-5
        np.testing.assert_allclose(s["agg"], s["qp"].sum(0), rtol=tol, atol=tol * np.abs(s["qp"]).max())
    assert some_skip


def test_laq_with_many_bits_and_zero_weights_is_gradient_descent():
    """"If enough bits are used and all xi_d are 0, LAQ reduces to GD" (text after Eq. (8))."""
    w = workloads.c0()
    N = sum(w.N)
    o = oracle.OracleLaq(64, oracle.MODEL_LOGREG_BIN, w.M, w.p, N=w.N, n_features=w.n_features,
                         alpha=w.alpha, lam=w.lam, b=30, D=w.D, xi=np.zeros(w.D), tbar=w.tbar)
    for m in range(w.M):
        o.set_shard(m, w.X[m], w.y[m])
    theta = np.zeros(w.p)
    Xall, yall = np.concatenate(w.X), np.concatenate(w.y)
    skipped = 0
    for k in range(200):
        _, g = oracle.grad_logreg_bin(Xall, yall, theta, 1.0 / N, 1.0, w.lam)   # pinned separately
        theta = theta - w.alpha * g                                              # Eq. (2)
        st = o.step()
        if np.linalg.norm(g) > 1e-7:
            skipped += int(st["skip"].sum())
    th = o.state(big=False)["theta"]
    assert skipped == 0
    assert np.linalg.norm(th - theta) / np.linalg.norm(theta) <= 1e-7


@pytest.mark.parametrize("precision", [64, 32])
def test_trigger_off_is_qgd(precision):
    """Algorithm 1: every worker uploads every iteration; theta follows Eq. (3)."""
    rng = np.random.default_rng(1)
    M, p, K, b, alpha = 4, 16, 30, 4, 0.125
    _, grad = _quadratic_problem(rng, M, p, rng.uniform(0.5, 1.5, M))
    o = oracle.OracleLaq(precision, oracle.MODEL_GIVEN, M, p, alpha=alpha, b=b, D=3, tbar=10,
                         flags=oracle.FLAG_TRIGGER_OFF)
    dt = np.float64 if precision == 64 else np.float32
    theta = np.zeros(p, dt)
    Q = np.zeros((M, p), dt)
    for k in range(K):
        g = grad(theta.astype(np.float64)).astype(dt)
        o.step_given(g)
        for m in range(M):
            Q[m] = oracle.quantize(g[m], Q[m], b, dt)["qnew"]
        theta = (theta - dt(alpha) * Q.sum(0, dtype=dt)).astype(dt)     # Eq. (3)
        th = o.state(big=False)["theta"]
        np.testing.assert_allclose(th, theta, rtol=1e-12 if precision == 64 else 1e-5, atol=1e-12 if precision == 64 else 1e-6)
    s = o.state(big=False)
    assert s["uploads"] == M * K
    assert s["bits"] == M * K * (32 + b * p)          # cost of a message, text after Eq. (6)


def test_quantizer_and_trigger_off_is_gradient_descent():
    """Eq. (2): with no quantizer and no skipping, theta^{k+1} = theta^k - alpha sum_m grad f_m(theta^k)."""
    rng = np.random.default_rng(5)
    M, p, K, alpha = 5, 12, 40, 0.0625
    _, grad = _quadratic_problem(rng, M, p, rng.uniform(0.5, 1.5, M))
    o = oracle.OracleLaq(64, oracle.MODEL_GIVEN, M, p, alpha=alpha, b=4, D=3, tbar=10,
                         flags=oracle.FLAG_TRIGGER_OFF | oracle.FLAG_QUANT_OFF)
    theta = np.zeros(p)
    for k in range(K):
        g = grad(theta)
        st = o.step_given(g)
        assert not st["skip"].any() and not st["n_eps"].any()
        np.testing.assert_allclose(st["R"], np.abs(g - (grad_prev if k else 0.0)).max(1), rtol=1e-12)
        grad_prev = g
        theta = theta - alpha * g.sum(0)
        np.testing.assert_allclose(o.state(big=False)["theta"], theta, rtol=1e-11, atol=1e-13)
    s = o.state()
    np.testing.assert_array_equal(s["qp"], grad_prev)           # the server holds the exact last gradients
    assert s["uploads"] == M * K and s["bits"] == M * K * 32 * p


def test_quantizer_off_is_lazily_aggregated_gradient_descent():
    """Without the quantizer the skip rule (7a) has eps = 0 and reads
    ||grad f_m(theta^k) - grad f_m(theta_hat_m)||^2 <= (1 / (alpha^2 M^2)) sum_d xi_d ||theta^{k+1-d} - theta^{k-d}||^2,
    the worker-side rule of the lazily aggregated gradient method that Sec. 4 compares with; simulated here directly."""
    rng = np.random.default_rng(6)
    M, p, K, alpha, D, tbar = 6, 10, 80, 0.0625, 4, 7
    xi = np.array([0.3, 0.2, 0.15, 0.1])
    _, grad = _quadratic_problem(rng, M, p, rng.uniform(0.1, 2.0, M))
    o = oracle.OracleLaq(64, oracle.MODEL_GIVEN, M, p, alpha=alpha, b=4, D=D, xi=xi, tbar=tbar,
                         flags=oracle.FLAG_QUANT_OFF)
    theta = np.zeros(p)
    held = np.zeros((M, p))                  # grad f_m(theta_hat_m) as the server holds it
    clock = np.full(M, tbar + 1)
    diffs = [0.0] * D                        # newest first
    total_skips = 0
    for k in range(K):
        g = grad(theta)
        st = o.step_given(g)
        rhs = float(np.dot(xi, diffs)) / (alpha * alpha * M * M)
        skip = np.zeros(M, bool)
        for m in range(M):
            skip[m] = (np.sum((g[m] - held[m]) ** 2) <= rhs) and clock[m] <= tbar
            if skip[m]:
                clock[m] += 1
            else:
                held[m] = g[m]
                clock[m] = 0
        np.testing.assert_array_equal(st["skip"].astype(bool), skip)
        new_theta = theta - alpha * held.sum(0)
        diffs = [float(np.sum((new_theta - theta) ** 2))] + diffs[:-1]
        theta = new_theta
        np.testing.assert_allclose(o.state(big=False)["theta"], theta, rtol=1e-10, atol=1e-13)
        total_skips += int(skip.sum())
    assert 0 < total_skips < M * K
    s = o.state(big=False)
    assert s["uploads"] == M * K - total_skips and s["bits"] == s["uploads"] * 32 * p


def test_first_iteration_uploads_and_staleness_clock():
    rng = np.random.default_rng(2)
    M, p = 6, 20
    # nearly flat workers: (7a) always holds after the first upload, so only the clock forces uploads
    _, grad = _quadratic_problem(rng, M, p, np.full(M, 1e-6))
    for tbar, mode, max_run in ((3, 0, 4), (0, 0, 1), (-1, 0, 0), (3, 1, 2), (1, 1, 0), (2, 1, 1)):
        o = oracle.OracleLaq(64, oracle.MODEL_GIVEN, M, p, alpha=0.5, b=8, D=2, xi=[0.4, 0.4], tbar=tbar,
                             clock_mode=mode)
        skips = _run_given(o, grad, 40, np.ones(p))
        assert not skips[0].any()                          # every worker uploads at k = 1
        for m in range(M):
            run = best = 0
            for s in skips[:, m]:
                run = run + 1 if s else 0
                best = max(best, run)
            assert best == max_run, (tbar, mode, best)     # Eq. (7b): bounded staleness, and attained here
        up = o.state(big=False)["uploads"]
        assert up == int((1 - skips).sum())


def test_tbar_one_never_skips_under_the_strict_clock():
    rng = np.random.default_rng(3)
    M, p = 5, 12
    _, grad = _quadratic_problem(rng, M, p, rng.uniform(1e-6, 1.0, M))
    o = oracle.OracleLaq(64, oracle.MODEL_GIVEN, M, p, alpha=0.3, b=4, D=1, xi=[0.8], tbar=1, clock_mode=1)
    assert not _run_given(o, grad, 50, np.ones(p)).any()


def test_proposition_1_upload_bound():
    """Worker m with L_m^2 <= xi_d / (3 alpha^2 M^2 D) for d <= d_m uploads at most k/(d_m+1) times
    (Proposition 1); the forced upload at k = 1 adds at most one."""
    rng = np.random.default_rng(4)
    M, p, D, alpha, K = 3, 10, 10, 0.05, 400
    xi = np.array([0.08] * 3 + [0.0008] * 7)                 # non-increasing
    thr = lambda d: np.sqrt(xi[d - 1] / (3 * alpha ** 2 * M ** 2 * D))
    Lm = np.array([1.5 * thr(1), 0.99 * thr(3), 0.99 * thr(10)])     # d_m = 0, 3, 10
    d_m = []
    for L in Lm:
        ok = [d for d in range(1, D + 1) if L ** 2 <= xi[d - 1] / (3 * alpha ** 2 * M ** 2 * D)]
        d_m.append(max(ok) if ok else 0)
    assert d_m == [0, 3, 10]
    _, grad = _quadratic_problem(rng, M, p, Lm)
    o = oracle.OracleLaq(64, oracle.MODEL_GIVEN, M, p, alpha=alpha, b=6, D=D, xi=xi, tbar=100)
    skips = _run_given(o, grad, K, np.zeros(p))
    uploads = (1 - skips).sum(0)
    for m in range(M):
        assert uploads[m] <= K / (d_m[m] + 1) + 1
        # stronger, from the proof: after an upload the next d_m iterations are skips
        run_after_upload = [int(skips[k + 1:k + 1 + d_m[m], m].sum()) for k in range(K - d_m[m] - 1) if not skips[k, m]]
        assert all(r == d_m[m] for r in run_after_upload)
    assert uploads[0] > uploads[1] > uploads[2]


@pytest.mark.parametrize("precision", [64, 32])
def test_linear_convergence_on_a_tiny_strongly_convex_problem(precision):
    """Theorem 1: with xi_d = 1/(16 D) and alpha = 1/(8 L) the loss residual and the quantization
    error both decay geometrically."""
    rng = np.random.default_rng(5)
    M, p, D = 3, 4, 5
    A = rng.standard_normal((M, 6, p))
    bvec = rng.standard_normal((M, 6))
    H = sum(a.T @ a for a in A)
    theta_star = np.linalg.solve(H, sum(a.T @ bb for a, bb in zip(A, bvec)))   # normal equations
    f = lambda th: 0.5 * sum(np.sum((a @ th - bb) ** 2) for a, bb in zip(A, bvec))
    L = np.linalg.eigvalsh(H).max()
    grad = lambda th: np.stack([a.T @ (a @ th - bb) for a, bb in zip(A, bvec)])
    o = oracle.OracleLaq(precision, oracle.MODEL_GIVEN, M, p, alpha=1.0 / (8 * L), b=4, D=D,
                         xi=np.full(D, 1.0 / (16 * D)), tbar=20)
    theta = np.zeros(p)
    res, err = [], []
    K = 1500 if precision == 64 else 500
    for k in range(K):
        g = grad(theta)
        st = o.step_given(g)
        s = o.state()
        theta = s["theta"]
        res.append(f(theta) - f(theta_star))
        err.append(st["R"].max() / 15.0)                   # tau R_m bounds ||eps_m||_inf
    res, err = np.array(res), np.array(err)
    if precision == 64:
        assert res[-1] < 1e-12
        ks = np.arange(50, 900)
        ok = res[ks] > 1e-25
        slope_res = np.polyfit(ks[ok], np.log(res[ks][ok]), 1)[0]
        slope_err = np.polyfit(ks, np.log(err[ks] + 1e-300), 1)[0]
        assert slope_res < -0.01 and slope_err < -0.005
        # geometric envelope: the residual never climbs back above an earlier level by much
        assert np.all(res[200:] < res[100])
    else:
        assert res[-1] < 1e-9 * max(res[0], 1.0)
        assert err[-1] < 1e-3 * err[0]


# ------------------------------------------------------------------------------------------------
# the stochastic variant (minibatch tests of Sec. 4)
# ------------------------------------------------------------------------------------------------
def _tiny_logreg(rng, M, n_per, F):
    X = [rng.standard_normal((n_per[m], F)).astype(np.float32) for m in range(M)]
    y = [(rng.random(n_per[m]) < 0.5).astype(np.int32) for m in range(M)]
    return X, y


def test_minibatch_window_start_is_in_range_and_spread_out():
    n = 37
    starts = np.array([[oracle.batch_offset(12345, m, k, n) for k in range(1, 2001)] for m in range(3)])
    assert starts.min() >= 0 and starts.max() < n
    for m in range(3):                                   # every start occurs, about equally often
        counts = np.bincount(starts[m], minlength=n)
        assert counts.min() > 0.5 * 2000 / n and counts.max() < 1.6 * 2000 / n
    assert not np.array_equal(starts[0], starts[1])      # workers draw different windows
    assert oracle.batch_offset(1, 0, 5, n) != oracle.batch_offset(2, 0, 5, n) or \
        oracle.batch_offset(1, 0, 6, n) != oracle.batch_offset(2, 0, 6, n)   # the seed matters
    assert oracle.batch_offset(9, 4, 7, 1) == 0


def test_minibatch_gradient_is_the_scaled_window_sum_and_unbiased():
    """g_m = (N_m / B)(1/N) sum over the window + the worker's share of the regulariser: checked against the
    full-shard routine applied to the window's rows, and averaged over all N_m window positions (each sample
    lies in exactly B windows) it equals the full gradient."""
    rng = np.random.default_rng(11)
    M, F, B, lam, alpha = 3, 5, 4, 0.125, 0.0625
    n_per = [9, 6, 11]
    N = sum(n_per)
    X, y = _tiny_logreg(rng, M, n_per, F)
    theta0 = rng.standard_normal(F).astype(np.float32)
    o = oracle.OracleLaq(64, oracle.MODEL_LOGREG_BIN, M, F, N=n_per, n_features=F, alpha=alpha, lam=lam, b=8, D=2,
                         tbar=5, seed=77, theta0=theta0, batch=B, flags=oracle.FLAG_TRIGGER_OFF | oracle.FLAG_QUANT_OFF)
    for m in range(M):
        o.set_shard(m, X[m], y[m])
    theta = theta0.astype(np.float64)
    for k in range(1, 6):
        expect = np.zeros(F)
        for m in range(M):
            st = oracle.batch_offset(77, m, k, n_per[m])
            rows = [(st + j) % n_per[m] for j in range(B)]
            _, g = oracle.grad_logreg_bin(X[m][rows], y[m][rows], theta, (n_per[m] / B) / N, n_per[m] / N, lam)
            expect += g
        o.step()                                          # GD mode: theta -= alpha sum_m g_m
        theta = theta - alpha * expect
        np.testing.assert_allclose(o.state(big=False)["theta"], theta, rtol=1e-10, atol=1e-12)
    # unbiasedness by brute force over every window position of worker 0
    th = rng.standard_normal(F)
    n0 = n_per[0]
    _, full = oracle.grad_logreg_bin(X[0], y[0], th, 1.0 / N, n0 / N, lam)
    mean = np.zeros(F)
    for st in range(n0):
        rows = [(st + j) % n0 for j in range(B)]
        _, g = oracle.grad_logreg_bin(X[0][rows], y[0][rows], th, (n0 / B) / N, n0 / N, lam)
        mean += g / n0
    np.testing.assert_allclose(mean, full, rtol=1e-12, atol=1e-14)


def test_minibatch_as_large_as_the_shard_is_the_full_gradient():
    rng = np.random.default_rng(12)
    M, F = 2, 4
    n_per = [7, 5]
    X, y = _tiny_logreg(rng, M, n_per, F)
    kw = dict(N=n_per, n_features=F, alpha=0.125, lam=0.01, b=4, D=2, tbar=5, seed=3)
    a = oracle.OracleLaq(64, oracle.MODEL_LOGREG_BIN, M, F, batch=0, **kw)
    b = oracle.OracleLaq(64, oracle.MODEL_LOGREG_BIN, M, F, batch=100, **kw)    # B_m = min(batch, N_m)
    for m in range(M):
        a.set_shard(m, X[m], y[m])
        b.set_shard(m, X[m], y[m])
    for k in range(10):
        sa, sb = a.step(), b.step()
        np.testing.assert_array_equal(sa["skip"], sb["skip"])
        np.testing.assert_allclose(b.state(big=False)["theta"], a.state(big=False)["theta"], rtol=1e-11, atol=1e-13)


# ------------------------------------------------------------------------------------------------
# Lyapunov function of Sec. 3
# ------------------------------------------------------------------------------------------------
def test_lyapunov_hand_numbers():
    """D = 2, xi = (0.25, 0.5), alpha = 0.5: c_1 = (0.25 + 0.5) / 0.5 = 1.5, c_2 = 0.5 / 0.5 = 1.
    f = (10, 7, 5, 4), steps ||theta^{k+1} - theta^k||^2 = (4, 2, 1, .), f* = 3:
      V^1 = 7                         (no earlier step exists)
      V^2 = 4 + 1.5 * 4           = 10
      V^3 = 2 + 1.5 * 2 + 1 * 4   = 9
      V^4 = 1 + 1.5 * 1 + 1 * 2   = 4.5"""
    v = oracle.lyapunov([10.0, 7.0, 5.0, 4.0], [4.0, 2.0, 1.0, 99.0], [0.25, 0.5], 0.5, 3.0)
    np.testing.assert_allclose(v, [7.0, 10.0, 9.0, 4.5], rtol=0, atol=1e-15)
    # all weights zero: the Lyapunov function is the loss residual
    v0 = oracle.lyapunov([10.0, 7.0, 5.0], [4.0, 2.0, 1.0], [0.0, 0.0, 0.0], 0.5, 3.0)
    np.testing.assert_allclose(v0, [7.0, 4.0, 2.0], rtol=0, atol=0)


def test_lyapunov_function_decays_linearly_under_the_lemma_parameters():
    """Theorem 1 on a tiny least-squares problem with xi_d = 1/(16 D), alpha = 1/(8 L): V >= f - f* >= 0, and V
    shrinks by a constant factor per iteration on average (it need not be monotone: Lemma 1 has the
    quantization errors on its right-hand side)."""
    rng = np.random.default_rng(11)
    M, p, D = 3, 4, 5
    A = rng.standard_normal((M, 6, p))
    bvec = rng.standard_normal((M, 6))
    H = sum(a.T @ a for a in A)
    theta_star = np.linalg.solve(H, sum(a.T @ bb for a, bb in zip(A, bvec)))
    f = lambda th: 0.5 * sum(np.sum((a @ th - bb) ** 2) for a, bb in zip(A, bvec))
    L = np.linalg.eigvalsh(H).max()
    alpha, xi = 1.0 / (8 * L), np.full(D, 1.0 / (16 * D))
    o = oracle.OracleLaq(64, oracle.MODEL_GIVEN, M, p, alpha=alpha, b=4, D=D, xi=xi, tbar=20)
    theta = np.zeros(p)
    losses, d2s = [], []
    for k in range(700):
        losses.append(f(theta))
        st = o.step_given(np.stack([a.T @ (a @ theta - bb) for a, bb in zip(A, bvec)]))
        d2s.append(st["dtheta2"])
        theta = o.state()["theta"]
    v = oracle.lyapunov(losses, d2s, xi, alpha, f(theta_star))
    res = np.array(losses) - f(theta_star)
    assert np.all(v >= res - 1e-15) and np.all(res > -1e-12)
    ks = np.arange(20, 500)
    ok = v[ks] > 1e-24
    sigma = np.exp(np.polyfit(ks[ok], np.log(v[ks][ok]), 1)[0])
    assert 0.0 < sigma < 0.99
    assert v[600] < 1e-10 * v[0]
    assert np.all(v[100:] < v[50])
