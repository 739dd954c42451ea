"""Convergence diagnostics of Sec. 3 computed from the per-iteration report of the CUDA path.

The Lyapunov function of LAQ couples the loss residual with the last D squared parameter differences, the same
quantities the skip rule (7a) weighs:

    V(theta^k) = f(theta^k) - f(theta*) + sum_{d=1..D} c_d ||theta^{k+1-d} - theta^{k-d}||^2,
    c_d = (xi_d + xi_{d+1} + ... + xi_D) / alpha.

Lemma 1 bounds V(theta^{k+1}) by sigma_1 V(theta^k) plus the quantization errors, and Theorem 1 states that V and
the quantization error tau R_m >= ||eps_m||_inf decay at a linear rate when sum_d xi_d and alpha meet the lemma's
conditions (for instance xi_d = 1/(16 D), alpha = 1/(8 L)).  The kernels already report f(theta^k) and
||theta^{k+1} - theta^k||^2 every iteration, so the diagnostics are arithmetic on D + 1 numbers per iteration.

    python -m paper_1909_07588_b200.diagnostics --workload c0 --iters 400
"""
import argparse
import json

import numpy as np


def lyapunov_weights(xi, alpha):
    """c_d for d = 1..D: the tail sums of xi divided by alpha."""
    xi = np.asarray(xi, np.float64)
    return np.cumsum(xi[::-1])[::-1] / float(alpha)


def lyapunov(loss, dtheta2, xi, alpha, f_star):
    """V(theta^k) for k = 1..n.  loss[k-1] = f(theta^k) and dtheta2[k-1] = ||theta^{k+1} - theta^k||^2 are the
    `loss` and `dtheta2` columns of a trace that starts at the first iteration; differences from before the first
    iteration count as zero (the library's initial state)."""
    loss, d2 = np.asarray(loss, np.float64), np.asarray(dtheta2, np.float64)
    c = lyapunov_weights(xi, alpha)
    # past[k-1] = sum_d c_d d2[k-1-d]: a correlation of the difference history with the weights
    padded = np.concatenate([np.zeros(len(c)), d2])
    past = np.array([np.dot(c, padded[k + len(c) - 1::-1][:len(c)]) for k in range(len(d2))])
    return loss - float(f_star) + past


def quantization_error_bound(R, b):
    """(tau R_m)^2 >= ||eps_m^k||_inf^2 per iteration and worker, tau = 1 / (2^b - 1) (Theorem 1's second claim)."""
    tau = 1.0 / float((1 << int(b)) - 1)
    return (tau * np.asarray(R, np.float64)) ** 2


def linear_rate(v, lo=0, hi=None, floor=0.0):
    """Least-squares estimate of sigma in v_k ~ C sigma^k over k in [lo, hi), using the entries above `floor`."""
    v = np.asarray(v, np.float64)
    hi = len(v) if hi is None else hi
    ks = np.arange(lo, hi)
    ok = v[lo:hi] > floor
    if ok.sum() < 2:
        return float("nan")
    return float(np.exp(np.polyfit(ks[ok], np.log(v[lo:hi][ok]), 1)[0]))


def run(w, iters, f_star, chunk=512):
    """Runs `iters` LAQ iterations of workload w on the GPU and returns the diagnostics per iteration."""
    from . import laq
    ctx = laq.from_workload(w, trace_capacity=chunk)
    cols = {k: [] for k in ("loss", "dtheta2", "R", "uploads")}
    done = 0
    while done < iters:
        n = min(chunk, iters - done)
        tr = ctx.step(n, trace=True)
        for k in cols:
            cols[k].append(tr[k])
        done += n
    ctx.close()
    loss, d2 = np.concatenate(cols["loss"]), np.concatenate(cols["dtheta2"])
    R, up = np.concatenate(cols["R"]), np.concatenate(cols["uploads"])
    return {"V": lyapunov(loss, d2, w.xi, w.alpha, f_star), "residual": loss - f_star,
            "eps_bound": quantization_error_bound(R, w.b).max(axis=1), "uploads": up}


def main():
    from . import compare, workloads
    ap = argparse.ArgumentParser(description="Lyapunov function and quantization error of a LAQ run (Sec. 3)")
    ap.add_argument("--workload", default="c0", choices=["c0", "c1", "c2"])
    ap.add_argument("--iters", type=int, default=400)
    ap.add_argument("--fstar-iters", type=int, default=20000)
    a = ap.parse_args()
    w = {"c0": workloads.c0, "c1": workloads.c1, "c2": workloads.c2}[a.workload]()
    f_star = compare.optimal_loss(w, a.fstar_iters)
    d = run(w, a.iters, f_star)
    half = a.iters // 2
    print(json.dumps({"workload": w.name, "f_star": f_star, "V_first": float(d["V"][0]), "V_last": float(d["V"][-1]),
                      "rate_V": linear_rate(d["V"], 0, half, floor=1e-12),
                      "rate_eps_bound": linear_rate(d["eps_bound"], 0, half, floor=1e-30),
                      "uploads": int(d["uploads"].sum())}))


if __name__ == "__main__":
    main()
