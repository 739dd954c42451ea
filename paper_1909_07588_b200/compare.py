"""Iterations, uploads and bits of GD, QGD, LAG and LAQ on one workload (the quantities of Table 2, Sec. 4).

The four methods are modes of the same CUDA path:
    GD   Eq. (2)        LAQ_FLAG_QUANT_OFF | LAQ_FLAG_TRIGGER_OFF   every worker sends 32 p bits every iteration
    QGD  Algorithm 1    LAQ_FLAG_TRIGGER_OFF                        every worker sends 32 + b p bits every iteration
    LAG  (Sec. 4)       LAQ_FLAG_QUANT_OFF                          32 p bits, only when the skip rule fires
    LAQ  Algorithm 2    0                                           32 + b p bits, only when (7a)/(7b) fire
A run stops either after a fixed number of iterations (the paper's rule for the network) or at the first iteration
whose loss is within `residual` of f*, the loss GD reaches after `fstar_iters` iterations (the paper's rule for
logistic regression, residual 1e-6).  The inputs are the seeded synthetic stand-ins of `workloads`, so the counts are
not the paper's; the ordering of the methods is what carries over.  With --batch B every method uses minibatch
gradients of B samples per worker (the stochastic tests of Sec. 4: SGD and SLAQ are then the rows GD and LAQ; the
loss column is the minibatch estimate).

    python -m paper_1909_07588_b200.compare --workload c0 --residual 1e-6
    python -m paper_1909_07588_b200.compare --workload c1 --batch 500 --bits 3 --max-iters 1000
"""
import argparse
import json

import numpy as np

from . import laq, workloads

MODES = (("GD", laq.FLAG_QUANT_OFF | laq.FLAG_TRIGGER_OFF), ("QGD", laq.FLAG_TRIGGER_OFF),
         ("LAG", laq.FLAG_QUANT_OFF), ("LAQ", 0))


def _losses(ctx, n, chunk):
    """Yields (loss at theta^k, uploads of iteration k) for k = 1..n, stepping `chunk` iterations per call."""
    done = 0
    while done < n:
        c = min(chunk, n - done)
        tr = ctx.step(c, trace=True)
        for j in range(c):
            yield float(tr["loss"][j]), int(tr["uploads"][j])
        done += c


def optimal_loss(w, iters, chunk=512):
    """Smallest loss along `iters` iterations of gradient descent, Eq. (2)."""
    ctx = laq.from_workload(w, trace_capacity=chunk, flags=MODES[0][1])
    best = min(l for l, _ in _losses(ctx, iters, chunk))
    ctx.close()
    return best


def run_mode(w, flags, max_iters, f_star=None, residual=None, chunk=512, batch=0):
    """One method until the loss residual is reached (or for max_iters iterations when residual is None)."""
    ctx = laq.from_workload(w, trace_capacity=chunk, flags=flags, batch=batch)
    per_upload = 32 * w.p if flags & laq.FLAG_QUANT_OFF else 32 + w.b * w.p
    iters = uploads = 0
    loss = float("nan")
    reached = residual is None
    for loss, up in _losses(ctx, max_iters, chunk):
        if residual is not None and loss - f_star <= residual:
            reached = True            # theta^k already meets the target: iteration k's uploads are not needed
            break
        iters += 1
        uploads += up
    ctx.close()
    return {"iterations": iters, "uploads": uploads, "bits": uploads * per_upload, "loss": loss, "reached": reached}


def compare(w, max_iters, residual=None, fstar_iters=None, chunk=512, batch=0):
    f_star = None
    if residual is not None:
        f_star = optimal_loss(w, fstar_iters or 4 * max_iters, chunk)
    rows = {}
    for name, flags in MODES:
        rows[name] = run_mode(w, flags, max_iters, f_star, residual, chunk, batch)
    return {"workload": w.name, "M": w.M, "p": w.p, "b": w.b, "alpha": w.alpha, "f_star": f_star, "batch": batch,
            "residual": residual, "rows": rows}


def main():
    ap = argparse.ArgumentParser(description=__doc__.split("\n")[0])
    ap.add_argument("--workload", default="c0", choices=["c0", "c1", "c2", "c3"])
    ap.add_argument("--max-iters", type=int, default=20000)
    ap.add_argument("--residual", type=float, default=None, help="stop at loss - f* <= residual (else fixed iterations)")
    ap.add_argument("--fstar-iters", type=int, default=None)
    ap.add_argument("--bits", type=int, default=None, help="bits per coordinate (1, 2, 3, 4, 8 or 16)")
    ap.add_argument("--batch", type=int, default=0, help="minibatch size per worker (0 = full gradients)")
    ap.add_argument("--alpha", type=float, default=None, help="step size (default: the workload's)")
    ap.add_argument("--json", action="store_true")
    a = ap.parse_args()
    w = {"c0": workloads.c0, "c1": workloads.c1, "c2": workloads.c2, "c3": workloads.c3}[a.workload]()
    if a.bits:
        w.b = a.bits
    if a.alpha:
        w.alpha = a.alpha
    res = compare(w, a.max_iters, a.residual, a.fstar_iters, batch=a.batch)
    if a.json:
        print(json.dumps(res))
        return
    print("%s  M=%d p=%d b=%d alpha=%.4g batch=%d  f*=%s residual=%s" % (res["workload"], w.M, w.p, w.b, w.alpha,
                                                                        a.batch, res["f_star"], res["residual"]))
    print("%-5s %12s %14s %14s %14s" % ("", "iterations", "uploads", "bits", "loss"))
    for name, r in res["rows"].items():
        print("%-5s %12d %14d %14.3e %14.8f%s" % (name, r["iterations"], r["uploads"], r["bits"], r["loss"],
                                                  "" if r["reached"] else "  (residual not reached)"))


if __name__ == "__main__":
    main()
