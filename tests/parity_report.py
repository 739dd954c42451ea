"""First disagreement between the CUDA library and the free-running fp64 oracle, per workload, as a table.

    python -m tests.parity_report [--c2-iters N] [--c1-iters N] [--c3-iters N]      (needs a B200)

Runs the model-parity comparison of tests/test_gpu_parity.py (every assertion of it included) on the four model
workloads at full size and prints one markdown row each: iterations run, the first iteration at which a skip bit
differs from the oracle's, a code differs, theta or the loss leaves the 1e-4 band, and the counts of classified
near-ties.  The oracle's cost bounds the iteration counts of the softmax and network workloads.
"""
import argparse
import json
import time

from paper_1909_07588_b200 import workloads
from tests import test_gpu_parity as T


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--c2-iters", type=int, default=1000)
    ap.add_argument("--c1-iters", type=int, default=40)
    ap.add_argument("--c3-iters", type=int, default=4)
    ap.add_argument("--json", default=None)
    a = ap.parse_args()
    runs = [("C0", workloads.c0(), 200),
            ("C1", workloads.c1(iters=a.c1_iters), a.c1_iters),
            ("C2", workloads.c2(iters=a.c2_iters, theta0_scale=0.01), a.c2_iters),
            ("C3", workloads.c3(iters=a.c3_iters), a.c3_iters)]
    rows, recs = [], {}
    for name, w, iters in runs:
        t0 = time.time()
        rec = T._run_model_parity(w, iters)
        rec["seconds"] = time.time() - t0
        recs[name] = rec
        rows.append("| %s | %d | %s | %s | %s | %s | %d of %d | %d | %.2g |" % (
            name, iters, rec["first_disagreement"], rec["first_skip_diff"], rec["first_code_diff"],
            rec["first_band_exit"], rec["near_tie_flips"], rec["codes_compared"], rec["skip_ties"], rec["max_coord_err"]))
    print("| workload | iterations | first disagreement | first skip-bit difference | first code difference | "
          "left the 1e-4 band | near-tie codes (restarted comparison) | skip near-ties | largest gradient coordinate error |")
    print("|---|---|---|---|---|---|---|---|---|")
    print("\n".join(rows))
    if a.json:
        with open(a.json, "w") as f:
            json.dump(recs, f, indent=1)


if __name__ == "__main__":
    main()
