"""GD, QGD, LAG and LAQ as modes of the CUDA path: the ordering of Table 2 (Sec. 4) on the small logistic workload."""
import pytest

from paper_1909_07588_b200 import compare, workloads

pytestmark = pytest.mark.gpu


def test_table_2_ordering_on_the_small_logistic_workload():
    w = workloads.c0()
    res = compare.compare(w, max_iters=3000, residual=1e-6)
    r = res["rows"]
    assert all(v["reached"] for v in r.values())
    # GD and QGD upload from every worker at every iteration
    assert r["GD"]["uploads"] == w.M * r["GD"]["iterations"] and r["QGD"]["uploads"] == w.M * r["QGD"]["iterations"]
    assert r["GD"]["bits"] == r["GD"]["uploads"] * 32 * w.p
    assert r["QGD"]["bits"] == r["QGD"]["uploads"] * (32 + w.b * w.p)
    # the lazy rules save most of the rounds at about the same number of iterations
    for lazy in ("LAG", "LAQ"):
        assert r[lazy]["uploads"] < 0.5 * r["GD"]["uploads"]
        assert r[lazy]["iterations"] <= 1.5 * r["GD"]["iterations"]
    # and LAQ sends the fewest bits
    assert r["LAQ"]["bits"] < min(r["GD"]["bits"], r["QGD"]["bits"], r["LAG"]["bits"])


def test_fixed_iteration_budget_counts_every_upload():
    w = workloads.c0()
    res = compare.compare(w, max_iters=64)
    for name, row in res["rows"].items():
        assert row["iterations"] == 64 and row["reached"]
    assert res["rows"]["GD"]["uploads"] == 64 * w.M
