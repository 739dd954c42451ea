"""Workers spread over several contexts, on one GPU.

(1) The two halves of an iteration (laq_step_local + laq_apply_uploads) in a context that holds all workers equal
    laq_step bit for bit.
(2) Two contexts that play ranks 0 and 1 of a two-rank job (workers split round robin), with the exchange of the
    upload messages done by plain copies between their workspaces, reproduce the single-context run bit for bit:
    theta, the aggregated gradient, every worker's Q_m, clocks, counters.  The contexts' kernels run one after the
    other on one stream; nothing waits for anything.
The collective itself (torch.distributed) is covered on CPU by tests/test_sharded_exchange.py.
"""
import numpy as np
import pytest

from paper_1909_07588_b200 import laq, sharded, workloads

pytestmark = pytest.mark.gpu


def _cases():
    return {"synthetic": lambda: workloads.c4(M=7, p=150_001, b=4, iters=12),
            "synthetic_b3": lambda: workloads.c4(M=5, p=40_003, b=3, iters=12),
            "logreg": lambda: workloads.c0(iters=30),
            "softmax": lambda: workloads.c1(n_per=240, iters=15),
            "network": lambda: workloads.c3(n_per=300, M=5, iters=8)}


@pytest.mark.parametrize("name", list(_cases()))
def test_split_iteration_equals_laq_step(name):
    w = _cases()[name]()
    a = laq.from_workload(w)
    b = laq.from_workload(w)
    for _ in range(w.iters):
        a.step(1)
        b.step_local()
        m, R = b.local_uploads()
        b.apply_uploads(m, R)
    sa, sb = a.get_state(codes=True), b.get_state(codes=True)
    for key in ("theta", "agg", "qprev", "clock", "ring", "n_eps_hat", "counters", "codes"):
        np.testing.assert_array_equal(sa[key], sb[key])
    assert 0 < sa["uploads"] < w.M * w.iters or name == "network"
    a.close()
    b.close()


@pytest.mark.parametrize("world", [2, 3])
@pytest.mark.parametrize("name", list(_cases()))
def test_ranks_on_one_gpu_reproduce_the_single_context_run(name, world):
    w = _cases()[name]()
    ref = laq.from_workload(w)
    ranks = [laq.from_workload(w, world=world, rank=r) for r in range(world)]
    assert sum(c.M for c in ranks) == w.M
    sent_bits = 0
    for k in range(w.iters):
        ref.step(1)
        for c in ranks:
            c.step_local()
        ups = [c.local_uploads() for c in ranks]
        m_all = np.concatenate([u[0] for u in ups])
        R_all = np.concatenate([u[1] for u in ups])
        order = np.argsort(m_all)
        m_all, R_all = m_all[order], R_all[order]
        for m in m_all:                                  # the wire: owner's code row -> everybody else's mailbox
            src = ranks[sharded.owner_of(int(m), world)]
            row = src.code_row((int(m) - src.rank) // world)
            for c in ranks:
                if c is not src:
                    c.mailbox_row(int(m)).copy_(row)
            sent_bits += sharded.message_bits(w.b, w.p)
        for c in ranks:
            c.apply_uploads(m_all, R_all)
    s = ref.get_state()
    for c in ranks:
        t = c.get_state()
        np.testing.assert_array_equal(t["theta"], s["theta"])
        np.testing.assert_array_equal(t["agg"], s["agg"])
        np.testing.assert_array_equal(t["ring"], s["ring"])
        np.testing.assert_array_equal(t["counters"], s["counters"])          # uploads and bits count all workers
        np.testing.assert_array_equal(t["qprev"], s["qprev"][c.rank::world])
        np.testing.assert_array_equal(t["clock"], s["clock"][c.rank::world])
        np.testing.assert_array_equal(t["n_eps_hat"], s["n_eps_hat"][c.rank::world])
    assert s["bits"] == sent_bits                                           # what crossed the wire is what is counted
    for c in ranks:
        c.close()
    ref.close()


def test_spread_context_rejects_the_whole_iteration_call_and_bad_lists():
    w = workloads.c4(M=4, p=1000, b=4)
    c = laq.from_workload(w, world=2, rank=1)
    with pytest.raises(laq.LaqError) as e:
        c.step(1)
    assert e.value.status == laq.LAQ_ESTATE
    c.step_local()
    c.local_uploads()
    for bad in ([2, 1], [0, 0], [5], [-1]):
        with pytest.raises(laq.LaqError) as e:
            c.apply_uploads(bad, [1.0] * len(bad))
        assert e.value.status == laq.LAQ_EINVAL
    with pytest.raises(laq.LaqError):
        laq.Laq(model=laq.MODEL_SYNTH, M=4, p=100, b=4, world=2, rank=2)
    with pytest.raises(laq.LaqError):
        laq.Laq(model=laq.MODEL_SYNTH, M=4, p=100, b=4, world=2, rank=0, flags=laq.FLAG_QUANT_OFF)
    c.close()
