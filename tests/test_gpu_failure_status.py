"""Failure status of the C ABI on a GPU, without faulting or hanging the device.

A wait inside a kernel is bounded; when it runs out the kernel records it, stops waiting, returns, and the next
synchronising call reports LAQ_ETIMEOUT.  The branch is exercised in the one safe way: the loader that feeds the
waiting consumer is told (laq_tune "starve_copies") to issue none of its asynchronous copies and the consumer polls
with a short limit, so the wait runs out while nothing is in flight.
"""
import numpy as np
import pytest

import oracle
from paper_1909_07588_b200 import laq, workloads

pytestmark = pytest.mark.gpu


def test_starved_ring_wait_runs_out_and_is_reported_as_timeout():
    w = workloads.c4(M=4, p=300_007, b=8, iters=8)
    ctx = laq.from_workload(w, trace_capacity=4)
    ref = laq.from_workload(w, trace_capacity=4)
    ctx.step(2)
    ref.step(2)
    ctx.sync()
    before = ctx.get_state()
    ctx.tune("starve_copies", 1)
    with pytest.raises(laq.LaqError) as e:
        ctx.step(1, trace=True)
    assert e.value.status == laq.LAQ_ETIMEOUT and "bounded wait" in str(e.value)
    # frozen at that iteration: later steps change nothing, every synchronising call keeps reporting it
    ctx.step(3)
    with pytest.raises(laq.LaqError) as e:
        ctx.sync()
    assert e.value.status == laq.LAQ_ETIMEOUT
    with pytest.raises(laq.LaqError) as e:
        ctx.get_worker(0)
    assert e.value.status == laq.LAQ_ETIMEOUT
    # the device and its context are fine: another context keeps running
    tr_ref = ref.step(4, trace=True)
    # clearing the condition (laq_set_state) resumes the run from the frozen iteration, bit for bit
    ctx.tune("starve_copies", 0)
    ctx.set_state()
    after = ctx.get_state()
    assert after["k"] == before["k"] == 2
    for key in ("theta", "agg", "qprev", "clock", "ring", "n_eps_hat"):
        np.testing.assert_array_equal(after[key], before[key])
    tr = ctx.step(4, trace=True)
    for key in tr:
        np.testing.assert_array_equal(tr[key], tr_ref[key])
    a, b = ctx.get_state(codes=True), ref.get_state(codes=True)
    for key in ("theta", "agg", "qprev", "codes", "counters"):
        np.testing.assert_array_equal(a[key], b[key])
    ctx.close()
    ref.close()


def test_starved_tensor_core_stage_runs_out_and_is_reported_as_timeout():
    """The network's fused hidden-layer kernel: the loader of one block issues no tile copies, the tensor-core warp's
    wait for the first stage runs out, the block gives its tensor memory back and returns."""
    w = workloads.c3(n_per=300, M=3, iters=6)
    ctx = laq.from_workload(w, trace_capacity=4)
    ref = laq.from_workload(w, trace_capacity=4)
    ctx.step(2)
    ref.step(2)
    before = ctx.get_state()
    ctx.tune("starve_copies", 1)
    with pytest.raises(laq.LaqError) as e:
        ctx.step(1, trace=True)
    assert e.value.status == laq.LAQ_ETIMEOUT
    tr_ref = ref.step(3, trace=True)                  # the device is fine
    ctx.tune("starve_copies", 0)
    ctx.set_state()
    after = ctx.get_state()
    assert after["k"] == before["k"] == 2
    np.testing.assert_array_equal(after["theta"], before["theta"])
    tr = ctx.step(3, trace=True)
    for key in tr:
        np.testing.assert_array_equal(tr[key], tr_ref[key])
    np.testing.assert_array_equal(ctx.get_state()["theta"], ref.get_state()["theta"])
    ctx.close()
    ref.close()


def test_timeout_status_is_distinct_from_the_other_failures():
    assert len({laq.LAQ_OK, laq.LAQ_EINVAL, laq.LAQ_EWORKSPACE, laq.LAQ_ECUDA, laq.LAQ_ENONFINITE, laq.LAQ_ESTATE,
                laq.LAQ_ETIMEOUT}) == 7
    ctx = laq.Laq(model=laq.MODEL_SYNTH, M=2, p=1000, b=4)
    with pytest.raises(laq.LaqError):
        ctx.tune("starve_copies", 2)                  # outside the documented values
    assert ctx.query("sweep_threads") > 0
    with pytest.raises(laq.LaqError):
        ctx.query("no_such_key")
    ctx.close()


def test_invalid_clock_bound_and_weights_are_rejected():
    for bad in (dict(tbar=-2), dict(tbar=2 ** 31 - 1), dict(xi=[0.1, float("nan")]), dict(xi=[-0.1, 0.1])):
        kw = dict(model=laq.MODEL_SYNTH, M=2, p=100, b=4, D=2, xi=[0.1, 0.1], tbar=5)
        kw.update(bad)
        with pytest.raises(laq.LaqError) as e:
            laq.Laq(**kw)
        assert e.value.status == laq.LAQ_EINVAL
    with pytest.raises(laq.LaqError) as e:
        laq.Laq(model=laq.MODEL_EXTERNAL, M=2, p=100, b=4, flags=laq.FLAG_STORE_G)
    assert e.value.status == laq.LAQ_EINVAL
