"""The generalisations the paper names without using them (per-lag constants
{c_d} of Algorithm 1's input list, a step size alpha^k that depends on k,
computing-time laws other than the exponential) against the CPU oracle, and
checkpoints, all through the C ABI."""
import numpy as np
import pytest
import torch

from paper_2201_04301_b200 import binding
from paper_2201_04301_b200.workloads import make_workload

from parity import TOL_BF16, forced_parity, make_oracle, rel_l2, to_cuda

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("schedule,law", [(("poly", 7.0, 0.5), "pareto"), (("step", 5, 0.7), "uniform"),
                                          (("const",), "exp")])
def test_lag_weights_schedule_and_delay_law_against_the_oracle(schedule, law):
    w = make_workload("cfg1")
    c_d = [2.0, 1.5, 1.0, 0.8, 0.6, 0.4, 0.3, 0.2, 0.1, 0.05]
    flips, worst = forced_parity(w, 40, stream=torch.cuda.Stream(), c_d=c_d, schedule=schedule, delay_law=law)
    assert worst["theta"] <= 1e-5
    # free-running: same selections as the oracle (margins are wide on this workload)
    g = binding.from_workload(to_cuda(w), stream=torch.cuda.Stream(), c_d=c_d, schedule=schedule, delay_law=law)
    o = make_oracle(w, c_d=c_d, schedule=schedule, delay_law=law)
    g.step(40)
    for _ in range(40):
        o.step()
    masks = g.get_selection_mask(0, 40)
    if np.array_equal(masks, np.stack(o.masks)):
        assert rel_l2(g.get_theta(), o.theta) <= 1e-5
        assert abs(g.get_wallclock()[0] - o.wall) <= 1e-12 * o.wall
    g.close()


def test_equal_lag_weights_change_nothing():
    w = to_cuda(make_workload("cfg1"))
    a = binding.from_workload(w, stream=torch.cuda.Stream())
    b = binding.from_workload(w, stream=torch.cuda.Stream(), c_d=[w["c"]] * w["D"], schedule=("poly", 3.0, 0.0))
    a.step(60)
    b.step(60)
    assert np.array_equal(a.get_selection_mask(0, 60), b.get_selection_mask(0, 60))
    assert np.array_equal(a.get_theta(), b.get_theta())


def test_setter_validation():
    w = to_cuda(make_workload("cfg1"))
    g = binding.from_workload(w)
    for bad in (lambda: g.set_lag_weights([1.0, 2.0]), lambda: g.set_lag_weights([-1.0] * w["D"]),
                lambda: g.set_step_schedule("poly", 0.0, 1.0), lambda: g.set_step_schedule("step", 2.5, 0.5),
                lambda: g.set_step_schedule(7), lambda: g.set_delay_law(3)):
        with pytest.raises(binding.GCadaError) as e:
            bad()
        assert e.value.status == binding.EINVAL
    g.step(1)
    with pytest.raises(binding.GCadaError) as e:
        g.set_lag_weights([1.0] * w["D"])
    assert e.value.status == binding.ESTATE


def _workload(name):
    if name == "logistic":
        return make_workload("cfg1"), {}
    if name == "wide":
        return make_workload("cfg3", rows=64 * 520), {}
    if name == "mlp":
        return make_workload("cfg4", rows=5 * 400), {}
    if name == "mlp_bf16":
        return make_workload("cfg5", rows=3000, dims=(64, 128, 96, 40), M=6, M_G=2, D=3, batch=128, c=0.3), {}
    return make_workload("cfg5", rows=3000, dims=(64, 128, 40), M=6, M_G=2, D=3, batch=128, c=0.3), {binding.OPT_KEEP_STALE: 1.0}


@pytest.mark.parametrize("name", ["logistic", "wide", "mlp", "mlp_bf16", "mlp_bf16_inspect"])
def test_checkpoint_resumes_bit_for_bit(name):
    w, opts = _workload(name)
    w = to_cuda(w)
    a = binding.from_workload(w, stream=torch.cuda.Stream(), options=opts)
    a.step(17)
    ck = a.checkpoint_save()
    a.step(21)
    b = binding.from_workload(w, stream=torch.cuda.Stream(), options=opts)
    b.step(3)                      # a run of its own that the load replaces
    b.checkpoint_load(ck)
    assert b.get_iteration() == 17
    b.step(21)
    assert np.array_equal(a.get_theta(), b.get_theta())
    assert np.array_equal(a.get_selection_mask(0, 38), b.get_selection_mask(0, 38))
    assert a.get_comm_count() == b.get_comm_count() and a.get_wallclock() == b.get_wallclock()
    for what in (binding.DBG_AGG, binding.DBG_H, binding.DBG_VHAT, binding.DBG_TAU, binding.DBG_SRING):
        assert np.array_equal(a.get_debug(what), b.get_debug(what))
    # a context of another shape refuses the checkpoint and keeps its own state
    other = dict(w)
    other["D"] = w["D"] + 1
    c = binding.from_workload(other, stream=torch.cuda.Stream(), options=opts)
    c.step(2)
    with pytest.raises(binding.GCadaError) as e:
        c.checkpoint_load(ck)
    assert e.value.status == binding.EINVAL and c.get_iteration() == 2
    with pytest.raises(binding.GCadaError):
        b.checkpoint_load(ck[:-8])
