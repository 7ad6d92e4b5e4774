"""Degenerate and boundary shapes through the C ABI, against the oracle."""
import numpy as np
import pytest
import torch

from paper_2201_04301_b200 import binding
from paper_2201_04301_b200.workloads import make_workload

from parity import forced_parity, to_cuda

pytestmark = pytest.mark.gpu


def _stream():
    return torch.cuda.Stream()


def test_single_sample_batches_and_one_row_shards():
    # batch of one row per group; shards of exactly one row (every draw is that row)
    w = make_workload("cfg1", rows=3, dims=(9,), M=3, M_G=1, D=2, batch=1)
    forced_parity(w, 8, stream=_stream())
    w = make_workload("cfg1", rows=50, dims=(300,), M=2, M_G=1, D=2, batch=1)
    forced_parity(w, 6, stream=_stream())


def test_widest_supported_linear_model_and_the_first_unsupported():
    w = make_workload("cfg1", rows=200, dims=(4096,), M=4, M_G=2, D=2, batch=9)
    forced_parity(w, 5, stream=_stream())
    with pytest.raises(binding.GCadaError) as e:
        binding.GCada("logistic", (4097,), 4, 2, 2, 1.0, 0.01, 0.9, 0.99, 1e-8)
    assert e.value.status == binding.EINVAL


def test_misaligned_wide_rows_are_rejected_not_misread():
    w = to_cuda(make_workload("cfg1", rows=100, dims=(512,), M=2, M_G=1, D=2, batch=4))
    g = binding.GCada("logistic", (512,), 2, 1, 2, 1.0, 0.01, 0.9, 0.99, 1e-8)
    Xp = torch.zeros(100, 514, device="cuda")
    Xp[:, :512] = w["X"]
    with pytest.raises(binding.GCadaError) as e:
        g.set_data(Xp, w["y"], 4, ld=514)              # row stride not a multiple of 4 floats
    assert e.value.status == binding.EINVAL
    with pytest.raises(binding.GCadaError) as e:
        g.set_data(w["X"], w["y"], 4, ld=511)          # stride smaller than d
    assert e.value.status == binding.EINVAL
    with pytest.raises(binding.GCadaError) as e:
        g.set_data(w["X"][:1], w["y"][:1], 4)           # fewer rows than groups
    assert e.value.status == binding.EINVAL


def test_many_groups_and_workers_per_group():
    # 300 groups (more than one 256-group pass of the scheduling phase), 5 workers each; D = 1: everyone, always
    w = make_workload("cfg1", rows=300 * 4, dims=(6,), M=1500, M_G=5, D=1, batch=2)
    forced_parity(w, 4, stream=_stream())
    g = binding.from_workload(to_cuda(w), stream=_stream())
    g.step(5)
    assert g.get_selection_mask(0, 5).all()
    up, comm, comp = g.get_comm_count()
    assert (up, comm, comp) == (1500, 1500 * 6, 1500 * 5)


def test_zero_iterations_and_getters_before_stepping():
    w = to_cuda(make_workload("cfg1", rows=600))
    g = binding.from_workload(w, stream=_stream())
    g.step(0)
    assert g.get_iteration() == 0 and g.get_wallclock() == (0.0, 0.0) and g.get_comm_count() == (0, 0, 0)
    assert np.array_equal(g.get_theta(), w["theta0"].cpu().numpy())
    with pytest.raises(binding.GCadaError):
        g.get_selection_mask(0, 1)


def test_mlp_batch_not_a_multiple_of_the_tile_and_single_class_margin():
    w = make_workload("cfg4", rows=400, dims=(20, 3), M=2, M_G=1, D=2, batch=65, alpha=0.01)
    forced_parity(w, 6, stream=_stream())
    w = make_workload("cfg5", rows=900, dims=(24, 40, 8), M=3, M_G=1, D=2, batch=200)   # padded to 256 rows
    forced_parity(w, 5, tol=2e-2, stream=_stream(), rhs_tol=2e-2)
    with pytest.raises(binding.GCadaError) as e:                                        # beyond the bf16 path's limit
        h = binding.from_workload(to_cuda(make_workload("cfg5", rows=900, dims=(24, 8), M=3, M_G=1, D=2, batch=300)))
        h.step(1)
    assert e.value.status == binding.EINVAL


def test_special_cases_distributed_adam_and_cada():
    """c = 0: every group uploads every iteration (the 'distributed Adam' of Section V); M_G = 1: groups are
    single workers and the scheme is CADA (Section III).  Both against the oracle, and the mean simulated
    wall-clock of the first against the order-statistics formula (Eq. 10): with G groups of M_G workers,
    shift 1 and rate 1 the server waits 1 + H_G / M_G per iteration on average."""
    w = make_workload("cfg1", rows=3000, c=0.0)
    forced_parity(w, 30, stream=_stream())
    g = binding.from_workload(to_cuda(make_workload("cfg1", c=0.0)), stream=_stream())
    K = 6000
    g.step(K)
    assert g.get_selection_mask(K - 50, 50).all()
    assert g.get_comm_count() == (3 * K, 3 * 3 * K, 3 * 2 * K)
    mean = g.get_wallclock()[0] / K
    want = 1.0 + (1 + 1 / 2 + 1 / 3) / 2
    assert abs(mean - want) < 5 * 0.45 / np.sqrt(K), (mean, want)      # sd of the max of three Exp(2) is < 0.45
    w = make_workload("cfg1", rows=3000, M=5, M_G=1, c=2.0)
    forced_parity(w, 30, stream=_stream())
    h = binding.from_workload(to_cuda(w), stream=_stream())
    h.step(100)
    up, comm, comp = h.get_comm_count()
    assert comm == 2 * up and comp == up and 0 < up < 500               # Eqs. (18), (21) with equality


def test_forced_masks_that_starve_a_group_beyond_the_maximum_delay():
    """The rule itself never lets an age exceed D.  A forced mask can; the library then documents its own
    behaviour (it keeps D+1 iterates): the stale iterate is the oldest one kept, theta^{k-D}.  That is
    outside the method's domain, so the expectation is built here from the oracle's model and iterates,
    not taken from the oracle's step (which goes back the literal tau_g iterates).  Linear, wide linear,
    both MLPs."""
    import numpy as np
    from parity import TOL_BF16, TOL_FP32, make_oracle, rel_l2
    cases = [(make_workload("cfg1", rows=3000, D=3), TOL_FP32),
             (make_workload("cfg3", rows=3 * 300, M=6, M_G=2, D=3, batch=40), TOL_FP32),
             (make_workload("cfg4", rows=3 * 300, dims=(30, 16, 5), M=6, M_G=2, D=3, batch=24), 1e-4),
             (make_workload("cfg5", rows=3 * 300, dims=(64, 72, 10), M=6, M_G=2, D=3, batch=128), TOL_BF16)]
    for w, tol in cases:
        o = make_oracle(w)
        D = o.D
        g = binding.from_workload(to_cuda(w), stream=_stream(), options={binding.OPT_KEEP_STALE: 1.0})
        masks = np.ones((12, 3), dtype=np.uint8)
        masks[1:10, 1] = 0                       # group 1 is not selected for nine iterations, D = 3
        beyond = 0
        for k in range(12):
            _, Xb, yb = o.minibatch(1)
            tau1 = int(o.tau[1])
            rec = o.step(forced_mask=masks[k])
            g.step_forced(masks[k][None, :])
            assert np.array_equal(g.get_debug(binding.DBG_TAU), o.tau)
            if tau1 <= D:
                want_stale, want_lhs = rec["stale"][1], rec["lhs"][1]
            else:                                 # the library's documented choice: theta^{k-D}
                beyond += 1
                want_stale = o.model.grad(o.theta_at(k - D), Xb, yb, "mean")
                want_lhs = float(np.sum((rec["fresh"][1] - want_stale) ** 2))
                assert not np.array_equal(want_stale, rec["stale"][1])
            stale = g.get_debug(binding.DBG_STALE)
            assert rel_l2(stale[1], want_stale) <= tol, (w["name"], k)
            assert abs(g.get_debug(binding.DBG_LHS)[1] - want_lhs) <= 2 * tol * max(want_lhs, 1e-30) + 1e-30
        assert beyond == 7
        assert rel_l2(g.get_theta(), o.theta) <= tol
        g.close()
