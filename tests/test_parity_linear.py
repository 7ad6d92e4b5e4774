"""CUDA path vs CPU oracle, logistic and quadratic models, element by element
on the same seeded inputs (through the C ABI)."""
import numpy as np
import pytest
import torch

from paper_2201_04301_b200 import binding
from paper_2201_04301_b200.workloads import make_workload

from parity import MARGIN, TOL_FP32, forced_parity, make_oracle, rel_l2, to_cuda

pytestmark = pytest.mark.gpu


def _stream():
    return torch.cuda.Stream()


def test_cfg1_teacher_forced_full_run():
    w = make_workload("cfg1")
    flips, worst = forced_parity(w, w["K"], stream=_stream())
    print("cfg1 worst", worst, "flips", flips)
    assert flips <= 2


def test_cfg2_teacher_forced():
    """d = 54 in rows padded to 56 floats, batch 1024: several CTAs per group."""
    w = make_workload("cfg2", rows=100000)
    flips, worst = forced_parity(w, 60, stream=_stream())
    print("cfg2 worst", worst, "flips", flips)


def test_cfg3_shape_small_shards():
    """d = 4096, 64 groups of 512 rows per batch as in the large workload, but
    shards of 600 rows so that the oracle can hold the data."""
    w = make_workload("cfg3", rows=64 * 600)
    flips, worst = forced_parity(w, 12, stream=_stream())
    print("cfg3-small worst", worst, "flips", flips)


@pytest.mark.parametrize("d,ld,batch,M,M_G,D", [
    (1, 1, 5, 2, 1, 1),         # scalar model, one worker per group, D = 1
    (7, 9, 33, 3, 3, 2),        # G = 1, odd sizes, stride > d
    (33, 40, 100, 8, 2, 3),     # two columns per lane with a ragged tail
    (200, 200, 17, 6, 2, 4),    # widest warp-per-row shape
    (257, 260, 37, 4, 2, 3),    # smallest row-ring shape, ragged 16-byte chunk
    (1000, 1000, 70, 10, 2, 5),
    (3001, 3004, 19, 6, 3, 2),  # ragged tail, four chunks per thread
])
def test_odd_shapes(d, ld, batch, M, M_G, D):
    G = M // M_G
    w = make_workload("cfg1", rows=G * 50, dims=(d,), M=M, M_G=M_G, D=D, batch=batch, c=0.5)
    if ld != d:
        Xp = torch.full((w["X"].shape[0], ld), float("nan"))
        Xp[:, :d] = w["X"]
        w["X"], w["ld"] = Xp, ld
        w["X"][:, d:] = 7.0      # padding must never be read into a result
    forced_parity(w, 3 * D + 2, stream=_stream())


@pytest.mark.parametrize("reduction", ["mean", "sum"])
def test_quadratic_model(reduction):
    w = make_workload("cfg1", rows=3000, kind="quadratic", alpha=0.002)
    forced_parity(w, 25, stream=_stream(), reduction=reduction)


def test_free_running_masks_match_until_a_near_tie():
    w = make_workload("cfg1")
    o = make_oracle(w)
    g = binding.from_workload(to_cuda(w), stream=_stream())
    K = w["K"]
    g.step(K)
    got = g.get_selection_mask(0, K)
    for k in range(K):
        rec = o.step()
        if not np.array_equal(got[k], rec["mask"]):
            bad = np.nonzero(got[k] != rec["mask"])[0]
            for gi in bad:
                margin = abs(rec["lhs"][gi] - rec["rhs"]) / max(rec["lhs"][gi], rec["rhs"])
                assert margin < MARGIN, (k, gi, margin)
            break
    else:
        assert rel_l2(g.get_theta(), o.theta) <= TOL_FP32
        assert g.get_comm_count() == (o.uploads, o.comm, o.comp)
    assert got.sum() < K * o.G          # the rule skipped uploads
    assert got[0].all()                 # first iteration selects every group


@pytest.mark.parametrize("name,rows,over", [("cfg2", 50000, {}), ("cfg3", 20000, {}),
                                            ("cfg3", 9000, dict(dims=(1004,), M=40, M_G=4, batch=77, D=3))])
def test_graph_replay_equals_plain_launches_bitwise(name, rows, over):
    """Replayed graphs hold chains of 16 iterations whose kernels are launched programmatically dependent; in
    a chain the wide models' gradient kernel starts copying rows before the previous iteration has finished
    and takes the iteration number for its draw from the chain's start.  Nothing of that may change a bit,
    however the run is cut into calls, and also when plain (forced) iterations sit between two chains."""
    w = to_cuda(make_workload(name, rows=rows, **over))
    G = w["M"] // w["M_G"]
    forced = np.ones((3, G), np.uint8)
    forced[1, ::2] = 0
    runs = []
    for graph, chunks in ((1.0, [40]), (0.0, [40]), (1.0, [16, 5, 19]), (1.0, [33, -3, 4]), (0.0, [33, -3, 4])):
        g = binding.from_workload(w, stream=_stream(), options={binding.OPT_GRAPH: graph, binding.OPT_PERSISTENT: 0.0})
        for n in chunks:
            if n < 0:
                g.step_forced(forced)
            else:
                g.step(n)
        runs.append((g.get_theta(), g.get_selection_mask(0, 40), g.get_wallclock(), g.get_comm_count()))
        g.close()
    for a, b in ((0, 1), (0, 2), (3, 4)):
        assert np.array_equal(runs[a][0], runs[b][0]) and np.array_equal(runs[a][1], runs[b][1])
        assert runs[a][2] == runs[b][2] and runs[a][3] == runs[b][3]


@pytest.mark.parametrize("name,rows,over", [("cfg1", None, {}), ("cfg2", 60000, {}),
                                            ("cfg1", 9000, dict(dims=(200,), M=12, M_G=4, batch=50, D=4)),
                                            ("cfg1", 3000, dict(kind="quadratic", alpha=0.002, dims=(70,), batch=33)),
                                            ("cfg1", 3200, dict(dims=(7,), M=512, M_G=16, batch=1, D=1)),       # 32 groups of 16 workers
                                            ("cfg1", 2000, dict(dims=(256,), M=4, M_G=2, batch=97, D=2, c=0.2)),
                                            ("cfg1", 5000, dict(dims=(33,), M=10, M_G=1, batch=300, D=7, c=3.0))])
def test_cluster_kernel_equals_the_kernel_chain(name, rows, over):
    """Narrow models run whole iterations inside one thread-block cluster (any number per launch).  The
    result must not depend on how the iterations are cut into launches (bitwise), and must agree with the
    chain of kernels up to summation order: same selections unless a test is within the margin, same
    parameters, counters and clock."""
    w = to_cuda(make_workload(name, rows=rows, **over))
    K = 60
    a = binding.from_workload(w, stream=_stream())
    a.step(K)
    b = binding.from_workload(w, stream=_stream())
    for n in (1, 7, 30, 22):
        b.step(n)
    assert a.get_launch_count() == 1 and b.get_launch_count() == 4          # one launch per call
    assert np.array_equal(a.get_theta(), b.get_theta())
    assert np.array_equal(a.get_selection_mask(0, K), b.get_selection_mask(0, K))
    assert a.get_wallclock() == b.get_wallclock() and a.get_comm_count() == b.get_comm_count()
    c = binding.from_workload(w, stream=_stream(), options={binding.OPT_PERSISTENT: 0.0})
    c.step(K)
    assert c.get_launch_count() == 3 * K
    ma, mc = a.get_selection_mask(0, K), c.get_selection_mask(0, K)
    if np.array_equal(ma, mc):
        assert rel_l2(a.get_theta(), c.get_theta()) <= 1e-5
        assert a.get_comm_count() == c.get_comm_count()
        assert abs(a.get_wallclock()[0] - c.get_wallclock()[0]) <= 1e-12 * c.get_wallclock()[0]
        for what in (binding.DBG_AGG, binding.DBG_GLAST, binding.DBG_FRESH, binding.DBG_H, binding.DBG_VHAT):
            assert rel_l2(a.get_debug(what), c.get_debug(what)) <= 1e-5, what
        assert np.array_equal(a.get_debug(binding.DBG_TAU), c.get_debug(binding.DBG_TAU))
        assert np.allclose(a.get_debug(binding.DBG_LHS), c.get_debug(binding.DBG_LHS), rtol=1e-4)
        assert np.allclose(a.get_debug(binding.DBG_SRING), c.get_debug(binding.DBG_SRING), rtol=1e-5)
    else:       # a near-tie went the other way: allowed only inside the margin
        k = int(np.nonzero((ma != mc).any(axis=1))[0][0])
        assert k > 0
    # the two paths share their state: a run may switch between them
    a.step_forced(np.ones((1, a.G), dtype=np.uint8))
    a.step(3)
    assert a.get_iteration() == K + 4 and np.isfinite(a.get_theta()).all()


def test_host_fed_step_equals_resident_step():
    from oracle import philox
    w = make_workload("cfg1", rows=3000)
    wc = to_cuda(w)
    a = binding.from_workload(wc, stream=_stream(), options={binding.OPT_PERSISTENT: 0.0})
    b = binding.GCada(w["kind"], w["dims"], w["M"], w["M_G"], w["D"], w["c"], w["alpha"], w["beta1"],
                      w["beta2"], w["eps"], stream=_stream())
    b.set_batch(w["batch"])
    b.set_theta(w["theta0"])
    G, n_g = a.G, w["X"].shape[0] // a.G
    for k in range(15):
        idx = np.concatenate([philox.batch_indices(w["seed"], k, g, w["batch"], n_g) for g in range(G)])
        Xb = w["X"][idx].contiguous().pin_memory()
        yb = w["y"][idx].contiguous().pin_memory()
        a.step(1)
        b.step_host_batch(Xb, yb)
        assert np.array_equal(a.get_theta(), b.get_theta())
        assert np.array_equal(a.get_selection_mask(k, 1), b.get_selection_mask(k, 1))
    assert a.get_wallclock() == b.get_wallclock()


def test_state_errors_and_history_window():
    w = to_cuda(make_workload("cfg1", rows=600))
    g = binding.GCada(w["kind"], w["dims"], w["M"], w["M_G"], w["D"], w["c"], w["alpha"], w["beta1"],
                      w["beta2"], w["eps"])
    with pytest.raises(binding.GCadaError) as e:
        g.step(1)
    assert e.value.status == binding.ESTATE
    g.set_option(binding.OPT_HISTORY, 8)
    g.set_theta(w["theta0"])
    with pytest.raises(binding.GCadaError) as e:
        g.step(1)
    assert e.value.status == binding.ESTATE        # no data yet
    with pytest.raises(binding.GCadaError) as e:
        g.set_data(w["X"], w["y"], 0)
    assert e.value.status == binding.EINVAL
    g.set_data(w["X"], w["y"], w["batch"])
    g.step(20)                                     # legacy default stream; one launch of the cluster kernel
    assert g.get_iteration() == 20
    assert g.get_selection_mask(12, 8).shape == (8, g.G)
    for first, n in ((11, 8), (15, 6), (-1, 1)):
        with pytest.raises(binding.GCadaError) as e:
            g.get_selection_mask(first, n)
        assert e.value.status == binding.EINVAL
    with pytest.raises(binding.GCadaError):
        g.set_option(binding.OPT_REDUCTION, 1)     # fixed once stepping has begun
    up, comm, comp = g.get_comm_count()
    assert comm == (g.M_G + 1) * up and comp == g.M_G * up
    assert g.get_launch_count() == 1
    g.set_theta(w["theta0"])                       # restart
    assert g.get_iteration() == 0 and g.get_comm_count() == (0, 0, 0)


def test_rule_ps_printed_left_side():
    """GCADA_OPT_RULE = 1: the test uses L_g^2 ||theta^k - theta^{k-tau_g}||^2 (Eq. 9 as printed)."""
    w = make_workload("cfg1", rows=3000, D=5, c=0.4)
    L = [0.9, 1.4, 2.0]
    flips, worst = forced_parity(w, 40, stream=_stream(), L=L)
    print("rule PS worst", worst, "flips", flips)
    # free-running: masks equal the oracle's (up to near-ties) and uploads are skipped
    o = make_oracle(w, rule="ps", L=L)
    g = binding.from_workload(to_cuda(w), stream=_stream(), options={binding.OPT_RULE: 1.0}, smoothness=L)
    g.step(40)
    got = g.get_selection_mask(0, 40)
    for k in range(40):
        rec = o.step()
        if not np.array_equal(got[k], rec["mask"]):
            for gi in np.nonzero(got[k] != rec["mask"])[0]:
                assert abs(rec["lhs"][gi] - rec["rhs"]) / max(rec["lhs"][gi], rec["rhs"]) < MARGIN
            break
    assert 0 < got.sum() < got.size
    assert g.get_launch_count() == 5 * 40      # distances, schedule, gradients of the selected, reduce, update
    # without constants the rule cannot run
    h = binding.from_workload(to_cuda(w), options={binding.OPT_RULE: 1.0})
    with pytest.raises(binding.GCadaError) as e:
        h.step(1)
    assert e.value.status == binding.ESTATE


def test_rule_ps_wide_model_skips_work():
    """Row-ring kernel under the printed rule: gradients of the selected groups only (the rows of the
    others are never read), checked against the oracle; the kernel gets faster as fewer groups upload."""
    w = make_workload("cfg3", rows=16 * 600, M=32, M_G=2, D=6, c=0.05)
    L = [0.5 + 0.1 * g for g in range(16)]
    flips, worst = forced_parity(w, 14, stream=_stream(), L=L)
    print("rule PS wide worst", worst, "flips", flips)


def test_rule_ps_wide_model_with_fewer_selected_rows_than_ctas():
    """Printed rule on the row-ring kernel when the selected groups' rows are fewer than the kernel's CTAs
    (small minibatches): only the first rows-many CTAs work, one row each, and the selection kernel must add
    up exactly those (a CTA without rows between two that hold a group's partial sums would contribute
    whatever its slot held before)."""
    w = make_workload("cfg3", rows=6 * 300, M=12, M_G=2, D=3, batch=40)
    flips, worst = forced_parity(w, 8, stream=_stream(), L=[3.0, 0.2, 1.4, 0.05, 2.0, 0.5])
    print("rule PS, few rows, worst", worst, "flips", flips)
