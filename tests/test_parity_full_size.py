"""Parity at the full workload sizes, in the launch configuration the benchmark
times (graph replay on a stream): the CUDA path runs free, then sampled groups'
gradients are recomputed by the CPU oracle from the CUDA path's own iterate and
the rows it must have sampled, and properties that hold at any size are checked."""
import numpy as np
import pytest
import torch

from oracle import philox
from oracle.models import make_model
from paper_2201_04301_b200 import binding
from paper_2201_04301_b200.workloads import make_workload

from parity import LHS_TOL_BF16, TOL_BF16, TOL_FP32, rel_l2

pytestmark = pytest.mark.gpu


def _group_batch(w, k, g, G):
    n_g = w["X"].shape[0] // G
    idx = philox.batch_indices(w["seed"], k, g, w["batch"], n_g)
    t = torch.as_tensor(idx, device=w["X"].device)
    d = w["dims"][0]
    return w["X"].index_select(0, t)[:, :d].float().cpu().numpy().astype(np.float64), w["y"].index_select(0, t).cpu().numpy()


def test_cfg3_full_size_sampled_groups():
    """d = 4096, N = 2,000,000 (32.8 GB resident), 64 groups x 512 rows."""
    w = make_workload("cfg3", device="cuda")
    G = w["M"] // w["M_G"]
    g = binding.from_workload(w, stream=torch.cuda.Stream())
    model = make_model("logistic", w["dims"])
    K = 24
    for k in range(K):
        theta = g.get_theta().astype(np.float64)
        g.step(1)
        if k in (0, 7, 23):
            for gi in (0, 31, 63):
                Xb, yb = _group_batch(w, k, gi, G)
                want = model.grad(theta, Xb, yb, "mean")
                assert rel_l2(g.get_group_gradient(binding.DBG_FRESH, gi), want) <= TOL_FP32
    masks = g.get_selection_mask(0, K)
    up, comm, comp = g.get_comm_count()
    assert masks[0].all() and up == int(masks.sum()) and comm == (w["M_G"] + 1) * up and comp == w["M_G"] * up
    # no group goes D iterations without an upload
    for gi in range(G):
        gaps = np.diff(np.nonzero(masks[:, gi])[0])
        assert gaps.size == 0 or gaps.max() <= w["D"]
    # the aggregate equals the sum of the last uploaded gradients (Eq. 3)
    agg = g.get_debug(binding.DBG_AGG).astype(np.float64)
    assert rel_l2(agg, g.get_debug(binding.DBG_GLAST).astype(np.float64).sum(axis=0)) <= 1e-6
    g.step(200)                       # replayed graphs, 16 iterations each
    assert g.get_iteration() == K + 200 and np.isfinite(g.get_theta()).all()


def test_cfg5_full_size_sampled_groups():
    """1024-4096-4096-1000, bf16 operands, 256 groups x 128 rows.  The first iteration is forced to
    upload eight groups only: two of their gradients (rebuilt from the kept factors) are recomputed by
    the oracle, and the aggregate must be the sum of the eight (Eq. 3)."""
    w = make_workload("cfg5", device="cuda")
    G = w["M"] // w["M_G"]
    g = binding.from_workload(w, stream=torch.cuda.Stream())
    model = make_model("mlp", w["dims"], bf16=True)
    theta = g.get_theta().astype(np.float64)
    chosen = (3, 40, 77, 100, 131, 200, 201, 255)
    mask0 = np.zeros((1, G), dtype=np.uint8)
    mask0[0, list(chosen)] = 1
    g.step_forced(mask0)
    total = np.zeros(g.p, dtype=np.float64)
    for gi in chosen:
        got = g.get_group_gradient(binding.DBG_GLAST, gi)
        total += got
        if gi in (3, 200):
            Xb, yb = _group_batch(w, 0, gi, G)
            assert rel_l2(got, model.grad(theta, Xb, yb, "mean")) <= TOL_BF16
    assert rel_l2(g.get_debug(binding.DBG_AGG), total) <= 1e-5
    assert not g.get_group_gradient(binding.DBG_GLAST, 0).any()      # never uploaded
    g.step(12)
    masks = g.get_selection_mask(0, 13)
    assert masks[1, np.setdiff1d(np.arange(G), chosen)].all()        # the others' age passed D: selected by the age rule
    up, comm, comp = g.get_comm_count()
    assert up == int(masks.sum()) and comm == 5 * up and comp == 4 * up
    assert np.isfinite(g.get_theta()).all()


def test_cfg5_full_size_groups_at_different_ages():
    """1024-4096-4096-1000 at full size on the production path (norm-only weight-gradient pass, uploads
    kept as factors, running aggregate).  Forced masks leave the groups at ages 1, 2 and 3, so the row tiles
    of one launch read three different slots of the weight ring and the stale iterates differ from the
    fresh one.  For one group of each age the left side of the test and - where the group uploads - its
    gradient are recomputed by the oracle from the CUDA path's own iterates theta^k and theta^{k - tau_g}
    on the rows that must have been drawn.  The masks of iterations 1-3 select a third of the groups at an
    iteration that is not a multiple of 16: the aggregate is then updated in place (old uploads out, new
    ones in) and must still be the sum of the groups' last uploads (Eq. 3), checked on slices of every
    layer against all 256 uploads rebuilt from their factors."""
    w = make_workload("cfg5", device="cuda")
    G = w["M"] // w["M_G"]
    g = binding.from_workload(w, stream=torch.cuda.Stream())
    model = make_model("mlp", w["dims"], bf16=True)
    gs = np.arange(G)
    tau = np.full(G, w["D"])
    thetas = []
    probe = (3, 40, 77)                       # g % 3 = 0, 1, 2: ages 2, 3, 1 at iteration 3
    worst = dict(lhs=0.0, upload=0.0)
    for k in range(4):
        thetas.append(g.get_theta().astype(np.float64))
        mask = np.ones(G, dtype=np.uint8) if k == 0 else ((k + gs) % 3 == 1).astype(np.uint8)
        g.step_forced(mask[None, :])
        assert np.array_equal(g.get_debug(binding.DBG_TAU), np.where(mask, 1, tau + 1))
        if k >= 2:
            lhs = g.get_debug(binding.DBG_LHS)
            if k == 3:
                assert sorted(int(tau[gi]) for gi in probe) == [1, 2, 3]
            for gi in probe:
                Xb, yb = _group_batch(w, k, gi, G)
                fresh = model.grad(thetas[k], Xb, yb, "mean")
                stale = model.grad(thetas[k - int(tau[gi])], Xb, yb, "mean")
                want = float(np.sum((fresh - stale) ** 2))
                worst["lhs"] = max(worst["lhs"], abs(lhs[gi] - want) / want)
                if mask[gi]:
                    worst["upload"] = max(worst["upload"], rel_l2(g.get_group_gradient(binding.DBG_GLAST, gi), fresh))
        tau = np.where(mask, 1, tau + 1)
    print("cfg5 full size, groups at ages 1-3: worst", worst)
    assert worst["lhs"] <= LHS_TOL_BF16 and worst["upload"] <= TOL_BF16 and worst["upload"] > 0
    # Eq. (3) after three in-place updates of the aggregate: slices of every layer's weights and biases
    dims, o, slices = w["dims"], 0, []
    for l in range(1, len(dims)):
        n_w = dims[l] * dims[l - 1]
        slices += [slice(o, o + 50000), slice(o + n_w // 2, o + n_w // 2 + 50000), slice(o + n_w - 4096, o + n_w + dims[l])]
        o += n_w + dims[l]
    idx = np.concatenate([np.arange(sl.start, sl.stop) for sl in slices])
    total = np.zeros(idx.size, dtype=np.float64)
    for gi in range(G):
        total += g.get_group_gradient(binding.DBG_GLAST, gi)[idx]
    agg = g.get_debug(binding.DBG_AGG)[idx].astype(np.float64)
    err = rel_l2(agg, total)
    print("cfg5 full size: aggregate vs sum of the 256 rebuilt uploads on %d entries: %.2e" % (idx.size, err))
    # the aggregate is ONE product per layer whose reduction runs over all 256 x 128 rows with fp32
    # accumulation in tensor memory: 2048 accumulation steps of 16 rows, each rounding to 2^-24 relative,
    # give up to 2048 * 2^-24 = 1.2e-4 (measured 8.7e-5); the rebuilt uploads are summed in double here
    assert err <= 2e-4


@pytest.mark.parametrize("name,tol", [("cfg1", TOL_FP32), ("cfg2", TOL_FP32), ("cfg4", TOL_FP32)])
def test_small_workloads_at_full_size(name, tol):
    """The latency-bound workloads at their full sizes, free-running under graph replay: every group's
    fresh gradient at sampled iterations against the oracle's gradient at the CUDA path's own iterate on
    the rows it must have drawn; counters and Eq. (3) throughout."""
    w = make_workload(name, device="cuda")
    G = w["M"] // w["M_G"]
    g = binding.from_workload(w, stream=torch.cuda.Stream())
    model = make_model(w["kind"], w["dims"])
    K = 40
    for k in range(K):
        theta = g.get_theta().astype(np.float64)
        g.step(1)
        if k in (0, 11, 39):
            for gi in range(G):
                Xb, yb = _group_batch(w, k, gi, G)
                want = model.grad(theta, Xb, yb, "mean")
                got = g.get_group_gradient(binding.DBG_FRESH, gi)
                kinks = w["kind"] == "mlp" and model.near_kinks(theta, Xb, 2e-6)
                assert rel_l2(got, want) <= (tol if not kinks else 1e-3), (k, gi)
    masks = g.get_selection_mask(0, K)
    up, comm, comp = g.get_comm_count()
    assert masks[0].all() and up == int(masks.sum()) and comm == (w["M_G"] + 1) * up and comp == w["M_G"] * up
    agg = g.get_debug(binding.DBG_AGG).astype(np.float64)
    assert rel_l2(agg, g.get_debug(binding.DBG_GLAST).astype(np.float64).sum(axis=0)) <= 1e-6
    g.step(w["K"] - K)                # the rest of the workload's run, 16 iterations per replayed graph
    assert g.get_iteration() == w["K"] and np.isfinite(g.get_theta()).all()
