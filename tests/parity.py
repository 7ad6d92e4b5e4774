"""Helpers shared by the GPU parity tests: build the CPU oracle and the CUDA
context from the same seeded workload and compare them step by step."""
import numpy as np
import torch

from oracle.gcada import GCadaOracle
from oracle.models import make_model
from paper_2201_04301_b200 import binding

TOL_FP32 = 1e-5      # relative L2, gradients and parameters, fp32 paths
TOL_BF16 = 2e-2      # relative L2 with bf16 operands
MARGIN = 1e-4        # selection test: relative margin below which a flip is allowed
MARGIN_BF16 = 4 * TOL_BF16   # the same with bf16 operands: both sides of the test carry up to 2 * TOL_BF16
LHS_TOL_FP32 = 1e-4  # relative error of the left side of the test (a squared norm), fp32 paths
LHS_TOL_BF16 = 4e-2  # ... with bf16 operands


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a))


class DeviceRows:
    """Rows of a CUDA matrix fetched on demand (for data sets too large to copy)."""

    def __init__(self, X, d):
        self.X, self.d = X, d

    def __getitem__(self, idx):
        t = torch.as_tensor(np.asarray(idx), device=self.X.device)
        return self.X.index_select(0, t)[:, :self.d].float().cpu().numpy()


def make_oracle(w, lazy=False, **kw):
    d = w["dims"][0]
    model = make_model(w["kind"], w["dims"], bf16=(w["compute"] == "bf16"))
    if lazy:
        X, y = DeviceRows(w["X"], d), DeviceRows(w["y"].reshape(-1, 1), 1)

        class _Y:
            def __init__(self, t):
                self.t = t

            def __len__(self):
                return self.t.shape[0]

            def __getitem__(self, idx):
                i = torch.as_tensor(np.asarray(idx), device=self.t.device)
                return self.t.index_select(0, i).cpu().numpy()
        y = _Y(w["y"])
    else:
        X = w["X"][:, :d].float().cpu().numpy().astype(np.float64)
        y = w["y"].cpu().numpy()
    args = dict(X=X, y=y, batch=w["batch"], theta0=w["theta0"].cpu().numpy().astype(np.float64),
                seed=w["seed"], shift=w["shift"], rate=w["rate"])
    args.update(kw)
    return GCadaOracle(model, w["M"], w["M_G"], w["D"], w["c"], w["alpha"], w["beta1"], w["beta2"], w["eps"],
                       **args)


def to_cuda(w):
    w = dict(w)
    for key in ("X", "y", "theta0"):
        w[key] = w[key].cuda()
    return w


def _kink_match(o, got, theta, Xb, yb, reduction, tol, kink_tol):
    """A ReLU unit whose pre-activation is zero to within rounding may be
    switched either way; both gradients are valid.  True if `got` equals the
    oracle gradient for some admissible choice on the (few) such units."""
    import itertools
    ks = o.model.near_kinks(theta, Xb, kink_tol)
    if not ks or len(ks) > 8:
        return False
    for n in range(1, len(ks) + 1):
        for sub in itertools.combinations(ks, n):
            if rel_l2(got, o.model.grad(theta, Xb, yb, reduction, flip=sub)) <= tol:
                return True
    return False


def forced_parity(w, K, tol=TOL_FP32, stream=None, reduction="mean", check_stale=True, kink_tol=2e-6,
                  margin=None, rhs_tol=1e-4, L=None, c_d=None, schedule=None, delay_law=None, lhs_tol=None,
                  options=None):
    """Run the oracle free for K steps and the CUDA path teacher-forced with the
    oracle's masks; compare every step.  Returns the number of steps at which
    the CUDA path's own test outcome differed from the oracle's (only allowed
    within the margin: MARGIN for fp32 arithmetic, MARGIN_BF16 with bf16
    operands) and the worst relative errors seen.  The left side of the test
    is compared too: within `lhs_tol` relative, plus - where the two gradients
    are formed separately in fp32 and subtracted (the fp32 MLP) - what their
    rounding leaves of a small difference."""
    bf16 = w["compute"] == "bf16"
    if margin is None:
        margin = MARGIN_BF16 if bf16 else MARGIN
    if lhs_tol is None:
        lhs_tol = LHS_TOL_BF16 if bf16 else LHS_TOL_FP32
    extra = {"rule": "ps", "L": L} if L is not None else {}
    if c_d is not None:
        extra["c_d"] = c_d
    if schedule is not None:
        extra["schedule"] = schedule
    if delay_law is not None:
        extra["delay_law"] = delay_law
    o = make_oracle(w, reduction=reduction, **extra)
    wc = to_cuda(w)
    opts = {binding.OPT_KEEP_STALE: 1.0, binding.OPT_REDUCTION: 0.0 if reduction == "mean" else 1.0}
    if L is not None:
        opts[binding.OPT_RULE] = 1.0
    opts.update(options or {})
    g = binding.from_workload(wc, stream=stream, options=opts, smoothness=L, c_d=c_d, schedule=schedule,
                              delay_law=delay_law)
    flips = 0
    worst = dict(fresh=0.0, stale=0.0, theta=0.0, lhs=0.0, kinks=0)
    is_mlp = w["kind"] == "mlp"
    for k in range(K):
        tau_before = g.get_debug(binding.DBG_TAU)
        batches = [o.minibatch(gi) for gi in range(o.G)] if is_mlp else None
        th_now = o.thetas[o.k]
        th_old = [o.theta_at(o.k - int(o.tau[gi])) for gi in range(o.G)]
        rec = o.step()
        g.step_forced(rec["mask"][None, :])
        fresh, stale = g.get_debug(binding.DBG_FRESH), g.get_debug(binding.DBG_STALE)
        for gi in range(o.G):
            for name, got, want, th in (("fresh", fresh[gi], rec["fresh"][gi], th_now),
                                        ("stale", stale[gi], rec["stale"][gi], th_old[gi])):
                if name == "stale" and not check_stale:
                    continue
                # printed rule on a linear model: only the selected groups compute, and only at theta^k
                if L is not None and not is_mlp and (name == "stale" or not rec["mask"][gi]):
                    continue
                e = rel_l2(got, want)
                if e > tol and is_mlp and _kink_match(o, got, th, batches[gi][1], batches[gi][2], reduction, tol, kink_tol):
                    worst["kinks"] += 1
                    continue
                worst[name] = max(worst[name], e)
                assert e <= tol, (name, k, gi, e)
        lhs, rhs = g.get_debug(binding.DBG_LHS), g.get_debug(binding.DBG_RHS)[0]
        assert np.array_equal(tau_before, rec["tau"]), (k, tau_before, rec["tau"])
        assert abs(rhs - rec["rhs"]) <= rhs_tol * max(rec["rhs"], 1e-300), (k, rhs, rec["rhs"])
        # the CUDA path's own decision, from its own numbers
        own = (tau_before >= o.D) | (lhs > rhs)
        for gi in range(o.G):
            if bool(own[gi]) != bool(rec["mask"][gi]):
                rel = abs(rec["lhs"][gi] - rec["rhs"]) / max(rec["lhs"][gi], rec["rhs"], 1e-300)
                assert rel < margin, ("mask", k, gi, lhs[gi], rhs, rec["lhs"][gi], rec["rhs"])
                flips += 1
            if rec["lhs"][gi] > 0 and L is None:
                # fp32 MLP: fresh and stale gradients are rounded to fp32 before they are subtracted, so an
                # absolute error e ~ 2^-23 (|fresh| + |stale|) stays in the difference whatever its size
                e_abs = 0.0
                if is_mlp and not bf16:
                    e_abs = 2.0 ** -22 * (np.linalg.norm(rec["fresh"][gi]) + np.linalg.norm(rec["stale"][gi]))
                slack = 2.0 * np.sqrt(rec["lhs"][gi]) * e_abs + e_abs * e_abs
                err = max(abs(lhs[gi] - rec["lhs"][gi]) - slack, 0.0) / rec["lhs"][gi]
                worst["lhs"] = max(worst["lhs"], err)
                assert err <= lhs_tol or worst["kinks"] > 0, ("lhs", k, gi, lhs[gi], rec["lhs"][gi])
            elif L is not None and rec["lhs"][gi] > 0:
                err = abs(lhs[gi] - rec["lhs"][gi]) / rec["lhs"][gi]
                worst["lhs"] = max(worst["lhs"], err)
                assert err <= lhs_tol, ("lhs (printed rule)", k, gi, lhs[gi], rec["lhs"][gi])
        e = rel_l2(g.get_theta(), rec["theta"])
        worst["theta"] = max(worst["theta"], e)
        # after a differing (equally valid) ReLU choice the two runs carry different gradients
        assert e <= (tol if worst["kinks"] == 0 else 30 * tol), ("theta", k, e)
        assert np.allclose(g.get_debug(binding.DBG_TGROUP), rec["t_g"], rtol=1e-12, atol=0)
    assert np.array_equal(g.get_selection_mask(0, K), np.stack(o.masks))
    assert g.get_comm_count() == (o.uploads, o.comm, o.comp)
    wall, last = g.get_wallclock()
    assert abs(wall - o.wall) <= 1e-12 * max(o.wall, 1.0) and abs(last - rec["dt"]) <= 1e-12 * max(rec["dt"], 1.0)
    assert g.get_iteration() == K
    assert rel_l2(g.get_debug(binding.DBG_AGG), rec["agg"]) <= (tol if worst["kinks"] == 0 else 1e-2)
    g.close()
    return flips, worst
