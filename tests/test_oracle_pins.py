"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA path.  Each one is meant to fail for a
plausible mistake somewhere in oracle/: a dropped term, a wrong sign or index,
a transposed operand, a wrong recursion.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import philox
from oracle.gcada import GCadaOracle
from oracle.models import MLP, Logistic, Quadratic, round_to_bf16

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# --------------------------------------------------------------------------
# random numbers
# --------------------------------------------------------------------------
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        v = [int(x, 16) for x in r]
        out = philox.philox4x32_10(*v[:6])
        assert [int(o) for o in out] == v[6:]


def test_batch_indices_stay_in_shard_and_are_uniform():
    n_g, B = 1000, 4096
    for g in (0, 3):
        idx = philox.batch_indices(7, 5, g, B, n_g)
        assert idx.min() >= g * n_g and idx.max() < (g + 1) * n_g
    # chi-square against the uniform law over 50 bins, many iterations
    counts = np.zeros(50)
    for k in range(20):
        idx = philox.batch_indices(0, k, 2, B, n_g) - 2 * n_g
        counts += np.bincount(idx * 50 // n_g, minlength=50)
    expected = counts.sum() / 50
    chi2 = ((counts - expected) ** 2 / expected).sum()
    assert chi2 < 100.0            # 49 dof: P(chi2 > 100) ~ 2e-5
    # different (k, g, seed) give different batches; same arguments repeat
    a = philox.batch_indices(0, 1, 0, 64, n_g)
    assert np.array_equal(a, philox.batch_indices(0, 1, 0, 64, n_g))
    assert not np.array_equal(a, philox.batch_indices(0, 2, 0, 64, n_g))
    assert not np.array_equal(a % n_g, philox.batch_indices(0, 1, 1, 64, n_g) % n_g)
    assert not np.array_equal(a, philox.batch_indices(1, 1, 0, 64, n_g))
    # word j of the stream is the same whatever the batch length
    assert np.array_equal(a[:10], philox.batch_indices(0, 1, 0, 10, n_g))


def test_delays_follow_the_shifted_exponential_law():
    from scipy import stats
    o = _toy_oracle(M=8, M_G=2, shift=1.0, rate=2.0)
    T = []
    for k in range(600):
        o.k = k
        T.append(o.delays())
    T = np.concatenate(T)
    assert T.min() > 1.0
    # Section II-B: exponential computing time (here shifted by 1, mean 1/rate)
    assert stats.kstest(T - 1.0, "expon", args=(0, 0.5)).pvalue > 1e-3
    # independent across workers: correlation of two workers' streams ~ 0
    T = T.reshape(600, 8)
    assert abs(np.corrcoef(T[:, 0], T[:, 1])[0, 1]) < 0.15


# --------------------------------------------------------------------------
# model gradients: central finite differences of the written-out loss
# --------------------------------------------------------------------------
def _fd(model, theta, Xb, yb, reduction):
    g = np.zeros_like(theta)
    for i in range(len(theta)):
        e = np.zeros_like(theta)
        e[i] = 1e-6
        g[i] = (model.loss(theta + e, Xb, yb, reduction) - model.loss(theta - e, Xb, yb, reduction)) / 2e-6
    return g


@pytest.mark.parametrize("reduction", ["mean", "sum"])
def test_gradients_match_finite_differences(reduction):
    rng = np.random.default_rng(0)
    Xb = rng.normal(size=(7, 5))
    for model, yb in ((Logistic(5), rng.integers(0, 2, 7).astype(float)),
                      (Quadratic(5), rng.normal(size=7))):
        theta = rng.normal(size=5)
        g = model.grad(theta, Xb, yb, reduction)
        assert np.allclose(g, _fd(model, theta, Xb, yb, reduction), rtol=1e-6, atol=1e-8)
    mlp = MLP((5, 4, 6, 3))
    theta = rng.normal(size=mlp.p) * 0.5
    yb = rng.integers(0, 3, 7)
    g = mlp.grad(theta, Xb, yb, reduction)
    assert g.shape == (mlp.p,) and mlp.p == 5 * 4 + 4 + 4 * 6 + 6 + 6 * 3 + 3
    assert np.allclose(g, _fd(mlp, theta, Xb, yb, reduction), rtol=1e-5, atol=1e-8)


def test_logistic_and_mlp_gradients_match_autograd():
    """The library routine: torch autograd of binary / softmax cross-entropy."""
    rng = np.random.default_rng(1)
    Xb = rng.normal(size=(9, 6))
    yb = rng.integers(0, 2, 9).astype(float)
    th = torch.tensor(rng.normal(size=6), requires_grad=True)
    loss = torch.nn.functional.binary_cross_entropy_with_logits(
        torch.tensor(Xb) @ th, torch.tensor(yb), reduction="mean")
    loss.backward()
    assert np.allclose(Logistic(6).grad(th.detach().numpy(), Xb, yb, "mean"), th.grad.numpy(), rtol=1e-10)

    mlp = MLP((6, 5, 4))
    theta = rng.normal(size=mlp.p)
    cls = rng.integers(0, 4, 9)
    t = torch.tensor(theta, requires_grad=True)
    W1 = t[:30].reshape(5, 6)
    b1 = t[30:35]
    W2 = t[35:55].reshape(4, 5)
    b2 = t[55:59]
    z = torch.relu(torch.tensor(Xb) @ W1.T + b1) @ W2.T + b2
    torch.nn.functional.cross_entropy(z, torch.tensor(cls), reduction="sum").backward()
    assert np.allclose(mlp.grad(theta, Xb, cls, "sum"), t.grad.numpy(), rtol=1e-10, atol=1e-12)


def test_bf16_rounding():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, 1.0 + 3 * 2 ** -8, -0.1, 3.0e38, 1e-3])
    want = torch.tensor(x, dtype=torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(round_to_bf16(x), want)
    # ties go to even: 1 + 2^-8 lies midway between 1 and 1 + 2^-7
    assert round_to_bf16(np.array([1.0 + 2 ** -8]))[0] == 1.0
    assert round_to_bf16(np.array([1.0 + 3 * 2 ** -8]))[0] == 1.0 + 2 ** -6


# --------------------------------------------------------------------------
# Eq. (8a-c): the update
# --------------------------------------------------------------------------
def test_update_closed_form_under_a_constant_gradient():
    g = np.array([0.5, -2.0, 1e-3])
    a, b1, b2, eps = 0.01, 0.9, 0.99, 1e-8
    th, h, vh = np.zeros(3), np.zeros(3), np.zeros(3)
    for k in range(1, 30):
        new, h, vh = GCadaOracle.amsgrad(th, h, vh, g, a, b1, b2, eps)
        assert np.allclose(h, (1 - b1 ** k) * g, rtol=1e-12)
        assert np.allclose(vh, (1 - b2 ** k) * g * g, rtol=1e-12)
        assert np.allclose(th - new, a * (1 - b1 ** k) * g / np.sqrt(eps + (1 - b2 ** k) * g * g), rtol=1e-12)
        th = new


def test_update_equals_library_amsgrad_while_v_grows():
    """While the gradient magnitude does not shrink, v^{k+1} >= v-hat^k, so
    Eq. (8) coincides with textbook AMSGrad; torch's implementation applies
    bias corrections, undone here through the step size, and puts epsilon
    outside the root, so epsilon is taken negligible on both sides."""
    a, b1, b2 = 0.01, 0.9, 0.99
    grads = [np.array([0.1 * (k + 1), -0.3 * (k + 1) ** 0.5]) for k in range(12)]
    t = torch.zeros(2, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([t], lr=a, betas=(b1, b2), eps=0.0, amsgrad=True)
    th, h, vh = np.zeros(2), np.zeros(2), np.zeros(2)
    for k, g in enumerate(grads, start=1):
        for grp in opt.param_groups:
            grp["lr"] = a * (1 - b1 ** k) / math.sqrt(1 - b2 ** k)
        t.grad = torch.tensor(g)
        opt.step()
        th, h, vh = GCadaOracle.amsgrad(th, h, vh, g, a, b1, b2, 1e-300)
        assert np.allclose(th, t.detach().numpy(), rtol=1e-9)


def test_update_uses_vhat_in_the_second_moment_as_printed():
    """Eq. (8b) builds v^{k+1} from v-hat^k.  Gradients 1, 0, 0 by hand:
    v-hat stays at (1-b2) because b2*(1-b2) < (1-b2); textbook AMSGrad would
    carry v = b2^2 (1-b2) but the same v-hat, so the check is on h and on the
    step, plus a sequence where the two recursions differ in v-hat."""
    a, b1, b2, eps = 0.1, 0.5, 0.5, 1e-12
    th, h, vh = np.zeros(1), np.zeros(1), np.zeros(1)
    seq = [1.0, 0.0, 0.9]
    # by hand, paper's recursion: vh1 = .5 ; v2 = .25 -> vh2 = .5 ;
    # v3 = .5*.5 + .5*.81 = .655 -> vh3 = .655
    # textbook: v2 = .25, v3 = .125 + .405 = .53 -> vh3 = .53 (different)
    want_vh = [0.5, 0.5, 0.655]
    want_h = [0.5, 0.25, 0.575]
    for g, wv, wh in zip(seq, want_vh, want_h):
        new, h, vh = GCadaOracle.amsgrad(th, h, vh, np.array([g]), a, b1, b2, eps)
        assert vh[0] == pytest.approx(wv, rel=1e-12)
        assert h[0] == pytest.approx(wh, rel=1e-12)
        assert (th - new)[0] == pytest.approx(a * wh / math.sqrt(eps + wv), rel=1e-12)
        th = new


def test_vhat_is_monotone_on_a_real_run():
    o = _toy_oracle()
    prev = o.vhat.copy()
    for _ in range(25):
        o.step()
        assert np.all(o.vhat >= prev)
        prev = o.vhat.copy()


# --------------------------------------------------------------------------
# selection rule, aggregation, AoI
# --------------------------------------------------------------------------
def _toy_oracle(M=6, M_G=2, D=4, c=1.0, N=600, d=5, batch=8, kind="logistic", seed=3, **kw):
    rng = np.random.default_rng(11)
    X = rng.normal(size=(N, d))
    if kind == "logistic":
        y = (rng.random(N) < 0.5).astype(float)
        model = Logistic(d)
    else:
        y = X @ rng.normal(size=d) + 0.1 * rng.normal(size=N)
        model = Quadratic(d)
    args = dict(X=X, y=y, batch=batch, theta0=np.zeros(d), seed=seed)
    args.update(kw)
    return GCadaOracle(model, M, M_G, D, c, 0.01, 0.9, 0.99, 1e-8, **args)


def test_quadratic_innovation_closed_form():
    """For the quadratic loss the gradient change on a fixed minibatch is
    (X_B^T X_B / B)(theta - theta_old), whatever the labels."""
    o = _toy_oracle(kind="quadratic", c=5.0)
    for _ in range(8):
        k = o.k
        tau = o.tau.copy()
        batches = [o.minibatch(g) for g in range(o.G)]
        rec = o.step()
        for g in range(o.G):
            _, Xb, _ = batches[g]
            dth = o.thetas[k] - o.theta_at(k - tau[g])
            delta = Xb.T @ (Xb @ dth) / len(Xb)
            assert rec["lhs"][g] == pytest.approx(float(delta @ delta), rel=1e-9, abs=1e-30)


def test_logistic_innovation_obeys_the_smoothness_bound():
    """||delta_g|| <= L ||theta^k - theta_old|| with L = max_i ||x_i||^2 / 4
    (mean-reduced logistic loss): the sense in which Eq. (9)'s left side is an
    estimate of the gradient change."""
    o = _toy_oracle(c=50.0, D=6)
    for _ in range(15):
        k, tau = o.k, o.tau.copy()
        batches = [o.minibatch(g) for g in range(o.G)]
        rec = o.step()
        for g in range(o.G):
            Xb = batches[g][1]
            L = (Xb ** 2).sum(axis=1).max() / 4
            dth = o.thetas[k] - o.theta_at(k - tau[g])
            assert rec["lhs"][g] <= L * L * float(dth @ dth) * (1 + 1e-12) + 1e-30
    # same point twice gives exactly no innovation
    assert rec["lhs"].min() >= 0.0


def test_innovation_rule_reduces_to_eq9_for_scalar_unit_features():
    """d = 1, x = 1, quadratic loss: gradient = theta - mean(y_B), so the
    innovation is (theta^k - theta^{k-tau})^2, i.e. Eq. (9) with L_g = 1.
    Both rules must then produce the same masks and the same trajectory."""
    N = 40
    X = np.ones((N, 1))
    y = np.linspace(-1, 1, N)
    kw = dict(X=X, y=y, batch=4, theta0=np.array([0.3]), seed=5)
    a = GCadaOracle(Quadratic(1), 4, 2, 3, 0.8, 0.05, 0.9, 0.99, 1e-8, rule="innov", **kw)
    b = GCadaOracle(Quadratic(1), 4, 2, 3, 0.8, 0.05, 0.9, 0.99, 1e-8, rule="ps", L=[1.0, 1.0], **kw)
    skipped = 0
    for _ in range(40):
        ra, rb = a.step(), b.step()
        assert np.array_equal(ra["mask"], rb["mask"])
        assert np.allclose(ra["lhs"], rb["lhs"], rtol=1e-9, atol=1e-30)
        skipped += int((ra["mask"] == 0).sum())
    assert np.allclose(a.theta, b.theta, rtol=1e-12)
    assert skipped > 0          # the rule actually skipped something


def test_scalar_trajectory_by_hand():
    """Two groups, d = 1, x = 1, quadratic loss, constant labels (y = 1 in
    shard 0, y = -1 in shard 1) so minibatch gradients are theta - 1 and
    theta + 1 whatever the draw.  The whole run is then a scalar recursion,
    rewritten here with plain floats straight from Algorithm 1."""
    N = 20
    X = np.ones((N, 1))
    y = np.concatenate([np.ones(10), -np.ones(10)])
    D, c, alpha, b1, b2, eps = 3, 0.5, 0.1, 0.9, 0.99, 1e-8
    o = GCadaOracle(Quadratic(1), 2, 1, D, c, alpha, b1, b2, eps,
                    X=X, y=y, batch=3, theta0=np.array([0.25]), seed=0)
    th = [0.25]
    h = vh = 0.0
    tau = [D, D]
    last = [0.0, 0.0]
    off = [-1.0, 1.0]
    for k in range(30):
        rhs = c * sum((th[k + 1 - d] - th[k - d]) ** 2 for d in range(1, D + 1) if k - d >= 0)
        sel = []
        for g in range(2):
            old = th[max(k - tau[g], 0)]
            lhs = ((th[k] + off[g]) - (old + off[g])) ** 2
            sel.append(tau[g] >= D or lhs > rhs)
        for g in range(2):
            if sel[g]:
                last[g] = th[k] + off[g]
                tau[g] = 1
            else:
                tau[g] += 1
        agg = last[0] + last[1]
        h = b1 * h + (1 - b1) * agg
        v = b2 * vh + (1 - b2) * agg * agg
        vh = max(vh, v)
        th.append(th[k] - alpha * h / math.sqrt(eps + vh))
        rec = o.step()
        assert list(rec["mask"]) == [int(s) for s in sel]
        assert rec["rhs"] == pytest.approx(rhs, rel=1e-12, abs=1e-300)
        assert o.theta[0] == pytest.approx(th[-1], rel=1e-12)
    assert sum(int(m.sum()) for m in o.masks) < 60


@pytest.mark.parametrize("schedule", [("poly", 5.0, 0.5), ("step", 4, 0.5)])
def test_scalar_trajectory_by_hand_with_lag_weights_and_step_schedule(schedule):
    """The same scalar recursion with the two generalisations the paper names:
    per-lag constants c_d on the right side of Eq. (9) (Algorithm 1's input
    list) and a step size alpha^k that depends on k (Eq. 2, Eq. 8c)."""
    N = 20
    X = np.ones((N, 1))
    y = np.concatenate([np.ones(10), -np.ones(10)])
    D, alpha, b1, b2, eps = 3, 0.1, 0.9, 0.99, 1e-8
    c_d = [0.9, 0.3, 0.05]
    o = GCadaOracle(Quadratic(1), 2, 1, D, 123.0, alpha, b1, b2, eps, X=X, y=y, batch=3,
                    theta0=np.array([0.25]), seed=0, c_d=c_d, schedule=schedule)
    th = [0.25]
    h = vh = 0.0
    tau = [D, D]
    last = [0.0, 0.0]
    off = [-1.0, 1.0]
    for k in range(30):
        rhs = sum(c_d[d - 1] * (th[k + 1 - d] - th[k - d]) ** 2 for d in range(1, D + 1) if k - d >= 0)
        sel = []
        for g in range(2):
            old = th[max(k - tau[g], 0)]
            sel.append(tau[g] >= D or ((th[k] + off[g]) - (old + off[g])) ** 2 > rhs)
        for g in range(2):
            if sel[g]:
                last[g], tau[g] = th[k] + off[g], 1
            else:
                tau[g] += 1
        agg = last[0] + last[1]
        h = b1 * h + (1 - b1) * agg
        vh = max(vh, b2 * vh + (1 - b2) * agg * agg)
        a_k = alpha / math.sqrt(1 + k / 5.0) if schedule[0] == "poly" else alpha * 0.5 ** (k // 4)
        th.append(th[k] - a_k * h / math.sqrt(eps + vh))
        rec = o.step()
        assert list(rec["mask"]) == [int(v) for v in sel]
        assert rec["rhs"] == pytest.approx(rhs, rel=1e-12, abs=1e-300)
        assert o.theta[0] == pytest.approx(th[-1], rel=1e-12)


def test_equal_lag_weights_and_constant_schedule_are_the_printed_method():
    a, b = _toy_oracle(c=0.7), _toy_oracle(c=0.7, c_d=[0.7] * 4, schedule=("poly", 1.0, 0.0))
    for _ in range(25):
        ra, rb = a.step(), b.step()
        assert np.array_equal(ra["mask"], rb["mask"]) and np.array_equal(ra["theta"], rb["theta"])


@pytest.mark.parametrize("law", ["pareto", "uniform"])
def test_other_delay_laws(law):
    from scipy import stats
    o = _toy_oracle(M=8, M_G=2, shift=2.0, rate=3.0, delay_law=law)
    T = []
    for k in range(600):
        o.k = k
        T.append(o.delays())
    T = np.concatenate(T)
    if law == "pareto":     # P(T > t) = (shift / t)^rate
        assert T.min() >= 2.0 and stats.kstest(T, "pareto", args=(3.0, 0, 2.0)).pvalue > 1e-3
    else:                   # uniform on [shift, shift + 1/rate]
        assert T.min() >= 2.0 and T.max() <= 2.0 + 1 / 3.0
        assert stats.kstest(T, "uniform", args=(2.0, 1 / 3.0)).pvalue > 1e-3


def test_c_zero_is_synchronous_distributed_adam():
    """c = 0: every group with a non-zero innovation violates Eq. (9) (and at
    k = 0 all are forced), so the run is the 'distributed Adam' of Section V:
    every gradient fresh every iteration.  Independent loop: autograd
    gradients summed over groups, library AMSGrad state replaced by Eq. (8)
    in closed loop form."""
    o = _toy_oracle(c=0.0, D=5)
    X, y = o.X, o.y
    th = torch.zeros(5, dtype=torch.float64)
    h = torch.zeros(5, dtype=torch.float64)
    vh = torch.zeros(5, dtype=torch.float64)
    for k in range(12):
        total = torch.zeros(5, dtype=torch.float64)
        for g in range(o.G):
            idx = philox.batch_indices(o.seed, k, g, o.batch, o.n_g)
            t = th.clone().requires_grad_(True)
            torch.nn.functional.binary_cross_entropy_with_logits(
                torch.tensor(X[idx]) @ t, torch.tensor(y[idx]), reduction="mean").backward()
            total += t.grad
        h = 0.9 * h + 0.1 * total
        vh = torch.maximum(vh, 0.99 * vh + 0.01 * total * total)
        th = th - 0.01 * h / torch.sqrt(1e-8 + vh)
        rec = o.step()
        assert rec["mask"].all()
        assert np.allclose(rec["agg"], total.numpy(), rtol=1e-10)
        assert np.allclose(o.theta, th.numpy(), rtol=1e-10)
    assert o.uploads == 12 * o.G and o.comm == 12 * o.G * (o.M_G + 1) and o.comp == 12 * o.M


def test_group_size_one_is_cada():
    """M_G = 1: groups are single workers, the rule is the per-worker rule of
    Section III, and the server waits for the slowest selected worker."""
    o = _toy_oracle(M=4, M_G=1, D=4, c=2.0)
    assert o.G == 4
    for _ in range(20):
        rec = o.step()
        sel = rec["mask"].astype(bool)
        assert np.array_equal(rec["t_g"], rec["T"])
        assert rec["dt"] == (rec["T"][sel].max() if sel.any() else 0.0)
    assert o.comm == 2 * o.uploads and o.comp == o.uploads    # Eq. (18), (21) with equality


def test_aggregate_aoi_and_counter_invariants():
    o = _toy_oracle(D=4, c=3.0)
    last_sel = np.zeros(o.G, dtype=int) - 1
    total = 0
    for k in range(60):
        tau_before = o.tau.copy()
        rec = o.step()
        assert np.all(tau_before >= 1) and np.all(tau_before <= o.D)
        if k == 0:
            assert rec["mask"].all()               # initial AoI = D forces everyone
        # forced when the age reaches D
        assert np.all(rec["mask"][tau_before >= o.D] == 1)
        # the aggregate is the sum of the last uploaded gradients (Eq. 3)
        assert np.allclose(rec["agg"], o.g_last.sum(axis=0), rtol=1e-13)
        for g in range(o.G):
            if rec["mask"][g]:
                assert np.array_equal(o.g_last[g], rec["fresh"][g])
                assert o.tau[g] == 1
                last_sel[g] = k
            else:
                assert o.tau[g] == tau_before[g] + 1
            assert k - last_sel[g] < o.D           # never more than D-1 skips in a row
        total += int(rec["mask"].sum())
        assert o.uploads == total
        assert o.comm == (o.M_G + 1) * total       # Eq. (19) with the realised count
        assert o.comp == o.M_G * total             # Eq. (22), in gradients
    assert total < 60 * o.G                        # something was skipped


def test_mask_shrinks_as_c_grows_at_the_same_state():
    base = _toy_oracle(D=6, c=0.5)
    for _ in range(10):
        base.step()
    import copy
    prev = None
    for c in (0.0, 0.5, 5.0, 500.0):
        o = copy.deepcopy(base)
        o.c = c
        m = o.step()["mask"].astype(bool)
        if prev is not None:
            assert np.all(prev | ~m)               # m is a subset of prev
        prev = m


def test_forced_mask_is_obeyed():
    o = _toy_oracle()
    rec = o.step(forced_mask=[0, 1, 0])
    assert list(rec["mask"]) == [0, 1, 0]
    assert o.uploads == 1 and list(o.tau) == [o.D + 1, 1, o.D + 1]
    assert np.array_equal(o.g_last[0], np.zeros(5)) and np.array_equal(o.g_last[1], rec["fresh"][1])


# --------------------------------------------------------------------------
# wall-clock (Section II-B, Section V-A)
# --------------------------------------------------------------------------
def test_wallclock_on_a_hand_table():
    T = [5.0, 2.0, 9.0, 7.0, 1.0, 8.0]          # groups of two: mins 2, 7, 1
    dt, t_g = GCadaOracle.wallclock_increment(T, [1, 1, 1], 2)
    assert list(t_g) == [2.0, 7.0, 1.0] and dt == 7.0
    assert GCadaOracle.wallclock_increment(T, [1, 0, 1], 2)[0] == 2.0
    assert GCadaOracle.wallclock_increment(T, [0, 0, 0], 2)[0] == 0.0
    assert GCadaOracle.wallclock_increment(T, [1, 1, 1, 1, 1, 1], 1)[0] == 9.0


def test_mean_wallclock_matches_order_statistics():
    """All groups selected (c = 0): per iteration the server waits for the max
    over G of (min over M_G exponentials).  The min is exponential with mean
    1/(rate*M_G); Eq. (10) with a = b = G gives the mean of the max:
    shift + H_G / (rate * M_G) = 1 + (1 + 1/2 + 1/3)/2 for G = 3, M_G = 2."""
    o = _toy_oracle(c=0.0, M=6, M_G=2)
    K = 4000
    incs = []
    for k in range(K):
        o.k = k
        incs.append(GCadaOracle.wallclock_increment(o.delays(), [1, 1, 1], 2)[0])
    mean = float(np.mean(incs))
    want = 1 + 0.5 * (1 + 0.5 + 1 / 3)
    sd = float(np.std(incs)) / math.sqrt(K)
    assert abs(mean - want) < 5 * sd and sd < 0.02


def test_relu_kink_choices_are_the_one_sided_derivatives():
    """At a hidden pre-activation of exactly zero the ReLU derivative may be 0
    or 1.  The default is 0 (the left derivative); `flip` selects 1 (the right
    derivative).  Both are checked by one-sided finite differences in the
    unit's bias."""
    rng = np.random.default_rng(4)
    mlp = MLP((3, 2, 2))
    theta = rng.normal(size=mlp.p)
    Xb = rng.normal(size=(4, 3))
    yb = rng.integers(0, 2, 4)
    W1 = theta[:6].reshape(2, 3)
    theta[6] = -(Xb[1] @ W1[0])              # b_1[0]: unit 0 of sample 1 sits exactly on the kink
    kinks = mlp.near_kinks(theta, Xb, 1e-12)
    assert kinks == [(0, 1, 0)]
    e = np.zeros(mlp.p)
    e[6] = 1e-7
    base = mlp.loss(theta, Xb, yb, "sum")
    right = (mlp.loss(theta + e, Xb, yb, "sum") - base) / 1e-7
    left = (base - mlp.loss(theta - e, Xb, yb, "sum")) / 1e-7
    assert abs(right - left) > 1e-3           # the kink is real
    assert mlp.grad(theta, Xb, yb, "sum")[6] == pytest.approx(left, rel=1e-5)
    assert mlp.grad(theta, Xb, yb, "sum", flip=kinks)[6] == pytest.approx(right, rel=1e-5)


def test_bf16_mode_rounds_every_matrix_operand():
    """bf16 mode against torch autograd (library routine) with explicit
    bfloat16 casts of inputs, weights and hidden activations in the forward
    pass and gradient hooks that round the back-propagated errors."""
    rng = np.random.default_rng(7)
    mlp = MLP((6, 5, 4, 3), bf16=True)
    theta = rng.normal(size=mlp.p)
    Xb = rng.normal(size=(8, 6))
    yb = rng.integers(0, 3, 8)
    rb = lambda t: t.to(torch.float32).to(torch.bfloat16).to(torch.float64)

    class RoundGrad(torch.autograd.Function):
        @staticmethod
        def forward(ctx, x):
            return x

        @staticmethod
        def backward(ctx, g):
            return rb(g)

    class RoundValue(torch.autograd.Function):     # value rounded, gradient passed through
        @staticmethod
        def forward(ctx, x):
            return rb(x)

        @staticmethod
        def backward(ctx, g):
            return g

    t = torch.tensor(theta, requires_grad=True)
    tr = RoundValue.apply(t)
    o, a = 0, rb(torch.tensor(Xb))
    dims = mlp.dims
    for l in range(1, len(dims)):
        W = tr[o:o + dims[l] * dims[l - 1]].reshape(dims[l], dims[l - 1])
        o += dims[l] * dims[l - 1]
        b = tr[o:o + dims[l]]
        o += dims[l]
        z = RoundGrad.apply(a @ W.T + b)
        a = RoundValue.apply(torch.relu(z)) if l < len(dims) - 1 else z
    torch.nn.functional.cross_entropy(a, torch.tensor(yb), reduction="mean").backward()
    got = mlp.grad(theta, Xb, yb, "mean")
    assert np.allclose(got, t.grad.numpy(), rtol=1e-9, atol=1e-12)
    # and it stays close to the unrounded gradient
    exact = MLP((6, 5, 4, 3)).grad(theta, Xb, yb, "mean")
    assert 1e-5 < np.linalg.norm(got - exact) / np.linalg.norm(exact) < 3e-2


def test_bf16_operands_mode_rounds_features_and_weight_matrices_only():
    """The narrower reading of "bf16 inputs/weights": features and weight
    matrices rounded, everything else exact.  Against torch autograd (library
    routine) on explicitly cast leaves; the gradient is with respect to the
    unrounded parameters, the rounding passing gradients through unchanged."""
    rng = np.random.default_rng(11)
    dims = (7, 6, 5, 3)
    mlp = MLP(dims, bf16="operands")
    theta = rng.normal(size=mlp.p)
    Xb = rng.normal(size=(9, 7))
    yb = rng.integers(0, 3, 9)
    rb = lambda t: t.to(torch.float32).to(torch.bfloat16).to(torch.float64)
    t = torch.tensor(theta, requires_grad=True)
    o, a = 0, rb(torch.tensor(Xb))
    for l in range(1, len(dims)):
        W = t[o:o + dims[l] * dims[l - 1]].reshape(dims[l], dims[l - 1])
        o += dims[l] * dims[l - 1]
        b = t[o:o + dims[l]]
        o += dims[l]
        Wr = W + (rb(W.detach()) - W.detach())          # value rounded, gradient passed through
        z = a @ Wr.T + b
        a = torch.relu(z) if l < len(dims) - 1 else z
    torch.nn.functional.cross_entropy(a, torch.tensor(yb), reduction="mean").backward()
    got = mlp.grad(theta, Xb, yb, "mean")
    assert np.allclose(got, t.grad.numpy(), rtol=1e-9, atol=1e-12)
    # the three readings are distinct and ordered: exact -> operands -> every operand
    exact = MLP(dims).grad(theta, Xb, yb, "mean")
    every = MLP(dims, bf16=True).grad(theta, Xb, yb, "mean")
    n = np.linalg.norm(exact)
    assert 1e-5 < np.linalg.norm(got - exact) / n < 3e-2
    assert 1e-5 < np.linalg.norm(every - got) / n < 3e-2
    # rounding the inputs by hand and calling the unrounded model gives the same thing
    th_r = theta.copy()
    o = 0
    for l in range(1, len(dims)):
        n_w = dims[l] * dims[l - 1]
        th_r[o:o + n_w] = round_to_bf16(theta[o:o + n_w])
        o += n_w + dims[l]
    assert np.array_equal(got, MLP(dims).grad(th_r, round_to_bf16(Xb), yb, "mean"))


def test_stale_iterate_is_the_literal_one_under_forced_masks():
    """Eq. (3) / Section IV: the stale iterate of a group is theta^{k - tau_g}, whatever tau_g is.  The
    method's own rule keeps tau_g <= D; a forced mask can starve a group for longer, and the oracle then
    still goes back tau_g iterates (to theta^0 at the earliest)."""
    o = _toy_oracle(D=2)
    masks = [[1, 1, 1], [1, 0, 1], [1, 0, 1], [1, 0, 1], [1, 0, 1]]
    for k, m in enumerate(masks):
        assert o.tau[1] == (2 if k == 0 else k)       # initial age D, then 1, 2, 3, 4: beyond D = 2 from k = 3
        _, Xb, yb = o.minibatch(1)
        want = o.model.grad(o.thetas[max(k - int(o.tau[1]), 0)], Xb, yb, "mean")
        rec = o.step(forced_mask=m)
        assert np.array_equal(rec["stale"][1], want)
        if k >= 1:
            assert np.array_equal(want, o.model.grad(o.thetas[0], Xb, yb, "mean"))   # last upload was at k = 0
