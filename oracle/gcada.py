"""Plain fp64 CPU oracle of one G-CADA run (test infrastructure only).

Only tests, the smoke check and the CPU-baseline leg of the benchmark may use
this module; the product path never does.  It shares no code with the CUDA
implementation and is deliberately slow and literal: it keeps every iterate
theta^0..theta^k and evaluates each formula of the paper from that history.

What is followed (Zhu, Zhang, Simeone, Wang: "Adaptive Worker Grouping for
Communication-Efficient and Straggler-Tolerant Distributed SGD"):

  * Algorithm 1 gives the order of one iteration.
  * Section IV: G = M / M_G groups, disjoint equal shards, one age of
    information (AoI) tau_g per group kept by the server.
  * Eq. (9): a group is selected when it violates
        LHS_g <= c * sum_{d=1..D} ||theta^{k+1-d} - theta^{k-d}||^2 ,
    or when tau_g >= D.  Rule "innov" takes for LHS_g the quantity that the
    printed left side estimates (Section III, text after Eq. 7): the squared
    norm of the change of the group's minibatch gradient between theta^k and
    theta^{k - tau_g}, on the SAME fresh minibatch.  Rule "ps" takes the
    printed left side L_g^2 ||theta^k - theta^{k-tau_g}||^2.
  * Eq. (3) / the aggregate written out in Section IV: fresh gradients of the
    selected groups plus the last uploaded gradient of every other group.
  * Eq. (8a-c): the AMSGrad-style update, with v^{k+1} built from v-hat^k as
    printed and epsilon inside the square root.
  * Section II-B, Eqs. (4)-(6) and Section V: per-worker computing times,
    wall-clock = slowest selected group, a group being as fast as its fastest
    worker; communication load |M_D| + |M_U|; computation load |M_D|
    (counted in minibatch gradients).

Readings where the paper is silent or inconsistent: initial AoI = D (so the
first iteration selects everyone); unselected AoI grows by one (Algorithm 1);
iterates before theta^0 equal theta^0 and their differences are zero; ties
(LHS == RHS) do not select; h^0 = v-hat^0 = 0; constant step size; a single
constant c; minibatch = `batch` uniform draws with replacement from the
group's shard, shared by the workers of the group; computing time
T = shift - ln(1-u)/rate (shift 0, rate 1/eta is the paper's exponential).

Optional generalisations the paper names without using them: per-lag constants
{c_d} (Algorithm 1's input list) weight the D terms of the right side of
Eq. (9) individually; the step size alpha^k (Eq. 2, Eq. 8c) may follow a
schedule; computing times may follow another law than the exponential of
Section II-B (the analysis of Section V only needs i.i.d. times).

parity unpinned: free-running trajectories longer than the pinned special
cases (near-ties in the selection test may legitimately flip).
"""
import numpy as np

from . import philox


class GCadaOracle:
    def __init__(self, model, M, M_G, D, c, alpha, beta1, beta2, eps, *,
                 X, y, batch, theta0, seed=0, shift=1.0, rate=1.0,
                 rule="innov", reduction="mean", L=None, c_d=None, schedule=("const",),
                 delay_law="exp"):
        if M <= 0 or M_G <= 0 or M % M_G or D < 1 or c < 0 or alpha <= 0 \
                or not (0 < beta1 < 1) or not (0 < beta2 < 1) or eps <= 0:
            raise ValueError("invalid G-CADA parameters")
        self.model = model
        self.M, self.M_G, self.G = M, M_G, M // M_G
        self.D, self.c = D, float(c)
        self.alpha, self.beta1, self.beta2, self.eps = map(float, (alpha, beta1, beta2, eps))
        self.X, self.y = X, y
        self.N = len(y)
        self.n_g = self.N // self.G            # trailing N mod G rows unused
        self.batch = int(batch)
        self.seed, self.shift, self.rate = seed, float(shift), float(rate)
        self.rule, self.reduction = rule, reduction
        self.L = None if L is None else np.asarray(L, dtype=np.float64)
        # c_d[d-1] multiplies ||theta^{k+1-d} - theta^{k-d}||^2; the printed Eq. (9) has c_d = c for all d
        self.c_d = np.full(D, self.c) if c_d is None else np.asarray(c_d, dtype=np.float64).reshape(D)
        self.schedule = tuple(schedule)
        self.delay_law = delay_law
        p = model.p
        self.thetas = [np.array(theta0, dtype=np.float64).reshape(p)]   # theta^0..theta^k
        self.h = np.zeros(p)
        self.vhat = np.zeros(p)
        self.g_last = np.zeros((self.G, p))     # last uploaded gradient per group
        self.tau = np.full(self.G, D, dtype=np.int64)
        self.k = 0
        self.uploads = 0
        self.comm = 0
        self.comp = 0
        self.wall = 0.0
        self.masks = []

    # -- pieces, each one formula ------------------------------------------
    def theta_at(self, j):
        """theta^j, with theta^j = theta^0 for j < 0."""
        return self.thetas[max(j, 0)]

    def rhs(self):
        """sum_{d=1..D} c_d ||theta^{k+1-d} - theta^{k-d}||^2  (Eq. 9, right side; c_d = c as printed)."""
        k, total = self.k, 0.0
        for d in range(1, self.D + 1):
            if k - d < 0:
                continue
            diff = self.thetas[k + 1 - d] - self.thetas[k - d]
            total += self.c_d[d - 1] * float(diff @ diff)
        return total

    def step_size(self, k):
        """alpha^k of Eq. (8c).  ("const",): alpha;  ("poly", t0, q): alpha / (1 + k/t0)^q;
        ("step", every, factor): alpha * factor^floor(k / every)."""
        kind = self.schedule[0]
        if kind == "const":
            return self.alpha
        if kind == "poly":
            _, t0, q = self.schedule
            return self.alpha / (1.0 + k / float(t0)) ** float(q)
        if kind == "step":
            _, every, factor = self.schedule
            return self.alpha * float(factor) ** (k // int(every))
        raise ValueError(kind)

    def minibatch(self, g):
        idx = philox.batch_indices(self.seed, self.k, g, self.batch, self.n_g)
        Xb = np.asarray(self.X[idx], dtype=np.float64)
        yb = np.asarray(self.y[idx])
        return idx, Xb, yb

    def delays(self):
        """T_m^k for all M workers (Section II-B)."""
        u = philox.uniform01(self.seed, self.k, np.arange(self.M))
        if self.delay_law == "exp":         # Section II-B (shift 0): exponential with mean 1/rate
            return self.shift - np.log1p(-u) / self.rate
        if self.delay_law == "pareto":      # heavy tail: P(T > t) = (shift/t)^rate for t >= shift
            return self.shift * np.exp(-np.log1p(-u) / self.rate)
        if self.delay_law == "uniform":     # bounded: uniform on [shift, shift + 1/rate]
            return self.shift + u / self.rate
        raise ValueError(self.delay_law)

    @staticmethod
    def wallclock_increment(T, mask, M_G):
        """Slowest selected group, each group as fast as its fastest worker;
        zero when no group is selected (Section IV; Section V-A)."""
        t_g = np.asarray(T, dtype=np.float64).reshape(-1, M_G).min(axis=1)
        sel = np.asarray(mask, dtype=bool)
        return (float(t_g[sel].max()) if sel.any() else 0.0), t_g

    @staticmethod
    def amsgrad(theta, h, vhat, grad, alpha, beta1, beta2, eps):
        """Eq. (8a)-(8c) exactly as printed."""
        h = beta1 * h + (1.0 - beta1) * grad
        v = beta2 * vhat + (1.0 - beta2) * grad * grad
        vhat = np.maximum(vhat, v)
        theta = theta - alpha * h / np.sqrt(eps + vhat)
        return theta, h, vhat

    # -- one iteration of Algorithm 1 --------------------------------------
    def step(self, forced_mask=None):
        k, G = self.k, self.G
        theta_k = self.thetas[k]
        rhs = self.rhs()
        fresh = np.zeros((G, self.model.p))
        stale = np.zeros((G, self.model.p))
        lhs = np.zeros(G)
        for g in range(G):
            _, Xb, yb = self.minibatch(g)
            theta_old = self.theta_at(k - int(self.tau[g]))      # theta^{k - tau_g} (Eq. 3, Section IV)
            fresh[g] = self.model.grad(theta_k, Xb, yb, self.reduction)
            stale[g] = self.model.grad(theta_old, Xb, yb, self.reduction)
            if self.rule == "innov":
                delta = fresh[g] - stale[g]
                lhs[g] = float(delta @ delta)
            elif self.rule == "ps":
                dth = theta_k - theta_old
                lhs[g] = self.L[g] ** 2 * float(dth @ dth)
            else:
                raise ValueError(self.rule)
        if forced_mask is None:
            mask = (self.tau >= self.D) | (lhs > rhs)
        else:
            mask = np.asarray(forced_mask, dtype=bool).reshape(G)
        # server: lazy aggregate = fresh (selected) + last uploaded (others)
        for g in range(G):
            if mask[g]:
                self.g_last[g] = fresh[g]
        agg = self.g_last.sum(axis=0)
        theta_next, self.h, self.vhat = self.amsgrad(
            theta_k, self.h, self.vhat, agg,
            self.step_size(k), self.beta1, self.beta2, self.eps)
        self.thetas.append(theta_next)
        tau_used = self.tau.copy()
        self.tau = np.where(mask, 1, self.tau + 1)
        # metrics
        T = self.delays()
        dt, t_g = self.wallclock_increment(T, mask, self.M_G)
        n_sel = int(mask.sum())
        self.wall += dt
        self.uploads += n_sel
        self.comm += (self.M_G + 1) * n_sel
        self.comp += self.M_G * n_sel
        self.masks.append(mask.astype(np.uint8))
        self.k += 1
        return dict(k=k, fresh=fresh, stale=stale, lhs=lhs, rhs=rhs, mask=mask.astype(np.uint8),
                    tau=tau_used, agg=agg, theta=theta_next, T=T, t_g=t_g, dt=dt)

    @property
    def theta(self):
        return self.thetas[-1]
