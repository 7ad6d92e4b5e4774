"""Per-sample losses and minibatch gradients for the CPU oracle (test
infrastructure only; fp64 numpy; shares nothing with the CUDA path).

The paper (Section II-A, Eq. 1) asks only for a smooth per-sample loss
l(theta; z) with z = (x, y); the local gradient of a worker is the gradient of
the loss summed over its minibatch.  `reduction="sum"` is that sum;
`reduction="mean"` divides by the minibatch size (the scale in which the
smoothness constants of Section IV are defined).  The three losses are the
ones of the workloads this library targets: logistic regression, the
quadratic loss of Section VI, and a ReLU multilayer perceptron with softmax
cross-entropy.

Every function is the textbook definition written out; nothing is blocked,
fused or reordered.
"""
import numpy as np


def _scale(reduction, rows):
    if reduction == "mean":
        return 1.0 / rows
    if reduction == "sum":
        return 1.0
    raise ValueError("reduction must be 'mean' or 'sum'")


def round_to_bf16(a):
    """Round fp64/fp32 values to the nearest bfloat16 (ties to even), returned
    as float64.  bfloat16 is the top 16 bits of an IEEE binary32."""
    f = np.asarray(a, dtype=np.float32)
    bits = f.view(np.uint32).astype(np.uint64)
    lsb = (bits >> np.uint64(16)) & np.uint64(1)
    bits = (bits + np.uint64(0x7FFF) + lsb) & np.uint64(0xFFFF0000)
    return bits.astype(np.uint32).view(np.float32).astype(np.float64).reshape(f.shape)


class Logistic:
    """l(theta; x, y) = -y ln s(x.theta) - (1-y) ln(1 - s(x.theta)), y in {0,1},
    s the logistic sigmoid, no intercept; theta in R^d."""
    kind = "logistic"

    def __init__(self, d):
        self.d = int(d)
        self.p = int(d)

    def loss(self, theta, Xb, yb, reduction="mean"):
        z = Xb @ theta
        # ln(1+e^z) - y z, written stably
        per = np.logaddexp(0.0, z) - yb * z
        return _scale(reduction, len(yb)) * per.sum()

    def grad(self, theta, Xb, yb, reduction="mean"):
        z = Xb @ theta
        r = 1.0 / (1.0 + np.exp(-z)) - yb
        return _scale(reduction, len(yb)) * (Xb.T @ r)


class Quadratic:
    """l(theta; x, y) = (x.theta - y)^2 / 2 (the quadratic error loss of the
    linear-regression experiment, Section VI); theta in R^d."""
    kind = "quadratic"

    def __init__(self, d):
        self.d = int(d)
        self.p = int(d)

    def loss(self, theta, Xb, yb, reduction="mean"):
        e = Xb @ theta - yb
        return _scale(reduction, len(yb)) * 0.5 * (e @ e)

    def grad(self, theta, Xb, yb, reduction="mean"):
        e = Xb @ theta - yb
        return _scale(reduction, len(yb)) * (Xb.T @ e)


class MLP:
    """Fully connected network dims = (n_0, n_1, ..., n_L): a_0 = x,
    z_l = W_l a_{l-1} + b_l, a_l = max(z_l, 0) for l < L, class scores z_L,
    loss = -ln softmax(z_L)[y] with y an integer class.

    theta is the concatenation over l = 1..L of W_l (n_l rows of n_{l-1}
    values, row-major) followed by b_l (n_l values).

    With bf16=True every matrix-product operand is a bfloat16 value: the
    inputs, the weights (biases included), the hidden activations a_l and
    the back-propagated errors dz_l are rounded to bfloat16 (ties to even)
    before they are used; products, sums, the softmax and the loss are fp64.
    This is the reading of "bf16 inputs/weights with fp32 accumulation" for a
    multi-layer network: the input of layer l+1 is the bf16 output of layer l,
    so both sides take each ReLU on/off decision from the same numbers.

    With bf16="operands" only what the workload statement names is rounded:
    the input features and the weight matrices W_l (the copy of the iterate
    the products read); biases, hidden activations, back-propagated errors
    and all arithmetic stay fp64.  This is the narrower reading of the same
    phrase; the two differ by the rounding of the intermediate operands."""
    kind = "mlp"

    def __init__(self, dims, bf16=False):
        self.dims = tuple(int(n) for n in dims)
        if isinstance(bf16, str) and bf16 != "operands":
            raise ValueError("bf16 must be False, True or 'operands'")
        self.bf16_operands = isinstance(bf16, str)            # features and weight matrices only
        self.bf16 = bool(bf16) and not self.bf16_operands     # every matrix-product operand rounded
        self.p = sum(self.dims[l] * self.dims[l - 1] + self.dims[l]
                     for l in range(1, len(self.dims)))

    def unpack(self, theta):
        out, o = [], 0
        for l in range(1, len(self.dims)):
            n_in, n_out = self.dims[l - 1], self.dims[l]
            W = theta[o:o + n_in * n_out].reshape(n_out, n_in)
            o += n_in * n_out
            b = theta[o:o + n_out]
            o += n_out
            out.append((W, b))
        return out

    def _forward(self, theta, Xb):
        if self.bf16:
            theta = round_to_bf16(theta)
            Xb = round_to_bf16(Xb)
        layers = self.unpack(np.asarray(theta, dtype=np.float64))
        if self.bf16_operands:
            Xb = round_to_bf16(Xb)
            layers = [(round_to_bf16(W), b) for W, b in layers]
        acts = [np.asarray(Xb, dtype=np.float64)]
        zs = []
        for l, (W, b) in enumerate(layers):
            z = acts[-1] @ W.T + b
            zs.append(z)
            if l < len(layers) - 1:
                a = np.maximum(z, 0.0)
                acts.append(round_to_bf16(a) if self.bf16 else a)
        return layers, acts, zs

    def loss(self, theta, Xb, yb, reduction="mean"):
        _, _, zs = self._forward(theta, Xb)
        s = zs[-1]
        s = s - s.max(axis=1, keepdims=True)
        logp = s - np.log(np.exp(s).sum(axis=1, keepdims=True))
        per = -logp[np.arange(len(yb)), np.asarray(yb, dtype=np.int64)]
        return _scale(reduction, len(yb)) * per.sum()

    def near_kinks(self, theta, Xb, tol):
        """Hidden units (layer index, row, unit) whose pre-activation is within
        `tol` of zero: there the ReLU derivative is a matter of rounding, and
        either choice (0 or 1) is a valid subgradient."""
        _, _, zs = self._forward(theta, Xb)
        out = []
        for l, z in enumerate(zs[:-1]):
            r, u = np.nonzero(np.abs(z) <= tol)
            out += [(l, int(a), int(b)) for a, b in zip(r, u)]
        return out

    def grad(self, theta, Xb, yb, reduction="mean", flip=()):
        """Gradient of the minibatch loss.  `flip` lists hidden units
        (layer index, row, unit) whose ReLU derivative is taken as the other
        admissible value (see near_kinks); the forward pass is unaffected."""
        layers, acts, zs = self._forward(theta, Xb)
        s = zs[-1]
        s = s - s.max(axis=1, keepdims=True)
        prob = np.exp(s)
        prob /= prob.sum(axis=1, keepdims=True)
        dz = prob
        dz[np.arange(len(yb)), np.asarray(yb, dtype=np.int64)] -= 1.0
        dz *= _scale(reduction, len(yb))
        pieces = [None] * len(layers)
        for l in range(len(layers) - 1, -1, -1):
            W, _ = layers[l]
            if self.bf16:
                dz = round_to_bf16(dz)
            dW = dz.T @ acts[l]          # n_l x n_{l-1}
            db = dz.sum(axis=0)
            pieces[l] = (dW, db)
            if l > 0:
                da = dz @ W
                on = zs[l - 1] > 0.0
                for (fl, fr, fu) in flip:
                    if fl == l - 1:
                        on[fr, fu] = ~on[fr, fu]
                dz = da * on
        return np.concatenate([np.concatenate([dW.ravel(), db]) for dW, db in pieces])


def make_model(kind, dims, bf16=False):
    if kind == "logistic":
        return Logistic(dims[0])
    if kind == "quadratic":
        return Quadratic(dims[0])
    if kind == "mlp":
        return MLP(dims, bf16=bf16)
    raise ValueError(kind)
