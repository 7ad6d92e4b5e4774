"""Seeded synthetic inputs for the five G-CADA workloads.

This module only manufactures data (features, labels, initial parameters) and
the hyper-parameters of each workload.  It contains none of the method's
arithmetic, so that both the CUDA library and an independent checker can be
fed from it.  The sigmoid below is part of the label recipe, not of the
method.

Workloads (all synthetic; `cfg4` has the shape of a 28x28 ten-class image
benchmark and stands in for it, no item of any public dataset is used):

  cfg1  logistic, d=32,   N=20,000,    M=6,    M_G=2, batch 32,   K=200
  cfg2  logistic, d=54,   N=500,000,   M=20,   M_G=4, batch 1024, K=1000
        (10 Gaussian + 44 Bernoulli(0.1) columns; rows padded to 56 floats)
  cfg3  logistic, d=4096, N=2,000,000, M=256,  M_G=4, batch 512,  K=500
        (features N(0,1)/sqrt(d), planted labels with 5 % flips)
  cfg4  MLP 784-200-10 fp32, N=60,000, M=10,   M_G=2, batch 64,   K=2000
  cfg5  MLP 1024-4096-4096-1000, bf16 operands, N=1,048,576, M=1024, M_G=4,
        batch 128, K=200

  linreg784  the model class of the paper's own experiment (Section VI): linear
        regression with the quadratic loss on 784 features in [0,1] (the cfg4
        feature recipe), the class id 0..9 as the real-valued target, N=60,000,
        M=12 workers in G=3 groups of M_G=4, beta2=0.999, alpha=0.01, c=0.3,
        exponential computing times of mean 1e-4 s.  Batch size and D are not
        stated there; 64 and 10 are used.

`rows` shrinks N (keeping everything else) for quick checks.
"""
import math

import torch

CONFIGS = {
    "cfg1": dict(kind="logistic", dims=(32,), compute="fp32", N=20000, M=6, M_G=2, batch=32,
                 D=10, c=1.0, alpha=0.01, beta1=0.9, beta2=0.99, eps=1e-8, K=200),
    "cfg2": dict(kind="logistic", dims=(54,), compute="fp32", N=500000, M=20, M_G=4, batch=1024,
                 D=10, c=0.6, alpha=0.01, beta1=0.9, beta2=0.99, eps=1e-8, K=1000),
    "cfg3": dict(kind="logistic", dims=(4096,), compute="fp32", N=2000000, M=256, M_G=4, batch=512,
                 D=10, c=0.6, alpha=0.01, beta1=0.9, beta2=0.99, eps=1e-8, K=500),
    "cfg4": dict(kind="mlp", dims=(784, 200, 10), compute="fp32", N=60000, M=10, M_G=2, batch=64,
                 D=10, c=1.0, alpha=1e-3, beta1=0.9, beta2=0.99, eps=1e-8, K=2000),
    "cfg5": dict(kind="mlp", dims=(1024, 4096, 4096, 1000), compute="bf16", N=1048576, M=1024,
                 M_G=4, batch=128, D=10, c=0.6, alpha=1e-3, beta1=0.9, beta2=0.99, eps=1e-8, K=200),
}
for _c in CONFIGS.values():
    _c.update(seed=0, shift=1.0, rate=1.0)
CONFIGS["linreg784"] = dict(kind="quadratic", dims=(784,), compute="fp32", N=60000, M=12, M_G=4, batch=64,
                            D=10, c=0.3, alpha=0.01, beta1=0.9, beta2=0.999, eps=1e-8, K=2000,
                            seed=0, shift=0.0, rate=1.0e4)


def _gen(device, seed):
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _planted_labels(X, w, gen, flip=0.0):
    p = torch.sigmoid(X @ w)
    y = (torch.rand(p.shape, generator=gen, device=X.device) < p).to(torch.float32)
    if flip > 0:
        f = torch.rand(p.shape, generator=gen, device=X.device) < flip
        y = torch.where(f, 1.0 - y, y)
    return y


def mlp_theta0(dims, gen, device):
    """W_l ~ N(0, 1/fan_in) stored as n_l rows of n_{l-1}; biases zero;
    layers concatenated W_1, b_1, W_2, b_2, ..."""
    parts = []
    for l in range(1, len(dims)):
        n_in, n_out = dims[l - 1], dims[l]
        W = torch.randn(n_out, n_in, generator=gen, device=device) / math.sqrt(n_in)
        parts += [W.reshape(-1), torch.zeros(n_out, device=device)]
    return torch.cat(parts).contiguous()


def make_workload(name, device="cpu", rows=None, data_seed=0, **overrides):
    """Return a dict with the hyper-parameters of `name` plus tensors
    X [N, ld] (row stride ld >= d), y [N], theta0 [p] on `device`."""
    cfg = dict(CONFIGS[name])
    cfg.update(overrides)
    if rows is not None:
        cfg["N"] = int(rows)
    N, dims, kind = cfg["N"], cfg["dims"], cfg["kind"]
    dev = torch.device(device)
    gen = _gen(dev, data_seed)
    d = dims[0]
    cfg["name"] = name
    if kind in ("logistic", "quadratic"):
        if name == "linreg784":
            ld = d
            cls = torch.randint(0, 10, (N,), generator=gen, device=dev)
            mu = torch.rand(10, d, generator=gen, device=dev)
            X = (mu[cls] + 0.3 * torch.randn(N, d, generator=gen, device=dev)).clamp_(0, 1)
            w = None
            y = cls.to(torch.float32)
        elif name == "cfg2":
            ld = 56
            X = torch.zeros(N, ld, device=dev)
            X[:, :10] = torch.randn(N, 10, generator=gen, device=dev)
            X[:, 10:54] = (torch.rand(N, 44, generator=gen, device=dev) < 0.1).float()
            w = torch.randn(d, generator=gen, device=dev) / math.sqrt(d)
            y = _planted_labels(X[:, :d], w, gen)
        elif name == "cfg3":
            ld = d
            X = torch.empty(N, d, device=dev)
            chunk = 65536
            for s in range(0, N, chunk):
                e = min(N, s + chunk)
                X[s:e] = torch.randn(e - s, d, generator=gen, device=dev) / math.sqrt(d)
            w = torch.randn(d, generator=gen, device=dev)
            y = torch.empty(N, device=dev)
            for s in range(0, N, chunk):
                e = min(N, s + chunk)
                y[s:e] = _planted_labels(X[s:e], w, gen, flip=0.05)
        else:
            ld = d
            X = torch.randn(N, d, generator=gen, device=dev)
            w = torch.randn(d, generator=gen, device=dev) / math.sqrt(d)
            y = _planted_labels(X, w, gen)
        if kind == "quadratic" and w is not None:
            y = X[:, :d] @ w + 0.1 * torch.randn(N, generator=gen, device=dev)
        theta0 = torch.zeros(d, device=dev)
    elif kind == "mlp":
        ld = d
        n_cls = dims[-1]
        cls = torch.randint(0, n_cls, (N,), generator=gen, device=dev)
        if cfg["compute"] == "fp32":
            mu = torch.rand(n_cls, d, generator=gen, device=dev)
            X = torch.empty(N, d, device=dev)
            chunk = 65536
            for s in range(0, N, chunk):
                e = min(N, s + chunk)
                X[s:e] = (mu[cls[s:e]] + 0.3 * torch.randn(e - s, d, generator=gen, device=dev)).clamp_(0, 1)
        else:
            mu = torch.randn(n_cls, d, generator=gen, device=dev)
            X = torch.empty(N, d, device=dev, dtype=torch.bfloat16)
            chunk = 65536
            for s in range(0, N, chunk):
                e = min(N, s + chunk)
                X[s:e] = (mu[cls[s:e]] + torch.randn(e - s, d, generator=gen, device=dev)).to(torch.bfloat16)
        y = cls.to(torch.int32)
        theta0 = mlp_theta0(dims, gen, dev)
    else:
        raise ValueError(kind)
    cfg.update(X=X.contiguous(), y=y.contiguous(), theta0=theta0.contiguous(), ld=ld)
    return cfg
