"""Loss evaluation entry point against the oracle's loss, and the three-scheme
comparison (G-CADA, CADA = groups of one, distributed Adam = groups of one
with c = 0) on the synthetic linear-regression workload."""
import numpy as np
import pytest
import torch

from oracle.models import make_model
from paper_2201_04301_b200 import binding, compare
from paper_2201_04301_b200.workloads import make_workload

from parity import make_oracle, to_cuda

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,rows", [("cfg1", None), ("cfg2", 20000), ("linreg784", 6000)])
def test_eval_loss_matches_the_written_out_loss(name, rows):
    w = make_workload(name, rows=rows)
    g = binding.from_workload(to_cuda(w), stream=torch.cuda.Stream())
    model = make_model(w["kind"], w["dims"])
    d = w["dims"][0]
    X = w["X"][:, :d].double().numpy()
    y = w["y"].double().numpy()
    for first, n in ((0, 1), (0, 1000), (137, 2891)):
        for _ in range(2):
            theta = g.get_theta().astype(np.float64)
            want = model.loss(theta, X[first:first + n], y[first:first + n], "mean")
            assert g.eval_loss(first, n) == pytest.approx(want, rel=1e-9, abs=1e-12)
            g.step(7)
    with pytest.raises(binding.GCadaError):
        g.eval_loss(0, w["X"].shape[0] + 1)


def test_three_schemes():
    w = make_workload("linreg784", device="cuda", rows=12000)
    K, M = 300, w["M"]
    runs = {name: compare.run_scheme(w, kw["M_G"], kw["c"], K, 50, 4000, torch.cuda.Stream())
            for name, kw in compare.schemes(w, 2.0).items()}
    for name, recs in runs.items():
        assert [r["k"] for r in recs] == list(range(0, K + 1, 50))
        assert recs[-1]["loss"] < 0.5 * recs[0]["loss"], name                       # all three train
        assert all(b["wall"] >= a["wall"] and b["comm"] >= a["comm"] for a, b in zip(recs, recs[1:]))
    adam, cada, gc = runs["adam"][-1], runs["cada"][-1], runs["g-cada"][-1]
    assert adam["uploads"] == M * K and adam["comm"] == 2 * M * K and adam["comp"] == M * K
    assert cada["comm"] == 2 * cada["uploads"] and cada["uploads"] < adam["uploads"]  # CADA skips uploads
    assert gc["comm"] == (w["M_G"] + 1) * gc["uploads"] and gc["comp"] == w["M_G"] * gc["uploads"]
    # a group of M_G workers waits for its fastest one: per iteration G-CADA is faster than synchronous Adam
    assert gc["wall"] < adam["wall"]


def test_three_schemes_on_the_fp32_mlp():
    """The same comparison on the 784-200-10 network (loss through the MLP branch of gcada_eval_loss)."""
    w = make_workload("cfg4", device="cuda", rows=6000)
    K, M = 120, w["M"]
    runs = {name: compare.run_scheme(w, kw["M_G"], kw["c"], K, 40, 3000, torch.cuda.Stream())
            for name, kw in compare.schemes(w, 2.0).items()}
    for name, recs in runs.items():
        assert recs[-1]["loss"] < recs[0]["loss"], name
    adam, gc = runs["adam"][-1], runs["g-cada"][-1]
    assert adam["uploads"] == M * K and gc["comm"] == (w["M_G"] + 1) * gc["uploads"]


@pytest.mark.gpu
@pytest.mark.parametrize("name,kw", [
    ("cfg4", dict(rows=5 * 1300)),                                              # fp32, fused output layer
    ("cfg4", dict(rows=3 * 900, dims=(50, 70, 40, 30), M=6, M_G=2)),             # fp32, three layers, 30 classes
    ("cfg5", dict(rows=3 * 1500, dims=(64, 128, 96, 40), M=6, M_G=2, D=3, batch=128)),   # bf16 features
])
def test_mlp_loss_of_the_current_iterate(name, kw):
    """gcada_eval_loss on the MLPs: the mean softmax cross-entropy of the CUDA path's current iterate over a
    row range (ragged: whole 64-row chunks plus a remainder, and more than one slab) against the oracle's
    loss function evaluated at that iterate."""
    from oracle.models import make_model
    w = make_workload(name, **kw)
    g = binding.from_workload(to_cuda(w), stream=torch.cuda.Stream())
    g.step(7)
    theta = g.get_theta().astype(np.float64)
    model = make_model("mlp", w["dims"])                  # fp32 master parameters, no operand rounding
    X = w["X"].float().numpy().astype(np.float64)
    y = w["y"].numpy()
    for first, n in ((0, 64), (5, 1), (17, 1000), (0, X.shape[0])):
        want = model.loss(theta, X[first:first + n], y[first:first + n], "mean")
        got = g.eval_loss(first, n)
        assert abs(got - want) <= 2e-5 * abs(want), (first, n, got, want)
    g.step(3)                                             # the run goes on undisturbed
    assert g.get_iteration() == 10
    g.close()
