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
