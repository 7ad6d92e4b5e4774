"""CUDA path vs CPU oracle for the multilayer perceptron (through the C ABI)."""
import numpy as np
import pytest
import torch

from paper_2201_04301_b200 import binding
from paper_2201_04301_b200.workloads import make_workload

from parity import TOL_FP32, forced_parity, make_oracle, rel_l2, to_cuda

pytestmark = pytest.mark.gpu


def test_cfg4_teacher_forced():
    """784-200-10, fp32, 5 groups of 64 rows: the full small MLP workload."""
    w = make_workload("cfg4", rows=5 * 400)
    flips, worst = forced_parity(w, 40, stream=torch.cuda.Stream())
    print("cfg4 worst", worst, "flips", flips)


@pytest.mark.parametrize("dims,batch,M,M_G,D", [
    ((5, 3), 7, 2, 1, 2),                 # a single affine layer (softmax regression)
    ((33, 17, 9, 4), 10, 6, 2, 3),        # three layers, odd sizes
    ((70, 130, 65), 100, 3, 3, 4),        # sizes that straddle the 64-wide tiles, G = 1
    ((300, 70, 5), 33, 6, 2, 2),          # first layer split over a cluster of 4 (K shares 96, 96, 96, 12)
    ((600, 12), 20, 4, 2, 2),             # one layer of 12 outputs: warp-per-row product, K in three chunks
    ((520, 64, 40, 16), 64, 2, 1, 3),     # split of 8, a 16-column output layer
])
def test_odd_architectures(dims, batch, M, M_G, D):
    G = M // M_G
    w = make_workload("cfg4", rows=G * 150, dims=dims, M=M, M_G=M_G, D=D, batch=batch, c=0.3, alpha=0.01)
    forced_parity(w, 2 * D + 3, stream=torch.cuda.Stream())


def test_cfg4_free_running_counts_and_determinism():
    w = make_workload("cfg4", rows=5 * 400)
    wc = to_cuda(w)
    outs = []
    for _ in range(2):
        g = binding.from_workload(wc, stream=torch.cuda.Stream())
        g.step(50)
        outs.append((g.get_theta(), g.get_selection_mask(0, 50), g.get_comm_count(), g.get_wallclock()))
        g.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and np.array_equal(outs[0][1], outs[1][1])
    assert outs[0][2:] == outs[1][2:]
    up, comm, comp = outs[0][2]
    assert up == int(outs[0][1].sum()) and comm == 3 * up and comp == 2 * up
    assert outs[0][1][0].all() and up < 50 * 5


def test_printed_rule_computes_only_the_selected_groups():
    """Rule PS on the fp32 MLP: selection first, then only the selected groups run, at theta^k only.  The
    free-running masks equal the oracle's, the uploaded gradients equal the oracle's gradient at the CUDA
    path's own iterate, and the aggregate is the sum of the last uploads (Eq. 3)."""
    import numpy as np
    import torch
    from paper_2201_04301_b200 import binding
    from parity import make_oracle, rel_l2, to_cuda
    w = make_workload("cfg4", rows=5 * 400, D=5, c=1.0)
    G = 5
    L = [2.0, 0.1, 0.7, 0.02, 1.3]      # none with L_g^2 = c: at k = 1 the test is L_g^2 > c exactly
    o = make_oracle(w, rule="ps", L=L)
    g = binding.from_workload(to_cuda(w), stream=torch.cuda.Stream(), options={binding.OPT_RULE: 1.0}, smoothness=L)
    K = 20
    for k in range(K):
        theta_gpu = g.get_theta().astype(np.float64)
        batches = [o.minibatch(gi) for gi in range(G)]
        rec = o.step()
        g.step(1)
        mask = g.get_selection_mask(k, 1)[0]
        assert np.array_equal(mask, rec["mask"]), (k, mask, rec["mask"])
        assert np.allclose(g.get_debug(binding.DBG_LHS), rec["lhs"], rtol=1e-4, atol=1e-30)
        last = g.get_debug(binding.DBG_GLAST)
        for gi in np.nonzero(mask)[0]:
            want = o.model.grad(theta_gpu, batches[gi][1], batches[gi][2], "mean")
            assert rel_l2(last[gi], want) <= 5e-5, (k, gi)      # an occasional ReLU unit on its kink
        assert rel_l2(g.get_debug(binding.DBG_AGG), last.astype(np.float64).sum(axis=0)) <= 1e-6
        assert rel_l2(g.get_theta(), rec["theta"]) <= 1e-4
    masks = g.get_selection_mask(0, K)
    assert masks[0].all() and 0 < masks.sum() < masks.size
    assert g.get_comm_count() == (o.uploads, o.comm, o.comp)


@pytest.mark.parametrize("name,over", [("cfg4", dict(rows=5 * 400)),
                                       ("cfg5", dict(rows=6000, dims=(64, 128, 96, 40), M=12, M_G=2, D=5, batch=128, c=1.0))])
def test_graph_replay_equals_plain_launches_bitwise(name, over):
    """Inside a replayed chain of iterations the kernel that gathers the minibatch rows is launched programmatically
    dependent on the previous iteration's update kernel and runs beside it, with the iteration number of its
    draw taken from the chain's start.  The run must not depend on that in any bit, however it is cut into
    calls and with plain (forced) iterations between two chains."""
    w = to_cuda(make_workload(name, **over))
    G = w["M"] // w["M_G"]
    forced = np.ones((3, G), np.uint8)
    forced[1, ::2] = 0
    runs = []
    for graph, chunks in ((1.0, [40]), (0.0, [40]), (1.0, [16, 5, 19]), (1.0, [33, -3, 4]), (0.0, [33, -3, 4])):
        g = binding.from_workload(w, stream=torch.cuda.Stream(), options={binding.OPT_GRAPH: graph})
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
