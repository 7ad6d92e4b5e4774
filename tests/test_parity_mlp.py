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
