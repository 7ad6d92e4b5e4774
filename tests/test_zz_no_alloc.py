"""The no-allocation entry point against the ordinary path.

gcada_innovation_norms_noalloc serves callers that may not allocate device
memory (a process with a frozen memory pool, a latency-critical loop): its
scratch is a fixed array inside the library.  Here it is fed the two gradient
sets an ordinary context produced and must reproduce that context's own test
quantities (gcada_step + gcada_get_debug), on two calls in a row that share
the scratch array, with different data in each.

This file is named to be collected last, so that a run stopping at the first
failure has already run every other test.
"""
import numpy as np
import pytest
import torch

from paper_2201_04301_b200 import binding
from paper_2201_04301_b200.workloads import make_workload

from parity import MARGIN, to_cuda

pytestmark = pytest.mark.gpu


def test_two_calls_in_a_row_match_the_context_path():
    # a large step size keeps the gradient change well above fp32 rounding of the gradients
    w = to_cuda(make_workload("cfg1", rows=3000, kind="quadratic", alpha=0.2, c=1e9))
    stream = torch.cuda.Stream()
    g = binding.from_workload(w, stream=stream, options={binding.OPT_KEEP_STALE: 1.0})
    g.step(2)
    lhs_out = torch.full((g.G,), -1.0, dtype=torch.float64, device="cuda")   # caller-owned output
    for call in range(2):
        g.step(1)
        want = g.get_debug(binding.DBG_LHS)
        fresh = torch.from_numpy(g.get_debug(binding.DBG_FRESH)).cuda()
        stale = torch.from_numpy(g.get_debug(binding.DBG_STALE)).cuda()
        torch.cuda.synchronize()
        binding.innovation_norms_noalloc(fresh, stale, lhs_out, stream=stream)
        stream.synchronize()
        got = lhs_out.cpu().numpy()
        assert np.all(want > 0)
        assert np.all(np.abs(got - want) <= MARGIN * want), (call, got, want)
        # and exactly what the definition gives on those arrays
        ref = ((fresh - stale).double() ** 2).sum(dim=1).cpu().numpy()
        assert np.allclose(got, ref, rtol=1e-12)
    g.close()


def test_strided_rows_and_size_limit():
    G, p, ld = 5, 1001, 1024
    gen = torch.Generator(device="cuda").manual_seed(1)
    a = torch.randn(G, ld, generator=gen, device="cuda")
    b = torch.randn(G, ld, generator=gen, device="cuda")
    out = torch.zeros(G, dtype=torch.float64, device="cuda")
    binding.innovation_norms_noalloc(a[:, :p], b[:, :p], out)
    torch.cuda.synchronize()
    ref = ((a[:, :p] - b[:, :p]).double() ** 2).sum(dim=1)     # float difference, double sum, as documented
    assert torch.allclose(out, ref, rtol=1e-12)
    big = torch.zeros(binding.NOALLOC_MAX_GROUPS + 1, 4, device="cuda")
    with pytest.raises(binding.GCadaError) as e:
        binding.innovation_norms_noalloc(big, big, torch.zeros(big.shape[0], dtype=torch.float64, device="cuda"))
    assert e.value.status == binding.EINVAL and "at most" in str(e.value)
