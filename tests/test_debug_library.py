"""The bounds-checked twin of the library (libgcada_dbg.so: the same sources compiled with -DGCADA_DEBUG).

Every store whose position a kernel computes at run time is checked there against the size of its buffer; a
failed check skips the store and raises the run's device error word, which every getter reports.  The GPU
tests run odd shapes and edge cases of every path through that library against the oracle and require that
no check fired, and they exercise the reporting path (GCADA_ETIMEOUT for a device wait that gave up,
GCADA_ECUDA for a failed index check) by writing the error word from the host: no device-side failure is
provoked."""
import numpy as np
import pytest
import torch

from paper_2201_04301_b200 import binding, build
from paper_2201_04301_b200.workloads import make_workload

from parity import TOL_BF16, forced_parity, to_cuda


@pytest.fixture()
def debug_lib():
    build.build(debug=True)
    lib = binding.load(binding.DEBUG_LIB_PATH)      # contexts created from now on use the debug library
    assert lib.gcada_is_debug_build() == 1
    yield lib
    assert binding.load(binding.LIB_PATH).gcada_is_debug_build() == 0


def test_debug_library_builds_and_exports_the_same_interface():
    build.build()
    build.build(debug=True)
    rel = binding.load(binding.LIB_PATH)
    dbg = binding.load(binding.DEBUG_LIB_PATH)
    try:
        for name in binding.SIGNATURES:
            assert hasattr(dbg, name) and hasattr(rel, name)
        assert dbg.gcada_is_debug_build() == 1 and rel.gcada_is_debug_build() == 0
    finally:
        binding.load(binding.LIB_PATH)


@pytest.mark.gpu
def test_no_index_check_fires_on_odd_shapes_and_edge_cases(debug_lib):
    st = torch.cuda.Stream()
    # narrow linear (chain), groups of one, single-row batches, one-row shards
    forced_parity(make_workload("cfg1", rows=3, dims=(9,), M=3, M_G=1, D=2, batch=1), 6, stream=st)
    forced_parity(make_workload("cfg1", rows=3000), 12, stream=st)
    # d = 54 with padded rows, more groups than one pass of the scheduling phase
    forced_parity(make_workload("cfg2", rows=5 * 700), 6, stream=st)
    forced_parity(make_workload("cfg1", rows=300 * 4, dims=(6,), M=1500, M_G=5, D=1, batch=2), 3, stream=st)
    # wide linear: ragged width, a CTA that spans three groups, the full-width instantiation
    forced_parity(make_workload("cfg3", rows=7 * 90, dims=(1028,), M=7, M_G=1, D=3, batch=5), 5, stream=st)
    forced_parity(make_workload("cfg3", rows=64 * 40, M=128, M_G=2, D=3, batch=3), 4, stream=st)
    # printed rule, selection first (only the selected groups compute)
    forced_parity(make_workload("cfg3", rows=6 * 300, M=12, M_G=2, D=3, batch=40), 6, stream=st,
                  L=[3.0, 0.2, 1.4, 0.05, 2.0, 0.5])
    # fp32 MLP: batch not a multiple of the tile, cluster-split first layer
    forced_parity(make_workload("cfg4", rows=400, dims=(20, 3), M=2, M_G=1, D=2, batch=65, alpha=0.01), 5, stream=st)
    forced_parity(make_workload("cfg4", rows=5 * 200), 6, stream=st)
    # bf16 MLP: ragged K and N, padded minibatch, two row tiles per group; inspection and production paths
    forced_parity(make_workload("cfg5", rows=900, dims=(24, 40, 8), M=3, M_G=1, D=2, batch=200), 5, tol=TOL_BF16,
                  stream=st, rhs_tol=2e-2)
    w = to_cuda(make_workload("cfg5", rows=4 * 700, dims=(256, 300, 130), M=8, M_G=2, D=3, batch=200, c=0.3))
    g = binding.from_workload(w, stream=st)
    g.step(21)                                     # graph replay, running aggregate and a refresh
    assert np.isfinite(g.get_theta()).all() and g.get_iteration() == 21
    g.get_group_gradient(binding.DBG_GLAST, 2)
    g.close()
    # free-running cluster kernel and graph-replayed chain
    for name, opts in (("cfg1", {}), ("cfg2", {}), ("cfg2", {binding.OPT_PERSISTENT: 0.0})):
        g = binding.from_workload(to_cuda(make_workload(name, rows=5 * 2000)), stream=st, options=opts)
        g.step(40)
        assert g.get_iteration() == 40 and g.get_selection_mask(0, 40)[0].all()
        g.close()


@pytest.mark.gpu
def test_a_raised_error_word_reaches_every_getter(debug_lib):
    g = binding.from_workload(to_cuda(make_workload("cfg1", rows=3000)), stream=torch.cuda.Stream())
    g.step(3)
    g.get_theta()
    for word, status, text in ((1, binding.ETIMEOUT, "wait"), (2, binding.ECUDA, "index check"),
                               (3, binding.ECUDA, "chain of iterations")):
        g.debug_set_error(word)
        for call in (g.get_theta, g.get_iteration, g.get_comm_count, g.get_wallclock,
                     lambda: g.get_selection_mask(0, 1), lambda: g.get_debug(binding.DBG_LHS), g.checkpoint_save):
            with pytest.raises(binding.GCadaError) as e:
                call()
            assert e.value.status == status and text in str(e.value)
        g.debug_set_error(0)
        assert g.get_iteration() == 3
    with pytest.raises(binding.GCadaError) as e:
        g.debug_set_error(7)
    assert e.value.status == binding.EINVAL
    g.close()


@pytest.mark.gpu
def test_the_ordinary_library_has_no_error_setter():
    lib = binding.load(binding.LIB_PATH)
    assert lib.gcada_is_debug_build() == 0
    g = binding.from_workload(to_cuda(make_workload("cfg1", rows=3000)), stream=torch.cuda.Stream())
    with pytest.raises(binding.GCadaError) as e:
        g.debug_set_error(1)
    assert e.value.status == binding.ESTATE
    g.step(2)
    assert g.get_iteration() == 2
    g.close()
