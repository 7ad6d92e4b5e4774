"""The shared library loads on a machine without a GPU and exports every
symbol the header declares; argument checks that need no device work."""
import ctypes as C
import os
import re

import pytest

from paper_2201_04301_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def test_every_declared_symbol_is_exported(lib):
    text = open(os.path.join(ROOT, "include", "gcada.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(gcada_[a-z_]+)\s*\(", text))
    assert declared == set(binding.SIGNATURES), declared ^ set(binding.SIGNATURES)
    for name in declared:
        assert hasattr(lib, name)


def test_create_rejects_bad_arguments_before_touching_a_device(lib):
    dims = (C.c_int * 1)(8)
    m = binding.Model(binding.MODEL_LOGISTIC, 1, dims, 0)
    h = C.c_void_p()
    bad = [
        dict(M=6, M_G=4),            # M not divisible by M_G
        dict(M=0), dict(M_G=0), dict(D=0), dict(c=-1.0), dict(alpha=0.0),
        dict(beta1=1.0), dict(beta2=0.0), dict(eps=0.0),
    ]
    base = dict(M=6, M_G=2, D=10, c=1.0, alpha=0.01, beta1=0.9, beta2=0.99, eps=1e-8)
    for b in bad:
        a = dict(base, **b)
        st = lib.gcada_create(C.byref(m), a["M"], a["M_G"], a["D"], a["c"], a["alpha"], a["beta1"], a["beta2"],
                              a["eps"], C.byref(h))
        assert st == binding.EINVAL and not h.value
        assert lib.gcada_last_error(None)
    dims_big = (C.c_int * 1)(5000)
    m2 = binding.Model(binding.MODEL_LOGISTIC, 1, dims_big, 0)
    assert lib.gcada_create(C.byref(m2), 6, 2, 10, 1.0, .01, .9, .99, 1e-8, C.byref(h)) == binding.EINVAL
    m3 = binding.Model(7, 1, dims, 0)
    assert lib.gcada_create(C.byref(m3), 6, 2, 10, 1.0, .01, .9, .99, 1e-8, C.byref(h)) == binding.EINVAL


def test_no_device_means_an_error_not_a_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    dims = (C.c_int * 1)(8)
    m = binding.Model(binding.MODEL_LOGISTIC, 1, dims, 0)
    h = C.c_void_p()
    st = lib.gcada_create(C.byref(m), 6, 2, 10, 1.0, .01, .9, .99, 1e-8, C.byref(h))
    assert st == binding.ECUDA and not h.value


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(FileNotFoundError):
        binding.load(str(tmp_path / "libgcada.so"))
