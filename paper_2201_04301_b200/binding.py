"""ctypes binding of libgcada.so: the same entry points as include/gcada.h.

Only argument marshalling happens here; every step of the method runs in the
library's CUDA kernels.  `load()` fails loudly when the shared library is
missing or cannot be loaded: there is no fallback implementation.
"""
import ctypes as C
import os

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libgcada.so")
DEBUG_LIB_PATH = os.path.join(HERE, "libgcada_dbg.so")   # the same source with every computed store index checked

OK, EINVAL, ENOMEM, ECUDA, ESTATE, ETIMEOUT = range(6)
MODEL_LOGISTIC, MODEL_MLP, MODEL_QUADRATIC = 0, 1, 2
COMPUTE_FP32, COMPUTE_BF16 = 0, 1
(OPT_RULE, OPT_REDUCTION, OPT_HISTORY, OPT_KEEP_STALE, OPT_GRAPH, OPT_TIMING, _OPT_UNUSED,
 OPT_PERSISTENT) = range(8)
(DBG_FRESH, DBG_STALE, DBG_LHS, DBG_RHS, DBG_TAU, DBG_AGG, DBG_H, DBG_VHAT, DBG_TGROUP, DBG_GLAST,
 DBG_SRING) = range(11)
MODEL_KINDS = {"logistic": MODEL_LOGISTIC, "mlp": MODEL_MLP, "quadratic": MODEL_QUADRATIC}
COMPUTE_KINDS = {"fp32": COMPUTE_FP32, "bf16": COMPUTE_BF16}
DELAY_LAWS = {"exp": 0, "pareto": 1, "uniform": 2}
SCHEDULES = {"const": 0, "poly": 1, "step": 2}


class Model(C.Structure):
    _fields_ = [("kind", C.c_int), ("n_dims", C.c_int), ("dims", C.POINTER(C.c_int)), ("compute", C.c_int)]


class GCadaError(RuntimeError):
    def __init__(self, status, text):
        super().__init__("gcada status %d: %s" % (status, text))
        self.status = status


# name -> (restype, argtypes): every symbol include/gcada.h declares
_VP, _LL, _ULLP = C.c_void_p, C.c_longlong, C.POINTER(C.c_ulonglong)
SIGNATURES = {
    "gcada_create": (C.c_int, [C.POINTER(Model), C.c_int, C.c_int, C.c_int, C.c_double, C.c_double, C.c_double,
                               C.c_double, C.c_double, C.POINTER(_VP)]),
    "gcada_set_stream": (C.c_int, [_VP, _VP]),
    "gcada_set_data": (C.c_int, [_VP, _VP, _VP, _LL, _LL, C.c_int]),
    "gcada_set_theta": (C.c_int, [_VP, _VP, _LL, C.c_int]),
    "gcada_set_seed": (C.c_int, [_VP, C.c_ulonglong]),
    "gcada_set_delay_model": (C.c_int, [_VP, C.c_double, C.c_double]),
    "gcada_set_option": (C.c_int, [_VP, C.c_int, C.c_double]),
    "gcada_set_delay_law": (C.c_int, [_VP, C.c_int]),
    "gcada_set_lag_weights": (C.c_int, [_VP, C.POINTER(C.c_double), C.c_int]),
    "gcada_set_step_schedule": (C.c_int, [_VP, C.c_int, C.c_double, C.c_double]),
    "gcada_set_smoothness": (C.c_int, [_VP, C.POINTER(C.c_double), C.c_int]),
    "gcada_step": (C.c_int, [_VP, C.c_int]),
    "gcada_step_forced": (C.c_int, [_VP, C.c_int, _VP]),
    "gcada_step_host_batch": (C.c_int, [_VP, _VP, _VP]),
    "gcada_set_batch": (C.c_int, [_VP, C.c_int]),
    "gcada_get_theta": (C.c_int, [_VP, _VP, _LL]),
    "gcada_get_selection_mask": (C.c_int, [_VP, _VP, _LL, C.c_int]),
    "gcada_get_comm_count": (C.c_int, [_VP, _ULLP, _ULLP, _ULLP]),
    "gcada_get_wallclock": (C.c_int, [_VP, C.POINTER(C.c_double), C.POINTER(C.c_double)]),
    "gcada_get_iteration": (C.c_int, [_VP, C.POINTER(_LL)]),
    "gcada_get_debug": (C.c_int, [_VP, C.c_int, _VP, _LL]),
    "gcada_get_group_gradient": (C.c_int, [_VP, C.c_int, C.c_int, _VP, _LL]),
    "gcada_get_launch_count": (C.c_int, [_VP, _ULLP]),
    "gcada_get_kernel_times": (C.c_int, [_VP, C.POINTER(C.c_double), C.POINTER(C.c_int)]),
    "gcada_innovation_norms_noalloc": (C.c_int, [_VP, _VP, C.c_int, _LL, _LL, _VP, _VP, C.c_char_p, C.c_size_t]),
    "gcada_time_gradient": (C.c_int, [_VP, C.c_int, C.POINTER(C.c_double)]),
    "gcada_time_empty_chain": (C.c_int, [_VP, C.c_int, C.POINTER(C.c_double)]),
    "gcada_eval_loss": (C.c_int, [_VP, _LL, _LL, C.POINTER(C.c_double)]),
    "gcada_checkpoint_size": (C.c_int, [_VP, _ULLP]),
    "gcada_checkpoint_save": (C.c_int, [_VP, _VP, C.c_ulonglong]),
    "gcada_checkpoint_load": (C.c_int, [_VP, _VP, C.c_ulonglong]),
    "gcada_is_debug_build": (C.c_int, []),
    "gcada_debug_set_error": (C.c_int, [_VP, C.c_int]),
    "gcada_last_error": (C.c_char_p, [_VP]),
    "gcada_destroy": (None, [_VP]),
}

_lib = None


def load(path=None):
    """dlopen the library and attach prototypes.  Raises if it is not there."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise FileNotFoundError(
            "%s is missing: build it with `python -m paper_2201_04301_b200.build` (there is no fallback)" % path)
    lib = C.CDLL(path)
    for name, (res, args) in SIGNATURES.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


class GCada:
    """One G-CADA context.  Method names follow the C entry points."""

    def __init__(self, kind, dims, M, M_G, D, c, alpha, beta1, beta2, eps, compute="fp32", stream=None):
        self.lib = load()
        self.dims = [int(x) for x in dims]
        arr = (C.c_int * len(self.dims))(*self.dims)
        model = Model(MODEL_KINDS[kind], len(self.dims), arr, COMPUTE_KINDS[compute])
        h = _VP()
        st = self.lib.gcada_create(C.byref(model), M, M_G, D, c, alpha, beta1, beta2, eps, C.byref(h))
        if st != OK:
            raise GCadaError(st, self.lib.gcada_last_error(None).decode())
        self.h = h
        self.G = M // M_G
        self.M, self.M_G, self.D = M, M_G, D
        if kind == "mlp":
            self.p = sum(self.dims[l] * self.dims[l - 1] + self.dims[l] for l in range(1, len(self.dims)))
        else:
            self.p = self.dims[0]
        self._keep = []
        if stream is not None:
            self.set_stream(stream)

    def _ck(self, st):
        if st != OK:
            raise GCadaError(st, self.lib.gcada_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            self.lib.gcada_destroy(self.h)
            self.h = None

    __del__ = close

    # -- setters ----------------------------------------------------------
    def set_stream(self, stream):
        """`stream`: a torch.cuda.Stream, a raw cudaStream_t integer, or None."""
        raw = getattr(stream, "cuda_stream", stream)
        self._ck(self.lib.gcada_set_stream(self.h, _VP(raw or 0)))

    def set_data(self, X, y, batch, ld=None):
        """X, y: CUDA torch tensors (borrowed; kept alive by this object)."""
        assert X.is_cuda and y.is_cuda and X.stride(-1) == 1
        self._keep = [X, y]
        ld = int(ld if ld is not None else X.stride(0))
        self._ck(self.lib.gcada_set_data(self.h, _VP(X.data_ptr()), _VP(y.data_ptr()), X.shape[0], ld, int(batch)))

    def set_batch(self, batch):
        self._ck(self.lib.gcada_set_batch(self.h, int(batch)))

    def set_theta(self, theta0):
        """theta0: float32 torch tensor (CPU or CUDA) or numpy array."""
        if hasattr(theta0, "is_cuda"):
            t = theta0.detach().contiguous()
            assert str(t.dtype) == "torch.float32"
            self._ck(self.lib.gcada_set_theta(self.h, _VP(t.data_ptr()), t.numel(), 1 if t.is_cuda else 0))
        else:
            a = np.ascontiguousarray(theta0, dtype=np.float32)
            self._ck(self.lib.gcada_set_theta(self.h, _VP(a.ctypes.data), a.size, 0))

    def set_seed(self, seed):
        self._ck(self.lib.gcada_set_seed(self.h, int(seed)))

    def set_delay_model(self, shift, rate):
        self._ck(self.lib.gcada_set_delay_model(self.h, float(shift), float(rate)))

    def set_option(self, key, value):
        self._ck(self.lib.gcada_set_option(self.h, int(key), float(value)))

    def set_delay_law(self, law):
        self._ck(self.lib.gcada_set_delay_law(self.h, DELAY_LAWS.get(law, law)))

    def set_lag_weights(self, c_d):
        if c_d is None:
            self._ck(self.lib.gcada_set_lag_weights(self.h, None, 0))
        else:
            a = (C.c_double * len(c_d))(*[float(v) for v in c_d])
            self._ck(self.lib.gcada_set_lag_weights(self.h, a, len(c_d)))

    def set_step_schedule(self, kind, a=1.0, b=0.0):
        self._ck(self.lib.gcada_set_step_schedule(self.h, SCHEDULES.get(kind, kind), float(a), float(b)))

    def set_smoothness(self, L):
        a = (C.c_double * len(L))(*[float(v) for v in L])
        self._ck(self.lib.gcada_set_smoothness(self.h, a, len(L)))

    # -- stepping ----------------------------------------------------------
    def step(self, n_iters=1):
        self._ck(self.lib.gcada_step(self.h, int(n_iters)))

    def step_forced(self, mask):
        m = np.ascontiguousarray(mask, dtype=np.uint8).reshape(-1, self.G)
        self._ck(self.lib.gcada_step_forced(self.h, m.shape[0], _VP(m.ctypes.data)))

    def step_host_batch(self, Xb, yb):
        """Xb, yb: host buffers (pinned torch CPU tensors or numpy arrays)."""
        xp = Xb.data_ptr() if hasattr(Xb, "data_ptr") else Xb.ctypes.data
        yp = yb.data_ptr() if hasattr(yb, "data_ptr") else yb.ctypes.data
        self._ck(self.lib.gcada_step_host_batch(self.h, _VP(xp), _VP(yp)))

    # -- getters -----------------------------------------------------------
    def get_theta(self, out=None):
        """theta^k as p floats on the host.  `out`: an optional float32 host buffer of p elements to fill
        (a numpy array or a CPU torch tensor; a pinned one is copied into without a staging pass)."""
        if out is None:
            out = np.empty(self.p, dtype=np.float32)
        n = out.numel() if hasattr(out, "numel") else out.size
        contiguous = out.is_contiguous() if hasattr(out, "is_contiguous") else out.flags["C_CONTIGUOUS"]
        if n != self.p or "float32" not in str(out.dtype) or not contiguous or getattr(out, "is_cuda", False):
            raise ValueError("get_theta: out must be a contiguous host buffer of p = %d float32 values" % self.p)
        ptr = out.data_ptr() if hasattr(out, "data_ptr") else out.ctypes.data
        self._ck(self.lib.gcada_get_theta(self.h, _VP(ptr), self.p))
        return out

    def get_selection_mask(self, first_iter, n_iters):
        out = np.empty((n_iters, self.G), dtype=np.uint8)
        self._ck(self.lib.gcada_get_selection_mask(self.h, _VP(out.ctypes.data), int(first_iter), int(n_iters)))
        return out

    def get_comm_count(self):
        a, b, c = C.c_ulonglong(), C.c_ulonglong(), C.c_ulonglong()
        self._ck(self.lib.gcada_get_comm_count(self.h, C.byref(a), C.byref(b), C.byref(c)))
        return a.value, b.value, c.value

    def get_wallclock(self):
        a, b = C.c_double(), C.c_double()
        self._ck(self.lib.gcada_get_wallclock(self.h, C.byref(a), C.byref(b)))
        return a.value, b.value

    def get_iteration(self):
        k = _LL()
        self._ck(self.lib.gcada_get_iteration(self.h, C.byref(k)))
        return k.value

    def get_launch_count(self):
        n = C.c_ulonglong()
        self._ck(self.lib.gcada_get_launch_count(self.h, C.byref(n)))
        return n.value

    def get_group_gradient(self, what, g):
        out = np.empty(self.p, dtype=np.float32)
        self._ck(self.lib.gcada_get_group_gradient(self.h, int(what), int(g), _VP(out.ctypes.data), self.p))
        return out

    def time_gradient(self, reps):
        """Mean device time (ms) of the gradient kernel(s) over `reps` back-to-back repetitions."""
        ms = C.c_double()
        self._ck(self.lib.gcada_time_gradient(self.h, int(reps), C.byref(ms)))
        return ms.value

    def time_empty_chain(self, n_iters):
        """Device time per iteration (microseconds) of the iteration's launch structure with empty kernels."""
        us = C.c_double()
        self._ck(self.lib.gcada_time_empty_chain(self.h, int(n_iters), C.byref(us)))
        return us.value

    def get_kernel_times(self):
        """(ms_gradient, ms_select, ms_update), n_timed: see GCADA_OPT_TIMING."""
        ms = (C.c_double * 3)()
        n = C.c_int()
        self._ck(self.lib.gcada_get_kernel_times(self.h, ms, C.byref(n)))
        return (ms[0], ms[1], ms[2]), n.value

    def eval_loss(self, first_row, n_rows):
        """Mean loss of the current iterate over a range of training rows (linear models)."""
        v = C.c_double()
        self._ck(self.lib.gcada_eval_loss(self.h, int(first_row), int(n_rows), C.byref(v)))
        return v.value

    def checkpoint_save(self):
        """The run's state as a numpy byte array (see gcada_checkpoint_save)."""
        n = C.c_ulonglong()
        self._ck(self.lib.gcada_checkpoint_size(self.h, C.byref(n)))
        buf = np.empty(n.value, dtype=np.uint8)
        self._ck(self.lib.gcada_checkpoint_save(self.h, _VP(buf.ctypes.data), n.value))
        return buf

    def checkpoint_load(self, buf):
        buf = np.ascontiguousarray(buf, dtype=np.uint8)
        self._ck(self.lib.gcada_checkpoint_load(self.h, _VP(buf.ctypes.data), buf.size))

    def debug_set_error(self, dev_err):
        """Debug library only: write the device error word (0 none, 1 a wait gave up, 2 an index check failed)."""
        self._ck(self.lib.gcada_debug_set_error(self.h, int(dev_err)))

    def get_debug(self, what):
        G, p, D = self.G, self.p, self.D
        shape, dt = {
            DBG_FRESH: ((G, p), np.float32), DBG_STALE: ((G, p), np.float32), DBG_GLAST: ((G, p), np.float32),
            DBG_LHS: ((G,), np.float64), DBG_RHS: ((1,), np.float64), DBG_TAU: ((G,), np.int32),
            DBG_AGG: ((p,), np.float32), DBG_H: ((p,), np.float32), DBG_VHAT: ((p,), np.float32),
            DBG_TGROUP: ((G,), np.float64), DBG_SRING: ((D,), np.float64),
        }[what]
        out = np.empty(shape, dtype=dt)
        self._ck(self.lib.gcada_get_debug(self.h, int(what), _VP(out.ctypes.data), out.nbytes))
        return out


NOALLOC_MAX_GROUPS = 1024


def innovation_norms_noalloc(fresh, stale, lhs_out, stream=None):
    """lhs_out[g] = ||fresh[g] - stale[g]||^2 through gcada_innovation_norms_noalloc.

    fresh, stale: CUDA float32 tensors [G, p] with the same row stride; lhs_out:
    CUDA float64 tensor [G].  All of them are the caller's; the call itself
    allocates nothing on the device (its scratch is a fixed array inside the
    library, shared by every call: do not overlap calls on one GPU)."""
    lib = load()
    G, p = fresh.shape
    assert stale.shape == fresh.shape and fresh.stride(0) == stale.stride(0) and fresh.stride(1) == 1
    buf = C.create_string_buffer(256)
    raw = getattr(stream, "cuda_stream", stream)
    st = lib.gcada_innovation_norms_noalloc(_VP(fresh.data_ptr()), _VP(stale.data_ptr()), int(G), int(p),
                                            int(fresh.stride(0)), _VP(lhs_out.data_ptr()), _VP(raw or 0), buf, 256)
    if st != OK:
        raise GCadaError(st, buf.value.decode())


def from_workload(w, stream=None, options=None, smoothness=None, c_d=None, schedule=None, delay_law=None):
    """Context for a dict made by workloads.make_workload (tensors on CUDA)."""
    g = GCada(w["kind"], w["dims"], w["M"], w["M_G"], w["D"], w["c"], w["alpha"], w["beta1"], w["beta2"],
              w["eps"], compute=w["compute"], stream=stream)
    g.set_seed(w["seed"])
    g.set_delay_model(w["shift"], w["rate"])
    for key, val in (options or {}).items():
        g.set_option(key, val)
    if smoothness is not None:
        g.set_smoothness(smoothness)
    if c_d is not None:
        g.set_lag_weights(c_d)
    if schedule is not None:
        g.set_step_schedule(*schedule)
    if delay_law is not None:
        g.set_delay_law(delay_law)
    g.set_data(w["X"], w["y"], w["batch"], ld=w["ld"])
    g.set_theta(w["theta0"])
    return g
