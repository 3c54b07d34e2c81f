"""ctypes view of the CPU oracle (oracle/zoa_oracle.c).

Test infrastructure only: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg, never by the product.  This module only owns the
numpy arrays and marshals pointers; every arithmetic step of the method is in
the C file, next to the passage of the paper it follows.
"""
import ctypes as C
import importlib.util
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))


def _load():
    spec = importlib.util.spec_from_file_location("_zoa_oracle_build", os.path.join(_HERE, "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    return C.CDLL(mod.build())


_lib = _load()

ONEBIT, IDENTITY = 0, 1


def _state_struct(real):
    p_real = C.POINTER(real)
    p_u32 = C.POINTER(C.c_uint32)

    class State(C.Structure):
        _fields_ = [
            ("d", C.c_int64), ("n", C.c_int32), ("chunk", C.c_int64),
            ("beta1", real), ("beta2", real), ("eps", real),
            ("compressor", C.c_int32), ("literal_momentum", C.c_int32),
            ("x", p_real), ("m", p_real), ("u", p_real), ("delta", p_real),
            ("v", p_real), ("delta_bar", p_real), ("x_sync", p_real),
            ("z_hat", p_real), ("u_bar", p_real),
            ("words_worker", p_u32), ("scales_worker", p_real),
            ("words_server", p_u32), ("scales_server", p_real),
            ("gamma_sum", C.c_double), ("t_sync", C.c_int64),
        ]
    return State


_KINDS = {
    np.dtype(np.float32): ("_f32", C.c_float, _state_struct(C.c_float)),
    np.dtype(np.float64): ("_f64", C.c_double, _state_struct(C.c_double)),
}


def _fn(name, suffix):
    f = getattr(_lib, name + suffix)
    return f


def _ptr(a, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def compress(a, chunk):
    """Eq. 3 per chunk.  Returns (a_hat, words uint32, scales)."""
    a = np.ascontiguousarray(a)
    suffix, real, _ = _KINDS[a.dtype]
    d = a.size
    a_hat = np.empty_like(a)
    words = np.empty((d + 31) // 32, np.uint32)
    scales = np.empty((d + chunk - 1) // chunk, a.dtype)
    f = _fn("zo_compress", suffix)
    f.restype = None
    f(_ptr(a, real), C.c_int64(d), C.c_int64(chunk), _ptr(a_hat, real),
      _ptr(words, C.c_uint32), _ptr(scales, real))
    return a_hat, words, scales


def allreduce(g):
    """Algorithm 4: mean over the workers.  g is [n][d]."""
    g = np.ascontiguousarray(g)
    suffix, real, _ = _KINDS[g.dtype]
    n, d = g.shape
    out = np.empty(d, g.dtype)
    f = _fn("zo_allreduce", suffix)
    f.restype = None
    f(_ptr(g, real), C.c_int32(n), C.c_int64(d), _ptr(out, real))
    return out


class Oracle:
    """State of Algorithm 1 for n workers over a d-dimensional model."""

    def __init__(self, d, n, chunk, beta1=0.9, beta2=0.999, eps=1e-8, dtype=np.float32,
                 compressor=ONEBIT, literal_momentum=False):
        self.dtype = np.dtype(dtype)
        self._suffix, self._real, State = _KINDS[self.dtype]
        self.d, self.n, self.chunk = int(d), int(n), int(chunk)
        self.n_words = (self.d + 31) // 32
        self.n_chunks = (self.d + self.chunk - 1) // self.chunk
        z = lambda *shape: np.zeros(shape, self.dtype)
        self.x, self.m, self.u, self.delta = z(n, d), z(n, d), z(n, d), z(n, d)
        self.v, self.delta_bar, self.x_sync = z(d), z(d), z(d)
        self.z_hat, self.u_bar = z(n, d), z(d)
        self.words_worker = np.zeros((n, self.n_words), np.uint32)
        self.scales_worker = z(n, self.n_chunks)
        self.words_server = np.zeros(self.n_words, np.uint32)
        self.scales_server = z(self.n_chunks)
        self._g_bar = z(d)
        r, u32 = self._real, C.c_uint32
        self._st = State(
            d=self.d, n=self.n, chunk=self.chunk,
            beta1=self.dtype.type(beta1), beta2=self.dtype.type(beta2), eps=self.dtype.type(eps),
            compressor=int(compressor), literal_momentum=int(bool(literal_momentum)),
            x=_ptr(self.x, r), m=_ptr(self.m, r), u=_ptr(self.u, r), delta=_ptr(self.delta, r),
            v=_ptr(self.v, r), delta_bar=_ptr(self.delta_bar, r), x_sync=_ptr(self.x_sync, r),
            z_hat=_ptr(self.z_hat, r), u_bar=_ptr(self.u_bar, r),
            words_worker=_ptr(self.words_worker, u32), scales_worker=_ptr(self.scales_worker, r),
            words_server=_ptr(self.words_server, u32), scales_server=_ptr(self.scales_server, r),
            gamma_sum=0.0, t_sync=0)

    # -- state access ------------------------------------------------------
    def set_params(self, x0):
        """Same initial model on every worker; it is also x_{t'} until the first sync."""
        x0 = np.asarray(x0, self.dtype).reshape(self.d)
        self.x[:] = x0
        self.x_sync[:] = x0

    @property
    def gamma_sum(self):
        return self._st.gamma_sum

    @property
    def t_sync(self):
        return self._st.t_sync

    def _g(self, g):
        g = np.ascontiguousarray(g, self.dtype)
        assert g.shape == (self.n, self.d)
        return g

    # -- Algorithm 1 ---------------------------------------------------------
    def half_step(self, g, gamma):
        g = self._g(g)
        f = _fn("zo_alg1_half_step", self._suffix)
        f.restype = None
        f(C.byref(self._st), _ptr(g, self._real), self._real(gamma))

    def sync(self, t):
        f = _fn("zo_alg1_sync", self._suffix)
        f.restype = C.c_int
        return f(C.byref(self._st), C.c_int64(t))

    def variance(self, g):
        g = self._g(g)
        f = _fn("zo_alg1_variance", self._suffix)
        f.restype = None
        f(C.byref(self._st), _ptr(g, self._real), _ptr(self._g_bar, self._real))

    def step(self, g, gamma, t, in_T_u, in_T_v):
        g = self._g(g)
        f = _fn("zo_alg1_step", self._suffix)
        f.restype = C.c_int
        return f(C.byref(self._st), _ptr(g, self._real), self._real(gamma), C.c_int64(t),
                 C.c_int(bool(in_T_u)), C.c_int(bool(in_T_v)), _ptr(self._g_bar, self._real))

    # -- Algorithm 2 ---------------------------------------------------------
    def alg2_step(self, g, gamma, in_T_v):
        g = self._g(g)
        f = _fn("zo_alg2_step", self._suffix)
        f.restype = None
        f(C.byref(self._st), _ptr(g, self._real), self._real(gamma), C.c_int(bool(in_T_v)),
          _ptr(self._g_bar, self._real))

    # -- Algorithm 3 on an arbitrary buffer ------------------------------------
    def onebit_allreduce(self, z):
        """Runs Algorithm 3 on z [n][d] with this state's errors; returns z_bar."""
        z = self._g(z)
        f = _fn("zo_onebit_allreduce", self._suffix)
        f.restype = None
        f(C.byref(self._st), _ptr(z, self._real))
        return self.u_bar.copy()
