"""ctypes front end of the CPU oracle (oracle/dmx_oracle.cpp).

TEST INFRASTRUCTURE: imported only by the tests, the smoke check and the CPU-baseline leg of
the benchmark. It imports nothing from the CUDA package and the CUDA package never imports it.
The shared object is compiled next to the source on first use (g++ -O2, no fast-math, so the
compensated sums keep their meaning).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dmx_oracle.cpp")
_LIB = os.path.join(_HERE, "libdmx_oracle.so")
_lock = threading.Lock()
_lib = None

F32, BF16 = 0, 1
BLOCK = 1 << 20

# out_state indices (typed again here; see the layout in the oracle source)
ST = dict(B=0, A=1, TRS=2, G2=3, GNS=4, COS=5, DOT=6, PP=7, SIG2=8, SIG=9, WQ=10, FLAGS=11, HDR=16)


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or older than the source."""
    with _lock:
        stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
        if force or stale:
            tmp = _LIB + ".tmp.%d" % os.getpid()
            subprocess.check_call(
                ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-pthread", _SRC, "-o", tmp])
            os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_float
        L.dmxo_create.argtypes = [i32, i64, vp, i32, i32, ctypes.POINTER(vp)]
        L.dmxo_state_len.argtypes = [vp]
        L.dmxo_begin.argtypes = [vp, vp, f32, f32]
        L.dmxo_range.argtypes = [vp, i64, i64, vp, vp, vp, vp, i32]
        L.dmxo_end.argtypes = [vp, vp]
        L.dmxo_step.argtypes = [vp, vp, vp, vp, vp, f32, f32, vp, vp, i32]
        L.dmxo_destroy.argtypes = [vp]
        L.dmxo_begin_adam.argtypes = [vp, vp, f32, f32, f32, f32, i64]
        L.dmxo_range_adam.argtypes = [vp, i64, i64, vp, vp, vp, vp, vp, i32]
        L.dmxo_step_adam.argtypes = [vp, vp, vp, vp, vp, vp, f32, f32, f32, f32, i64, vp, vp, i32]
        L.dmxo_window_stats.argtypes = [vp, i32, i32, vp]
        L.dmxo_window_stats.restype = i32
        for f in (L.dmxo_create, L.dmxo_state_len, L.dmxo_begin, L.dmxo_range, L.dmxo_end,
                  L.dmxo_step, L.dmxo_destroy, L.dmxo_begin_adam, L.dmxo_range_adam, L.dmxo_step_adam):
            f.restype = i32
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code):
        super().__init__("oracle returned %d" % code)
        self.code = code


def _ptr(a: np.ndarray) -> int:
    return a.ctypes.data


def window_stats(states: np.ndarray) -> np.ndarray:
    """Mean and population std per entry over the rows of `states` (k x n float32); 2n floats."""
    st = np.ascontiguousarray(states, dtype=np.float32)
    k, n = st.shape
    out = np.empty(2 * n, dtype=np.float32)
    rc = lib().dmxo_window_stats(_ptr(st), k, n, _ptr(out))
    if rc != 0:
        raise OracleError(rc)
    return out


class Oracle:
    """One (K, P, segment table, dtype) problem; `step` advances host arrays in place.

    Gradients are numpy arrays: float32 for F32, uint16 (raw bf16 bit patterns) for BF16.
    """

    def __init__(self, K, P, seg_offsets, dtype=F32):
        self.K, self.P, self.dtype = int(K), int(P), int(dtype)
        self.seg = np.ascontiguousarray(seg_offsets, dtype=np.int64)
        self.S = len(self.seg) - 1
        h = ctypes.c_void_p()
        rc = lib().dmxo_create(self.K, self.P, _ptr(self.seg), self.S, self.dtype, ctypes.byref(h))
        if rc != 0:
            raise OracleError(rc)
        self._h = h
        self.state_len = lib().dmxo_state_len(self._h)

    def close(self):
        if getattr(self, "_h", None):
            lib().dmxo_destroy(self._h)
            self._h = None

    __del__ = close

    def _check_grads(self, grads, n):
        want = np.float32 if self.dtype == F32 else np.uint16
        assert len(grads) == self.K
        for g in grads:
            assert g.dtype == want and g.flags.c_contiguous and g.shape == (n,), (g.dtype, g.shape)
        return (ctypes.c_void_p * self.K)(*[_ptr(g) for g in grads])

    @staticmethod
    def _check_state(n, *arrs):
        for a in arrs:
            assert a.dtype == np.float32 and a.flags.c_contiguous and a.shape == (n,)

    def step(self, grads, batch_sizes, params, momentum, lr, beta, prev_agg, nthreads=1):
        """Whole step on full-length host arrays; returns out_state (float32)."""
        gp = self._check_grads(grads, self.P)
        self._check_state(self.P, params, momentum, prev_agg)
        b = np.ascontiguousarray(batch_sizes, dtype=np.int32)
        assert b.shape == (self.K,)
        out = np.empty(self.state_len, dtype=np.float32)
        rc = lib().dmxo_step(self._h, gp, _ptr(b), _ptr(params), _ptr(momentum), lr, beta,
                             _ptr(prev_agg), _ptr(out), int(nthreads))
        if rc != 0:
            raise OracleError(rc)
        return out

    def step_adam(self, grads, batch_sizes, params, first, second, lr, beta1, beta2, eps, t, prev_agg, nthreads=1):
        """Whole Adam step (t = 1-based step count) on full-length host arrays; returns out_state."""
        gp = self._check_grads(grads, self.P)
        self._check_state(self.P, params, first, second, prev_agg)
        b = np.ascontiguousarray(batch_sizes, dtype=np.int32)
        assert b.shape == (self.K,)
        out = np.empty(self.state_len, dtype=np.float32)
        rc = lib().dmxo_step_adam(self._h, gp, _ptr(b), _ptr(params), _ptr(first), _ptr(second), lr, beta1, beta2, eps,
                                  int(t), _ptr(prev_agg), _ptr(out), int(nthreads))
        if rc != 0:
            raise OracleError(rc)
        return out

    def begin_adam(self, batch_sizes, lr, beta1, beta2, eps, t):
        b = np.ascontiguousarray(batch_sizes, dtype=np.int32)
        assert b.shape == (self.K,)
        rc = lib().dmxo_begin_adam(self._h, _ptr(b), lr, beta1, beta2, eps, int(t))
        if rc != 0:
            raise OracleError(rc)

    def range_adam(self, j0, grads, params, first, second, prev_agg, nthreads=1):
        n = len(params)
        gp = self._check_grads(grads, n)
        self._check_state(n, params, first, second, prev_agg)
        rc = lib().dmxo_range_adam(self._h, int(j0), n, gp, _ptr(params), _ptr(first), _ptr(second), _ptr(prev_agg),
                                   int(nthreads))
        if rc != 0:
            raise OracleError(rc)

    # streaming form, for problems whose gradients do not fit in host memory at once
    def begin(self, batch_sizes, lr, beta):
        b = np.ascontiguousarray(batch_sizes, dtype=np.int32)
        assert b.shape == (self.K,)
        rc = lib().dmxo_begin(self._h, _ptr(b), lr, beta)
        if rc != 0:
            raise OracleError(rc)

    def range(self, j0, grads, params, momentum, prev_agg, nthreads=1):
        """Elements [j0, j0+n): all arrays have length n and hold that range."""
        n = len(params)
        gp = self._check_grads(grads, n)
        self._check_state(n, params, momentum, prev_agg)
        rc = lib().dmxo_range(self._h, int(j0), n, gp, _ptr(params), _ptr(momentum),
                              _ptr(prev_agg), int(nthreads))
        if rc != 0:
            raise OracleError(rc)

    def end(self):
        out = np.empty(self.state_len, dtype=np.float32)
        rc = lib().dmxo_end(self._h, _ptr(out))
        if rc != 0:
            raise OracleError(rc)
        return out
