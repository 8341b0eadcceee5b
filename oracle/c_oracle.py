"""Loader for the C twin of the CPU oracle (oracle/abs_oracle.c).

TEST INFRASTRUCTURE ONLY: used by tests (cross-check against the NumPy oracle) and by the
benchmark's CPU-baseline leg.  Never imported by the CUDA path.
"""

from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "abs_oracle.c")
_LIB = os.path.join(_HERE, "libabs_oracle.so")


def build(force: bool = False) -> str:
    """Compile oracle/abs_oracle.c with gcc (OpenMP) into oracle/libabs_oracle.so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, f32p, i32p = ctypes.c_void_p, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32)
        lib.abs_oracle_create.restype = vp
        lib.abs_oracle_create.argtypes = [ctypes.c_size_t, ctypes.c_int, f32p, ctypes.c_double,
                                          ctypes.c_double, ctypes.c_double, ctypes.c_double]
        lib.abs_oracle_destroy.argtypes = [vp]
        lib.abs_oracle_accumulate.restype = ctypes.c_int
        lib.abs_oracle_accumulate.argtypes = [vp, ctypes.c_int, vp, ctypes.c_int]
        lib.abs_oracle_sync_step.restype = ctypes.c_int64
        lib.abs_oracle_sync_step.argtypes = [vp, i32p]
        lib.abs_oracle_params.argtypes = [vp, f32p]
        lib.abs_oracle_momentum.argtypes = [vp, ctypes.POINTER(ctypes.c_double)]
        lib.abs_oracle_state.argtypes = [vp, i32p, i32p, ctypes.POINTER(ctypes.c_int64)]
        lib.abs_oracle_set_lr.argtypes = [vp, ctypes.c_double]
        _lib = lib
    return _lib


class AbsSgdOracleC:
    """Same interface as oracle.abs_oracle.AbsSgdOracle, backed by the C implementation."""

    def __init__(self, x0, W, lr, momentum=0.0, weight_decay=0.0, lambda_dc=0.0):
        lib = _load()
        x0 = np.ascontiguousarray(x0, dtype=np.float32)
        self.P, self.W = x0.shape[0], int(W)
        self._h = lib.abs_oracle_create(self.P, self.W, x0.ctypes.data_as(ctypes.POINTER(ctypes.c_float)),
                                        lr, momentum, weight_decay, lambda_dc)
        if not self._h:
            raise MemoryError("abs_oracle_create failed")
        self.consumed = []

    def accumulate(self, i, g):
        g = np.ascontiguousarray(g)
        assert g.shape == (self.P,)
        if g.dtype == np.uint16:
            dt = 1
        else:
            g = g.astype(np.float32, copy=False)
            dt = 0
        rc = _load().abs_oracle_accumulate(self._h, int(i), g.ctypes.data, dt)
        assert rc == 0

    def sync_step(self):
        b = np.zeros(self.W, dtype=np.int32)
        B = _load().abs_oracle_sync_step(self._h, b.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)))
        self.consumed.append(b)
        return int(B)

    def params(self):
        out = np.empty(self.P, dtype=np.float32)
        _load().abs_oracle_params(self._h, out.ctypes.data_as(ctypes.POINTER(ctypes.c_float)))
        return out

    @property
    def v(self):
        out = np.empty(self.P, dtype=np.float64)
        _load().abs_oracle_momentum(self._h, out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
        return out

    def counters(self):
        cnt = np.zeros((2, self.W), dtype=np.int32)
        cur = ctypes.c_int32(0)
        t = ctypes.c_int64(0)
        _load().abs_oracle_state(self._h, cnt.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                 ctypes.byref(cur), ctypes.byref(t))
        return cnt, int(cur.value), int(t.value)

    @property
    def cur(self):
        return self.counters()[1]

    @property
    def t(self):
        return self.counters()[2]

    def set_lr(self, lr):
        _load().abs_oracle_set_lr(self._h, float(lr))

    def close(self):
        if self._h:
            _load().abs_oracle_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
