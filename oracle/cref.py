"""ctypes wrapper of the plain-C oracle (oracle/gptq2d_oracle.c).

TEST INFRASTRUCTURE ONLY.  ``build()`` compiles the C file with gcc into
liboracle_gptq2d.so beside it; the functions below marshal numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gptq2d_oracle.c")
_LIB = os.path.join(_HERE, "liboracle_gptq2d.so")
_lib = None


def build(force=False):
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        # -ffp-contract=off: every product and sum is rounded separately, as written
        subprocess.check_call(["gcc", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-o", _LIB, _SRC, "-lm"])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        dp = ctypes.POINTER(ctypes.c_double)
        ip = ctypes.POINTER(ctypes.c_int64)
        _lib.oracle_vec_sweep.argtypes = [ctypes.c_int, ctypes.c_int, dp, dp, dp, ip, dp, ctypes.c_int64, ctypes.c_int64]
        _lib.oracle_alg3.argtypes = [ctypes.c_int, ctypes.c_int, dp, dp, dp, dp, ip, dp, ctypes.c_int, ctypes.c_int]
        _lib.oracle_nested.argtypes = [ctypes.c_int, ctypes.c_int, dp, dp, dp, ip, dp]
        for f in (_lib.oracle_vec_sweep, _lib.oracle_alg3, _lib.oracle_nested):
            f.restype = None
    return _lib


def _d(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _i(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def _prep(X, L, U):
    X = np.ascontiguousarray(X, dtype=np.float64)
    L = np.ascontiguousarray(L, dtype=np.float64)
    U = np.ascontiguousarray(U, dtype=np.float64)
    m, n = X.shape
    assert L.shape == (m, m) and U.shape == (n, n)
    return X, L, U, m, n


def _result(Z, E, done=None):
    Ed = E if done is None else E[done]
    return {"Z": Z, "E": E, "margin": float(0.5 - np.max(np.abs(Ed))) if Ed.size else 0.5}


def vec_sweep(X, L, U, k_end=None):
    """Quartic Algorithm 1 over vec(X); the first k_end coordinates only if given."""
    X, L, U, m, n = _prep(X, L, U)
    Y = X.copy()
    Z = np.zeros((m, n), dtype=np.int64)
    E = np.zeros((m, n))
    k_end = m * n if k_end is None else int(k_end)
    _load().oracle_vec_sweep(m, n, _d(Y), _d(L), _d(U), _i(Z), _d(E), 0, k_end)
    return _result(Z, E)


def alg3(X, L, U, s_end=None):
    """Algorithm 3 literally; the first s_end anti-diagonals only if given."""
    X, L, U, m, n = _prep(X, L, U)
    Y = X.copy()
    C = np.zeros((m, n))
    Z = np.zeros((m, n), dtype=np.int64)
    E = np.zeros((m, n))
    s_end = m + n - 1 if s_end is None else int(s_end)
    _load().oracle_alg3(m, n, _d(Y), _d(C), _d(L), _d(U), _i(Z), _d(E), 0, s_end)
    out = _result(Z, E)
    out["C"] = C
    return out


def nested(X, L, U):
    """Algorithm 5."""
    X, L, U, m, n = _prep(X, L, U)
    Y = X.copy()
    Z = np.zeros((m, n), dtype=np.int64)
    E = np.zeros((m, n))
    _load().oracle_nested(m, n, _d(Y), _d(L), _d(U), _i(Z), _d(E))
    return _result(Z, E)
