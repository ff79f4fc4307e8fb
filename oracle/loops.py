"""ctypes loader for the scalar-loop C twin (oracle/mdbf_loops.c).

TEST INFRASTRUCTURE ONLY (see mdbf_oracle.py).  `build()` compiles the C file
with gcc next to this module; nothing here touches the CUDA library.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mdbf_loops.c")
_LIB = os.path.join(_HERE, "libmdbf_loops.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", "-O2", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _prep(S_A, S_B, U_A, V_A, U_B, V_B):
    S_A = np.ascontiguousarray(S_A, dtype=np.int8)
    S_B = np.ascontiguousarray(S_B, dtype=np.int8)
    fs = [np.ascontiguousarray(a, dtype=np.float64) for a in (U_A, V_A, U_B, V_B)]
    d_out, k = S_A.shape
    k2, d_in = S_B.shape
    l = fs[0].shape[1]
    assert k == k2 and fs[0].shape == (d_out, l) and fs[1].shape == (k, l)
    assert fs[2].shape == (k, l) and fs[3].shape == (d_in, l)
    return S_A, S_B, fs, d_out, d_in, k, l


def reconstruct(S_A, S_B, U_A, V_A, U_B, V_B):
    S_A, S_B, fs, d_out, d_in, k, l = _prep(S_A, S_B, U_A, V_A, U_B, V_B)
    W = np.empty((d_out, d_in), dtype=np.float64)
    rc = _load().mdbf_loops_reconstruct(
        _p(S_A, ctypes.c_int8), _p(S_B, ctypes.c_int8),
        *[_p(f, ctypes.c_double) for f in fs],
        d_out, d_in, k, l, _p(W, ctypes.c_double))
    if rc:
        raise ValueError("sign matrix entries must be +1 or -1")
    return W


def forward(S_A, S_B, U_A, V_A, U_B, V_B, X):
    S_A, S_B, fs, d_out, d_in, k, l = _prep(S_A, S_B, U_A, V_A, U_B, V_B)
    X = np.ascontiguousarray(X, dtype=np.float64)
    assert X.ndim == 2 and X.shape[0] == d_in
    T = X.shape[1]
    W = np.empty((d_out, d_in), dtype=np.float64)
    Y = np.empty((d_out, T), dtype=np.float64)
    rc = _load().mdbf_loops_forward(
        _p(S_A, ctypes.c_int8), _p(S_B, ctypes.c_int8),
        *[_p(f, ctypes.c_double) for f in fs],
        d_out, d_in, k, l, _p(X, ctypes.c_double), T,
        _p(W, ctypes.c_double), _p(Y, ctypes.c_double))
    if rc:
        raise ValueError("sign matrix entries must be +1 or -1")
    return Y


def pack_signs(S):
    S = np.ascontiguousarray(S, dtype=np.int8)
    rows, cols = S.shape
    out = np.empty((rows, (cols + 31) // 32), dtype=np.uint32)
    lib = _load()
    lib.mdbf_loops_pack.argtypes = [ctypes.POINTER(ctypes.c_int8), ctypes.c_int64,
                                    ctypes.c_int64, ctypes.POINTER(ctypes.c_uint32)]
    rc = lib.mdbf_loops_pack(_p(S, ctypes.c_int8), rows, cols, _p(out, ctypes.c_uint32))
    if rc:
        raise ValueError("sign matrix entries must be +1 or -1")
    return out
