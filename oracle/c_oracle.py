"""Loader for the plain-C float64 oracle (oracle/xconv_oracle.c): test infrastructure, not product code.

Builds the C file with gcc (-O2 -fopenmp) into oracle/libxconv_oracle.so and wraps its loop nests for numpy arrays
in the logical (batch, channel, y, x) layout.  Same function names and argument order as the numpy oracle
(oracle/xconv_oracle.py), of which this is an independent second statement: the two are compared with each other and
pinned by the same brute-force and closed-form tests.  Only tests, the smoke check and the benchmark's CPU-baseline
leg may import this module.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "xconv_oracle.c")
_SO = os.path.join(_HERE, "libxconv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """gcc -O2 -fopenmp -shared; rebuilt when the source is newer than the library."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", _SRC, "-o", _SO], check=True)
    return _SO


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _d(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _p(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def conv_forward(X, W):
    X, W = _d(X), _d(W)
    B, Cin, H, Wd = X.shape
    Cout, _, KH, KW = W.shape
    Y = np.empty((B, Cout, H, Wd))
    lib().xo_conv_forward(_p(X), _p(W), _p(Y), B, Cin, Cout, H, Wd, KH, KW)
    return Y


def dx_exact(dY, W):
    dY, W = _d(dY), _d(W)
    B, Cout, H, Wd = dY.shape
    _, Cin, KH, KW = W.shape
    dX = np.empty((B, Cin, H, Wd))
    lib().xo_dx_exact(_p(dY), _p(W), _p(dX), B, Cin, Cout, H, Wd, KH, KW)
    return dX


def dw_exact(X, dY, KH=3, KW=3):
    X, dY = _d(X), _d(dY)
    B, Cin, H, Wd = X.shape
    Cout = dY.shape[1]
    dW = np.empty((Cout, Cin, KH, KW))
    lib().xo_dw_exact(_p(X), _p(dY), _p(dW), B, Cin, Cout, H, Wd, KH, KW)
    return dW


def sketch(X, Z):
    X, Z = _d(X), _d(Z)
    B, r = X.shape[0], Z.shape[0]
    S = np.empty((r, B))
    lib().xo_sketch(_p(X), _p(Z), _p(S), B, r, ctypes.c_size_t(X[0].size))
    return S


def backprobe(S, dY):
    S, dY = _d(S), _d(dY)
    r, B = S.shape
    L = np.empty((r,) + dY.shape[1:])
    lib().xo_backprobe(_p(S), _p(dY), _p(L), r, B, ctypes.c_size_t(dY[0].size))
    return L


def wgrad_contract(L, Z, KH=3, KW=3, scale=None):
    L, Z = _d(L), _d(Z)
    r, Cout, H, Wd = L.shape
    Cin = Z.shape[1]
    sc = _d(np.full(Cin, 1.0 / r) if scale is None else scale)
    dW = np.empty((Cout, Cin, KH, KW))
    lib().xo_wgrad_contract(_p(L), _p(Z), _p(sc), _p(dW), r, Cin, Cout, H, Wd, KH, KW)
    return dW


def wgrad_estimate(S, dY, Z, KH=3, KW=3, scale=None):
    """Algorithm 1 backward steps 3-4."""
    return wgrad_contract(backprobe(S, dY), Z, KH, KW, scale)


def threads() -> int:
    """OpenMP threads the loop nests run on."""
    try:
        return len(os.sched_getaffinity(0)) if "OMP_NUM_THREADS" not in os.environ else int(os.environ["OMP_NUM_THREADS"])
    except Exception:
        return os.cpu_count() or 1
