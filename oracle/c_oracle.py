"""ctypes access to the plain C oracle (oracle/lightkv_oracle.c), built by __graft_entry__.build().

TEST INFRASTRUCTURE ONLY, like the rest of oracle/: the tests compare this second, separately written oracle
with the numpy one, and bench.py may time it as the single-threaded CPU baseline.  Argument marshalling only."""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lightkv_oracle.c")
_LIB_PATH = os.path.join(_HERE, "liboracle_c.so")
_LIB = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB_PATH) or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC):
        subprocess.run(["gcc", "-O2", "-std=c99", "-shared", "-fPIC", "-o", _LIB_PATH, _SRC, "-lm"], check=True)
    return _LIB_PATH


def _lib():
    global _LIB
    if _LIB is None:
        _LIB = C.CDLL(build())
    return _LIB


def _d(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def _i(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _p(a, t):
    return a.ctypes.data_as(C.POINTER(t))


def xi(q, k, vis_begin, n_vis, ranges, causal=True):
    """q [H, N, dh], k [H_kv, N, dh] -> xi [n_vis]."""
    q, k = _d(q), _d(k)
    r = _i(np.asarray(ranges).reshape(-1, 2))
    out = np.zeros(n_vis)
    _lib().oracle_c_xi(_p(q, C.c_double), _p(k, C.c_double), C.c_int(q.shape[0]), C.c_int(k.shape[0]), C.c_int(q.shape[1]),
                       C.c_int(q.shape[2]), C.c_int(vis_begin), C.c_int(n_vis), _p(r, C.c_int), C.c_int(len(r)),
                       C.c_int(int(causal)), _p(out, C.c_double))
    return out


def compress(x, pos, xi_, tiles, w, keep):
    """One stage on one sample's vision tokens -> dict like the numpy oracle's compress_vision."""
    x, pos, xi_ = _d(x), _i(pos), _d(xi_)
    n, d = x.shape
    t = _i(np.asarray(tiles).reshape(-1, 2))
    x_out, pos_out = np.zeros((n, d)), np.zeros(n, dtype=np.int32)
    dst, weight, n_out = np.zeros(n, dtype=np.int32), np.zeros(n), C.c_int(0)
    _lib().oracle_c_compress(_p(x, C.c_double), _p(pos, C.c_int), _p(xi_, C.c_double), C.c_int(n), C.c_int(d), _p(t, C.c_int),
                             C.c_int(len(t)), C.c_int(w), C.c_double(keep), _p(x_out, C.c_double), _p(pos_out, C.c_int),
                             _p(dst, C.c_int), _p(weight, C.c_double), C.byref(n_out))
    m = n_out.value
    return {"x_out": x_out[:m], "pos_out": pos_out[:m].astype(np.int64), "dst": dst.astype(np.int64), "weight": weight,
            "n_out": m}


def compact(kv, dst, weight, n_out):
    """kv [H, n, dh] -> [H, n_out, dh]."""
    kv, dst, weight = _d(kv), _i(dst), _d(weight)
    out = np.zeros((kv.shape[0], n_out, kv.shape[2]))
    _lib().oracle_c_compact(_p(kv, C.c_double), C.c_int(kv.shape[0]), C.c_int(kv.shape[1]), C.c_int(kv.shape[2]), _p(dst, C.c_int),
                            _p(weight, C.c_double), C.c_int(n_out), _p(out, C.c_double))
    return out
