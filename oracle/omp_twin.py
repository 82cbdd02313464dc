"""ctypes front of oracle/kvswap_oracle_omp.cpp -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

`build()` compiles the C++/OpenMP twin of the oracle with g++ (in-tree, next to this file);
`score_select` and `attend` have the signatures of the numpy oracle's functions of the same name.
The numpy oracle stays the parity authority; this twin exists so that the benchmark's CPU
baseline times the method on all host cores rather than the Python interpreter."""
from __future__ import annotations

import ctypes
import os
import shutil
import subprocess

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
SRC = os.path.join(_DIR, "kvswap_oracle_omp.cpp")
LIB = os.path.join(_DIR, "libkvswap_oracle_omp.so")
_lib = None


def build(force: bool = False) -> str:
    if not force and os.path.exists(LIB) and os.path.getmtime(LIB) >= os.path.getmtime(SRC):
        return LIB
    gxx = shutil.which("g++")
    if gxx is None:
        raise RuntimeError("g++ not found: the OpenMP twin of the oracle cannot be built")
    res = subprocess.run([gxx, "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c++17", SRC, "-o", LIB],
                         capture_output=True, text=True)
    if res.returncode != 0:
        raise RuntimeError(f"g++ failed on {SRC}:\n{res.stderr}")
    return LIB


def load() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        F, I32, D = ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_double)
        i = ctypes.c_int
        lib.kvo_threads.restype = i
        lib.kvo_score_select.restype = i
        lib.kvo_score_select.argtypes = [F, F, F, i, i, i, i, i, i, i, i, i, i, I32, D]
        lib.kvo_attend.restype = i
        lib.kvo_attend.argtypes = [F, F, F, I32, i, i, i, i, i, i, i, i, D, D]
        _lib = lib
    return _lib


def threads() -> int:
    return int(load().kvo_threads())


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


_SCOPE = {"kv_head": 0, "all_heads": 1}


def score_select(q, proj, meta, G, M, scope="kv_head"):
    """(idx [B,S,M'], R [B,S,NG]) as oracle.kvswap_oracle.score_select (raw-logit reading)."""
    q, qp = _f32(q)
    proj, pp = _f32(proj)
    meta, mp = _f32(meta)
    B, Hq, d = q.shape
    Hkv, _, r = proj.shape
    Hm, N = meta.shape[1], meta.shape[2]
    S = Hkv if scope == "kv_head" else 1
    NG = N // G
    Mp = min(M, NG)
    idx = np.empty((B, S, Mp), dtype=np.int32)
    R = np.empty((B, S, NG), dtype=np.float64)
    rc = load().kvo_score_select(qp, pp, mp, B, Hq, Hkv, d, r, Hm, N, G, M, _SCOPE[scope],
                                 idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                 R.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    if rc != 0:
        raise ValueError("kvo_score_select: invalid shape")
    return idx, R


def attend(q, K, V, idx, G, scope="kv_head"):
    """(out [B,H_q,d], lse [B,H_q]) as oracle.kvswap_oracle.attend."""
    q, qp = _f32(q)
    K, Kp = _f32(K)
    V, Vp = _f32(V)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    B, Hq, d = q.shape
    Hkv, N = K.shape[1], K.shape[2]
    out = np.empty((B, Hq, d), dtype=np.float64)
    lse = np.empty((B, Hq), dtype=np.float64)
    rc = load().kvo_attend(qp, Kp, Vp, idx.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), idx.shape[2], B, Hq, Hkv, d,
                           N, G, _SCOPE[scope], out.ctypes.data_as(ctypes.POINTER(ctypes.c_double)),
                           lse.ctypes.data_as(ctypes.POINTER(ctypes.c_double)))
    if rc != 0:
        raise ValueError("kvo_attend: invalid shape")
    return out, lse
