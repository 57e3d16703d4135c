"""CPU fp64 oracle for delta-rule linear-attention prefill.  TEST INFRASTRUCTURE ONLY.

Only tests, the smoke check and the bench's CPU-baseline leg may import this
package.  It shares no code with the CUDA library and imports nothing from it.

``recurrent`` wraps the plain C token-by-token recurrence (ha_la_oracle.c);
``chunked`` (chunked.py) is an independently written chunkwise fp64 evaluation
used to cross-check the recurrence on small inputs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ha_la_oracle.c")
_LIB = os.path.join(_HERE, "libha_la_oracle.so")
_lib = None


class _Args(ctypes.Structure):
    _fields_ = [
        ("variant", ctypes.c_int32),
        ("num_seqs", ctypes.c_int32),
        ("num_qk_heads", ctypes.c_int32),
        ("num_v_heads", ctypes.c_int32),
        ("d_k", ctypes.c_int32),
        ("d_v", ctypes.c_int32),
        ("scale", ctypes.c_double),
        ("cu_seqlens", ctypes.c_void_p),
        ("q", ctypes.c_void_p),
        ("k", ctypes.c_void_p),
        ("v", ctypes.c_void_p),
        ("g", ctypes.c_void_p),
        ("beta", ctypes.c_void_p),
        ("h0", ctypes.c_void_p),
        ("o", ctypes.c_void_p),
        ("hT", ctypes.c_void_p),
        ("pairs", ctypes.c_void_p),
        ("num_pairs", ctypes.c_int32),
    ]


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (OpenMP) next to its source; returns the .so path."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.ha_la_oracle.argtypes = [ctypes.POINTER(_Args), ctypes.c_int, ctypes.POINTER(ctypes.c_int)]
        lib.ha_la_oracle.restype = ctypes.c_int
        _lib = lib
    return _lib


def _f32(x, shape=None):
    a = np.ascontiguousarray(np.asarray(x), dtype=np.float32)
    if shape is not None:
        assert a.shape == tuple(shape), (a.shape, shape)
    return a


def recurrent(q, k, v, g, beta, *, variant="gdn", h0=None, cu_seqlens=None, scale=1.0,
              pairs=None, num_threads=0, want_hT=True):
    """Token-by-token fp64 recurrence (the definition of the result).

    q, k : [T, HK, d_k]   v : [T, HV, d_v]   beta : [T, HV]
    g    : [T, HV] for "gdn", [T, HV, d_k] for "kda"  (log-gate)
    h0   : [N, HV, d_k, d_v] or None;  cu_seqlens : int [N+1] or None (one sequence)
    pairs: optional list of (sequence, V-head) to compute; other entries of the
           outputs are left at zero.
    Returns (o [T, HV, d_v] float64, hT [N, HV, d_k, d_v] float64 or None, threads_used).
    """
    lib = _load()
    q = _f32(q); k = _f32(k); v = _f32(v); beta = _f32(beta); g = _f32(g)
    T, HK, dk = q.shape
    _, HV, dv = v.shape
    assert k.shape == (T, HK, dk) and v.shape[0] == T and beta.shape == (T, HV)
    var = {"gdn": 0, "kda": 1}[variant]
    assert g.shape == ((T, HV) if var == 0 else (T, HV, dk)), g.shape
    if cu_seqlens is None:
        cu = np.array([0, T], dtype=np.int64)
    else:
        cu = np.ascontiguousarray(np.asarray(cu_seqlens), dtype=np.int64)
        assert cu[0] == 0 and cu[-1] == T
    N = len(cu) - 1
    h0a = None if h0 is None else _f32(h0, (N, HV, dk, dv))
    o = np.zeros((T, HV, dv), dtype=np.float64)
    hT = np.zeros((N, HV, dk, dv), dtype=np.float64) if want_hT else None
    pa = None
    if pairs is not None:
        pa = np.ascontiguousarray(np.asarray(pairs, dtype=np.int32).reshape(-1, 2))

    def ptr(a):
        return None if a is None else a.ctypes.data

    args = _Args(var, N, HK, HV, dk, dv, float(scale), ptr(cu), ptr(q), ptr(k), ptr(v), ptr(g),
                 ptr(beta), ptr(h0a), ptr(o), ptr(hT), ptr(pa), 0 if pa is None else len(pa))
    used = ctypes.c_int(0)
    rc = lib.ha_la_oracle(ctypes.byref(args), int(num_threads), ctypes.byref(used))
    if rc != 0:
        raise RuntimeError(f"ha_la_oracle failed with code {rc}")
    return o, hT, used.value
