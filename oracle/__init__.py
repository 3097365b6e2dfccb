"""CPU oracle for HDT hierarchical attention.  TEST INFRASTRUCTURE ONLY.

Loads (building with gcc when needed) the plain fp64 C implementation in
``hdt_oracle.c`` and exposes numpy wrappers.  Nothing under this package is
imported by the CUDA path; only tests, the smoke check and the benchmark's
CPU-baseline legs use it.  See the header of ``hdt_oracle.c`` for what each
function computes and which passage of the paper it follows.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "hdt_oracle.c")
_LIB = os.path.join(_HERE, "libhdt_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile hdt_oracle.c with gcc (OpenMP) into libhdt_oracle.so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        for name in ("hdt_oracle_mask", "hdt_oracle_fwd", "hdt_oracle_bwd", "hdt_oracle_rows",
                     "hdt_oracle_cols", "hdt_oracle_probs", "hdt_oracle_threads"):
            getattr(_lib, name).restype = ctypes.c_int
    return _lib


def threads() -> int:
    return int(lib().hdt_oracle_threads())


def _p(a):
    return ctypes.c_void_p(a.ctypes.data) if a is not None else ctypes.c_void_p(0)


def _struct(level, parent, cu):
    level = np.ascontiguousarray(level, np.int8)
    parent = np.ascontiguousarray(parent, np.int32)
    cu = np.ascontiguousarray(cu, np.int32)
    return level, parent, cu


def _inputs(*xs):
    """All inputs as one dtype: fp32 if every array is fp32, else fp64."""
    f32 = all(x is None or x.dtype == np.float32 for x in xs)
    dt = np.float32 if f32 else np.float64
    return [None if x is None else np.ascontiguousarray(x, dt) for x in xs], int(f32)


class _Directions:
    """Sets the oracle's direction bits (1 = child attends parent, 2 = siblings attend each other,
    4 = parent attends children; the diagonal always stays) for the calls inside the block."""

    def __init__(self, bits):
        self.bits = 7 if bits is None else int(bits)

    def __enter__(self):
        lib().hdt_oracle_set_directions(ctypes.c_int(self.bits))

    def __exit__(self, *a):
        lib().hdt_oracle_set_directions(ctypes.c_int(7))


def default_scale(d: int) -> float:
    return 1.0 / float(np.sqrt(d))


def mask(level, parent, cu, b: int, directions=None) -> np.ndarray:
    """Dense 0/1 mask (uint8 [n, n]) of sequence b from the parent/sibling/child rule."""
    level, parent, cu = _struct(level, parent, cu)
    n = int(cu[b + 1] - cu[b])
    out = np.zeros((n, n), np.uint8)
    with _Directions(directions):
        lib().hdt_oracle_mask(_p(level), _p(parent), _p(cu), ctypes.c_int(b), _p(out))
    return out


def forward(level, parent, cu, q, k, v, scale=None, directions=None):
    """O fp64 [T,H,d] and LSE fp64 [H,T] of masked softmax attention."""
    level, parent, cu = _struct(level, parent, cu)
    (q, k, v), f32 = _inputs(q, k, v)
    T, H, d = q.shape
    scale = default_scale(d) if scale is None else scale
    o = np.zeros((T, H, d), np.float64)
    lse = np.full((H, T), -np.inf, np.float64)
    with _Directions(directions):
        rc = lib().hdt_oracle_fwd(_p(level), _p(parent), _p(cu), ctypes.c_int(len(cu) - 1),
                                  ctypes.c_int(H), ctypes.c_int(d), _p(q), _p(k), _p(v),
                                  ctypes.c_int(f32), ctypes.c_double(scale), _p(o), _p(lse))
    assert rc == 0
    return o, lse


def backward(level, parent, cu, q, k, v, do, scale=None, directions=None):
    """dQ, dK, dV fp64 [T,H,d]."""
    level, parent, cu = _struct(level, parent, cu)
    (q, k, v, do), f32 = _inputs(q, k, v, do)
    T, H, d = q.shape
    scale = default_scale(d) if scale is None else scale
    dq = np.zeros((T, H, d), np.float64)
    dk = np.zeros((T, H, d), np.float64)
    dv = np.zeros((T, H, d), np.float64)
    with _Directions(directions):
        rc = lib().hdt_oracle_bwd(_p(level), _p(parent), _p(cu), ctypes.c_int(len(cu) - 1),
                                  ctypes.c_int(H), ctypes.c_int(d), _p(q), _p(k), _p(v), _p(do),
                                  ctypes.c_int(f32), ctypes.c_double(scale), _p(dq), _p(dk), _p(dv))
    assert rc == 0
    return dq, dk, dv


def rows(level, parent, cu, q, k, v, rows, do=None, scale=None, directions=None):
    """Sampled rows (global token ids): O [r,H,d], LSE [r,H] and, with do, dQ [r,H,d]."""
    level, parent, cu = _struct(level, parent, cu)
    (q, k, v, do), f32 = _inputs(q, k, v, do)
    T, H, d = q.shape
    scale = default_scale(d) if scale is None else scale
    rows = np.ascontiguousarray(rows, np.int32)
    o = np.zeros((len(rows), H, d), np.float64)
    lse = np.zeros((len(rows), H), np.float64)
    dq = np.zeros((len(rows), H, d), np.float64) if do is not None else None
    with _Directions(directions):
        rc = lib().hdt_oracle_rows(_p(level), _p(parent), _p(cu), ctypes.c_int(len(cu) - 1),
                                   ctypes.c_int(H), ctypes.c_int(d), _p(q), _p(k), _p(v), _p(do),
                                   ctypes.c_int(f32), ctypes.c_double(scale), _p(rows),
                                   ctypes.c_int(len(rows)), _p(o), _p(lse), _p(dq))
    assert rc == 0
    return o, lse, dq


def cols(level, parent, cu, q, k, v, do, cols, scale=None, directions=None):
    """Sampled keys (global token ids): dK, dV [c,H,d]."""
    level, parent, cu = _struct(level, parent, cu)
    (q, k, v, do), f32 = _inputs(q, k, v, do)
    T, H, d = q.shape
    scale = default_scale(d) if scale is None else scale
    cols = np.ascontiguousarray(cols, np.int32)
    dk = np.zeros((len(cols), H, d), np.float64)
    dv = np.zeros((len(cols), H, d), np.float64)
    with _Directions(directions):
        rc = lib().hdt_oracle_cols(_p(level), _p(parent), _p(cu), ctypes.c_int(len(cu) - 1),
                                   ctypes.c_int(H), ctypes.c_int(d), _p(q), _p(k), _p(v), _p(do),
                                   ctypes.c_int(f32), ctypes.c_double(scale), _p(cols),
                                   ctypes.c_int(len(cols)), _p(dk), _p(dv))
    assert rc == 0
    return dk, dv


def probs(level, parent, cu, q, k, b: int, h: int, scale=None, directions=None) -> np.ndarray:
    """Dense softmax matrix S fp64 [n, n] of sequence b, head h."""
    level, parent, cu = _struct(level, parent, cu)
    (q, k), f32 = _inputs(q, k)
    T, H, d = q.shape
    scale = default_scale(d) if scale is None else scale
    n = int(cu[b + 1] - cu[b])
    S = np.zeros((n, n), np.float64)
    with _Directions(directions):
        rc = lib().hdt_oracle_probs(_p(level), _p(parent), _p(cu), ctypes.c_int(b), ctypes.c_int(H),
                                    ctypes.c_int(d), _p(q), _p(k), ctypes.c_int(f32),
                                    ctypes.c_double(scale), ctypes.c_int(h), _p(S))
    assert rc == 0
    return S
