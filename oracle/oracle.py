"""ORACLE -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.

ctypes front end of ``oracle.c``: the plain double-precision CPU statement of the
exact filter gradient and of the paper's approximation methods (Section 2.1 zero,
2.2 random, 2.3 / Algorithm 1 max-gradient).  Only ``tests/``, the smoke check and
the benchmark's CPU-baseline leg may import this module; the CUDA library and its
Python binding never do.

All arrays are numpy float64 in logical order: x [N,C,H,W], dy [N,K,P,Q],
dw [K,C,R,S].  Inputs of lower precision are widened exactly by the caller, so the
oracle sees the very values the GPU reads.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")


def build(force: bool = False) -> str:
    """Compile oracle.c with gcc (portable x86-64 code, OpenMP over output channels)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class _Shape(ctypes.Structure):
    _fields_ = [(f, ctypes.c_int) for f in
                ("n", "c", "h", "w", "k", "r", "s", "stride_h", "stride_w", "pad_h", "pad_w", "p", "q")]


@dataclass(frozen=True)
class Shape:
    """Convolution geometry as the oracle sees it (its own copy; not shared with the product)."""
    n: int
    c: int
    h: int
    w: int
    k: int
    r: int
    s: int
    stride_h: int = 1
    stride_w: int = 1
    pad_h: int = 0
    pad_w: int = 0

    @property
    def p(self) -> int:
        return (self.h + 2 * self.pad_h - self.r) // self.stride_h + 1

    @property
    def q(self) -> int:
        return (self.w + 2 * self.pad_w - self.s) // self.stride_w + 1

    def c_struct(self) -> _Shape:
        return _Shape(self.n, self.c, self.h, self.w, self.k, self.r, self.s,
                      self.stride_h, self.stride_w, self.pad_h, self.pad_w, self.p, self.q)


_lib = None
_dp = ctypes.POINTER(ctypes.c_double)
_ip = ctypes.POINTER(ctypes.c_int32)
_up = ctypes.POINTER(ctypes.c_uint32)


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_dw_exact.restype = ctypes.c_int
        _lib.oracle_dw_top1.restype = ctypes.c_int
        _lib.oracle_dw_sparse.restype = ctypes.c_int
        _lib.oracle_dw_topk.restype = ctypes.c_int
    return _lib


def _d(a):
    return None if a is None else a.ctypes.data_as(_dp)


def _f64(a, shape):
    a = np.ascontiguousarray(a, dtype=np.float64)
    assert a.shape == tuple(shape), (a.shape, shape)
    return a


def dw_exact(x, dy, g: Shape, alpha: float = 1.0):
    """Exact filter gradient and its normaliser sum|products|: returns (dw, dnorm), each [K,C,R,S]."""
    x = _f64(x, (g.n, g.c, g.h, g.w)); dy = _f64(dy, (g.n, g.k, g.p, g.q))
    dw = np.empty((g.k, g.c, g.r, g.s)); dn = np.empty_like(dw)
    rc = lib().oracle_dw_exact(_d(x), _d(dy), _d(dw), _d(dn), ctypes.byref(g.c_struct()), ctypes.c_double(alpha))
    if rc:
        raise ValueError("oracle_dw_exact rejected the shape")
    return dw, dn


def dw_exact_at(x, dy, g: Shape, k: int, c: int, r: int, s: int, alpha: float = 1.0):
    """One element of the exact filter gradient: returns (value, normaliser)."""
    x = _f64(x, (g.n, g.c, g.h, g.w)); dy = _f64(dy, (g.n, g.k, g.p, g.q))
    v = ctypes.c_double(); nrm = ctypes.c_double()
    lib().oracle_dw_exact_at(_d(x), _d(dy), ctypes.byref(g.c_struct()), ctypes.c_double(alpha),
                             k, c, r, s, ctypes.byref(v), ctypes.byref(nrm))
    return v.value, nrm.value


def top1_select(dy):
    """Selection step of Algorithm 1: returns (idx int32 [N,K], sum [N,K], abssum [N,K])."""
    dy = np.ascontiguousarray(dy, dtype=np.float64)
    n, k, p, q = dy.shape
    idx = np.empty((n, k), dtype=np.int32); s = np.empty((n, k)); a = np.empty((n, k))
    lib().oracle_top1_select(_d(dy), n, k, p * q, idx.ctypes.data_as(_ip), _d(s), _d(a))
    return idx, s, a


def dw_top1(x, dy, g: Shape, alpha: float = 1.0):
    """Algorithm 1 (max gradient approximation): returns (dw, dnorm)."""
    x = _f64(x, (g.n, g.c, g.h, g.w)); dy = _f64(dy, (g.n, g.k, g.p, g.q))
    dw = np.empty((g.k, g.c, g.r, g.s)); dn = np.empty_like(dw)
    rc = lib().oracle_dw_top1(_d(x), _d(dy), _d(dw), _d(dn), ctypes.byref(g.c_struct()), ctypes.c_double(alpha))
    if rc:
        raise ValueError("oracle_dw_top1 rejected the shape")
    return dw, dn


def topk_select(dy, topk: int):
    """Selection of the top-k variant: returns (idx int32 [N,K,topk] in order of selection, sum [N,K], abssum [N,K])."""
    dy = np.ascontiguousarray(dy, dtype=np.float64)
    n, k, p, q = dy.shape
    t = min(topk, p * q)
    idx = np.empty((n, k, t), dtype=np.int32); s = np.empty((n, k)); a = np.empty((n, k))
    lib().oracle_topk_select(_d(dy), n, k, p * q, t, idx.ctypes.data_as(_ip), _d(s), _d(a))
    return idx, s, a


def dw_topk(x, dy, g: Shape, topk: int, alpha: float = 1.0):
    """Top-k variant of Algorithm 1 (each retained entry gets sum/topk): returns (dw, dnorm)."""
    x = _f64(x, (g.n, g.c, g.h, g.w)); dy = _f64(dy, (g.n, g.k, g.p, g.q))
    dw = np.empty((g.k, g.c, g.r, g.s)); dn = np.empty_like(dw)
    rc = lib().oracle_dw_topk(_d(x), _d(dy), _d(dw), _d(dn), ctypes.byref(g.c_struct()), ctypes.c_double(alpha), int(topk))
    if rc:
        raise ValueError("oracle_dw_topk rejected its arguments (code %d)" % rc)
    return dw, dn


def dw_sparse(x, entries, g: Shape, alpha: float = 1.0):
    """Filter gradient of a list of retained entries [(n, k, p, q, value), ...]."""
    x = _f64(x, (g.n, g.c, g.h, g.w))
    cols = [np.ascontiguousarray([e[i] for e in entries], dtype=np.int32) for i in range(4)]
    val = np.ascontiguousarray([e[4] for e in entries], dtype=np.float64)
    dw = np.empty((g.k, g.c, g.r, g.s))
    rc = lib().oracle_dw_sparse(_d(x), *[c_.ctypes.data_as(_ip) for c_ in cols], _d(val),
                                ctypes.c_size_t(len(entries)), _d(dw), ctypes.byref(g.c_struct()),
                                ctypes.c_double(alpha))
    if rc:
        raise ValueError("oracle_dw_sparse rejected its arguments (code %d)" % rc)
    return dw


def sparsify(idx, s, pq: int):
    """Dense sparse-version of dy: the channel sum at the selected position, zero elsewhere. [N,K,PQ]."""
    idx = np.ascontiguousarray(idx, dtype=np.int32); s = np.ascontiguousarray(s, dtype=np.float64)
    n, k = idx.shape
    out = np.empty((n, k, pq))
    lib().oracle_sparsify(idx.ctypes.data_as(_ip), _d(s), n, k, pq, _d(out))
    return out


def dw_zero(count: int):
    out = np.full(count, np.nan)
    lib().oracle_dw_zero(_d(out), ctypes.c_size_t(count))
    return out


def philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*ctr); k = (ctypes.c_uint32 * 2)(*key); o = (ctypes.c_uint32 * 4)()
    lib().oracle_philox4x32_10(c, k, o)
    return [int(v) for v in o]


def random_words(seed: int, count: int):
    out = np.empty(count, dtype=np.uint32)
    lib().oracle_random_words(ctypes.c_uint64(seed), ctypes.c_size_t(count), out.ctypes.data_as(_up))
    return out


def dw_random(count: int, seed: int, std: float):
    """Random gradient (Section 2.2): count values std * z_i in logical [K,C,R,S] order."""
    out = np.empty(count)
    lib().oracle_dw_random(_d(out), ctypes.c_size_t(count), ctypes.c_uint64(seed), ctypes.c_double(std))
    return out


def num_threads() -> int:
    return int(lib().oracle_num_threads())
