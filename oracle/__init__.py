"""CPU oracle (fp64, dense iteration space) -- TEST INFRASTRUCTURE ONLY.

Thin numpy/ctypes front end of ``st_oracle.c``.  It is independent of the CUDA
library: nothing here imports the GPU package, and the GPU package never
imports this.  Only the tests, the smoke check and the CPU-baseline leg of the
benchmark call it.

Every function follows the dense definition of the operation (the paper's
method is lossless, Section 6: the structured result must equal the dense
one), and returns ``(T, S)`` where ``S`` is the sum of the absolute values of
the terms of each output, the normaliser of the error metric.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "st_oracle.c")
_LIB = os.path.join(_HERE, "_st_oracle.so")

KIND_TRI, KIND_TET, KIND_BAND, KIND_BLOCKDIAG, KIND_FIXED_ROW, KIND_FIXED_COL, KIND_SIMPLEX4 = 0, 1, 2, 3, 4, 5, 6
FILL_ZERO, FILL_SYMMETRIC = 0, 1

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP over output indices only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
        lib.oracle_num_threads.restype = ci
        lib.oracle_set_threads.argtypes = [ci]
        lib.oracle_moment2.argtypes = [vp, i64, i64, i64, vp, vp]
        lib.oracle_moment2_at.argtypes = [vp, i64, i64, i64, vp, vp, i64, vp, vp]
        lib.oracle_moment3.argtypes = [vp, i64, i64, i64, vp, vp]
        lib.oracle_moment3_at.argtypes = [vp, i64, i64, i64, vp, vp, vp, i64, vp, vp]
        lib.oracle_moment4.argtypes = [vp, i64, i64, i64, vp, vp]
        lib.oracle_moment4_at.argtypes = [vp, i64, i64, i64, vp, vp, vp, vp, i64, vp, vp]
        lib.oracle_mttkrp.argtypes = [vp, i64, i64, i64, vp, vp, i64, i64, i64, vp, vp]
        lib.oracle_ttm.argtypes = [vp, i64, i64, vp, i64, vp, vp]
        lib.oracle_pack.argtypes = [ci, i64, i64, i64, i64, i64, i64, i64, vp, vp]
        lib.oracle_pack.restype = i64
        lib.oracle_unpack.argtypes = [ci, i64, i64, i64, i64, i64, i64, i64, ci, vp, vp]
        lib.oracle_unpack.restype = i64
        lib.oracle_locate.argtypes = [ci, i64, i64, i64, i64, i64, i64, i64, i64, i64]
        lib.oracle_locate.restype = i64
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_threads(n: int) -> None:
    _load().oracle_set_threads(int(n))


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a


def _ptr(a):
    return a.ctypes.data_as(ctypes.c_void_p)


def _x2d(X):
    X = np.asarray(X)
    if X.dtype != np.float32:
        raise TypeError("X must be float32 (widen bf16 to float32 first: the widening is exact)")
    if X.ndim != 2:
        raise ValueError("X must be [N, d]")
    X = np.ascontiguousarray(X)
    return X, X.shape[0], X.shape[1], X.shape[1]


def moment2(X):
    """T[i,j] = sum_n X[n,i] X[n,j] for all (i,j); Section 3, Sigma = x (x) x."""
    X, N, d, ldx = _x2d(X)
    T = np.zeros((d, d), np.float64)
    S = np.zeros((d, d), np.float64)
    _load().oracle_moment2(_ptr(X), N, d, ldx, _ptr(T), _ptr(S))
    return T, S


def moment2_at(X, ii, jj):
    """The same sums for sampled entries (ii[e], jj[e]) only."""
    X, N, d, ldx = _x2d(X)
    ii = np.ascontiguousarray(ii, dtype=np.int64)
    jj = np.ascontiguousarray(jj, dtype=np.int64)
    assert ii.shape == jj.shape and ii.ndim == 1
    if ii.size and (ii.min() < 0 or jj.min() < 0 or ii.max() >= d or jj.max() >= d):
        raise IndexError("sample index out of range")
    T = np.zeros(ii.size, np.float64)
    S = np.zeros(ii.size, np.float64)
    _load().oracle_moment2_at(_ptr(X), N, d, ldx, _ptr(ii), _ptr(jj), ii.size, _ptr(T), _ptr(S))
    return T, S


def moment3(X):
    """T[i,j,k] = sum_n X[n,i] X[n,j] X[n,k] for all (i,j,k); Section 3, term M2."""
    X, N, d, ldx = _x2d(X)
    T = np.zeros((d, d, d), np.float64)
    S = np.zeros((d, d, d), np.float64)
    _load().oracle_moment3(_ptr(X), N, d, ldx, _ptr(T), _ptr(S))
    return T, S


def moment3_at(X, ii, jj, kk):
    """The same sums for sampled entries (ii[e], jj[e], kk[e]) only."""
    X, N, d, ldx = _x2d(X)
    idx = [np.ascontiguousarray(a, dtype=np.int64) for a in (ii, jj, kk)]
    assert idx[0].ndim == 1 and idx[0].shape == idx[1].shape == idx[2].shape
    for a in idx:
        if a.size and (a.min() < 0 or a.max() >= d):
            raise IndexError("sample index out of range")
    T = np.zeros(idx[0].size, np.float64)
    S = np.zeros(idx[0].size, np.float64)
    _load().oracle_moment3_at(_ptr(X), N, d, ldx, _ptr(idx[0]), _ptr(idx[1]), _ptr(idx[2]), idx[0].size,
                              _ptr(T), _ptr(S))
    return T, S


def moment4(X):
    """T[i,j,k,l] = sum_n X[n,i] X[n,j] X[n,k] X[n,l]; Section 3, term M3."""
    X, N, d, ldx = _x2d(X)
    T = np.zeros((d, d, d, d), np.float64)
    S = np.zeros((d, d, d, d), np.float64)
    _load().oracle_moment4(_ptr(X), N, d, ldx, _ptr(T), _ptr(S))
    return T, S


def moment4_at(X, ii, jj, kk, ll):
    """The same sums for sampled entries (ii[e], jj[e], kk[e], ll[e]) only."""
    X, N, d, ldx = _x2d(X)
    idx = [np.ascontiguousarray(a, dtype=np.int64) for a in (ii, jj, kk, ll)]
    assert idx[0].ndim == 1 and all(a.shape == idx[0].shape for a in idx)
    for a in idx:
        if a.size and (a.min() < 0 or a.max() >= d):
            raise IndexError("sample index out of range")
    T = np.zeros(idx[0].size, np.float64)
    S = np.zeros(idx[0].size, np.float64)
    _load().oracle_moment4_at(_ptr(X), N, d, ldx, *[_ptr(a) for a in idx], idx[0].size, _ptr(T), _ptr(S))
    return T, S


def mttkrp(B, C, D, i0: int = 0, i1: int | None = None):
    """A[i,r] = sum_{j,k} B[i,j,k] C[j,r] D[k,r] over a dense B (Table 1, MTTKRP).

    Rows i0 <= i < i1 only (default: all)."""
    B, C, D = _f32(B), _f32(C), _f32(D)
    I, J, K = B.shape
    R = C.shape[1]
    assert C.shape == (J, R) and D.shape == (K, R)
    i1 = I if i1 is None else i1
    assert 0 <= i0 <= i1 <= I
    A = np.zeros((i1 - i0, R), np.float64)
    S = np.zeros((i1 - i0, R), np.float64)
    _load().oracle_mttkrp(_ptr(B), I, J, K, _ptr(C), _ptr(D), R, i0, i1, _ptr(A), _ptr(S))
    return A, S


def ttm(B, U):
    """A[..., r] = sum_k B[..., k] U[k, r] (Table 1, TTM) for every mode-3 fibre of B."""
    B, U = _f32(B), _f32(U)
    K, R = U.shape
    assert B.shape[-1] == K
    rows = int(np.prod(B.shape[:-1], dtype=np.int64))
    A = np.zeros((rows, R), np.float64)
    S = np.zeros((rows, R), np.float64)
    _load().oracle_ttm(_ptr(B), rows, K, _ptr(U), R, _ptr(A), _ptr(S))
    shp = tuple(B.shape[:-1]) + (R,)
    return A.reshape(shp), S.reshape(shp)


def thp(B, C):
    """A = B * C element by element (Table 1, THP) over the full dense iteration space."""
    B, C = _f32(B), _f32(C)
    assert B.shape == C.shape
    A = B.astype(np.float64) * C.astype(np.float64)
    return A, np.abs(A)


def _dense_rows(kind, d):
    return {KIND_TET: d ** 3, KIND_SIMPLEX4: d ** 4}.get(kind, d * d)


def packed_rows(kind, d, kl=0, ku=0, nb=0, bs=0) -> int:
    """Number of packed positions, counted by walking the unique set."""
    return int(_load().oracle_pack(kind, d, 1, kl, ku, nb, bs, 1, None, None))


def pack(dense, kind, d, inner=1, kl=0, ku=0, nb=0, bs=0):
    """T_C = T * T_U stored contiguously in lexicographic order of T_U (Section 4)."""
    dense = np.ascontiguousarray(dense)
    es = dense.dtype.itemsize
    assert dense.size == _dense_rows(kind, d) * inner, "dense size does not match the layout"
    rows = packed_rows(kind, d, kl, ku, nb, bs)
    if rows < 0:
        raise ValueError("unsupported layout")
    out = np.empty(rows * inner, dense.dtype)
    _load().oracle_pack(kind, d, inner, kl, ku, nb, bs, es, _ptr(dense), _ptr(out))
    return out


def unpack(packed, kind, d, inner=1, kl=0, ku=0, nb=0, bs=0, fill=FILL_ZERO):
    """T = T_C + T_R * T_C (Section 6, Property 5); zeros where T_R is empty."""
    packed = np.ascontiguousarray(packed)
    es = packed.dtype.itemsize
    rows = packed_rows(kind, d, kl, ku, nb, bs)
    if rows < 0:
        raise ValueError("unsupported layout")
    assert packed.size == rows * inner, "packed size does not match the layout"
    out = np.empty(_dense_rows(kind, d) * inner, packed.dtype)
    r = _load().oracle_unpack(kind, d, inner, kl, ku, nb, bs, es, fill, _ptr(packed), _ptr(out))
    if r < 0:
        raise ValueError("unsupported layout / fill")
    shape = {KIND_TET: (d, d, d), KIND_SIMPLEX4: (d, d, d, d)}.get(kind, (d, d))
    if inner != 1:
        shape = shape + (inner,)
    return out.reshape(shape)


def locate(kind, d, a, b, c=0, e=0, kl=0, ku=0, nb=0, bs=0) -> int:
    """Packed position of one index tuple, by walking T_U from the start (the fixed index of the
    one-row / one-column kinds is passed in kl)."""
    return int(_load().oracle_locate(kind, d, kl, ku, nb, bs, a, b, c, e))


def rel_err(got, T, S):
    """max |got - T| / S over entries with S > 0; entries with S == 0 must be exactly 0."""
    got = np.asarray(got, dtype=np.float64)
    T = np.asarray(T, dtype=np.float64)
    S = np.asarray(S, dtype=np.float64)
    assert got.shape == T.shape == S.shape, (got.shape, T.shape, S.shape)
    zero = S == 0
    if np.any(got[zero] != 0):
        return float("inf")
    if np.all(zero):
        return 0.0
    return float(np.max(np.abs(got[~zero] - T[~zero]) / S[~zero]))
