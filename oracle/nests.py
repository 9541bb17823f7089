"""ctypes front end of ``nests.c``: the paper's scheduled loop nests on the CPU.

TEST INFRASTRUCTURE ONLY (tests and the CPU-baseline leg of bench.py); the product code never imports it.
The compressed storage the nests walk is built here from the COO input with numpy alone (a lexicographic sort and
run boundaries per level, Section 2.1 of the paper), independently of the library's own builder.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "nests.c")
_LIB = os.path.join(_HERE, "libnests.so")
_lib = None
_i64 = ctypes.c_int64
_p = ctypes.c_void_p


def build(force=False):
    """Compile nests.c into libnests.so if missing or older than the source."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _arr(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a, a.ctypes.data_as(_p)


def csf_from_coo(coords, vals):
    """Sorted CSF of an order-n COO tensor with distinct coordinates: (levels, vals) where levels[d] = (pos, crd);
    pos of level 0 is None (its crd lists the non-empty slices), pos of level d > 0 has one entry per node of level
    d - 1 plus one."""
    coords = np.asarray(coords)
    nnz, order = coords.shape
    perm = np.lexsort([coords[:, d] for d in range(order - 1, -1, -1)]) if nnz else np.zeros(0, dtype=np.int64)
    c = coords[perm]
    v = np.asarray(vals, dtype=np.float32)[perm]
    levels = []
    starts_prev = None
    for d in range(order):
        if nnz == 0:
            starts = np.zeros(0, dtype=np.int64)
        elif d == order - 1:
            starts = np.arange(nnz, dtype=np.int64)
        else:
            new = np.ones(nnz, dtype=bool)
            new[1:] = (c[1:, :d + 1] != c[:-1, :d + 1]).any(axis=1)
            starts = np.flatnonzero(new).astype(np.int64)
        crd = c[starts, d].astype(np.int32)
        if d == 0:
            pos = None
        else:
            # node x of level d - 1 starts at nonzero starts_prev[x]; its children are the level-d nodes from there on
            pos = np.searchsorted(starts, np.append(starts_prev, nnz)).astype(np.int64)
        levels.append((pos, crd))
        starts_prev = starts
    return levels, v


def csr_from_coo(coords, vals, I):
    """(pos, crd, vals) of a matrix given as COO with distinct coordinates: dense row level, compressed columns."""
    coords = np.asarray(coords)
    perm = np.lexsort([coords[:, 1], coords[:, 0]]) if coords.shape[0] else np.zeros(0, dtype=np.int64)
    c = coords[perm]
    pos = np.zeros(I + 1, dtype=np.int64)
    np.add.at(pos, c[:, 0].astype(np.int64) + 1, 1)
    return np.cumsum(pos), c[:, 1].astype(np.int32), np.asarray(vals, dtype=np.float32)[perm]


def _check(rc):
    if rc != 0:
        raise MemoryError("nests: allocation failed")


def spttm_ttm3(levels, vals, I, C, D, threads=0):
    (_, s_i), (pos1, crd1), (pos2, crd2) = levels
    C, Cp = _arr(C, np.float32)
    D, Dp = _arr(D, np.float32)
    L, M = C.shape[1], D.shape[1]
    A = np.zeros((I, L, M), dtype=np.float64)
    keep = [_arr(s_i, np.int32), _arr(pos1, np.int64), _arr(crd1, np.int32), _arr(pos2, np.int64), _arr(crd2, np.int32),
            _arr(vals, np.float32)]
    _check(_load().nest_spttm_ttm3(_i64(keep[0][0].shape[0]), *[k[1] for k in keep], _i64(L), _i64(M), Cp, Dp,
                                   A.ctypes.data_as(_p), ctypes.c_int(threads)))
    return A


def spttm_ttm4(levels, vals, I, C, D, E, threads=0):
    (_, s_i), (pos1, crd1), (pos2, crd2), (pos3, crd3) = levels
    C, Cp = _arr(C, np.float32)
    D, Dp = _arr(D, np.float32)
    E, Ep = _arr(E, np.float32)
    L, M, N = C.shape[1], D.shape[1], E.shape[1]
    A = np.zeros((I, L, M, N), dtype=np.float64)
    keep = [_arr(s_i, np.int32), _arr(pos1, np.int64), _arr(crd1, np.int32), _arr(pos2, np.int64), _arr(crd2, np.int32),
            _arr(pos3, np.int64), _arr(crd3, np.int32), _arr(vals, np.float32)]
    _check(_load().nest_spttm_ttm4(_i64(keep[0][0].shape[0]), *[k[1] for k in keep], _i64(L), _i64(M), _i64(N), Cp, Dp, Ep,
                                   A.ctypes.data_as(_p), ctypes.c_int(threads)))
    return A


def ttmc3(levels, vals, C, D, E, threads=0):
    (_, s_i), (pos1, crd1), (pos2, crd2) = levels
    C, Cp = _arr(C, np.float32)
    D, Dp = _arr(D, np.float32)
    E, Ep = _arr(E, np.float32)
    L, M, N = C.shape[1], D.shape[1], E.shape[1]
    A = np.zeros((L, M, N), dtype=np.float64)
    keep = [_arr(s_i, np.int32), _arr(pos1, np.int64), _arr(crd1, np.int32), _arr(pos2, np.int64), _arr(crd2, np.int32),
            _arr(vals, np.float32)]
    _check(_load().nest_ttmc3(_i64(keep[0][0].shape[0]), *[k[1] for k in keep], _i64(L), _i64(M), _i64(N), Cp, Dp, Ep,
                              A.ctypes.data_as(_p), ctypes.c_int(threads)))
    return A


def sddmm_spmm(pos, crd, vals, C, D, E, threads=0):
    C, Cp = _arr(C, np.float32)
    D, Dp = _arr(D, np.float32)
    E, Ep = _arr(E, np.float32)
    I, K, L = C.shape[0], C.shape[1], E.shape[1]
    A = np.zeros((I, L), dtype=np.float64)
    keep = [_arr(pos, np.int64), _arr(crd, np.int32), _arr(vals, np.float32)]
    _check(_load().nest_sddmm_spmm(_i64(I), *[k[1] for k in keep], _i64(K), _i64(L), Cp, Dp, Ep, A.ctypes.data_as(_p),
                                   ctypes.c_int(threads)))
    return A


def spmm_gemm(pos, crd, vals, C, D, order="left", threads=0):
    C, Cp = _arr(C, np.float32)
    D, Dp = _arr(D, np.float32)
    I, J, L, M = pos.shape[0] - 1, C.shape[0], C.shape[1], D.shape[1]
    A = np.zeros((I, M), dtype=np.float64)
    keep = [_arr(pos, np.int64), _arr(crd, np.int32), _arr(vals, np.float32)]
    if order == "left":
        rc = _load().nest_spmm_gemm_left(_i64(I), *[k[1] for k in keep], _i64(L), _i64(M), Cp, Dp, A.ctypes.data_as(_p),
                                         ctypes.c_int(threads))
    else:
        tmp = np.empty((J, M), dtype=np.float64)
        rc = _load().nest_spmm_gemm_right(_i64(I), _i64(J), *[k[1] for k in keep], _i64(L), _i64(M), Cp, Dp,
                                          tmp.ctypes.data_as(_p), A.ctypes.data_as(_p), ctypes.c_int(threads))
    _check(rc)
    return A


def sddmm_spmm_gemm(pos, crd, vals, C, D, E, F, threads=0):
    C, Cp = _arr(C, np.float32)
    D, Dp = _arr(D, np.float32)
    E, Ep = _arr(E, np.float32)
    F, Fp = _arr(F, np.float32)
    I, K, L, M = C.shape[0], C.shape[1], E.shape[1], F.shape[1]
    A = np.zeros((I, M), dtype=np.float64)
    keep = [_arr(pos, np.int64), _arr(crd, np.int32), _arr(vals, np.float32)]
    _check(_load().nest_sddmm_spmm_gemm(_i64(I), *[k[1] for k in keep], _i64(K), _i64(L), _i64(M), Cp, Dp, Ep, Fp,
                                        A.ctypes.data_as(_p), ctypes.c_int(threads)))
    return A


def spmmh_gemm(pos, crd, vals, C, D, E, threads=0):
    C, Cp = _arr(C, np.float32)
    D, Dp = _arr(D, np.float32)
    E, Ep = _arr(E, np.float32)
    I, L, M = pos.shape[0] - 1, C.shape[1], E.shape[1]
    A = np.zeros((I, M), dtype=np.float64)
    keep = [_arr(pos, np.int64), _arr(crd, np.int32), _arr(vals, np.float32)]
    _check(_load().nest_spmmh_gemm(_i64(I), *[k[1] for k in keep], _i64(L), _i64(M), Cp, Dp, Ep, A.ctypes.data_as(_p),
                                   ctypes.c_int(threads)))
    return A


def mttkrp_gemm(levels, vals, I, C, D, E, threads=0):
    (_, s_i), (pos1, crd1), (pos2, crd2) = levels
    C, Cp = _arr(C, np.float32)
    D, Dp = _arr(D, np.float32)
    E, Ep = _arr(E, np.float32)
    R, M = C.shape[1], E.shape[1]
    A = np.zeros((I, M), dtype=np.float64)
    keep = [_arr(s_i, np.int32), _arr(pos1, np.int64), _arr(crd1, np.int32), _arr(pos2, np.int64), _arr(crd2, np.int32),
            _arr(vals, np.float32)]
    _check(_load().nest_mttkrp_gemm(_i64(keep[0][0].shape[0]), *[k[1] for k in keep], _i64(R), _i64(M), Cp, Dp, Ep,
                                    A.ctypes.data_as(_p), ctypes.c_int(threads)))
    return A


def spttm_spttm(levels, vals, C, D, threads=0):
    """One output row per (i,j) fiber, in lexicographic order of the pairs."""
    (_, _s), (_pos1, crd1), (pos2, crd2) = levels
    C, Cp = _arr(C, np.float32)
    D, Dp = _arr(D, np.float32)
    L, M = C.shape[1], D.shape[1]
    F = crd1.shape[0]
    A = np.zeros((F, M), dtype=np.float64)
    keep = [_arr(pos2, np.int64), _arr(crd2, np.int32), _arr(vals, np.float32)]
    _check(_load().nest_spttm_spttm(_i64(F), *[k[1] for k in keep], _i64(L), _i64(M), Cp, Dp, A.ctypes.data_as(_p),
                                    ctypes.c_int(threads)))
    return A


def prepare(w, order="left", threads=0):
    """Builds the compressed storage of the workload's sparse operand and returns a function that runs the chain's
    nest on it (so that a caller can time the nest without the sort)."""
    if w.expr in ("spttm_ttm3", "spttm_ttm4", "ttmc3", "mttkrp_gemm", "spttm_spttm"):
        levels, v = csf_from_coo(w.coords, w.vals)
        if w.expr == "mttkrp_gemm":
            return lambda: mttkrp_gemm(levels, v, int(w.dims[0]), *w.dense, threads=threads)
        if w.expr == "spttm_spttm":
            return lambda: spttm_spttm(levels, v, *w.dense, threads=threads)
        if w.expr == "spttm_ttm3":
            return lambda: spttm_ttm3(levels, v, int(w.dims[0]), *w.dense, threads=threads)
        if w.expr == "spttm_ttm4":
            return lambda: spttm_ttm4(levels, v, int(w.dims[0]), *w.dense, threads=threads)
        return lambda: ttmc3(levels, v, *w.dense, threads=threads)
    if w.expr in ("sddmm_spmm", "spmm_gemm", "sddmm_spmm_gemm", "spmmh_gemm"):
        pos, crd, v = csr_from_coo(w.coords, w.vals, int(w.dims[0]))
        if w.expr == "sddmm_spmm_gemm":
            return lambda: sddmm_spmm_gemm(pos, crd, v, *w.dense, threads=threads)
        if w.expr == "spmmh_gemm":
            return lambda: spmmh_gemm(pos, crd, v, *w.dense, threads=threads)
        if w.expr == "sddmm_spmm":
            return lambda: sddmm_spmm(pos, crd, v, *w.dense, threads=threads)
        return lambda: spmm_gemm(pos, crd, v, *w.dense, order=order, threads=threads)
    raise ValueError("no scheduled nest for " + w.expr)


def evaluate(w, order="left", threads=0):
    """The workload's chain by the paper's nest, from its COO input; returns A as float64 (full output)."""
    return prepare(w, order=order, threads=threads)()
