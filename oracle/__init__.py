"""ctypes front end of the CPU oracle (``oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle evaluates each contraction chain as its unfused
Einsum definition over COO input with fp64 accumulation (Table of kernels, Section 6 of
the paper); the product code never imports this package.  ``liboracle.so`` is compiled
from ``oracle.c`` by :func:`build` (plain ``gcc -O2 -fopenmp``).

``oracle.nests`` (``nests.c``) holds a second CPU evaluation, the paper's scheduled loop nests over compressed
storage; the tests hold the two against each other and bench.py times both.
"""
import ctypes
import os
import subprocess
import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lib = None


def build(force=False):
    """Compile oracle.c into liboracle.so if missing or older than the source."""
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
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def max_threads():
    return int(_load().oracle_max_threads())


_i64 = ctypes.c_int64
_p = ctypes.c_void_p


def _f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return a, a.ctypes.data_as(_p)


def _coords(coords, order):
    c = np.ascontiguousarray(coords, dtype=np.int32)
    assert c.ndim == 2 and c.shape[1] == order
    return c, c.ctypes.data_as(_p)


def _sel(sel, I):
    if sel is None:
        return None, None, 0, I
    s = np.ascontiguousarray(sel, dtype=np.int64)
    assert len(set(s.tolist())) == s.shape[0], "selected slices must be distinct"
    return s, s.ctypes.data_as(_p), s.shape[0], s.shape[0]


def _check(rc):
    if rc == -2:
        raise ValueError("oracle: coordinate or selection out of range")
    if rc != 0:
        raise MemoryError("oracle: allocation failed")


def spttm_ttm3(coords, vals, dims, C, D, sel=None, with_abs=True, threads=0):
    """A(i,l,m) = sum_{j,k} B(i,j,k) C(j,l) D(k,m).  Returns (A, S) as float64."""
    I, J, K = (int(d) for d in dims)
    c, cp = _coords(coords, 3)
    v, vp = _f32(vals)
    C, Cp = _f32(C)
    D, Dp = _f32(D)
    assert C.shape[0] == J and D.shape[0] == K
    L, M = C.shape[1], D.shape[1]
    s, sp, n_sel, n_out = _sel(sel, I)
    A = np.empty((n_out, L, M), dtype=np.float64)
    S = np.empty_like(A) if with_abs else None
    rc = _load().oracle_spttm_ttm3(_i64(v.shape[0]), cp, vp, _i64(I), _i64(J), _i64(K), _i64(L), _i64(M),
                                   Cp, Dp, _i64(n_sel), sp, A.ctypes.data_as(_p),
                                   S.ctypes.data_as(_p) if with_abs else None, ctypes.c_int(threads))
    _check(rc)
    return A, S


def spttm_ttm4(coords, vals, dims, C, D, E, sel=None, with_abs=True, threads=0):
    """A(i,l,m,n) = sum_{j,k,o} B(i,j,k,o) C(j,l) D(k,m) E(o,n).  Returns (A, S)."""
    I, J, K, O = (int(d) for d in dims)
    c, cp = _coords(coords, 4)
    v, vp = _f32(vals)
    C, Cp = _f32(C)
    D, Dp = _f32(D)
    E, Ep = _f32(E)
    assert C.shape[0] == J and D.shape[0] == K and E.shape[0] == O
    L, M, N = C.shape[1], D.shape[1], E.shape[1]
    s, sp, n_sel, n_out = _sel(sel, I)
    A = np.empty((n_out, L, M, N), dtype=np.float64)
    S = np.empty_like(A) if with_abs else None
    rc = _load().oracle_spttm_ttm4(_i64(v.shape[0]), cp, vp, _i64(I), _i64(J), _i64(K), _i64(O),
                                   _i64(L), _i64(M), _i64(N), Cp, Dp, Ep, _i64(n_sel), sp,
                                   A.ctypes.data_as(_p), S.ctypes.data_as(_p) if with_abs else None,
                                   ctypes.c_int(threads))
    _check(rc)
    return A, S


def sddmm_spmm(coords, vals, dims, C, D, E, sel=None, with_abs=True, with_sampled=False, threads=0):
    """A(i,l) = sum_{j,k} B(i,j) C(i,k) D(j,k) E(j,l).  Returns (A, S, P).

    P (if requested) holds, per stored nonzero in input order, the sampled value
    B(i,j) * sum_k C(i,k) D(j,k); entries of rows outside ``sel`` are NaN.
    """
    I, J = (int(d) for d in dims)
    c, cp = _coords(coords, 2)
    v, vp = _f32(vals)
    C, Cp = _f32(C)
    D, Dp = _f32(D)
    E, Ep = _f32(E)
    assert C.shape[0] == I and D.shape[0] == J and E.shape[0] == J and C.shape[1] == D.shape[1]
    K, L = C.shape[1], E.shape[1]
    s, sp, n_sel, n_out = _sel(sel, I)
    A = np.empty((n_out, L), dtype=np.float64)
    S = np.empty_like(A) if with_abs else None
    P = np.full(v.shape[0], np.nan, dtype=np.float64) if with_sampled else None
    rc = _load().oracle_sddmm_spmm(_i64(v.shape[0]), cp, vp, _i64(I), _i64(J), _i64(K), _i64(L),
                                   Cp, Dp, Ep, _i64(n_sel), sp, A.ctypes.data_as(_p),
                                   S.ctypes.data_as(_p) if with_abs else None,
                                   P.ctypes.data_as(_p) if with_sampled else None, ctypes.c_int(threads))
    _check(rc)
    return A, S, P


def sddmm_spmm_gemm(coords, vals, dims, C, D, E, F, sel=None, with_abs=True, threads=0):
    """A(i,m) = sum_{j,k,l} B(i,j) C(i,k) D(j,k) E(j,l) F(l,m).  Returns (A, S)."""
    I, J = (int(d) for d in dims)
    c, cp = _coords(coords, 2)
    v, vp = _f32(vals)
    C, Cp = _f32(C)
    D, Dp = _f32(D)
    E, Ep = _f32(E)
    F, Fp = _f32(F)
    assert C.shape[0] == I and D.shape[0] == J and E.shape[0] == J and C.shape[1] == D.shape[1] and F.shape[0] == E.shape[1]
    K, L, M = C.shape[1], E.shape[1], F.shape[1]
    s, sp, n_sel, n_out = _sel(sel, I)
    A = np.empty((n_out, M), dtype=np.float64)
    S = np.empty_like(A) if with_abs else None
    rc = _load().oracle_sddmm_spmm_gemm(_i64(v.shape[0]), cp, vp, _i64(I), _i64(J), _i64(K), _i64(L), _i64(M),
                                        Cp, Dp, Ep, Fp, _i64(n_sel), sp, A.ctypes.data_as(_p),
                                        S.ctypes.data_as(_p) if with_abs else None, ctypes.c_int(threads))
    _check(rc)
    return A, S


def spmm_gemm(coords, vals, dims, C, D, sel=None, with_abs=True, threads=0):
    """A(i,m) = sum_{j,l} B(i,j) C(j,l) D(l,m).  Returns (A, S)."""
    I, J = (int(d) for d in dims)
    c, cp = _coords(coords, 2)
    v, vp = _f32(vals)
    C, Cp = _f32(C)
    D, Dp = _f32(D)
    assert C.shape[0] == J and D.shape[0] == C.shape[1]
    L, M = C.shape[1], D.shape[1]
    s, sp, n_sel, n_out = _sel(sel, I)
    A = np.empty((n_out, M), dtype=np.float64)
    S = np.empty_like(A) if with_abs else None
    rc = _load().oracle_spmm_gemm(_i64(v.shape[0]), cp, vp, _i64(I), _i64(J), _i64(L), _i64(M),
                                  Cp, Dp, _i64(n_sel), sp, A.ctypes.data_as(_p),
                                  S.ctypes.data_as(_p) if with_abs else None, ctypes.c_int(threads))
    _check(rc)
    return A, S


def spmmh_gemm(coords, vals, dims, C, D, E, sel=None, with_abs=True, threads=0):
    """Kernel 3: A(i,m) = sum_{j,l} B(i,j) C(j,l) D(j,l) E(l,m).  Returns (A, S)."""
    I, J = (int(d) for d in dims)
    c, cp = _coords(coords, 2)
    v, vp = _f32(vals)
    C, Cp = _f32(C)
    D, Dp = _f32(D)
    E, Ep = _f32(E)
    assert C.shape[0] == J and D.shape == C.shape and E.shape[0] == C.shape[1]
    L, M = C.shape[1], E.shape[1]
    s, sp, n_sel, n_out = _sel(sel, I)
    A = np.empty((n_out, M), dtype=np.float64)
    S = np.empty_like(A) if with_abs else None
    rc = _load().oracle_spmmh_gemm(_i64(v.shape[0]), cp, vp, _i64(I), _i64(J), _i64(L), _i64(M),
                                   Cp, Dp, Ep, _i64(n_sel), sp, A.ctypes.data_as(_p),
                                   S.ctypes.data_as(_p) if with_abs else None, ctypes.c_int(threads))
    _check(rc)
    return A, S


def mttkrp_gemm(coords, vals, dims, C, D, E, sel=None, with_abs=True, threads=0):
    """Kernel 8: A(i,m) = sum_{j,k,r} B(i,j,k) C(j,r) D(k,r) E(r,m).  Returns (A, S)."""
    I, J, K = (int(d) for d in dims)
    c, cp = _coords(coords, 3)
    v, vp = _f32(vals)
    C, Cp = _f32(C)
    D, Dp = _f32(D)
    E, Ep = _f32(E)
    assert C.shape[0] == J and D.shape[0] == K and D.shape[1] == C.shape[1] and E.shape[0] == C.shape[1]
    R, M = C.shape[1], E.shape[1]
    s, sp, n_sel, n_out = _sel(sel, I)
    A = np.empty((n_out, M), dtype=np.float64)
    S = np.empty_like(A) if with_abs else None
    rc = _load().oracle_mttkrp_gemm(_i64(v.shape[0]), cp, vp, _i64(I), _i64(J), _i64(K), _i64(R), _i64(M),
                                    Cp, Dp, Ep, _i64(n_sel), sp, A.ctypes.data_as(_p),
                                    S.ctypes.data_as(_p) if with_abs else None, ctypes.c_int(threads))
    _check(rc)
    return A, S


def fiber_keys(coords, dims):
    """The (i,j) pairs that occur in B, sorted lexicographically, and for every nonzero the index of its pair."""
    c = np.asarray(coords)
    key = c[:, 0].astype(np.int64) * int(dims[1]) + c[:, 1].astype(np.int64)
    uniq, inv = np.unique(key, return_inverse=True)
    keys = np.stack([uniq // int(dims[1]), uniq % int(dims[1])], axis=1)
    return keys, inv.reshape(-1)


def spttm_spttm(coords, vals, dims, C, D, sel=None, with_abs=True, threads=0):
    """Kernel 7 <SpTTM,SpTTM>: A(i,j,m) = sum_{k,l} B(i,j,k) C(k,l) D(l,m)  (Table of kernels, Description
    column with the two contracted indices k and l summed).  The output is sparse with the pattern of B's
    (i,j) pairs: row f of the result belongs to the f-th pair in lexicographic order (see fiber_keys).
    ``sel`` lists the rows wanted.  Plain definition in fp64: every nonzero adds v C(k,l) D(l,m) for all l, m.
    Returns (A, S) with S the sum of the absolute values of the terms."""
    I, J, K = (int(d) for d in dims)
    c = np.asarray(coords)
    v = np.asarray(vals, dtype=np.float64)
    C = np.asarray(C, dtype=np.float64)
    D = np.asarray(D, dtype=np.float64)
    assert C.shape[0] == K and D.shape[0] == C.shape[1]
    if c.shape[0] and (c.min() < 0 or (c.max(axis=0) >= np.array([I, J, K])).any()):
        raise ValueError("coordinate out of range")
    M = D.shape[1]
    keys, inv = fiber_keys(c, dims)
    if sel is None:
        row_of, n_out, pick = inv, keys.shape[0], np.arange(c.shape[0])
    else:
        sel = np.asarray(sel, dtype=np.int64)
        where = np.full(keys.shape[0], -1, dtype=np.int64)
        where[sel] = np.arange(sel.shape[0])
        row_of = where[inv]
        pick = np.nonzero(row_of >= 0)[0]
        n_out = sel.shape[0]
    A = np.zeros((n_out, M), dtype=np.float64)
    S = np.zeros((n_out, M), dtype=np.float64) if with_abs else None
    for a in range(0, pick.shape[0], 4096):
        p = pick[a:a + 4096]
        term = v[p, None, None] * C[c[p, 2], :, None] * D[None, :, :]        # [nonzero, l, m]
        np.add.at(A, row_of[p], term.sum(axis=1))
        if with_abs:
            np.add.at(S, row_of[p], np.abs(term).sum(axis=1))
    return A, S

def ttmc3(coords, vals, dims, C, D, E, sel=None, with_abs=True, threads=0):
    """A(l,m,n) = sum_{i,j,k} B(i,j,k) C(i,l) D(j,m) E(k,n).  Returns (A, S) of shape (L, M, N), or of
    shape (len(sel),) when ``sel`` lists flat output indices (l*M + m)*N + n."""
    I, J, K = (int(d) for d in dims)
    c, cp = _coords(coords, 3)
    v, vp = _f32(vals)
    C, Cp = _f32(C)
    D, Dp = _f32(D)
    E, Ep = _f32(E)
    assert C.shape[0] == I and D.shape[0] == J and E.shape[0] == K
    L, M, N = C.shape[1], D.shape[1], E.shape[1]
    if sel is None:
        s, sp, n_sel, shape = None, None, 0, (L, M, N)
    else:
        s = np.ascontiguousarray(sel, dtype=np.int64)
        sp, n_sel, shape = s.ctypes.data_as(_p), s.shape[0], (s.shape[0],)
    A = np.empty(shape, dtype=np.float64)
    S = np.empty_like(A) if with_abs else None
    rc = _load().oracle_ttmc3(_i64(v.shape[0]), cp, vp, _i64(I), _i64(J), _i64(K), _i64(L), _i64(M), _i64(N),
                              Cp, Dp, Ep, _i64(n_sel), sp, A.ctypes.data_as(_p),
                              S.ctypes.data_as(_p) if with_abs else None, ctypes.c_int(threads))
    _check(rc)
    return A, S


def evaluate(w, sel=None, with_abs=True, threads=0):
    """Evaluate a workload object (``workloads.configs.Workload``) -> (A, S)."""
    if w.expr == "spttm_ttm3":
        return spttm_ttm3(w.coords, w.vals, w.dims, *w.dense, sel=sel, with_abs=with_abs, threads=threads)
    if w.expr == "spttm_ttm4":
        return spttm_ttm4(w.coords, w.vals, w.dims, *w.dense, sel=sel, with_abs=with_abs, threads=threads)
    if w.expr == "ttmc3":
        return ttmc3(w.coords, w.vals, w.dims, *w.dense, sel=sel, with_abs=with_abs, threads=threads)
    if w.expr == "sddmm_spmm_gemm":
        return sddmm_spmm_gemm(w.coords, w.vals, w.dims, *w.dense, sel=sel, with_abs=with_abs, threads=threads)
    if w.expr == "sddmm_spmm":
        return sddmm_spmm(w.coords, w.vals, w.dims, *w.dense, sel=sel, with_abs=with_abs, threads=threads)[:2]
    if w.expr == "spttm_spttm":
        return spttm_spttm(w.coords, w.vals, w.dims, *w.dense, sel=sel, with_abs=with_abs, threads=threads)
    if w.expr == "mttkrp_gemm":
        return mttkrp_gemm(w.coords, w.vals, w.dims, *w.dense, sel=sel, with_abs=with_abs, threads=threads)
    if w.expr == "spmmh_gemm":
        return spmmh_gemm(w.coords, w.vals, w.dims, *w.dense, sel=sel, with_abs=with_abs, threads=threads)
    if w.expr == "spmm_gemm":
        return spmm_gemm(w.coords, w.vals, w.dims, *w.dense, sel=sel, with_abs=with_abs, threads=threads)
    raise ValueError(w.expr)
