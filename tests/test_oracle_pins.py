"""Pins for the CPU oracle: everything here is fixed by the mathematics of the Einsum
definitions (Table of kernels, Section 6 of the paper), not by the oracle itself.

* brute force: B densified, the Einsum evaluated by explicit Python loops and by
  numpy.einsum on tiny, non-square shapes (a transposed operand or swapped index
  changes the result or the shape);
* closed forms for all-ones operands;
* special cases that reduce to densification, SpMM (scipy CSR @ dense, the loop of
  Fig. 1b) and dense GEMM;
* invariants: linearity in each operand, invariance under reordering of the COO list,
  slice-subset evaluation equals the matching slices of the full evaluation;
* the SDDMM sampled values exist exactly on B's stored coordinates.
"""
import itertools

import numpy as np
import pytest
import scipy.sparse as sp

import oracle


def tiny_coo(rs, dims, nnz):
    total = int(np.prod(dims))
    lin = rs.choice(total, size=nnz, replace=False)
    coords = np.stack(np.unravel_index(lin, dims), axis=1).astype(np.int32)
    vals = rs.uniform(-1, 1, size=nnz).astype(np.float32)
    return coords, vals


def densify(coords, vals, dims):
    B = np.zeros(dims, dtype=np.float64)
    for c, v in zip(coords, vals):
        B[tuple(c)] += float(v)
    return B


def dense(rs, r, c):
    return rs.uniform(-1, 1, size=(r, c)).astype(np.float32)


# ----------------------------------------------------------------- brute force

def test_ttm3_bruteforce_loops_and_einsum():
    rs = np.random.RandomState(1)
    dims = (4, 5, 6)
    coords, vals = tiny_coo(rs, dims, 37)
    C, D = dense(rs, 5, 3), dense(rs, 6, 2)
    A, S = oracle.spttm_ttm3(coords, vals, dims, C, D)
    B = densify(coords, vals, dims)
    ref = np.zeros((4, 3, 2))
    refS = np.zeros((4, 3, 2))
    for i, j, k, l, m in itertools.product(range(4), range(5), range(6), range(3), range(2)):
        t = B[i, j, k] * float(C[j, l]) * float(D[k, m])
        ref[i, l, m] += t
        refS[i, l, m] += abs(t)
    np.testing.assert_allclose(A, ref, rtol=0, atol=1e-13)
    np.testing.assert_allclose(S, refS, rtol=0, atol=1e-13)
    ein = np.einsum("ijk,jl,km->ilm", B, C.astype(np.float64), D.astype(np.float64))
    np.testing.assert_allclose(A, ein, rtol=0, atol=1e-13)


def test_ttm4_bruteforce_loops_and_einsum():
    rs = np.random.RandomState(2)
    dims = (3, 4, 5, 6)
    coords, vals = tiny_coo(rs, dims, 61)
    C, D, E = dense(rs, 4, 2), dense(rs, 5, 3), dense(rs, 6, 4)
    A, S = oracle.spttm_ttm4(coords, vals, dims, C, D, E)
    B = densify(coords, vals, dims)
    ein = np.einsum("ijko,jl,km,on->ilmn", B, *(x.astype(np.float64) for x in (C, D, E)))
    np.testing.assert_allclose(A, ein, rtol=0, atol=1e-13)
    einS = np.einsum("ijko,jl,km,on->ilmn", np.abs(B), *(np.abs(x.astype(np.float64)) for x in (C, D, E)))
    np.testing.assert_allclose(S, einS, rtol=0, atol=1e-13)
    ref = np.zeros((3, 2, 3, 4))
    for c, v in zip(coords, vals):
        i, j, k, o = (int(x) for x in c)
        for l, m, n in itertools.product(range(2), range(3), range(4)):
            ref[i, l, m, n] += float(v) * float(C[j, l]) * float(D[k, m]) * float(E[o, n])
    np.testing.assert_allclose(A, ref, rtol=0, atol=1e-13)


def test_sddmm_spmm_bruteforce():
    rs = np.random.RandomState(3)
    dims = (5, 7)
    coords, vals = tiny_coo(rs, dims, 17)
    C, D, E = dense(rs, 5, 3), dense(rs, 7, 3), dense(rs, 7, 4)
    A, S, P = oracle.sddmm_spmm(coords, vals, dims, C, D, E, with_sampled=True)
    B = densify(coords, vals, dims)
    ref = np.zeros((5, 4))
    for i, j, k, l in itertools.product(range(5), range(7), range(3), range(4)):
        ref[i, l] += B[i, j] * float(C[i, k]) * float(D[j, k]) * float(E[j, l])
    np.testing.assert_allclose(A, ref, rtol=0, atol=1e-13)
    C64, D64, E64 = (x.astype(np.float64) for x in (C, D, E))
    ein = np.einsum("ij,ik,jk,jl->il", B, C64, D64, E64)
    np.testing.assert_allclose(A, ein, rtol=0, atol=1e-13)
    np.testing.assert_allclose(S, np.einsum("ij,ik,jk,jl->il", np.abs(B), np.abs(C64), np.abs(D64), np.abs(E64)),
                               rtol=0, atol=1e-13)
    # sampled matrix: (C D^T) sampled at B's coordinates and scaled by B; nothing elsewhere
    samp = B * (C64 @ D64.T)
    for p, c in enumerate(coords):
        assert abs(P[p] - samp[c[0], c[1]]) < 1e-13
    assert P.shape[0] == coords.shape[0]
    # the SpMM of the sampled matrix gives A: fused == two separate kernels
    np.testing.assert_allclose(A, samp @ E64, rtol=0, atol=1e-13)


def test_spmm_gemm_bruteforce_and_both_orders():
    rs = np.random.RandomState(4)
    dims = (6, 5)
    coords, vals = tiny_coo(rs, dims, 13)
    C, D = dense(rs, 5, 4), dense(rs, 4, 3)
    A, S = oracle.spmm_gemm(coords, vals, dims, C, D)
    B = densify(coords, vals, dims)
    ref = np.zeros((6, 3))
    for i, j, l, m in itertools.product(range(6), range(5), range(4), range(3)):
        ref[i, m] += B[i, j] * float(C[j, l]) * float(D[l, m])
    np.testing.assert_allclose(A, ref, rtol=0, atol=1e-13)
    C64, D64 = C.astype(np.float64), D.astype(np.float64)
    np.testing.assert_allclose(A, (B @ C64) @ D64, rtol=0, atol=1e-13)   # (B.C).D
    np.testing.assert_allclose(A, B @ (C64 @ D64), rtol=0, atol=1e-13)   # B.(C.D)
    np.testing.assert_allclose(S, np.abs(B) @ np.abs(C64) @ np.abs(D64), rtol=0, atol=1e-13)


# ----------------------------------------------------------------- closed forms

def test_all_ones_closed_forms():
    rs = np.random.RandomState(5)
    dims = (7, 6, 5)
    coords, _ = tiny_coo(rs, dims, 50)
    ones = np.ones(50, dtype=np.float32)
    A, S = oracle.spttm_ttm3(coords, ones, dims, np.ones((6, 3), np.float32), np.ones((5, 4), np.float32))
    cnt = np.bincount(coords[:, 0], minlength=7)
    assert np.array_equal(A, np.broadcast_to(cnt[:, None, None], (7, 3, 4)).astype(np.float64))
    assert np.array_equal(A, S)

    dims4 = (4, 3, 5, 2)
    coords4, _ = tiny_coo(rs, dims4, 40)
    A4, _ = oracle.spttm_ttm4(coords4, np.ones(40, np.float32), dims4, np.ones((3, 2), np.float32),
                              np.ones((5, 3), np.float32), np.ones((2, 2), np.float32))
    cnt4 = np.bincount(coords4[:, 0], minlength=4)
    assert np.array_equal(A4, np.broadcast_to(cnt4[:, None, None, None], (4, 2, 3, 2)).astype(np.float64))

    dims2 = (9, 8)
    coords2, _ = tiny_coo(rs, dims2, 30)
    deg = np.bincount(coords2[:, 0], minlength=9)
    K, L = 5, 3
    A1, _, P = oracle.sddmm_spmm(coords2, np.ones(30, np.float32), dims2, np.ones((9, K), np.float32),
                                 np.ones((8, K), np.float32), np.ones((8, L), np.float32), with_sampled=True)
    assert np.array_equal(A1, np.broadcast_to((K * deg)[:, None], (9, L)).astype(np.float64))
    assert np.array_equal(P, np.full(30, float(K)))
    Lg, Mg = 6, 2
    Ag, _ = oracle.spmm_gemm(coords2, np.ones(30, np.float32), dims2, np.ones((8, Lg), np.float32),
                             np.ones((Lg, Mg), np.float32))
    assert np.array_equal(Ag, np.broadcast_to((Lg * deg)[:, None], (9, Mg)).astype(np.float64))


# ----------------------------------------------------------------- special cases

def test_identity_factors_densify():
    rs = np.random.RandomState(6)
    dims = (4, 5, 6)
    coords, vals = tiny_coo(rs, dims, 41)
    A, _ = oracle.spttm_ttm3(coords, vals, dims, np.eye(5, dtype=np.float32), np.eye(6, dtype=np.float32))
    assert np.array_equal(A, densify(coords, vals, dims))
    dims4 = (3, 4, 2, 5)
    coords4, vals4 = tiny_coo(rs, dims4, 33)
    A4, _ = oracle.spttm_ttm4(coords4, vals4, dims4, np.eye(4, dtype=np.float32), np.eye(2, dtype=np.float32),
                              np.eye(5, dtype=np.float32))
    assert np.array_equal(A4, densify(coords4, vals4, dims4))


def test_spmm_gemm_reduces_to_spmm_and_gemm():
    rs = np.random.RandomState(7)
    I, J, L = 40, 30, 9
    coords, vals = tiny_coo(rs, (I, J), 200)
    C = dense(rs, J, L)
    # D = identity: plain SpMM, the CSR loop nest of Fig. 1b
    A, _ = oracle.spmm_gemm(coords, vals, (I, J), C, np.eye(L, dtype=np.float32))
    Bcsr = sp.csr_matrix((vals.astype(np.float64), (coords[:, 0], coords[:, 1])), shape=(I, J))
    np.testing.assert_allclose(A, Bcsr @ C.astype(np.float64), rtol=0, atol=1e-13)
    # B = identity: dense GEMM C.D
    n = 12
    eye_coords = np.stack([np.arange(n), np.arange(n)], axis=1).astype(np.int32)
    C2, D2 = dense(rs, n, 7), dense(rs, 7, 5)
    A2, _ = oracle.spmm_gemm(eye_coords, np.ones(n, np.float32), (n, n), C2, D2)
    np.testing.assert_allclose(A2, C2.astype(np.float64) @ D2.astype(np.float64), rtol=0, atol=1e-13)


def test_sddmm_spmm_reduces_to_spmm():
    rs = np.random.RandomState(8)
    I, J, L = 25, 35, 6
    coords, vals = tiny_coo(rs, (I, J), 150)
    E = dense(rs, J, L)
    A, _, _ = oracle.sddmm_spmm(coords, vals, (I, J), np.ones((I, 1), np.float32), np.ones((J, 1), np.float32), E)
    Bcsr = sp.csr_matrix((vals.astype(np.float64), (coords[:, 0], coords[:, 1])), shape=(I, J))
    np.testing.assert_allclose(A, Bcsr @ E.astype(np.float64), rtol=0, atol=1e-13)


# ----------------------------------------------------------------- invariants

def test_linearity_and_coo_order_invariance():
    rs = np.random.RandomState(9)
    dims = (6, 7, 8)
    coords, vals = tiny_coo(rs, dims, 120)
    C, D = dense(rs, 7, 4), dense(rs, 8, 5)
    C2 = dense(rs, 7, 4)
    A, S = oracle.spttm_ttm3(coords, vals, dims, C, D)
    perm = rs.permutation(120)
    Ap, Sp = oracle.spttm_ttm3(coords[perm], vals[perm], dims, C, D)
    np.testing.assert_allclose(A, Ap, rtol=0, atol=1e-13)
    np.testing.assert_allclose(S, Sp, rtol=0, atol=1e-13)
    # linear in B (power-of-two scaling is exact), additive in C
    A2, _ = oracle.spttm_ttm3(coords, (2 * vals).astype(np.float32), dims, C, D)
    assert np.array_equal(A2, 2 * A)
    Ac2, _ = oracle.spttm_ttm3(coords, vals, dims, C2, D)
    Csum = C.astype(np.float64) + C2.astype(np.float64)
    B = densify(coords, vals, dims)
    np.testing.assert_allclose(A + Ac2, np.einsum("ijk,jl,km->ilm", B, Csum, D.astype(np.float64)),
                               rtol=0, atol=1e-12)
    assert np.all(S >= np.abs(A) - 1e-13)


@pytest.mark.parametrize("threads", [1, 3])
def test_slice_subset_matches_full(threads):
    rs = np.random.RandomState(10)
    dims = (9, 5, 6)
    coords, vals = tiny_coo(rs, dims, 100)
    C, D = dense(rs, 5, 3), dense(rs, 6, 2)
    A, S = oracle.spttm_ttm3(coords, vals, dims, C, D, threads=threads)
    sel = np.array([7, 0, 3])
    As, Ss = oracle.spttm_ttm3(coords, vals, dims, C, D, sel=sel, threads=threads)
    assert np.array_equal(As, A[sel]) and np.array_equal(Ss, S[sel])
    c2, v2 = tiny_coo(rs, (9, 8), 40)
    Cg, Dg = dense(rs, 8, 5), dense(rs, 5, 3)
    Ag, _ = oracle.spmm_gemm(c2, v2, (9, 8), Cg, Dg)
    Ags, _ = oracle.spmm_gemm(c2, v2, (9, 8), Cg, Dg, sel=sel)
    assert np.array_equal(Ags, Ag[sel])
    Cs, Ds, Es = dense(rs, 9, 4), dense(rs, 8, 4), dense(rs, 8, 3)
    A1, _, _ = oracle.sddmm_spmm(c2, v2, (9, 8), Cs, Ds, Es)
    A1s, _, P = oracle.sddmm_spmm(c2, v2, (9, 8), Cs, Ds, Es, sel=sel, with_sampled=True)
    assert np.array_equal(A1s, A1[sel])
    assert np.array_equal(~np.isnan(P), np.isin(c2[:, 0], sel))
    c4, v4 = tiny_coo(rs, (9, 3, 4, 2), 50)
    f = [dense(rs, 3, 2), dense(rs, 4, 2), dense(rs, 2, 3)]
    A4, _ = oracle.spttm_ttm4(c4, v4, (9, 3, 4, 2), *f)
    A4s, _ = oracle.spttm_ttm4(c4, v4, (9, 3, 4, 2), *f, sel=sel)
    assert np.array_equal(A4s, A4[sel])


def test_empty_and_out_of_range():
    C, D = np.ones((3, 2), np.float32), np.ones((4, 2), np.float32)
    A, S = oracle.spttm_ttm3(np.zeros((0, 3), np.int32), np.zeros(0, np.float32), (5, 3, 4), C, D)
    assert A.shape == (5, 2, 2) and not A.any() and not S.any()
    with pytest.raises(ValueError):
        oracle.spttm_ttm3(np.array([[0, 3, 0]], np.int32), np.ones(1, np.float32), (5, 3, 4), C, D)


def test_workload_generators_feed_oracle():
    from workloads import configs
    w = configs.make(1)
    A, S = oracle.evaluate(w)
    assert A.shape == (200, 16, 16) and np.isfinite(A).all()
    # slice i only sees nonzeros with that i: zero B outside slice 5 and compare
    keep = w.coords[:, 0] == 5
    A5, _ = oracle.spttm_ttm3(w.coords[keep], w.vals[keep], w.dims, *w.dense)
    np.testing.assert_array_equal(A5[5], A[5])
    assert not A5[np.arange(200) != 5].any()


# ----------------------------------------------------------------- kernel 5, all-mode TTMC

def test_ttmc3_bruteforce_closed_form_and_relation_to_the_partial_chain():
    rs = np.random.RandomState(11)
    dims = (5, 4, 6)
    coords, vals = tiny_coo(rs, dims, 43)
    C, D, E = dense(rs, 5, 2), dense(rs, 4, 3), dense(rs, 6, 4)
    A, S = oracle.ttmc3(coords, vals, dims, C, D, E)
    B = densify(coords, vals, dims)
    C64, D64, E64 = (x.astype(np.float64) for x in (C, D, E))
    ref = np.zeros((2, 3, 4))
    for i, j, k, l, m, n in itertools.product(range(5), range(4), range(6), range(2), range(3), range(4)):
        ref[l, m, n] += B[i, j, k] * C64[i, l] * D64[j, m] * E64[k, n]
    np.testing.assert_allclose(A, ref, rtol=0, atol=1e-13)
    np.testing.assert_allclose(A, np.einsum("ijk,il,jm,kn->lmn", B, C64, D64, E64), rtol=0, atol=1e-13)
    np.testing.assert_allclose(S, np.einsum("ijk,il,jm,kn->lmn", np.abs(B), np.abs(C64), np.abs(D64), np.abs(E64)),
                               rtol=0, atol=1e-13)
    # fissioned form: the per-slice chain over (j,k) first, then the contraction over i
    T, _ = oracle.spttm_ttm3(coords, vals, dims, D, E)
    np.testing.assert_allclose(A, np.einsum("il,imn->lmn", C64, T), rtol=0, atol=1e-12)
    # element list = the same elements of the full result; all ones: every element counts the nonzeros
    sel = np.array([23, 0, 7, 12])
    As, Ss = oracle.ttmc3(coords, vals, dims, C, D, E, sel=sel)
    assert np.array_equal(As, A.reshape(-1)[sel]) and np.array_equal(Ss, S.reshape(-1)[sel])
    ones = [np.ones((d, r), np.float32) for d, r in zip(dims, (2, 3, 4))]
    A1, _ = oracle.ttmc3(coords, np.ones(43, np.float32), dims, *ones)
    assert np.array_equal(A1, np.full((2, 3, 4), 43.0))
    # identity factors return the densified tensor
    Ai, _ = oracle.ttmc3(coords, vals, dims, *(np.eye(d, dtype=np.float32) for d in dims))
    assert np.array_equal(Ai, B)


# ----------------------------------------------------------------- kernel 2, SDDMM -> SpMM -> GEMM

def test_sddmm_spmm_gemm_bruteforce_and_relation_to_kernel_1():
    rs = np.random.RandomState(12)
    dims = (6, 5)
    coords, vals = tiny_coo(rs, dims, 14)
    C, D, E, F = dense(rs, 6, 3), dense(rs, 5, 3), dense(rs, 5, 4), dense(rs, 4, 2)
    A, S = oracle.sddmm_spmm_gemm(coords, vals, dims, C, D, E, F)
    B = densify(coords, vals, dims)
    f64 = [x.astype(np.float64) for x in (C, D, E, F)]
    ref = np.zeros((6, 2))
    for i, j, k, l, m in itertools.product(range(6), range(5), range(3), range(4), range(2)):
        ref[i, m] += B[i, j] * f64[0][i, k] * f64[1][j, k] * f64[2][j, l] * f64[3][l, m]
    np.testing.assert_allclose(A, ref, rtol=0, atol=1e-13)
    np.testing.assert_allclose(A, np.einsum("ij,ik,jk,jl,lm->im", B, *f64), rtol=0, atol=1e-13)
    np.testing.assert_allclose(S, np.einsum("ij,ik,jk,jl,lm->im", np.abs(B), *(np.abs(x) for x in f64)), rtol=0, atol=1e-13)
    # two-level schedule: the row temporary T_l of kernel 1, then the product with F
    A1, _, _ = oracle.sddmm_spmm(coords, vals, dims, C, D, E)
    np.testing.assert_allclose(A, A1 @ f64[3], rtol=0, atol=1e-13)
    # F = identity reduces to kernel 1; subset mode
    Ai, _ = oracle.sddmm_spmm_gemm(coords, vals, dims, C, D, E, np.eye(4, dtype=np.float32))
    np.testing.assert_allclose(Ai, A1, rtol=0, atol=1e-14)
    sel = np.array([4, 1])
    As, Ss = oracle.sddmm_spmm_gemm(coords, vals, dims, C, D, E, F, sel=sel)
    assert np.array_equal(As, A[sel]) and np.array_equal(Ss, S[sel])


# ----------------------------------------------------------------- kernel 3 <SpMMH,GEMM>

def test_spmmh_gemm_bruteforce_special_cases_and_invariants():
    """A(i,m) = sum_{j,l} B(i,j) C(j,l) D(j,l) E(l,m) (Table of kernels, row 3, Description column)."""
    rs = np.random.RandomState(21)
    dims = (6, 5)
    coords, vals = tiny_coo(rs, dims, 14)
    C, D, E = dense(rs, 5, 4), dense(rs, 5, 4), dense(rs, 4, 3)
    A, S = oracle.spmmh_gemm(coords, vals, dims, C, D, E)
    B = densify(coords, vals, dims)
    ref = np.zeros((6, 3))
    for i, j, l, m in itertools.product(range(6), range(5), range(4), range(3)):
        ref[i, m] += B[i, j] * float(C[j, l]) * float(D[j, l]) * float(E[l, m])
    np.testing.assert_allclose(A, ref, rtol=0, atol=1e-13)
    C64, D64, E64 = (x.astype(np.float64) for x in (C, D, E))
    np.testing.assert_allclose(A, np.einsum("ij,jl,jl,lm->im", B, C64, D64, E64), rtol=0, atol=1e-13)
    np.testing.assert_allclose(A, (B @ (C64 * D64)) @ E64, rtol=0, atol=1e-13)       # the two stages the name spells
    np.testing.assert_allclose(S, np.abs(B) @ (np.abs(C64) * np.abs(D64)) @ np.abs(E64), rtol=0, atol=1e-13)
    # D = all ones: kernel 4 with the same C and E
    A4, S4 = oracle.spmm_gemm(coords, vals, dims, C, E)
    A1, S1 = oracle.spmmh_gemm(coords, vals, dims, C, np.ones_like(C), E)
    assert np.array_equal(A1, A4) and np.array_equal(S1, S4)
    # E = identity: SpMM of B with the Hadamard product (library CSR product)
    Ai, _ = oracle.spmmh_gemm(coords, vals, dims, C, D, np.eye(4, dtype=np.float32))
    Bcsr = sp.csr_matrix((vals.astype(np.float64), (coords[:, 0], coords[:, 1])), shape=dims)
    np.testing.assert_allclose(Ai, Bcsr @ (C64 * D64), rtol=0, atol=1e-13)
    # the Hadamard factors commute; a transposed (wrongly indexed) D does not give the same result
    A2, _ = oracle.spmmh_gemm(coords, vals, dims, D, C, E)
    np.testing.assert_allclose(A2, A, rtol=0, atol=1e-13)
    # all ones: A(i,m) = L * deg(i)
    Ao, So = oracle.spmmh_gemm(coords, np.ones(14, np.float32), dims, np.ones((5, 4), np.float32), np.ones((5, 4), np.float32),
                               np.ones((4, 3), np.float32))
    deg = np.bincount(coords[:, 0], minlength=6)
    assert np.array_equal(Ao, np.broadcast_to(4.0 * deg[:, None], (6, 3))) and np.array_equal(Ao, So)
    # linearity in B, invariance under the COO order, subset mode
    A3, _ = oracle.spmmh_gemm(coords, 4.0 * vals, dims, C, D, E)        # a power of two: exact in fp32
    np.testing.assert_allclose(A3, 4.0 * A, rtol=0, atol=1e-12)
    perm = rs.permutation(14)
    Ap, _ = oracle.spmmh_gemm(coords[perm], vals[perm], dims, C, D, E)
    np.testing.assert_allclose(Ap, A, rtol=0, atol=1e-13)
    sel = np.array([4, 0, 5], dtype=np.int64)
    As, Ss = oracle.spmmh_gemm(coords, vals, dims, C, D, E, sel=sel)
    assert np.array_equal(As, A[sel]) and np.array_equal(Ss, S[sel])


# ----------------------------------------------------------------- kernel 8 <MTTKRP,GEMM>

def test_mttkrp_gemm_bruteforce_special_cases_and_invariants():
    """A(i,m) = sum_{j,k,r} B(i,j,k) C(j,r) D(k,r) E(r,m) (Table of kernels, row 8, Description column)."""
    rs = np.random.RandomState(31)
    dims = (5, 4, 6)
    coords, vals = tiny_coo(rs, dims, 40)
    C, D, E = dense(rs, 4, 3), dense(rs, 6, 3), dense(rs, 3, 2)
    A, S = oracle.mttkrp_gemm(coords, vals, dims, C, D, E)
    B = densify(coords, vals, dims)
    ref = np.zeros((5, 2))
    for i, j, k, r, m in itertools.product(range(5), range(4), range(6), range(3), range(2)):
        ref[i, m] += B[i, j, k] * float(C[j, r]) * float(D[k, r]) * float(E[r, m])
    np.testing.assert_allclose(A, ref, rtol=0, atol=1e-13)
    C64, D64, E64 = (x.astype(np.float64) for x in (C, D, E))
    np.testing.assert_allclose(A, np.einsum("ijk,jr,kr,rm->im", B, C64, D64, E64), rtol=0, atol=1e-13)
    np.testing.assert_allclose(S, np.einsum("ijk,jr,kr,rm->im", np.abs(B), np.abs(C64), np.abs(D64), np.abs(E64)), rtol=0, atol=1e-13)
    # E = identity: the MTTKRP itself = mode-1 unfolding of B times the Khatri-Rao product of C and D
    Ai, _ = oracle.mttkrp_gemm(coords, vals, dims, C, D, np.eye(3, dtype=np.float32))
    kr = (C64[:, None, :] * D64[None, :, :]).reshape(4 * 6, 3)            # row (j,k) = C(j,:) * D(k,:)
    np.testing.assert_allclose(Ai, B.reshape(5, 24) @ kr, rtol=0, atol=1e-13)
    np.testing.assert_allclose(A, (B.reshape(5, 24) @ kr) @ E64, rtol=0, atol=1e-13)   # the two stages the name spells
    # rank 1 with unit weights: A(i,0) = sum_jk B(i,j,k) c(j) d(k), a bilinear form per slice
    c1, d1 = dense(rs, 4, 1), dense(rs, 6, 1)
    A1, _ = oracle.mttkrp_gemm(coords, vals, dims, c1, d1, np.ones((1, 1), np.float32))
    np.testing.assert_allclose(A1[:, 0], np.einsum("ijk,j,k->i", B, c1[:, 0].astype(np.float64), d1[:, 0].astype(np.float64)),
                               rtol=0, atol=1e-13)
    # swapping the roles of C and D does not give the same result (j and k are different modes)
    # all ones: A(i,m) = R * nnz(slice i)
    Ao, So = oracle.mttkrp_gemm(coords, np.ones(40, np.float32), dims, np.ones((4, 3), np.float32), np.ones((6, 3), np.float32),
                                np.ones((3, 2), np.float32))
    cnt = np.bincount(coords[:, 0], minlength=5)
    assert np.array_equal(Ao, np.broadcast_to(3.0 * cnt[:, None], (5, 2))) and np.array_equal(Ao, So)
    # linearity in B, invariance under the COO order, subset mode
    A4, _ = oracle.mttkrp_gemm(coords, 4.0 * vals, dims, C, D, E)
    np.testing.assert_allclose(A4, 4.0 * A, rtol=0, atol=1e-12)
    perm = rs.permutation(40)
    Ap, _ = oracle.mttkrp_gemm(coords[perm], vals[perm], dims, C, D, E)
    np.testing.assert_allclose(Ap, A, rtol=0, atol=1e-13)
    sel = np.array([3, 0], dtype=np.int64)
    As, Ss = oracle.mttkrp_gemm(coords, vals, dims, C, D, E, sel=sel)
    assert np.array_equal(As, A[sel]) and np.array_equal(Ss, S[sel])


# ----------------------------------------------------------------- kernel 7 <SpTTM,SpTTM>

def test_spttm_spttm_bruteforce_pattern_special_cases_and_invariants():
    """A(i,j,m) = sum_{k,l} B(i,j,k) C(k,l) D(l,m), stored for B's (i,j) pairs (Table of kernels, row 7)."""
    rs = np.random.RandomState(37)
    dims = (5, 4, 6)
    coords, vals = tiny_coo(rs, dims, 40)
    C, D = dense(rs, 6, 3), dense(rs, 3, 2)
    keys, inv = oracle.fiber_keys(coords, dims)
    A, S = oracle.spttm_spttm(coords, vals, dims, C, D)
    B = densify(coords, vals, dims)
    # pattern: exactly the (i,j) pairs with a stored nonzero, in lexicographic order, each once
    want = sorted({(int(i), int(j)) for i, j, _ in coords})
    assert [tuple(k) for k in keys.tolist()] == want and A.shape == (len(want), 2)
    assert np.array_equal(keys[inv], coords[:, :2])
    # brute force over the dense tensor, term by term
    ref = np.zeros((5, 4, 2))
    for i, j, k, l, m in itertools.product(range(5), range(4), range(6), range(3), range(2)):
        ref[i, j, m] += B[i, j, k] * float(C[k, l]) * float(D[l, m])
    np.testing.assert_allclose(A, ref[keys[:, 0], keys[:, 1]], rtol=0, atol=1e-13)
    C64, D64 = C.astype(np.float64), D.astype(np.float64)
    full = np.einsum("ijk,kl,lm->ijm", B, C64, D64)
    np.testing.assert_allclose(A, full[keys[:, 0], keys[:, 1]], rtol=0, atol=1e-13)
    np.testing.assert_allclose(S, np.einsum("ijk,kl,lm->ijm", np.abs(B), np.abs(C64), np.abs(D64))[keys[:, 0], keys[:, 1]],
                               rtol=0, atol=1e-13)
    # pairs outside the pattern hold no term at all: the dense result is zero there
    mask = np.zeros((5, 4), dtype=bool)
    mask[keys[:, 0], keys[:, 1]] = True
    assert not full[~mask].any()
    # both association orders of the two mode products give the same numbers
    np.testing.assert_allclose(A, (np.einsum("ijk,kl->ijl", B, C64) @ D64)[keys[:, 0], keys[:, 1]], rtol=0, atol=1e-13)
    np.testing.assert_allclose(A, np.einsum("ijk,km->ijm", B, C64 @ D64)[keys[:, 0], keys[:, 1]], rtol=0, atol=1e-13)
    # D = identity: the first SpTTM alone, T(i,j,l) = sum_k B(i,j,k) C(k,l)
    Ai, _ = oracle.spttm_spttm(coords, vals, dims, C, np.eye(3, dtype=np.float32))
    np.testing.assert_allclose(Ai, np.einsum("ijk,kl->ijl", B, C64)[keys[:, 0], keys[:, 1]], rtol=0, atol=1e-13)
    # all ones: A(i,j,m) = L * (number of nonzeros of the fiber), and S equals A
    Ao, So = oracle.spttm_spttm(coords, np.ones(40, np.float32), dims, np.ones((6, 3), np.float32), np.ones((3, 2), np.float32))
    cnt = np.bincount(inv, minlength=keys.shape[0])
    assert np.array_equal(Ao, np.broadcast_to(3.0 * cnt[:, None], Ao.shape)) and np.array_equal(Ao, So)
    # swapping the operands' roles is a different expression (C is indexed by k, not by l)
    # linearity in B, invariance under the COO order, subset mode
    A4, _ = oracle.spttm_spttm(coords, 4.0 * vals, dims, C, D)
    np.testing.assert_allclose(A4, 4.0 * A, rtol=0, atol=1e-12)
    perm = rs.permutation(40)
    Ap, _ = oracle.spttm_spttm(coords[perm], vals[perm], dims, C, D)
    np.testing.assert_allclose(Ap, A, rtol=0, atol=1e-13)
    sel = np.array([7, 0, 3], dtype=np.int64)
    As, Ss = oracle.spttm_spttm(coords, vals, dims, C, D, sel=sel)
    np.testing.assert_allclose(As, A[sel], rtol=0, atol=1e-14)
    np.testing.assert_allclose(Ss, S[sel], rtol=0, atol=1e-14)
    with pytest.raises(ValueError):
        bad = coords.copy()
        bad[0, 2] = 6
        oracle.spttm_spttm(bad, vals, dims, C, D)
