"""The paper's scheduled loop nests on the CPU (oracle/nests.c) against the unfused definition (oracle/oracle.c).

Section 4 of the paper: fission and fusion change the loop structure and the temporaries, not the result.  The two
evaluations share nothing but the inputs: one walks the COO list with one perfectly nested loop per nonzero, the
other walks compressed storage it builds itself (numpy sort, run boundaries) with the branched nests of the Table of
kernels and their temporaries.  Agreement to rounding pins each of them by the other; the storage builder is checked
against scipy and against a brute-force description of the format (Section 2.1)."""
import numpy as np
import pytest
import scipy.sparse as sp

import oracle
from oracle import nests
from workloads import configs


def _close(A, A_ref, S, what):
    assert A.shape == A_ref.shape
    assert not A[S == 0].any(), what + ": element without terms is not zero"
    assert (np.abs(A - A_ref) <= 1e-12 * S).all(), what


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5, 6, 7, 8, 9, 10])
def test_nests_agree_with_the_definition_on_the_mini_configurations(cfg):
    w = configs.make(cfg, "mini")
    A_ref, S = oracle.evaluate(w)
    for order in (("left", "right") if w.expr == "spmm_gemm" else ("left",)):
        _close(nests.evaluate(w, order=order), A_ref, S, "%s/%s" % (w.name, order))
    # the thread count does not matter (every i owns its rows; kernel 5 adds per-thread copies)
    A1 = nests.evaluate(w, threads=1)
    _close(A1, A_ref, S, w.name + " single thread")


def test_nests_on_random_small_tensors_with_empty_slices_and_single_entries():
    rs = np.random.RandomState(5)
    for case in range(12):
        I, J, K, O = (int(rs.randint(1, 9)) for _ in range(4))
        L, M, N = (int(rs.randint(1, 5)) for _ in range(3))
        dense = rs.rand(I, J, K, O) < rs.choice([0.05, 0.3, 0.9])
        coords = np.argwhere(dense).astype(np.int32)
        rs.shuffle(coords)
        vals = rs.uniform(-1, 1, coords.shape[0]).astype(np.float32)
        C, D, E = (rs.uniform(-1, 1, s).astype(np.float32) for s in ((J, L), (K, M), (O, N)))
        levels, v = nests.csf_from_coo(coords, vals)
        A = nests.spttm_ttm4(levels, v, I, C, D, E)
        B = np.zeros((I, J, K, O))
        B[tuple(coords.T)] = vals
        ref = np.einsum("ijko,jl,km,on->ilmn", B, C.astype(np.float64), D.astype(np.float64), E.astype(np.float64))
        assert np.allclose(A, ref, rtol=0, atol=1e-12), case
        # order 3 on the (i,j,k) projection with summed duplicates removed: take o = 0 only
        c3 = coords[coords[:, 3] == 0][:, :3]
        v3 = vals[coords[:, 3] == 0]
        lv3, vv3 = nests.csf_from_coo(c3, v3)
        A3 = nests.spttm_ttm3(lv3, vv3, I, C, D)
        ref3 = np.einsum("ijk,jl,km->ilm", B[:, :, :, 0], C.astype(np.float64), D.astype(np.float64))
        assert np.allclose(A3, ref3, rtol=0, atol=1e-12), case
        # kernel 5 with all-ones D (J x M) and E (K x 1): A(l,m,0) = sum_i C(i,l) * (sum of slice i's values)
        Ci = rs.uniform(-1, 1, (I, L)).astype(np.float32)
        A5 = nests.ttmc3(lv3, vv3, Ci, np.ones((J, M), np.float32), np.ones((K, 1), np.float32))
        vsum_i = B[:, :, :, 0].sum(axis=(1, 2))
        assert np.allclose(A5[:, :, 0], (Ci.astype(np.float64).T @ vsum_i)[:, None] * np.ones((1, M)), atol=1e-12), case


def test_compressed_storage_matches_the_format_description_and_scipy():
    rs = np.random.RandomState(11)
    # matrix: rows dense, columns compressed, sorted
    I, J = 40, 30
    dense = rs.rand(I, J) < 0.2
    coords = np.argwhere(dense).astype(np.int32)
    rs.shuffle(coords)
    vals = rs.uniform(-1, 1, coords.shape[0]).astype(np.float32)
    pos, crd, v = nests.csr_from_coo(coords, vals, I)
    ref = sp.csr_matrix((vals, (coords[:, 0], coords[:, 1])), shape=(I, J))
    ref.sort_indices()
    assert np.array_equal(pos, ref.indptr) and np.array_equal(crd, ref.indices) and np.array_equal(v, ref.data)
    # order-3 tensor: level 0 lists the non-empty slices, level d + 1 the distinct children of every level-d node
    dims = (7, 6, 5)
    dense = rs.rand(*dims) < 0.25
    dense[3] = False                                            # an empty slice
    coords = np.argwhere(dense).astype(np.int32)
    rs.shuffle(coords)
    vals = rs.uniform(-1, 1, coords.shape[0]).astype(np.float32)
    (p0, c0), (p1, c1), (p2, c2) = nests.csf_from_coo(coords, vals)[0]
    assert p0 is None and c0.tolist() == [i for i in range(dims[0]) if dense[i].any()]
    f = 0
    for s, i in enumerate(c0):
        js = [j for j in range(dims[1]) if dense[i, j].any()]
        assert c1[p1[s]:p1[s + 1]].tolist() == js
        for j in js:
            assert c2[p2[f]:p2[f + 1]].tolist() == [k for k in range(dims[2]) if dense[i, j, k]]
            f += 1
    assert f == c1.shape[0] and p2[-1] == coords.shape[0]
    # empty input
    lv, v = nests.csf_from_coo(np.zeros((0, 3), dtype=np.int32), np.zeros(0, dtype=np.float32))
    assert all(c.shape[0] == 0 for _, c in lv) and lv[1][0].tolist() == [0] and v.shape[0] == 0
    assert not nests.spttm_ttm3(lv, v, 4, np.ones((6, 2), np.float32), np.ones((5, 3), np.float32)).any()
