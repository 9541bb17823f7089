"""The cost side: iteration complexities, auxiliary memory and the run-time choice between schedules.

The paper prints no contraction output, but it does print cost figures: the iteration complexity of five
schedules of kernel 5 (captions of the figure with the five loop nests, Section 3), ratios between them for four
concrete sets of loop bounds (the four cases of Section 3) and sizes of temporaries (Case 2; the table of
auxiliary memory in the comparison with SpTTN-Cyclops; the table of auxiliary memory requirements per kernel).
A small evaluator of branched loop nests, written here, is pinned against those printed figures and then tells
what the library's own nests must cost, which is compared with what sa_schedule_cost reports."""
import os

import numpy as np
import pytest

import paper_2311_09549_b200 as sa
from workloads import configs

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "paper_cost_figures.txt")


def golden(kind):
    """Records of one kind from the file of figures the paper prints (fields split at '|', stripped)."""
    out = []
    with open(GOLDEN) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            fields = [x.strip() for x in line.split("|")]
            if fields[0] == kind:
                out.append(fields[1:])
    return out


def iterations(nest):
    """Iteration complexity of a branched loop nest: a nest is (extent, [children]); a leaf runs `extent` times,
    an inner node runs its children, one after the other, `extent` times (footnote on iteration complexity,
    Section 3).  Loops over a sparse operand are given as one loop over its stored entries."""
    extent, children = nest
    return extent * (sum(iterations(c) for c in children) if children else 1)


def fig2(I, J, K, L, M, N, nnz):
    """The five schedules of the figure with the loop nests of kernel 5, written as nests from its listings."""
    return {
        "a": (L * M * N, [(nnz, [])]),                                          # one perfectly nested loop
        "b": (L * M, [(nnz, []), (N * K, [])]),                                 # T(k)
        "c": (L, [(nnz, []), (J * M * K * N, [])]),                             # T(k,j), one consumer nest
        "d": (L, [(nnz, []), (M * K, [(J, []), (N, [])])]),                     # T(k,j) and a scalar: two levels
        "e": (L, [(nnz, []), (J * M * K, []), (M * K * N, [])]),                # T(k,j) and T(m,k)
    }


def test_nest_evaluator_reproduces_the_printed_complexity_formulas():
    # captions of the figure: LMN nnz | LM (nnz + NK) | L (nnz + JMKN) | L (nnz + MK (J + N)) twice
    I, J, K, L, M, N, nnz = 7, 11, 13, 3, 5, 2, 101
    f = {k: iterations(v) for k, v in fig2(I, J, K, L, M, N, nnz).items()}
    assert f["a"] == L * M * N * nnz
    assert f["b"] == L * M * (nnz + N * K)
    assert f["c"] == L * (nnz + J * M * K * N)
    assert f["d"] == L * (nnz + M * K * (J + N)) == f["e"]


def test_nest_evaluator_reproduces_the_printed_ratios_of_the_four_cases():
    """Section 3, Cases 1, 2 and 4, from tests/golden/paper_cost_figures.txt (which also states the two readings:
    a tenth of the sparsities printed for Cases 1 and 2, and the exchanged ratio labels of Case 4)."""
    cases = golden("case")
    assert len(cases) == 3
    for name, bounds, _printed, sparsity, *ratios in cases:
        I, J, K, L, M, N = (int(x) for x in bounds.split())
        f = {k: iterations(v) for k, v in fig2(I, J, K, L, M, N, float(sparsity) * I * J * K).items()}
        for r in ratios:
            lhs, value = (x.strip() for x in r.split("="))
            num, den = lhs.split("/")
            assert f[num] / f[den] == pytest.approx(float(value), rel=4e-2), (name, r, f[num] / f[den])
    # the printed sparsities of Cases 1 and 2 do not give the printed ratios (which is why they are not taken)
    name, bounds, printed, *_ = cases[0]
    I, J, K, L, M, N = (int(x) for x in bounds.split())
    f = {k: iterations(v) for k, v in fig2(I, J, K, L, M, N, float(printed) * I * J * K).items()}
    assert abs(f["a"] / f["d"] - 237.5) > 50
    # the temporary T(k,j) of the two-level schedule (4-byte elements)
    for K, J, mb in (x[0].split() for x in golden("temp_mb")):
        assert int(K) * int(J) * 4 / 2**20 == pytest.approx(float(mb), abs=0.005)


def _host_tensor(w):
    return sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSR if w.fmt == "csr" else sa.SA_FMT_CSF, device=-1)


def _ops(w):
    return [(16, d.shape[0], d.shape[1], d.shape[1]) for d in w.dense]


def test_library_iteration_counts_are_those_of_its_nests():
    """sa_schedule_cost.iterations against the evaluator applied to the nests the kernels run (headers of the
    kernel sources; Table of kernels, Section 6, with the scalar temporaries widened to vectors)."""
    # kernel 4, both association orders
    w = configs.make(4, "mini")
    t = _host_tensor(w)
    I, J = w.dims
    L, M = w.dense[0].shape[1], w.dense[1].shape[1]
    nnz = w.nnz
    left = sa.sa_schedule_cost(t.handle, sa.SA_EXPR_SPMM_GEMM, sa.SA_SCHED_ASSOC_LEFT, _ops(w))
    right = sa.sa_schedule_cost(t.handle, sa.SA_EXPR_SPMM_GEMM, sa.SA_SCHED_ASSOC_RIGHT, _ops(w))
    # i < T(l) ; j', l : T += B C , m, l : A += T D >   with the loop over i unrolled into its total extents
    assert left["iterations"] == iterations((1, [(nnz * L, []), (I * L * M, [])]))
    # < E(j,m) ; j, l, m : E += C D , i, j', m : A += B E >
    assert right["iterations"] == iterations((1, [(J * L * M, []), (nnz * M, [])]))
    assert left["temp_elements"] == L and right["temp_elements"] == J * M
    assert right["workspace_bytes"] >= J * M * 4 > left["workspace_bytes"]
    # kernel 6 and the order-4 chain: fibers and subtrees come from the level counts
    w = configs.make(2, "mini")
    t = _host_tensor(w)
    _, counts, _ = t.info()
    L, M = w.dense[0].shape[1], w.dense[1].shape[1]
    c = sa.sa_schedule_cost(t.handle, sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_FUSED, _ops(w))
    assert c["iterations"] == iterations((1, [(w.nnz * M, []), (int(counts[1]) * L * M, [])])) and c["temp_elements"] == M
    w = configs.make(5, "mini")
    t = _host_tensor(w)
    _, counts, _ = t.info()
    c = sa.sa_schedule_cost(t.handle, sa.SA_EXPR_SPTTM_TTM4, sa.SA_SCHED_FUSED, _ops(w))
    assert c["iterations"] == w.nnz * 16 + int(counts[2]) * 256 + int(counts[1]) * 4096
    # the temporaries of the two-level nest are t(n) and T2(m,n): N + M N elements, the element count that the
    # paper's table of auxiliary memory (comparison with SpTTN-Cyclops) lists in bytes for 16 .. 128
    assert c["temp_elements"] == 16 + 16 * 16
    table = golden("aux_bytes")
    assert len(table) == 4
    for rank, own, cyclops in table:
        n = int(rank)
        assert (n + n * n) * 4 == int(cyclops)          # t(n) and T(m,n): this library's widened temporaries
        assert (1 + n) * 4 == int(own)                  # scalar + T(m): the paper's own schedule
    # kernels 1 and 2: scalar temporary, and scalar + row temporary (table of auxiliary memory requirements)
    printed = dict((k, v) for k, v in golden("aux_elements"))
    assert printed["kernel1"] == "1" and printed["kernel2"] == "1 to 1+L"
    w = configs.make(3, "mini")
    t = _host_tensor(w)
    assert sa.sa_schedule_cost(t.handle, sa.SA_EXPR_SDDMM_SPMM, sa.SA_SCHED_FUSED, _ops(w))["temp_elements"] == 1
    w = configs.make(7, "mini")
    t = _host_tensor(w)
    assert sa.sa_schedule_cost(t.handle, sa.SA_EXPR_SDDMM_SPMM_GEMM, sa.SA_SCHED_FUSED, _ops(w))["temp_elements"] == 1 + w.dense[2].shape[1]


def _csr(I, J, nnz, seed):
    rs = np.random.RandomState(seed)
    flat = np.unique(rs.randint(0, I * J, int(nnz * 1.2) + 16, dtype=np.int64))
    flat = rs.permutation(flat)[:nnz]
    assert flat.shape[0] == nnz
    coords = np.stack([flat // J, flat % J], axis=1).astype(np.int32)
    return sa.SparseTensor((I, J), coords, np.ones(nnz, np.float32), sa.SA_FMT_CSR, device=-1)


def test_default_schedule_takes_fewer_bytes_within_the_auxiliary_memory_cap():
    """Stage 4 of Section 5.2, recast: least moved bytes among the schedules whose workspace fits the cap."""
    E4 = sa.SA_EXPR_SPMM_GEMM
    L, M = 256, 64
    # few nonzeros, many columns: B.(C.D) would form C.D for 50 000 rows that are hardly used
    J = 50_000
    sparse = _csr(100, J, 500, 3)
    ops = [(16, J, L, L), (16, L, M, M)]
    c = {s: sa.sa_schedule_cost(sparse.handle, E4, s, ops) for s in (sa.SA_SCHED_DEFAULT, sa.SA_SCHED_ASSOC_LEFT, sa.SA_SCHED_ASSOC_RIGHT)}
    assert c[sa.SA_SCHED_ASSOC_LEFT]["moved_bytes"] < c[sa.SA_SCHED_ASSOC_RIGHT]["moved_bytes"]
    assert c[sa.SA_SCHED_DEFAULT]["resolved"] == sa.SA_SCHED_ASSOC_LEFT
    assert sa.sa_workspace_size(sparse.handle, E4, sa.SA_SCHED_DEFAULT, ops) == c[sa.SA_SCHED_ASSOC_LEFT]["workspace_bytes"]
    # many nonzeros per column: one gathered 1 KB row of C per nonzero costs more than reading C once to form E = C.D
    J = 400_000
    dense = _csr(2000, J, 1_500_000, 4)
    ops = [(16, J, L, L), (16, L, M, M)]
    c = {s: sa.sa_schedule_cost(dense.handle, E4, s, ops) for s in (sa.SA_SCHED_DEFAULT, sa.SA_SCHED_ASSOC_LEFT, sa.SA_SCHED_ASSOC_RIGHT)}
    nnz = 1_500_000
    assert c[sa.SA_SCHED_ASSOC_LEFT]["moved_bytes"] == pytest.approx(nnz * (8 + 4 * L) + 4 * 2001 + 4 * L * M + 4 * 2000 * M)
    assert c[sa.SA_SCHED_ASSOC_RIGHT]["moved_bytes"] < c[sa.SA_SCHED_ASSOC_LEFT]["moved_bytes"]
    assert c[sa.SA_SCHED_DEFAULT]["resolved"] == sa.SA_SCHED_ASSOC_RIGHT
    # ... unless its J x M temporary (102 MB) is above the caller's cap: then the order without it runs
    sa.sa_tensor_set_aux_limit(dense.handle, 64 << 20)
    capped = sa.sa_schedule_cost(dense.handle, E4, sa.SA_SCHED_DEFAULT, ops)
    assert capped["resolved"] == sa.SA_SCHED_ASSOC_LEFT and capped["workspace_bytes"] <= 64 << 20
    assert sa.sa_workspace_size(dense.handle, E4, sa.SA_SCHED_DEFAULT, ops) == capped["workspace_bytes"]
    # naming a schedule overrides the cap; lifting the cap restores the choice by bytes
    assert sa.sa_schedule_cost(dense.handle, E4, sa.SA_SCHED_ASSOC_RIGHT, ops)["resolved"] == sa.SA_SCHED_ASSOC_RIGHT
    sa.sa_tensor_set_aux_limit(dense.handle, 2**62)
    assert sa.sa_schedule_cost(dense.handle, E4, sa.SA_SCHED_DEFAULT, ops)["resolved"] == sa.SA_SCHED_ASSOC_RIGHT


def test_kernel5_default_is_fissioned_until_its_temporaries_exceed_the_cap():
    """Kernel 5: the fissioned schedule (slice temporaries I x M x N in the workspace) is the default; when the
    caller caps auxiliary memory below that, the schedule with the temporaries on chip runs instead (Stage 4's
    memory condition, Section 5.2; Stage 1 of the paper prunes temporaries of three dimensions altogether)."""
    rs = np.random.RandomState(9)
    I = 200_000
    coords = np.unique(np.stack([rs.randint(0, I, 5000), rs.randint(0, 50, 5000), rs.randint(0, 60, 5000)], axis=1), axis=0).astype(np.int32)
    t = sa.SparseTensor((I, 50, 60), coords, np.ones(len(coords), np.float32), sa.SA_FMT_CSF, device=-1)
    ops = [(16, I, 16, 16), (16, 50, 16, 16), (16, 60, 16, 16)]
    E5 = sa.SA_EXPR_TTMC3
    fis = sa.sa_schedule_cost(t.handle, E5, sa.SA_SCHED_FISSIONED, ops)
    fus = sa.sa_schedule_cost(t.handle, E5, sa.SA_SCHED_FUSED, ops)
    assert fis["workspace_bytes"] >= I * 256 * 4 > fus["workspace_bytes"]
    assert fis["temp_elements"] == 16 + I * 256 and fus["temp_elements"] == 16 + 256
    assert fis["iterations"] == fus["iterations"] and fis["moved_bytes"] == fus["moved_bytes"] + 8 * I * 256
    assert sa.sa_schedule_cost(t.handle, E5, sa.SA_SCHED_DEFAULT, ops)["resolved"] == sa.SA_SCHED_FISSIONED
    sa.sa_tensor_set_aux_limit(t.handle, 100 << 20)
    assert sa.sa_schedule_cost(t.handle, E5, sa.SA_SCHED_DEFAULT, ops)["resolved"] == sa.SA_SCHED_FUSED
    assert sa.sa_workspace_size(t.handle, E5, sa.SA_SCHED_DEFAULT, ops) == fus["workspace_bytes"]
