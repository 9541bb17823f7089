"""Randomised parity sweep: many small seeded tensors of varying shape, skew and fiber length per chain, each
compared with the oracle element by element.  The shapes are drawn from a fixed seed, so every run tests the same
cases; they are chosen to move the boundaries the kernels care about (round and tile tails, slices split over
several blocks or fitting one warp, subtrees on both sides of the small/large limit, empty slices and rows)."""
import numpy as np
import pytest

import oracle
from workloads import configs
from util import TOL_FP32, TOL_TF32, assert_close, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sa():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    import paper_2311_09549_b200 as sa
    return sa


def _rs(family, case):
    return np.random.RandomState(1000 * family + case)


def _pick(rs, lo, hi):
    return int(rs.randint(lo, hi + 1))


def _one(rs, values):
    return values[int(rs.randint(len(values)))]


@pytest.mark.parametrize("case", range(12))
def test_order3_chain_random_shapes(sa, case):
    rs = _rs(1, case)
    I, J, K = _pick(rs, 3, 600), _pick(rs, 40, 700), _pick(rs, 17, 900)
    mean_fiber = _one(rs, [1.0, 2.0, 5.0, 12.0, 40.0])
    nnz = min(_pick(rs, 1, 90_000), J * K // 4)
    alpha = _one(rs, [0.0, 0.8, 1.2, 1.6])
    L, M = _one(rs, [(16, 16), (16, 32), (32, 16), (32, 32)])
    w = configs.make_ttm3_zipf("random3-%d" % case, 4000 + case, I, J, K, nnz, alpha, mean_fiber, L, M)
    A_ref, S = oracle.evaluate(w)
    A, t = run_gpu(sa, w)
    assert_close(A, A_ref, S, TOL_FP32, w.name)
    # kernel 8's first stage and kernel 5 share the producer: same tensor through kernel 5, both schedules
    if case % 3 == 0:
        w5 = configs.make_ttmc3_zipf("random5-%d" % case, 4000 + case, I, J, K, nnz, alpha, mean_fiber, 16, 16, M)
        A5_ref, S5 = oracle.evaluate(w5)
        for sched in (sa.SA_SCHED_FISSIONED, sa.SA_SCHED_FUSED):
            A5, _ = run_gpu(sa, w5, sched=sched)
            assert_close(A5, A5_ref, S5, TOL_FP32, "%s/%d" % (w5.name, sched))


@pytest.mark.parametrize("case", range(8))
def test_order4_chain_random_shapes(sa, case):
    rs = _rs(2, case)
    I, J, K, O = _pick(rs, 2, 300), _pick(rs, 30, 300), _pick(rs, 20, 200), _pick(rs, 16, 400)
    mean_fiber = _one(rs, [1.5, 3.0, 6.0, 14.0])
    nnz = min(_pick(rs, 1, 120_000), J * K * O // 8)
    alpha = _one(rs, [0.0, 1.0, 1.4, 2.0])              # alpha 2 puts most nonzeros into one slice: large subtrees
    w = configs.make_ttm4_zipf("random4-%d" % case, 5000 + case, I, J, K, O, nnz, alpha, mean_fiber, 16, 16, 16)
    A_ref, S = oracle.evaluate(w)
    for sched in (sa.SA_SCHED_FISSIONED, sa.SA_SCHED_FUSED):
        A, _ = run_gpu(sa, w, sched=sched)
        assert_close(A, A_ref, S, TOL_FP32, "%s/%d" % (w.name, sched))


@pytest.mark.parametrize("case", range(8))
def test_sddmm_spmm_random_shapes(sa, case):
    rs = _rs(3, case)
    I, J = _pick(rs, 1, 5000), _pick(rs, 64, 6000)
    nnz = min(_pick(rs, 1, 150_000), I * min(J, 3000) // 2)
    alpha = _one(rs, [0.0, 0.6, 1.1])
    cap = _one(rs, [8, 200, 3000])
    nnz = max(1, min(nnz, I * min(cap, J)))
    K, L = _one(rs, [32, 64, 128]), _one(rs, [32, 64, 128])
    w = configs.make_sddmm_spmm("random-sddmm-%d" % case, 6000 + case, I, J, nnz, alpha, cap, K, L)
    A_ref, S = oracle.evaluate(w)
    A, _ = run_gpu(sa, w)
    assert_close(A, A_ref, S, TOL_FP32, w.name)


@pytest.mark.parametrize("case", range(8))
def test_spmm_gemm_random_shapes(sa, case):
    rs = _rs(4, case)
    I, J = _pick(rs, 1, 6000), _pick(rs, 32, 5000)
    nnz = min(_pick(rs, 1, 120_000), I * J // 4 + 1)
    L, M = _one(rs, [128, 256]), _one(rs, [32, 64])
    w = configs.make_spmm_gemm("random-spmm-gemm-%d" % case, 7000 + case, I, J, nnz, L, M)
    A_ref, S = oracle.evaluate(w)
    for sched in (sa.SA_SCHED_ASSOC_LEFT, sa.SA_SCHED_ASSOC_RIGHT):
        A, _ = run_gpu(sa, w, sched=sched)
        # both orders contain a tensor-core stage over split operands (error about 2^-20 per product)
        assert_close(A, A_ref, S, TOL_FP32, "%s/%d" % (w.name, sched))
