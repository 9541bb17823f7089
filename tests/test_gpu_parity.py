"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same
seeded inputs, element by element."""
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


@pytest.mark.parametrize("cfg", [1, 2, 5, 6])
def test_ttm_chains_mini(sa, cfg):
    w = configs.make(cfg, "mini")
    A_ref, S_ref = oracle.evaluate(w)
    A, _ = run_gpu(sa, w)
    assert_close(A, A_ref, S_ref, TOL_FP32, w.name)


@pytest.mark.parametrize("cfg", [3, 7])
def test_sddmm_spmm_mini(sa, cfg):
    w = configs.make(cfg, "mini")
    A_ref, S_ref = oracle.evaluate(w)
    A, _ = run_gpu(sa, w)
    assert_close(A, A_ref, S_ref, TOL_FP32, w.name)


@pytest.mark.parametrize("sched", ["left", "right", "default"])
def test_spmm_gemm_mini_both_orders(sa, sched):
    w = configs.make(4, "mini")
    A_ref, S_ref = oracle.evaluate(w)
    s = {"left": sa.SA_SCHED_ASSOC_LEFT, "right": sa.SA_SCHED_ASSOC_RIGHT, "default": sa.SA_SCHED_DEFAULT}[sched]
    A, _ = run_gpu(sa, w, sched=s)
    assert_close(A, A_ref, S_ref, TOL_FP32, w.name + "/" + sched)


def test_spmmh_gemm_mini(sa):
    w = configs.make(8, "mini")
    A_ref, S_ref = oracle.evaluate(w)
    A, _ = run_gpu(sa, w)
    assert_close(A, A_ref, S_ref, TOL_FP32, w.name)


def test_mttkrp_gemm_mini(sa):
    w = configs.make(9, "mini")
    A_ref, S_ref = oracle.evaluate(w)
    A, _ = run_gpu(sa, w)
    assert_close(A, A_ref, S_ref, TOL_FP32, w.name)


@pytest.mark.parametrize("sched", ["left", "right", "default"])
def test_spttm_spttm_mini_both_orders_and_pattern(sa, sched):
    """Kernel 7: values against the oracle, the output's index structure bit-exact against the (i,j) pairs of B."""
    w = configs.make(10, "mini")
    A_ref, S_ref = oracle.evaluate(w)
    keys, _ = oracle.fiber_keys(w.coords, w.dims)
    s = {"left": sa.SA_SCHED_ASSOC_LEFT, "right": sa.SA_SCHED_ASSOC_RIGHT, "default": sa.SA_SCHED_DEFAULT}[sched]
    A, t = run_gpu(sa, w, sched=s)
    assert_close(A, A_ref, S_ref, TOL_FP32, w.name + "/" + sched)
    nnz, counts, _ = t.info()
    pos0, crd0, _ = sa.sa_tensor_export(t.handle, 0, n_pos=2, n_crd=int(counts[0]))
    pos1, crd1, _ = sa.sa_tensor_export(t.handle, 1, n_pos=int(counts[0]) + 1, n_crd=int(counts[1]))
    i_of_fiber = np.repeat(crd0.astype(np.int64), np.diff(pos1))
    assert np.array_equal(np.stack([i_of_fiber, crd1.astype(np.int64)], axis=1), keys)
