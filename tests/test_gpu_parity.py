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


@pytest.mark.parametrize("sched", ["fused", "fissioned", "default"])
def test_ttm4_mini_every_schedule(sa, sched):
    """Order-4 chain: temporaries on chip (fused), through the workspace (fissioned), and the default, which is the
    fissioned schedule until a cap on auxiliary memory rules it out."""
    w = configs.make(5, "mini")
    A_ref, S_ref = oracle.evaluate(w)
    s = {"fused": sa.SA_SCHED_FUSED, "fissioned": sa.SA_SCHED_FISSIONED, "default": sa.SA_SCHED_DEFAULT}[sched]
    A, t = run_gpu(sa, w, sched=s)
    assert_close(A, A_ref, S_ref, TOL_FP32, w.name + "/" + sched)
    ops = [(16, d.shape[0], d.shape[1], d.shape[1]) for d in w.dense]
    E4 = sa.SA_EXPR_SPTTM_TTM4
    fus, fis = (sa.sa_schedule_cost(t.handle, E4, x, ops) for x in (sa.SA_SCHED_FUSED, sa.SA_SCHED_FISSIONED))
    n_sub = int(t.info()[1][1])
    assert fis["workspace_bytes"] >= n_sub * 1024 > fus["workspace_bytes"]
    assert fis["moved_bytes"] == fus["moved_bytes"] + 8 * n_sub * 256 and fis["iterations"] == fus["iterations"]
    assert sa.sa_schedule_cost(t.handle, E4, sa.SA_SCHED_DEFAULT, ops)["resolved"] == sa.SA_SCHED_FISSIONED
    if sched == "default":
        sa.sa_tensor_set_aux_limit(t.handle, n_sub * 1024 - 1)
        assert sa.sa_schedule_cost(t.handle, E4, sa.SA_SCHED_DEFAULT, ops)["resolved"] == sa.SA_SCHED_FUSED
        A2, _ = run_gpu(sa, w, sched=s, tensor=t)          # now the fused kernel runs
        assert_close(A2, A_ref, S_ref, TOL_FP32, w.name + "/default under a cap")


@pytest.mark.parametrize("ranks", [(16, 16, 16), (32, 16, 16), (16, 32, 16), (16, 16, 32), (32, 32, 16)])
def test_ttmc3_both_schedules(sa, ranks):
    """Kernel 5 with the loop over i fused (block accumulators in shared memory) and fissioned (slice temporaries in
    the workspace); the fused one exists while L M N <= 8192.  The tensor has slices split over several thread
    blocks, whose chunks the fused schedule adds without a fix-up pass."""
    L, M, N = ranks
    w = configs.make_ttmc3_zipf("ttmc3-%d-%d-%d" % ranks, 77, 300, 200, 250, 60_000, 1.2, 8.0, L, M, N)
    A_ref, S_ref = oracle.evaluate(w)
    A, t = run_gpu(sa, w, sched=sa.SA_SCHED_FISSIONED)
    assert_close(A, A_ref, S_ref, TOL_FP32, w.name + "/fissioned")
    A2, _ = run_gpu(sa, w, sched=sa.SA_SCHED_FISSIONED, tensor=t)
    assert np.array_equal(A, A2), "the fissioned schedule is bitwise reproducible"
    ops = [(16, d.shape[0], d.shape[1], d.shape[1]) for d in w.dense]
    if L * M * N <= 8192:
        A, _ = run_gpu(sa, w, sched=sa.SA_SCHED_FUSED, tensor=t)
        assert_close(A, A_ref, S_ref, TOL_FP32, w.name + "/fused")
        c = sa.sa_schedule_cost(t.handle, sa.SA_EXPR_TTMC3, sa.SA_SCHED_FUSED, ops)
        assert c["resolved"] == sa.SA_SCHED_FUSED and c["temp_elements"] == N + M * N
        # the default is the fissioned schedule until its I x M x N temporary is above the caller's cap
        assert sa.sa_schedule_cost(t.handle, sa.SA_EXPR_TTMC3, sa.SA_SCHED_DEFAULT, ops)["resolved"] == sa.SA_SCHED_FISSIONED
        sa.sa_tensor_set_aux_limit(t.handle, 300 * M * N * 4 - 1)
        assert sa.sa_schedule_cost(t.handle, sa.SA_EXPR_TTMC3, sa.SA_SCHED_DEFAULT, ops)["resolved"] == sa.SA_SCHED_FISSIONED, \
            "neither fits: stay with the default"
        sa.sa_tensor_set_aux_limit(t.handle, 2**62)
    else:
        with pytest.raises(sa.SaError) as e:
            sa.sa_workspace_size(t.handle, sa.SA_EXPR_TTMC3, sa.SA_SCHED_FUSED, ops)
        assert e.value.status == sa.SA_E_UNSUPPORTED
        assert sa.sa_schedule_cost(t.handle, sa.SA_EXPR_TTMC3, sa.SA_SCHED_DEFAULT, ops)["resolved"] == sa.SA_SCHED_FISSIONED


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
