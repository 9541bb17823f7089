"""The allocation-free entry point (sa_run_ttm3_static_scratch) against the oracle and the regular sa_run.

It exists for callers that cannot get device memory at call time (fixed memory plans, plug-ins
whose host owns allocation, loops that must not touch cudaMalloc) and therefore cannot pass a
workspace: the partial tiles of split slices go to a 4 MiB array inside the library.  The array
is shared by all calls and keeps old contents, so the check is repeated on two calls in a row,
the second one after a different tensor has used the same scratch.
"""
import numpy as np
import pytest

import oracle
from workloads import configs
from util import TOL_FP32, assert_close

pytestmark = pytest.mark.gpu


def _run_both(sa, torch, w):
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSF, device=0)
    ops_t = [torch.from_numpy(np.ascontiguousarray(x)).cuda() for x in w.dense]
    ops = [(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0)) for x in ops_t]
    ref, _ = t.run(w.expr, ops_t)
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream().cuda_stream

    def static_call(check_memory=False, _keep=ops_t):     # the operand tensors must outlive the raw pointers in `ops`
        out = torch.full(w.out_shape, float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        before = (torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
        sa.sa_run_ttm3_static_scratch(t.handle, ops, out.data_ptr(), stream)
        torch.cuda.synchronize()
        after = (torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
        if check_memory:
            # neither the driver's free memory nor torch's allocator moved: the call obtained no device memory
            assert after == before, (before, after)
        return out.cpu().numpy().astype(np.float64)

    return t, ref.cpu().numpy().astype(np.float64), static_call


def test_static_scratch_matches_sa_run_on_two_calls_in_a_row():
    import torch
    assert torch.cuda.is_available()
    import paper_2311_09549_b200 as sa
    w = configs.make(2, "mini")                       # has slices split over several thread blocks
    t, ref, static_call = _run_both(sa, torch, w)
    assert sa.sa_tensor_worklist(t.handle)[0][3] > 0, "the case must really use partial-tile slots"
    A_ref, S = oracle.evaluate(w)
    first = static_call()                             # the first call on a device also looks up the scratch's address
    assert_close(first, A_ref, S, TOL_FP32, "static scratch against the oracle, first call")
    assert_close(first, ref, S, TOL_FP32, "static scratch against sa_run, first call")
    # another tensor overwrites the shared scratch in between
    w5 = configs.make_ttm3_zipf("other", 99, 400, 300, 300, 120_000, 1.2, 8.0, 32, 32)
    t5, ref5, static_call5 = _run_both(sa, torch, w5)
    A5, S5 = oracle.evaluate(w5)
    assert_close(static_call5(check_memory=True), A5, S5, TOL_FP32, "static scratch against the oracle, other tensor")
    second = static_call(check_memory=True)
    assert_close(second, A_ref, S, TOL_FP32, "static scratch against the oracle, second call")
    assert_close(second, ref, S, TOL_FP32, "static scratch against sa_run, second call")
    assert np.array_equal(first, second)


def test_static_scratch_rejects_what_does_not_fit():
    import torch
    import paper_2311_09549_b200 as sa
    # 520 slices of 9000 nonzeros: each is cut into two chunks -> 1040 partial tiles of 4 KiB > 4 MiB
    n_slices, per = 520, 9000
    idx = np.arange(per)
    i = np.repeat(np.arange(n_slices), per)
    coords = np.stack([i, np.tile(idx // 100, n_slices), np.tile(idx % 100, n_slices)], axis=1).astype(np.int32)
    vals = np.ones(coords.shape[0], dtype=np.float32)
    t = sa.SparseTensor((n_slices, 90, 100), coords, vals, sa.SA_FMT_CSF, device=0)
    C = torch.ones(90, 32, device="cuda")
    D = torch.ones(100, 32, device="cuda")
    ops = [(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0)) for x in (C, D)]
    assert sa.sa_workspace_size(t.handle, sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_DEFAULT, ops) > 4 << 20
    out = torch.zeros(n_slices, 32, 32, device="cuda")
    with pytest.raises(sa.SaError) as e:
        sa.sa_run_ttm3_static_scratch(t.handle, ops, out.data_ptr(), torch.cuda.current_stream().cuda_stream)
    assert e.value.status == sa.SA_E_WORKSPACE
    torch.cuda.synchronize()
    assert not out.any(), "a rejected call enqueues nothing"
    # the regular entry point handles the same tensor
    ref, _ = t.run("spttm_ttm3", [C, D])
    torch.cuda.synchronize()
    assert float(ref.min()) == float(ref.max()) == float(per)
