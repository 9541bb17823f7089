"""Full-size parity: the benchmark configurations, run exactly as bench.py runs them (same
builder, same launch configuration), checked on sampled output slices / rows that the oracle
evaluates one by one in its subset mode."""
import numpy as np
import pytest

import oracle
from workloads import configs
from util import TOL_FP32, assert_close, fmt_of

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sa():
    import torch
    assert torch.cuda.is_available()
    import paper_2311_09549_b200 as sa
    return sa


def _sample(w, max_nnz, n_random):
    """The largest slice/row with at most max_nnz nonzeros, the smallest non-empty one, an empty
    one if any, and n_random seeded others."""
    I = w.dims[0]
    counts = np.bincount(w.coords[:, 0], minlength=I)
    ok = np.nonzero(counts <= max_nnz)[0]
    picks = [int(ok[np.argmax(counts[ok])])]
    nz = np.nonzero(counts > 0)[0]
    picks.append(int(nz[np.argmin(counts[nz])]))
    empty = np.nonzero(counts == 0)[0]
    if empty.size:
        picks.append(int(empty[0]))
    rnd = configs.rng.permutation(w.seed, 55, I)
    rnd = rnd[counts[rnd] <= max_nnz][:n_random]
    return np.unique(np.concatenate([np.array(picks, dtype=np.int64), rnd]))


def _run_full(sa, w, sched=None):
    import torch
    t = sa.SparseTensor(w.dims, w.coords, w.vals, fmt_of(sa, w), device=0)
    ops = [torch.from_numpy(x).cuda() for x in w.dense]
    out, _ = t.run(w.expr, ops, sched=sa.SA_SCHED_DEFAULT if sched is None else sched)
    torch.cuda.synchronize()
    assert sa.sa_last_device_status(t.handle, torch.cuda.current_stream().cuda_stream) == sa.SA_OK
    return out, t


def _compare(out, w, sel, what):
    import torch
    A_ref, S_ref = oracle.evaluate(w, sel=sel)
    got = out[torch.from_numpy(sel).cuda()].cpu().numpy().astype(np.float64)
    return assert_close(got, A_ref, S_ref, TOL_FP32, what)


def _compare_head_slice(out, w, what, parts=16):
    """The slice with the most nonzeros, which the sample above leaves out because the oracle evaluates a slice on
    one thread: its nonzeros are dealt to ``parts`` pseudo-slices (the contraction is linear in B, and so is the sum
    of absolute terms), the oracle evaluates those in parallel, and the sums are compared with the GPU's slice."""
    counts = np.bincount(w.coords[:, 0], minlength=w.dims[0])
    top = int(np.argmax(counts))
    rows = np.nonzero(w.coords[:, 0] == top)[0]
    coords = np.ascontiguousarray(w.coords[rows])
    coords[:, 0] = np.arange(rows.shape[0]) % parts
    sub = configs.Workload(w.name + "-head", w.expr, w.fmt, (parts,) + tuple(w.dims[1:]), coords,
                           np.ascontiguousarray(w.vals[rows]), w.dense, (parts,) + tuple(w.out_shape[1:]), w.seed)
    A_parts, S_parts = oracle.evaluate(sub)
    got = out[top].cpu().numpy().astype(np.float64)
    return assert_close(got, A_parts.sum(axis=0), S_parts.sum(axis=0), TOL_FP32, what + " head slice %d (%d nonzeros)" % (top, rows.shape[0]))


def test_cfg2_full_sampled(sa):
    import torch
    w = configs.make(2, "full")
    out, t = _run_full(sa, w)
    sel = _sample(w, 3_000_000, 300)                  # includes a slice split over ~50 thread blocks
    _compare(out, w, sel, w.name)
    _compare_head_slice(out, w, w.name)               # 19.6 % of B in one slice
    # whole-output properties that hold at any size: finite, and slices scale with B
    assert bool(torch.isfinite(out).all())
    del out, t
    torch.cuda.empty_cache()


def test_cfg3_full_sampled(sa):
    import torch
    w = configs.make(3, "full")
    out, t = _run_full(sa, w)
    sel = _sample(w, 50_000, 3000)                    # includes a 50 000-nonzero row cut into pieces
    _compare(out, w, sel, w.name)
    counts = np.bincount(w.coords[:, 0], minlength=w.dims[0])
    empty = torch.from_numpy(np.nonzero(counts == 0)[0]).cuda()
    assert not bool(out[empty].any()), "empty rows must be +0"
    del out, t
    torch.cuda.empty_cache()


@pytest.fixture(scope="module")
def cfg4():
    return configs.make(4, "full")


@pytest.mark.parametrize("sched", ["left", "right"])
def test_cfg4_full_sampled(sa, cfg4, sched):
    import torch
    w = cfg4
    s = sa.SA_SCHED_ASSOC_LEFT if sched == "left" else sa.SA_SCHED_ASSOC_RIGHT
    out, t = _run_full(sa, w, sched=s)
    sel = _sample(w, 10_000, 3000)
    _compare(out, w, sel, w.name + "/" + sched)
    del out, t
    torch.cuda.empty_cache()


@pytest.fixture(scope="module")
def cfg5():
    return configs.make(5, "full")


@pytest.mark.parametrize("sched", ["fused", "fissioned"])
def test_cfg5_full_sampled(sa, cfg5, sched):
    import torch
    w = cfg5
    out, t = _run_full(sa, w, sched=sa.SA_SCHED_FUSED if sched == "fused" else sa.SA_SCHED_FISSIONED)
    sel = _sample(w, 600_000, 150)                    # includes a slice split over several thread blocks
    _compare(out, w, sel, w.name + "/" + sched)
    _compare_head_slice(out, w, w.name + "/" + sched)  # 19.9 % of B in one slice
    del out, t
    torch.cuda.empty_cache()


def test_cfg6_ttmc_full_sampled(sa):
    """Kernel 5 on the nell-2-shaped tensor: every output element sums over all nonzeros, so the
    oracle evaluates a seeded sample of output elements one by one."""
    import torch
    w = configs.make(6, "full")
    out, t = _run_full(sa, w)
    n_out = int(np.prod(w.out_shape))
    sel = np.sort(configs.rng.permutation(w.seed, 56, n_out)[:48])
    A_ref, S_ref = oracle.evaluate(w, sel=sel)
    got = out.reshape(-1)[torch.from_numpy(sel).cuda()].cpu().numpy().astype(np.float64)
    assert_close(got, A_ref, S_ref, TOL_FP32, w.name)
    assert bool(torch.isfinite(out).all())
    del out, t
    torch.cuda.empty_cache()


def test_cfg7_sddmm_spmm_gemm_full_sampled(sa):
    import torch
    w = configs.make(7, "full")
    out, t = _run_full(sa, w)
    sel = _sample(w, 5_000, 1200)
    _compare(out, w, sel, w.name)
    del out, t
    torch.cuda.empty_cache()


def test_cfg8_spmmh_gemm_mid_sampled(sa):
    """Kernel 3 at a quarter of the benchmark size (the full size holds two 4 GB matrices on the host)."""
    import torch
    w = configs.make(8, "mid")
    out, t = _run_full(sa, w)
    sel = _sample(w, 10_000, 3000)
    _compare(out, w, sel, w.name)
    del out, t
    torch.cuda.empty_cache()


def test_cfg9_mttkrp_gemm_full_sampled(sa):
    import torch
    w = configs.make(9, "full")
    out, t = _run_full(sa, w)
    sel = _sample(w, 3_000_000, 300)                  # includes a slice split over many thread blocks
    _compare(out, w, sel, w.name)
    counts = np.bincount(w.coords[:, 0], minlength=w.dims[0])
    empty = torch.from_numpy(np.nonzero(counts == 0)[0]).cuda()
    assert not bool(out[empty].any()), "empty slices must be +0"
    del out, t
    torch.cuda.empty_cache()


def test_cfg10_spttm_spttm_full_sampled(sa):
    """Kernel 7 on the config-2 tensor: sampled fibers (the longest, the shortest, seeded others) against the
    oracle, and the number of output rows against the number of distinct (i,j) pairs."""
    import torch
    w = configs.make(10, "full")
    out, t = _run_full(sa, w)
    keys, inv = oracle.fiber_keys(w.coords, w.dims)
    assert tuple(out.shape) == (keys.shape[0], 32)
    lens = np.bincount(inv, minlength=keys.shape[0])
    sel = np.unique(np.concatenate([[int(np.argmax(lens)), int(np.argmin(lens))],
                                    configs.rng.permutation(w.seed, 57, keys.shape[0])[:4000]])).astype(np.int64)
    A_ref, S_ref = oracle.evaluate(w, sel=sel)
    got = out[torch.from_numpy(sel).cuda()].cpu().numpy().astype(np.float64)
    assert_close(got, A_ref, S_ref, TOL_FP32, w.name)
    assert bool(torch.isfinite(out).all())
    del out, t
    torch.cuda.empty_cache()
