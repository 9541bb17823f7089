"""GPU edge cases through the C ABI: empty and one-entry tensors, empty slices and rows, padded
leading dimensions, every compiled rank combination, fibers and rows around the split
thresholds, the SDDMM sampling pattern, run-to-run reproducibility and workspace errors."""
import numpy as np
import pytest

import oracle
from workloads import configs, rng
from util import TOL_FP32, assert_close, fmt_of, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sa():
    import torch
    assert torch.cuda.is_available()
    import paper_2311_09549_b200 as sa
    return sa


def _wl(expr, fmt, dims, coords, vals, dense, out_shape):
    return configs.Workload("edge", expr, fmt, tuple(dims), np.asarray(coords, np.int32).reshape(-1, len(dims)),
                            np.asarray(vals, np.float32), dense, tuple(out_shape), 0)


def _dense(seed, which, r, c):
    return configs.dense_uniform(seed, which, r, c)


def _random_coo(seed, dims, nnz):
    lin = rng.keyed_bijection(np.arange(nnz), int(np.prod(dims)), np.uint64(seed))
    coords = np.stack(np.unravel_index(lin, dims), axis=1).astype(np.int32)
    return coords, rng.uniform_f32(seed, 1, np.arange(nnz), -1.0, 1.0)


def _check(sa, w, sched=None, tol=TOL_FP32):
    A_ref, S_ref = oracle.evaluate(w)
    A, t = run_gpu(sa, w, sched=sched)
    assert_close(A, A_ref, S_ref, tol, w.expr)
    return A, t


@pytest.mark.parametrize("nnz", [0, 1])
def test_empty_and_single_entry_all_chains(sa, nnz):
    c3 = [[3, 2, 1]][:nnz]
    c4 = [[3, 2, 1, 0]][:nnz]
    c2 = [[3, 2]][:nnz]
    v = [0.5][:nnz]
    _check(sa, _wl("spttm_ttm3", "csf", (5, 4, 3), c3, v, [_dense(1, 0, 4, 16), _dense(1, 1, 3, 32)], (5, 16, 32)))
    _check(sa, _wl("spttm_ttm4", "csf", (5, 4, 3, 2), c4, v,
                   [_dense(1, 0, 4, 16), _dense(1, 1, 3, 16), _dense(1, 2, 2, 16)], (5, 16, 16, 16)))
    _check(sa, _wl("sddmm_spmm", "csr", (5, 4), c2, v, [_dense(1, 0, 5, 64), _dense(1, 1, 4, 64), _dense(1, 2, 4, 32)], (5, 32)))
    _check(sa, _wl("ttmc3", "csf", (5, 4, 3), c3, v, [_dense(1, 0, 5, 32), _dense(1, 1, 4, 16), _dense(1, 2, 3, 32)], (32, 16, 32)))
    _check(sa, _wl("sddmm_spmm_gemm", "csr", (5, 4), c2, v,
                   [_dense(1, 0, 5, 64), _dense(1, 1, 4, 64), _dense(1, 2, 4, 128), _dense(1, 3, 128, 32)], (5, 32)))
    w = _wl("spmm_gemm", "csr", (5, 4), c2, v, [_dense(1, 0, 4, 128), _dense(1, 1, 128, 32)], (5, 32))
    _check(sa, w, sched=sa.SA_SCHED_ASSOC_LEFT)
    _check(sa, w, sched=sa.SA_SCHED_ASSOC_RIGHT)
    _check(sa, _wl("spmmh_gemm", "csr", (5, 4), c2, v, [_dense(1, 0, 4, 128), _dense(1, 3, 4, 128), _dense(1, 1, 128, 32)], (5, 32)))


@pytest.mark.parametrize("L,M", [(16, 16), (16, 32), (32, 16), (32, 32)])
def test_ttm3_rank_combinations_with_empty_slices(sa, L, M):
    dims = (40, 37, 53)
    coords, vals = _random_coo(7, dims, 3000)
    keep = coords[:, 0] % 3 != 1                     # every third slice empty
    w = _wl("spttm_ttm3", "csf", dims, coords[keep], vals[keep], [_dense(2, 0, 37, L), _dense(2, 1, 53, M)], (40, L, M))
    A, _ = _check(sa, w)
    assert not A[1::3].any()


@pytest.mark.parametrize("M", [32, 64])
def test_mttkrp_gemm_empty_slices_and_split_slices(sa, M):
    # empty slices, small slices (several per warp task) and one slice large enough to be split over thread blocks
    dims = (40, 37, 530)
    coords, vals = _random_coo(9, dims, 400000)
    keep = (coords[:, 0] % 3 != 1) & ((coords[:, 0] == 5) | (np.arange(400000) % 40 == 0))
    w = _wl("mttkrp_gemm", "csf", dims, coords[keep], vals[keep],
            [_dense(5, 0, 37, 32), _dense(5, 1, 530, 32), _dense(5, 2, 32, M)], (40, M))
    A, t = _check(sa, w)
    assert not A[1::3].any()
    assert sa.sa_tensor_worklist(t.handle)[0][3] >= 2, "slice 5 must be split into chunks with partial rows"


def test_ttm3_one_slice_long_fibers_split_over_many_blocks(sa):
    # a single slice of 60 000 nonzeros in 12 fibers of 5000: pieces cut inside fibers, 8 partial tiles
    dims = (3, 12, 5000)
    j, k = np.divmod(np.arange(60000), 5000)
    coords = np.stack([np.full(60000, 1), j, k], axis=1)
    vals = rng.uniform_f32(3, 1, np.arange(60000), -1.0, 1.0)
    perm = rng.permutation(3, 3, 60000)
    w = _wl("spttm_ttm3", "csf", dims, coords[perm], vals[perm], [_dense(3, 0, 12, 32), _dense(3, 1, 5000, 32)], (3, 32, 32))
    A, t = _check(sa, w)
    counts, items, fix = sa.sa_tensor_worklist(t.handle)
    assert counts[3] >= 2 and not A[0].any() and not A[2].any()


@pytest.mark.parametrize("n", [1, 7, 8, 9, 31, 32, 33, 63, 65, 2048, 2049, 8192, 8193, 16385])
def test_ttm3_ragged_sizes_around_batch_and_split_thresholds(sa, n):
    # one slice with n nonzeros in fibers of length 1, 2, 3, ... : hits batch tails, groups of 8
    # fibers, the one-warp / one-block / many-block boundaries
    lens = []
    while sum(lens) < n:
        lens.append(min(len(lens) % 11 + 1, n - sum(lens)))
    j = np.repeat(np.arange(len(lens)), lens)
    k = np.concatenate([np.arange(x) for x in lens])
    dims = (2, len(lens), 12)
    coords = np.stack([np.ones(n, np.int64), j, k], axis=1)
    vals = rng.uniform_f32(n, 1, np.arange(n), -1.0, 1.0)
    w = _wl("spttm_ttm3", "csf", dims, coords, vals, [_dense(4, 0, len(lens), 32), _dense(4, 1, 12, 32)], (2, 32, 32))
    _check(sa, w)


def test_padded_leading_dimensions(sa):
    import torch
    w = configs.make(1)
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSF, device=0)
    big = [torch.zeros(x.shape[0], x.shape[1] + 12, device="cuda") for x in w.dense]
    views = []
    for b, x in zip(big, w.dense):
        b[:, 4:4 + x.shape[1]] = torch.from_numpy(x).cuda()
        views.append(b[:, 4:4 + x.shape[1]])          # 16-byte aligned start, ld = cols + 12
    out, _ = t.run(w.expr, views)
    torch.cuda.synchronize()
    A_ref, S_ref = oracle.evaluate(w)
    assert_close(out.cpu().numpy().astype(np.float64), A_ref, S_ref, TOL_FP32, "padded ld")
    # a misaligned view is refused before anything is launched
    with pytest.raises(sa.SaError) as e:
        t.run(w.expr, [big[0][:, 1:17], views[1]])
    assert e.value.status == sa.SA_E_SHAPE


@pytest.mark.parametrize("K,L", [(k, l) for k in (32, 64, 128) for l in (32, 64, 128)])
def test_sddmm_spmm_ranks_long_rows_and_sampled_pattern(sa, K, L):
    import torch
    I, J = 300, 6000
    deg = np.zeros(I, dtype=np.int64)
    deg[5] = 5000                                      # cut into pieces with partial rows
    deg[6] = 1024                                      # exactly at the threshold: one item
    deg[10:200:3] = 17
    deg[299] = 1
    cols = configs.distinct_children(11, 2, deg, J)
    rows = np.repeat(np.arange(I), deg)
    vals = rng.uniform_f32(11, 1, np.arange(rows.shape[0]), 0.0, 1.0)
    perm = rng.permutation(11, 3, rows.shape[0])
    coords = np.stack([rows, cols], axis=1)[perm].astype(np.int32)
    vals = vals[perm]
    dense = [configs.dense_normal(11, 0, I, K), configs.dense_normal(11, 1, J, K), configs.dense_normal(11, 2, J, L)]
    w = _wl("sddmm_spmm", "csr", (I, J), coords, vals, dense, (I, L))
    A, t = _check(sa, w)
    assert not A[0].any() and not A[298].any()        # empty rows are +0
    # debug schedule: sampled values land exactly on B's stored coordinates, in CSR order
    ops = [torch.from_numpy(x).cuda() for x in dense]
    tuples = [(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0)) for x in ops]
    need = sa.sa_workspace_size(t.handle, sa.SA_EXPR_SDDMM_SPMM, sa.SA_SCHED_DEBUG_MATERIALIZE, tuples)
    ws = torch.full((need // 4,), float("nan"), device="cuda")
    out, _ = t.run(w.expr, ops, sched=sa.SA_SCHED_DEBUG_MATERIALIZE, workspace=ws.view(torch.uint8))
    torch.cuda.synchronize()
    nnz = vals.shape[0]
    sampled = ws[-(((nnz * 4 + 255) // 256) * 64):][:nnz].cpu().numpy().astype(np.float64)
    _, _, P = oracle.sddmm_spmm(coords, vals, (I, J), *dense, with_sampled=True)
    _, crd, _ = sa.sa_tensor_export(t.handle, 1, n_crd=nnz)
    order = np.lexsort((coords[:, 1], coords[:, 0]))   # CSR order of the input entries
    assert np.array_equal(coords[order, 1], crd)
    Sabs = np.abs(vals[order].astype(np.float64)) * (np.abs(dense[0][coords[order, 0]].astype(np.float64)) *
                                                     np.abs(dense[1][coords[order, 1]].astype(np.float64))).sum(axis=1)
    assert np.isfinite(sampled).all() and (np.abs(sampled - P[order]) <= TOL_FP32 * Sabs).all()
    assert_close(out.cpu().numpy().astype(np.float64), *oracle.evaluate(w), TOL_FP32, "materialize schedule output")


@pytest.mark.parametrize("L,M", [(128, 32), (128, 64), (256, 32)])
def test_spmm_gemm_rank_combinations_and_long_rows(sa, L, M):
    I, J = 500, 6000
    deg = np.full(I, 3, dtype=np.int64)
    deg[::7] = 0
    deg[123] = 2900
    deg[124] = 5000                                    # above the long-row threshold: pieces + fix-up
    cols = configs.distinct_children(12, 2, deg, J)
    rows = np.repeat(np.arange(I), deg)
    vals = rng.uniform_f32(12, 1, np.arange(rows.shape[0]), -1.0, 1.0)
    coords = np.stack([rows, cols], axis=1).astype(np.int32)
    w = _wl("spmm_gemm", "csr", (I, J), coords, vals,
            [configs.dense_normal(12, 0, J, L), configs.dense_normal(12, 1, L, M)], (I, M))
    _check(sa, w, sched=sa.SA_SCHED_ASSOC_LEFT)
    _check(sa, w, sched=sa.SA_SCHED_ASSOC_RIGHT)
    # kernel 3 on the same tensor: empty rows, long rows cut into pieces, every rank combination
    wh = _wl("spmmh_gemm", "csr", (I, J), coords, vals,
             [w.dense[0], configs.dense_normal(12, 2, J, L), w.dense[1]], (I, M))
    _check(sa, wh)


def test_ttm4_ragged_and_split_slices(sa):
    # few level-1 fibers per slice: the head slice's (i,j) subtrees are above the size the fused kernel evaluates
    # itself, so the order-3 kernel writes their temporaries first (some split over several thread blocks, with
    # partial temporaries that the fix-up kernel sums) and items of kind 1 copy them into the pool
    w = configs.make_ttm4_zipf("edge4", 31, 90, 6, 130, 110, 150_000, 1.4, 5.0, 16, 16, 16)
    A, t = _check(sa, w, sched=sa.SA_SCHED_FUSED)
    assert sa.sa_tensor_worklist(t.handle, 0)[0][3] >= 2, "a large (i,j) subtree must be split over several thread blocks"
    kinds = sa.sa_tensor_worklist(t.handle, 2)[1][:, 7]
    assert (kinds == 1).any() and (kinds == 0).any()
    # many level-1 fibers per slice: the head slices span several pieces and leave partial slice tiles
    w = configs.make_ttm4_zipf("edge4b", 32, 90, 700, 50, 45, 150_000, 1.4, 5.0, 16, 16, 16)
    A, t = _check(sa, w, sched=sa.SA_SCHED_FUSED)
    assert sa.sa_tensor_worklist(t.handle, 1)[0][3] >= 2, "the head slice must be split into several pieces"
    # subtrees with more level-2 fibers than one batch holds next to small ones
    for w in (configs.make_ttm4_zipf("edge4c", 33, 90, 40, 160, 110, 150_000, 1.4, 5.0, 16, 16, 16),
              configs.make_ttm4_zipf("edge4d", 34, 400, 60, 150, 40, 200_000, 1.2, 3.0, 16, 16, 16)):
        A, t = _check(sa, w, sched=sa.SA_SCHED_FUSED)
        items = sa.sa_tensor_worklist(t.handle, 2)[1]
        nf = items[:, 3] - items[:, 2]
        assert ((items[:, 7] == 0) & (nf > 32)).any() and ((items[:, 7] == 0) & (nf <= 32) & (items[:, 1] - items[:, 0] > 1)).any()


def test_ttm4_fissioned_ragged_and_split_slices(sa):
    """The same tensors through the two-pass schedule (temporaries of all (i,j) subtrees in the workspace)."""
    F = sa.SA_SCHED_FISSIONED
    # few level-1 fibers per slice: the head slice's (i,j) subtrees exceed one thread block's chunk, so the
    # first pass writes partial temporaries that the fix-up kernel sums
    w = configs.make_ttm4_zipf("edge4", 31, 90, 6, 130, 110, 150_000, 1.4, 5.0, 16, 16, 16)
    A, t = _check(sa, w, sched=F)
    assert sa.sa_tensor_worklist(t.handle, 4)[0][3] >= 2, "a large (i,j) subtree must be split over several thread blocks"
    # many level-1 fibers per slice: the second pass cuts the head slices into pieces of 512 fibers
    w = configs.make_ttm4_zipf("edge4b", 32, 90, 700, 50, 45, 150_000, 1.4, 5.0, 16, 16, 16)
    A, t = _check(sa, w, sched=F)
    assert sa.sa_tensor_worklist(t.handle, 5)[0][3] >= 2, "the head slice must be split into several pieces"
    # both kernels of the first pass in one run: small subtrees (list 6) and large ones (list 4)
    for w in (configs.make_ttm4_zipf("edge4c", 33, 90, 40, 160, 110, 150_000, 1.4, 5.0, 16, 16, 16),
              configs.make_ttm4_zipf("edge4d", 34, 400, 60, 150, 40, 200_000, 1.2, 3.0, 16, 16, 16)):
        A, t = _check(sa, w, sched=F)
        n_main, n_sub = (int(sa.sa_tensor_worklist(t.handle, x)[0][0]) for x in (4, 6))
        assert n_main > 0 and n_sub > 0, (n_main, n_sub)


def test_results_are_reproducible_run_to_run(sa):
    w = configs.make(2, "mini")
    A1, t = run_gpu(sa, w)
    A2, _ = run_gpu(sa, w, tensor=t)
    assert np.array_equal(A1, A2)


def test_workspace_errors_enqueue_nothing(sa):
    import torch
    w = configs.make(2, "mini")
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSF, device=0)
    ops = [torch.from_numpy(x).cuda() for x in w.dense]
    tuples = [(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0)) for x in ops]
    need = sa.sa_workspace_size(t.handle, sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_DEFAULT, tuples)
    assert need > 0
    out = torch.zeros(w.out_shape, device="cuda")
    small = torch.empty(need - 256, dtype=torch.uint8, device="cuda")
    s = torch.cuda.current_stream().cuda_stream
    for ws_ptr, ws_bytes in [(small.data_ptr(), small.numel()), (None, 0), (small.data_ptr() + 16, need)]:
        with pytest.raises(sa.SaError) as e:
            sa.sa_run(t.handle, sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_DEFAULT, tuples, out.data_ptr(), ws_ptr, ws_bytes, s)
        assert e.value.status == sa.SA_E_WORKSPACE
    torch.cuda.synchronize()
    assert not out.any()
    assert sa.sa_last_device_status(t.handle, s) == sa.SA_OK


@pytest.mark.parametrize("L,M", [(32, 32), (32, 64), (64, 32), (64, 64)])
@pytest.mark.parametrize("sched", ["left", "right"])
def test_spttm_spttm_ranks_long_fibers_and_empty_slices(sa, L, M, sched):
    # short fibers, empty slices, and one fiber of 9000 nonzeros that is cut into pieces with partial rows
    dims = (40, 37, 9500)
    coords, vals = _random_coo(11, dims, 6000)
    keep = coords[:, 0] % 3 != 1
    longf = np.stack([np.full(9000, 6), np.full(9000, 3), np.arange(9000)], axis=1).astype(np.int32)
    keep &= ~((coords[:, 0] == 6) & (coords[:, 1] == 3))
    c = np.concatenate([coords[keep], longf])
    v = np.concatenate([vals[keep], rng.uniform_f32(12, 1, np.arange(9000), -1.0, 1.0)])
    perm = rng.permutation(13, 3, c.shape[0])
    keys, _ = oracle.fiber_keys(c, dims)
    w = _wl("spttm_spttm", "csf", dims, c[perm], v[perm], [_dense(6, 0, 9500, L), _dense(6, 1, L, M)], (keys.shape[0], M))
    s = sa.SA_SCHED_ASSOC_LEFT if sched == "left" else sa.SA_SCHED_ASSOC_RIGHT
    A, t = _check(sa, w, sched=s)
    assert A.shape == (keys.shape[0], M)
    assert sa.sa_tensor_worklist(t.handle, 1)[0][3] >= 1, "the long fiber must be split into pieces with partial rows"


@pytest.mark.parametrize("nnz", [0, 1])
def test_spttm_spttm_empty_and_single_entry(sa, nnz):
    w = _wl("spttm_spttm", "csf", (5, 4, 3), [[3, 2, 1]][:nnz], [0.5][:nnz], [_dense(1, 0, 3, 32), _dense(1, 1, 32, 64)], (nnz, 64))
    for s in (sa.SA_SCHED_ASSOC_LEFT, sa.SA_SCHED_ASSOC_RIGHT):
        A, _ = _check(sa, w, sched=s)
        assert A.shape == (nnz, 64)


@pytest.mark.parametrize("L,M", [(128, 32), (128, 64), (256, 32), (256, 64)])
def test_dense_stage_ragged_rows_and_padded_leading_dimensions(sa, L, M):
    """B.(C.D) with a number of columns J that is not a multiple of the dense stage's 128-row tile (the last
    tile is ragged, several tiles per thread block) and with C and D given as padded views."""
    import torch
    I, J = 700, 148 * 128 * 2 + 77
    coords, vals = _random_coo(21, (I, J), 30_000)
    C, D = configs.dense_normal(21, 0, J, L), configs.dense_normal(21, 1, L, M)
    w = _wl("spmm_gemm", "csr", (I, J), coords, vals, [C, D], (I, M))
    A_ref, S_ref = oracle.evaluate(w)
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSR, device=0)
    bigC = torch.zeros(J, L + 8, device="cuda")
    bigD = torch.zeros(L, M + 4, device="cuda")
    bigC[:, 4:4 + L] = torch.from_numpy(C).cuda()
    bigD[:, :M] = torch.from_numpy(D).cuda()
    out, _ = t.run("spmm_gemm", [bigC[:, 4:4 + L], bigD[:, :M]], sched=sa.SA_SCHED_ASSOC_RIGHT)
    torch.cuda.synchronize()
    assert sa.sa_last_device_status(t.handle, torch.cuda.current_stream().cuda_stream) == sa.SA_OK
    assert_close(out.cpu().numpy().astype(np.float64), A_ref, S_ref, TOL_FP32, "dense stage %dx%d" % (L, M))


def test_ttm4_padded_factor_matrices(sa):
    """Order-4 chain with the factor matrices given as padded views (leading dimension 20): the fused kernel's
    general-stride variant, and the subtree kernel's of the two-pass schedule."""
    import torch
    w = configs.make_ttm4_zipf("edge4e", 35, 300, 60, 150, 40, 120_000, 1.2, 3.0, 16, 16, 16)
    A_ref, S_ref = oracle.evaluate(w)
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSF, device=0)
    views = []
    for x in w.dense:
        b = torch.zeros(x.shape[0], 20, device="cuda")
        b[:, :16] = torch.from_numpy(x).cuda()
        views.append(b[:, :16])
    for sched in (sa.SA_SCHED_FUSED, sa.SA_SCHED_FISSIONED):
        out, _ = t.run(w.expr, views, sched=sched)
        torch.cuda.synchronize()
        assert sa.sa_last_device_status(t.handle, torch.cuda.current_stream().cuda_stream) == sa.SA_OK
        assert_close(out.cpu().numpy().astype(np.float64), A_ref, S_ref, TOL_FP32, "ttm4 padded ld, schedule %d" % sched)
    assert int(sa.sa_tensor_worklist(t.handle, 2)[0][0]) > 0 and int(sa.sa_tensor_worklist(t.handle, 6)[0][0]) > 0


def test_allocator_failure_at_every_upload_is_reported_and_leaks_nothing(sa):
    """The device allocator returns NULL at the k-th request, for every k up to the number of requests a tensor
    makes: create answers SA_E_ALLOC, hands out no handle, and every block it had obtained is released."""
    import ctypes
    import torch
    base = sa.TorchAllocator(0)

    class Failing:
        def __init__(self, fail_at):
            self.calls, self.fail_at, self.live = 0, fail_at, set()
            self._a = sa._ALLOC_FN(self.alloc)
            self._r = sa._RELEASE_FN(self.release)
            self.struct = sa.SaAllocator(self._a, self._r, None)

        def alloc(self, nbytes, ctx):
            self.calls += 1
            if self.calls - 1 == self.fail_at:
                return None
            p = base._do_alloc(nbytes, ctx)
            self.live.add(p)
            return p

        def release(self, ptr, ctx):
            self.live.discard(ptr)
            base._do_release(ptr, ctx)

    for cfg in (1, 3, 5):
        w = configs.make(cfg, "mini")
        fmt = fmt_of(sa, w)
        k = 0
        while True:
            a = Failing(k)
            try:
                h = sa.sa_tensor_create(len(w.dims), w.dims, len(w.vals), w.coords, w.vals, fmt, 0, a.struct)
            except sa.SaError as e:
                assert e.status == sa.SA_E_ALLOC, (cfg, k, e)
                assert a.calls == k + 1 and not a.live, "blocks obtained before the failure must be released"
                k += 1
                continue
            assert a.calls <= k, "with no failing request the tensor is created"
            assert len(a.live) == a.calls
            sa.sa_destroy(h)
            assert not a.live
            break
        assert k >= 8, "the loop really walked through the uploads"
    torch.cuda.synchronize()


def test_default_order_of_spmm_gemm_picks_the_faster_one_on_both_sides(sa):
    """The run-time choice between (B.C).D and B.(C.D) on two tensors where it goes opposite ways, checked against
    device timings: with few nonzeros on a huge C, forming C.D reads 2 GB that (B.C).D never touches; with many
    nonzeros per column, one gathered 1 KB row per nonzero is the larger cost."""
    import torch

    def both(I, J, nnz, seed):
        w = configs.make_spmm_gemm("order-%d" % J, seed, I, J, nnz, 256, 64)
        t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSR, device=0)
        ops = [torch.from_numpy(x).cuda() for x in w.dense]
        desc = [(x.data_ptr(), x.shape[0], x.shape[1], x.stride(0)) for x in ops]
        chosen = sa.sa_schedule_cost(t.handle, sa.SA_EXPR_SPMM_GEMM, sa.SA_SCHED_DEFAULT, desc)["resolved"]
        ms = {}
        for s in (sa.SA_SCHED_ASSOC_LEFT, sa.SA_SCHED_ASSOC_RIGHT):
            out, _ = t.run(w.expr, ops, sched=s)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                t.run(w.expr, ops, out=out, sched=s)
            e1.record()
            torch.cuda.synchronize()
            ms[s] = e0.elapsed_time(e1) / 10
        # the default really runs the chosen order (same launches, same result)
        a, _ = t.run(w.expr, ops, sched=sa.SA_SCHED_DEFAULT)
        b, _ = t.run(w.expr, ops, sched=chosen)
        torch.cuda.synchronize()
        assert torch.equal(a, b)
        t.close()
        return chosen, ms

    chosen, ms = both(5_000, 2_000_000, 200_000, 61)
    assert chosen == sa.SA_SCHED_ASSOC_LEFT and ms[sa.SA_SCHED_ASSOC_LEFT] < ms[sa.SA_SCHED_ASSOC_RIGHT], ms
    chosen, ms = both(20_000, 400_000, 1_500_000, 62)
    assert chosen == sa.SA_SCHED_ASSOC_RIGHT and ms[sa.SA_SCHED_ASSOC_RIGHT] < ms[sa.SA_SCHED_ASSOC_LEFT], ms


@pytest.mark.parametrize("K,L,M", [(64, 64, 32), (32, 128, 64), (128, 32, 32)])
def test_sddmm_spmm_gemm_rank_combinations(sa, K, L, M):
    """Kernel 2 over ranks the mini workload does not use: the tcgen05 dense stage at L = 64 with M = 32, the row
    temporaries of 32 and 128 floats."""
    w0 = configs.make_sddmm_spmm("k2-ranks", 91, 4_000, 4_000, 50_000, 1.5, 1_200, K, L)
    F = configs.dense_normal(91, 3, L, M)
    w = _wl("sddmm_spmm_gemm", "csr", w0.dims, w0.coords, w0.vals, w0.dense + [F], (w0.dims[0], M))
    _check(sa, w)
