"""Host builder of the C-ABI library, without a GPU (host-only handles, device = -1):
compressed levels bit for bit against an independent construction, work-list (partition)
invariants, error codes for malformed input, exported symbols."""
import ctypes
import re
import os

import numpy as np
import pytest

import paper_2311_09549_b200 as sa
from workloads import configs

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def independent_levels(coords, vals, dims, fmt):
    """pos/crd/vals per level built with plain Python containers from the sorted tuple list."""
    order = coords.shape[1]
    entries = sorted((tuple(int(x) for x in c), float(v)) for c, v in zip(coords, vals))
    out_vals = np.array([v for _, v in entries], dtype=np.float32)
    if fmt == "csr":
        pos = np.zeros(dims[0] + 1, dtype=np.int64)
        for (i, _), _ in entries:
            pos[i + 1] += 1
        return [(None, None), (np.cumsum(pos), np.array([c[1] for c, _ in entries], dtype=np.int32))], out_vals
    levels = []
    parents = [()]                      # distinct prefixes of the previous level, sorted
    for l in range(order):
        prefixes = sorted(set(c[:l + 1] for c, _ in entries))
        crd = np.array([p[l] for p in prefixes], dtype=np.int32)
        pos = np.zeros(len(parents) + 1, dtype=np.int64)
        index_of = {p: n for n, p in enumerate(parents)}
        for p in prefixes:
            pos[index_of[p[:l]] + 1] += 1
        levels.append((np.cumsum(pos), crd))
        parents = prefixes
    return levels, out_vals


def export_all(t, fmt):
    nnz, counts, _ = t.info()
    levels = []
    for l in range(t.order):
        if fmt == "csr" and l == 0:
            levels.append((None, None))
            continue
        n_pos = (1 if l == 0 else int(counts[l - 1])) + 1
        pos, crd, _ = sa.sa_tensor_export(t.handle, l, n_pos=n_pos, n_crd=int(counts[l]))
        levels.append((pos, crd if crd is not None else np.zeros(0, np.int32)))
    _, _, vals = sa.sa_tensor_export(t.handle, t.order - 1, n_vals=nnz)
    return levels, vals if vals is not None else np.zeros(0, np.float32)


def small(cfg):
    w = configs.make(cfg, "mini")
    keep = configs.rng.permutation(5, 5, w.nnz)[:4000]
    return w, w.coords[keep], w.vals[keep]


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_levels_match_independent_construction(cfg):
    w, coords, vals = small(cfg)
    t = sa.SparseTensor(w.dims, coords, vals, sa.SA_FMT_CSR if w.fmt == "csr" else sa.SA_FMT_CSF, device=-1)
    got, got_vals = export_all(t, w.fmt)
    want, want_vals = independent_levels(coords, vals, w.dims, w.fmt)
    for l, ((gp, gc), (wp, wc)) in enumerate(zip(got, want)):
        if wp is None:
            assert gp is None
            continue
        assert np.array_equal(gp, wp), "pos of level %d" % l
        assert np.array_equal(gc, wc), "crd of level %d" % l
    assert np.array_equal(got_vals, want_vals)


@pytest.mark.parametrize("cfg", [1, 2, 5])
def test_csf_worklist_partitions_every_nonzero_once(cfg):
    """Main list of a CSF tensor: the units of the order-3 kernel.  For an order-4 tensor its "slices" are the
    large (i,j) subtrees (more than 4096 nonzeros; output row = index among the large ones) and its fibers the
    (i,j,k) fibers; the other subtrees are covered by the items of the fused kernel."""
    w = configs.make(cfg, "mini")
    coords, vals = w.coords, w.vals
    if cfg == 5:
        # two (i,j) subtrees that the fused kernel does not evaluate itself (more than 4096 nonzeros), so that the
        # main list of the order-4 tensor is not empty; all the others are in the third list
        keep = ~(((coords[:, 0] == 3) & (coords[:, 1] == 5)) | ((coords[:, 0] == 200) & (coords[:, 1] == 7)))
        k, o = np.divmod(np.arange(4800), 40)
        extra = [np.stack([np.full(4800, i), np.full(4800, j), k, o], axis=1) for i, j in ((3, 5), (200, 7))]
        coords = np.concatenate([coords[keep]] + extra).astype(np.int32)
        vals = np.concatenate([vals[keep], np.ones(9600, np.float32)])
    nnz_all = coords.shape[0]
    t = sa.SparseTensor(w.dims, coords, vals, sa.SA_FMT_CSF, device=-1)
    levels, _ = export_all(t, "csf")
    counts, items, fix = sa.sa_tensor_worklist(t.handle)
    n_items, n_groups, n_fix, n_slots = (int(x) for x in counts)
    if t.order == 3:
        slice_rows, pos1, pos2 = levels[0][1], levels[1][0], levels[2][0]
        slice_pos = {int(c): n for n, c in enumerate(slice_rows)}
    else:
        pos1, pos2 = levels[2][0], levels[3][0]
        nz_sub = pos2[pos1[1:]] - pos2[pos1[:-1]]
        large = np.nonzero(nz_sub > 4096)[0]
        assert len(large) == 2
        slice_rows = np.arange(len(large))
        slice_pos = {n: int(r) for n, r in enumerate(large)}      # output row = index among the large subtrees
    covered = np.zeros(nnz_all, dtype=np.int32)
    if t.order == 4:
        sub = sa.sa_tensor_worklist(t.handle, 2)[1]
        assert len(sub) > 0 and n_items > 0
        for row, row_end, f0, f1, p0, p1, dest, kind in sub:
            if kind == 0:
                covered[p0:p1] += 1              # the other subtrees are evaluated from the third list
    slot_owner = {}
    G = 4                                   # warps (tasks) per thread block of the order-3 kernel
    task_start, stream_f0 = sa.sa_tensor_tasks(t.handle)
    group_items = int(task_start[n_groups * G])
    item_group = np.searchsorted(task_start, np.arange(n_items), side="right") - 1
    for n, (row, row_end, f0, f1, p0, p1, dest, spos) in enumerate(items):
        assert p0 < p1, "no empty units"
        s = slice_pos[int(row)]
        fa, fb = pos2[f0], pos2[f1]
        if n >= group_items:
            # a whole small slice
            assert int(spos) == s and (f0, f1) == (pos1[s], pos1[s + 1]) and (fa, fb) == (p0, p1)
            assert p1 - p0 <= 2048 and dest == -1
        else:
            assert pos1[s] <= f0 < f1 <= pos1[s + 1], "fibers stay inside the item's slice"
            assert fa <= p0 < p1 <= fb, "nonzero range lies inside the fiber range"
            # first and last fiber really intersect the clip range
            assert pos2[f0 + 1] > p0 and pos2[f1 - 1] < p1 and int(spos) == s
            lead = items[task_start[(item_group[n] // G) * G]]
            assert dest == lead[6] and row == lead[0], "a group works on one slice and one destination"
        covered[p0:p1] += 1
        if dest >= 0:
            slot_owner.setdefault(int(dest), int(row))
            assert slot_owner[int(dest)] == int(row)
    assert (covered == 1).all(), "every nonzero belongs to exactly one unit"
    # fix-up entries: split slices own disjoint slot ranges, empty slices are listed with count 0
    used = np.zeros(n_slots, dtype=np.int32)
    empties = set()
    for row, slot0, count, _ in fix:
        if count == 0:
            empties.add(int(row))
            continue
        used[slot0:slot0 + count] += 1
        assert all(slot_owner[s] == int(row) for s in range(slot0, slot0 + count))
    assert (used == 1).all() and set(slot_owner) == set(range(n_slots))
    if t.order == 3:
        assert empties == set(range(w.dims[0])) - set(int(c) for c in slice_rows)
    else:
        assert not empties, "every large subtree has nonzeros"
    # nonzero balance: no unit is larger than the small-slice bound / the piece size
    sizes = items[:, 5] - items[:, 4]
    assert sizes.max() <= max(4096, int(np.ceil(nnz_all / 8)))
    # tasks: a partition of the item list; group tasks hold at most one item and warp 0 of a group has one;
    # small-slice tasks hold at most 16 items and about 2048 nonzeros
    assert task_start[0] == 0 and task_start[-1] == n_items and (np.diff(task_start) >= 0).all()
    per_task = np.diff(task_start)
    assert (per_task[:n_groups * G] <= 1).all() and (per_task[:n_groups * G:G] == 1).all()
    assert (per_task[n_groups * G:] >= 1).all() and (per_task[n_groups * G:] <= 16).all()
    for a, b in zip(task_start[n_groups * G:-1], task_start[n_groups * G + 1:]):
        assert b - a == 1 or sizes[a:b].sum() <= 2048
    # stream starts: part q of an item begins in fiber stream_f0[n, q]
    for n, (row, row_end, f0, f1, p0, p1, dest, _) in enumerate(items):
        b8 = (p0 // 16) * 16
        slen = -(-(-(-(p1 - b8) // 4)) // 16) * 16
        for q in range(4):
            lo, hi = max(p0, b8 + q * slen), min(p1, b8 + (q + 1) * slen)
            f = int(stream_f0[n, q])
            if lo < hi:
                assert f0 <= f < f1 and pos2[f] <= lo < pos2[f + 1]
            else:
                assert f == f0


def _order4_lists(t):
    levels, _ = export_all(t, "csf")
    items = sa.sa_tensor_worklist(t.handle, 2)[1]
    counts3, pieces, supers = sa.sa_tensor_worklist(t.handle, 3)
    counts1, _, fix = sa.sa_tensor_worklist(t.handle, 1)
    return levels, items, pieces, supers, fix, int(counts3[1]), int(counts1[3])


def check_order4_fused_lists(t, dims0):
    """Items, super-items and pieces of the fused order-4 kernel: every (i,j) subtree belongs to exactly one item,
    the items of a super-item and the super-items of a piece are consecutive and fit the pool, and every slice
    has exactly one destination per piece it lies in."""
    levels, items, pieces, supers, fix, n_large, n_slots = _order4_lists(t)
    crd0, pos1, pos2, pos3 = levels[0][1], levels[1][0], levels[2][0], levels[3][0]
    F2 = len(pos1) and int(pos1[-1])
    nz_sub = pos3[pos2[1:]] - pos3[pos2[:-1]]
    is_large = nz_sub > 4096
    assert n_large == int(is_large.sum())
    large_ord = np.cumsum(is_large) - 1
    seen = np.zeros(F2, dtype=np.int32)
    for r0, r1, f0, f1, p0, p1, dest, kind in items:
        assert r0 < r1 <= F2 and r1 - r0 <= 32
        seen[r0:r1] += 1
        if kind == 0:
            assert not is_large[r0:r1].any()
            assert (f0, f1) == (pos2[r0], pos2[r1]) and (p0, p1) == (pos3[f0], pos3[f1])
        else:
            assert kind == 1 and is_large[r0:r1].all() and r1 - r0 <= 8
            assert f0 == large_ord[r0] and f1 - f0 == r1 - r0
    assert (seen == 1).all()
    # super-items: consecutive items, consecutive subtrees, at most 64 subtrees, at most 8 runs of small subtrees
    nxt_item, nxt_r = 0, 0
    for i0, i1, r0, r1 in supers:
        assert i0 == nxt_item and i1 > i0 and r0 == nxt_r and 0 < r1 - r0 <= 64
        assert items[i0][0] == r0 and items[i1 - 1][1] == r1
        assert all(items[k][1] == items[k + 1][0] for k in range(i0, i1 - 1))
        n_large_runs = sum(1 for k in range(i0, i1) if items[k][7] == 1)
        assert sum(1 for k in range(i0, i1) if items[k][7] == 0) <= 8 + n_large_runs
        nxt_item, nxt_r = i1, r1
    assert nxt_item == len(items) and nxt_r == F2
    # pieces: consecutive super-items; slices and destinations
    slot_user = {}
    nxt_sup = 0
    dests = {}
    for sup0, sup1, sa_, sb_, d_first, d_last, r0, r1 in pieces:
        assert sup0 == nxt_sup and sup1 > sup0 and supers[sup0][2] == r0 and supers[sup1 - 1][3] == r1
        nxt_sup = sup1
        assert pos1[sa_] <= r0 < pos1[sa_ + 1] and pos1[sb_] < r1 <= pos1[sb_ + 1] and sa_ <= sb_
        for s_ in range(sa_, sb_ + 1):
            whole = r0 <= pos1[s_] and pos1[s_ + 1] <= r1
            d = d_first if s_ == sa_ else d_last if s_ == sb_ else -1
            if whole:
                assert d == -1, "a slice inside one piece goes straight to the output"
            else:
                assert d >= 0 and d not in slot_user
                slot_user[d] = s_
            dests.setdefault(s_, []).append(d)
        if sa_ == sb_:
            assert d_first == d_last
    assert nxt_sup == len(supers)
    used = np.zeros(n_slots, dtype=np.int32)
    empties = set()
    for row, slot0, count, _ in fix:
        if count == 0:
            empties.add(int(row))
            continue
        s_ = int(np.nonzero(crd0 == row)[0][0])
        assert dests[s_] == list(range(slot0, slot0 + count)), "one partial tile per piece, in piece order"
        used[slot0:slot0 + count] += 1
    assert (used == 1).all() and set(slot_user) == set(range(n_slots))
    assert empties == set(range(dims0)) - set(int(c) for c in crd0)
    return items, pieces, supers


def test_order4_fused_worklists_cover_every_subtree_once():
    w = configs.make(5, "mini")
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSF, device=-1)
    items, pieces, supers = check_order4_fused_lists(t, w.dims[0])
    assert len(pieces) > 4, "the mini tensor spans several pieces"
    # a tensor with one slice: every piece is inside it and leaves a partial tile
    keep = w.coords[:, 0] == w.coords[0, 0]
    one = np.ascontiguousarray(w.coords[keep])
    t1 = sa.SparseTensor(w.dims, one, w.vals[keep], sa.SA_FMT_CSF, device=-1)
    check_order4_fused_lists(t1, w.dims[0])


def test_order4_large_and_many_fiber_subtrees():
    """A subtree above 4096 nonzeros is left to the order-3 lists (item of kind 1); one with 130 fibers but few
    nonzeros is part of an item of kind 0 that the kernel evaluates in batches."""
    k, o = np.divmod(np.arange(4800), 40)
    big = np.stack([np.zeros(4800), np.zeros(4800), k, o], axis=1).astype(np.int32)
    many = np.stack([np.ones(130), np.ones(130), np.arange(130), np.zeros(130)], axis=1).astype(np.int32)
    both = np.concatenate([big, many, np.array([[1, 2, 5, 1]], np.int32)])
    t2 = sa.SparseTensor((2, 3, 130, 40), both, np.ones(len(both), np.float32), sa.SA_FMT_CSF, device=-1)
    items, pieces, supers = check_order4_fused_lists(t2, 2)
    kinds = {(int(x[0]), int(x[1])): int(x[7]) for x in items}
    assert kinds == {(0, 1): 1, (1, 2): 0, (2, 3): 0}
    main = sa.sa_tensor_worklist(t2.handle, 0)[1]
    assert set(main[:, 0].tolist()) == {0} and (main[:, 5] - main[:, 4]).sum() == 4800


@pytest.mark.parametrize("cfg,which", [(3, 0), (4, 1), (4, 0)])
def test_csr_worklist_partitions_rows_and_nonzeros(cfg, which):
    w = configs.make(cfg, "mini")
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSR, device=-1)
    levels, _ = export_all(t, "csr")
    pos = levels[1][0]
    counts, items, fix = sa.sa_tensor_worklist(t.handle, which)
    covered = np.zeros(w.nnz, dtype=np.int32)
    rows = np.zeros(w.dims[0], dtype=np.int32)
    for row, row_end, _, _, p0, p1, dest, _ in items:
        if dest >= 0:
            assert row_end == row + 1 and pos[row] <= p0 < p1 <= pos[row + 1]
        else:
            assert (p0, p1) == (pos[row], pos[row_end])
            rows[row:row_end] += 1
        covered[p0:p1] += 1
    assert (covered == 1).all()
    for row, slot0, count, _ in fix:
        assert count >= 2
        rows[row] += 1
    assert (rows == 1).all(), "every row is written by exactly one range item or one fix-up entry"


def test_empty_and_single_entry_tensors():
    t = sa.SparseTensor((5, 4, 3), np.zeros((0, 3), np.int32), np.zeros(0, np.float32), sa.SA_FMT_CSF, device=-1)
    nnz, counts, chunks = t.info()
    assert nnz == 0 and not counts.any() and chunks == 0
    c, items, fix = sa.sa_tensor_worklist(t.handle)
    assert sorted(fix[:, 0].tolist()) == [0, 1, 2, 3, 4] and not fix[:, 2].any()
    t1 = sa.SparseTensor((5, 4, 3), np.array([[4, 3, 2]], np.int32), np.ones(1, np.float32), sa.SA_FMT_CSF, device=-1)
    assert t1.info()[1].tolist() == [1, 1, 1]
    t2 = sa.SparseTensor((3, 3), np.zeros((0, 2), np.int32), np.zeros(0, np.float32), sa.SA_FMT_CSR, device=-1)
    assert t2.info()[0] == 0


def _create_status(order, dims, coords, vals, fmt):
    try:
        t = sa.SparseTensor(dims, np.asarray(coords, np.int32).reshape(-1, order), np.asarray(vals, np.float32), fmt,
                            device=-1)
        t.close()
        return sa.SA_OK
    except sa.SaError as e:
        return e.status


def test_malformed_input_is_rejected_with_a_status():
    assert _create_status(3, (4, 4, 4), [[0, 0, 4]], [1.0], sa.SA_FMT_CSF) == sa.SA_E_COORD_RANGE
    assert _create_status(3, (4, 4, 4), [[0, -1, 0]], [1.0], sa.SA_FMT_CSF) == sa.SA_E_COORD_RANGE
    assert _create_status(3, (4, 4, 4), [[1, 2, 3], [0, 0, 0], [1, 2, 3]], [1.0, 2.0, 3.0], sa.SA_FMT_CSF) == sa.SA_E_COORD_DUP
    assert _create_status(3, (4, 4, 4), [[1, 2, 3]], [1.0], sa.SA_FMT_CSR) == sa.SA_E_FORMAT
    assert _create_status(2, (4, 4), [[1, 2]], [1.0], sa.SA_FMT_CSF) == sa.SA_E_FORMAT
    assert _create_status(3, (4, 0, 4), [[1, 0, 3]], [1.0], sa.SA_FMT_CSF) == sa.SA_E_ARG
    assert _create_status(3, (4, 4, 4), [[1, 2, 3]], [1.0], 7) == sa.SA_E_ARG
    big = (2**30, 2**30, 2**30)     # 90 bits of packed coordinate
    assert _create_status(3, big, [[1, 2, 3]], [1.0], sa.SA_FMT_CSF) == sa.SA_E_UNSUPPORTED
    # order outside 2..4
    h = ctypes.c_void_p()
    dims = np.array([2] * 5, dtype=np.int64)
    st = sa._lib.sa_tensor_create(5, dims.ctypes.data, 0, None, None, sa.SA_FMT_CSF, -1, None, ctypes.byref(h))
    assert st == sa.SA_E_FORMAT and not h.value
    assert sa._lib.sa_tensor_create(3, None, 0, None, None, sa.SA_FMT_CSF, -1, None, ctypes.byref(h)) == sa.SA_E_ARG


def test_run_argument_checks_need_no_device():
    w = configs.make(1)
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSF, device=-1)
    good = [(16, 200, 16, 16), (16, 200, 16, 16)]
    assert sa.sa_workspace_size(t.handle, sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_DEFAULT, good) >= 0
    for expr, sched, ops, want in [
        (sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_DEFAULT, [(16, 199, 16, 16), (16, 200, 16, 16)], sa.SA_E_SHAPE),
        (sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_DEFAULT, [(16, 200, 24, 24), (16, 200, 16, 16)], sa.SA_E_UNSUPPORTED),
        (sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_ASSOC_LEFT, good, sa.SA_E_UNSUPPORTED),
        (sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_DEFAULT, good[:1], sa.SA_E_ARG),
        (sa.SA_EXPR_SDDMM_SPMM, sa.SA_SCHED_DEFAULT, good + good[:1], sa.SA_E_FORMAT),
        (99, sa.SA_SCHED_DEFAULT, good, sa.SA_E_ARG),
    ]:
        with pytest.raises(sa.SaError) as e:
            sa.sa_workspace_size(t.handle, expr, sched, ops)
        assert e.value.status == want
    # a host-only handle cannot run
    with pytest.raises(sa.SaError) as e:
        sa.sa_run(t.handle, sa.SA_EXPR_SPTTM_TTM3, sa.SA_SCHED_DEFAULT, good, 256, None, 0, None)
    assert e.value.status == sa.SA_E_ARG
    sa.sa_destroy(None)            # NULL-safe
    assert sa.sa_status_string(sa.SA_E_COORD_DUP) == "duplicate coordinate"


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "sparseauto.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(sa_[a-z_0-9]+)\s*\(", header)))
    assert declared and set(declared) == set(sa.EXPORTED_SYMBOLS)
    lib = ctypes.CDLL(sa.LIB_PATH)
    for name in declared:
        assert hasattr(lib, name), name


def test_fiber_row_worklist_of_order3_csf_partitions_fibers_and_nonzeros():
    """Kernel 7 walks an order-3 CSF tensor as a sparse matrix with one row per (i,j) fiber: its work list
    (the second one of the tensor) covers every fiber and every nonzero once; a fiber longer than 4096
    nonzeros is cut into pieces with partial rows."""
    w = configs.make(10, "mini")
    longf = np.stack([np.full(5000, 7), np.full(5000, 3), np.arange(5000)], axis=1).astype(np.int32)
    base = w.coords[~((w.coords[:, 0] == 7) & (w.coords[:, 1] == 3))]
    dims = (w.dims[0], w.dims[1], 5000)
    coords = np.concatenate([base, longf])
    vals = np.ones(coords.shape[0], np.float32)
    t = sa.SparseTensor(dims, coords, vals, sa.SA_FMT_CSF, device=-1)
    levels, _ = export_all(t, "csf")
    pos = levels[2][0]
    n_fibers = int(t.info()[1][1])
    counts, items, fix = sa.sa_tensor_worklist(t.handle, 1)
    covered = np.zeros(coords.shape[0], dtype=np.int32)
    rows = np.zeros(n_fibers, dtype=np.int32)
    for row, row_end, q1, q2, p0, p1, dest, q3 in items:
        if dest >= 0:
            assert row_end == row + 1 and pos[row] <= p0 < p1 <= pos[row + 1]
        else:
            assert (p0, p1) == (pos[row], pos[row_end])
            rows[row:row_end] += 1
            # the rows in which the item's quarters (equal counts of nonzeros) start
            share = -(-(p1 - p0) // 4)
            for q, got in ((1, q1), (2, q2), (3, q3)):
                at = min(p0 + q * share, p1)
                want = min(int(np.searchsorted(pos, at, side="right")) - 1, row_end - 1)
                assert got == want and row <= got < row_end, (row, row_end, q, got, want)
        covered[p0:p1] += 1
    assert (covered == 1).all()
    assert len(fix) == 1 and fix[0][2] == 3          # 5000 nonzeros in pieces of 2048
    for row, slot0, count, _ in fix:
        assert pos[row + 1] - pos[row] == 5000
        rows[row] += 1
    assert (rows == 1).all()
    # default order: with rank-32 matrices B'.(C.D) moves fewer bytes unless the mode-3 dimension dwarfs the nonzeros
    ops = [(16, dims[2], 32, 32), (16, 32, 32, 32)]
    ws = {s: sa.sa_workspace_size(t.handle, sa.SA_EXPR_SPTTM_SPTTM, s, ops)
          for s in (sa.SA_SCHED_DEFAULT, sa.SA_SCHED_FUSED, sa.SA_SCHED_ASSOC_LEFT, sa.SA_SCHED_ASSOC_RIGHT)}
    assert ws[sa.SA_SCHED_FUSED] == ws[sa.SA_SCHED_ASSOC_LEFT] >= n_fibers * 32 * 4
    assert ws[sa.SA_SCHED_DEFAULT] == ws[sa.SA_SCHED_ASSOC_RIGHT] >= dims[2] * 32 * 4


def test_order4_fissioned_second_pass_worklist_covers_every_fiber_quarter_once():
    """Fissioned schedule of the order-4 chain, list 5: (piece of a slice) x (quarter of the temporaries' columns)."""
    w = configs.make(5, "mini")
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSF, device=-1)
    levels, _ = export_all(t, "csf")
    crd0, pos1 = levels[0][1], levels[1][0]
    counts, items, fix = sa.sa_tensor_worklist(t.handle, 5)
    slice_pos = {int(c): n for n, c in enumerate(crd0)}
    covered = np.zeros((len(levels[1][1]), 4), dtype=np.int32)
    pieces = {}
    for row, row_end, f0, f1, _, _, dest, quarter in items:
        s = slice_pos[int(row)]
        assert pos1[s] <= f0 < f1 <= pos1[s + 1] and f1 - f0 <= 512 and 0 <= quarter <= 4
        if quarter == 4:
            assert f1 - f0 <= 8, "only a piece of one tensor-core group takes all four quarters in one item"
            covered[f0:f1, :] += 1
        else:
            assert f1 - f0 > 8
            covered[f0:f1, quarter] += 1
        if dest >= 0:
            pieces.setdefault(int(row), set()).add(int(dest))
        else:
            assert (f0, f1) == (pos1[s], pos1[s + 1])
    assert (covered == 1).all()
    assert (np.diff(items[:, 3] - items[:, 2]) <= 0).all(), "largest items first"
    empties = set()
    used = np.zeros(int(counts[3]), dtype=np.int32)
    for row, slot0, count, _ in fix:
        if count == 0:
            empties.add(int(row))
            continue
        assert pieces[int(row)] == set(range(slot0, slot0 + count))
        used[slot0:slot0 + count] += 1
    assert (used == 1).all()
    assert empties == set(range(w.dims[0])) - set(int(c) for c in crd0)


def test_order4_fissioned_subtree_worklist_covers_every_subtree_once_within_its_limits():
    """Fissioned schedule of the order-4 chain, list 6: ranges of whole small (i,j) subtrees, at most 64 level-2 fibers and 32
    subtrees each; a larger subtree is left to list 4 (the order-3 lists over those subtrees)."""
    w = configs.make(5, "mini")
    t = sa.SparseTensor(w.dims, w.coords, w.vals, sa.SA_FMT_CSF, device=-1)
    levels, _ = export_all(t, "csf")
    pos2, pos3 = levels[2][0], levels[3][0]
    counts, items, fix = sa.sa_tensor_worklist(t.handle, 6)
    assert counts[0] > 0 and counts[2] == 0 and counts[3] == 0
    n_sub = int(t.info()[1][1])
    seen = np.zeros(n_sub, dtype=np.int32)
    for row, row_end, f0, f1, p0, p1, dest, _ in items:
        assert row_end > row and dest < 0
        assert (f0, f1) == (pos2[row], pos2[row_end]) and (p0, p1) == (pos3[f0], pos3[f1])
        assert f1 - f0 <= 64 and row_end - row <= 32
        seen[row:row_end] += 1
    # the others are the large ones, and the main list holds exactly those
    large = np.nonzero(seen == 0)[0]
    assert (seen <= 1).all()
    f3s, nz = np.diff(pos2), pos3[pos2[1:]] - pos3[pos2[:-1]]
    assert ((f3s[large] > 64) | (nz[large] > 4096)).all() and ((f3s[seen == 1] <= 64) & (nz[seen == 1] <= 4096)).all()
    assert set(sa.sa_tensor_worklist(t.handle, 4)[1][:, 0].tolist()) == set(large.tolist())
    # one (i,j) pair with 130 level-2 fibers next to a small one: the large one is in the main list only
    big = np.stack([np.zeros(130), np.zeros(130), np.arange(130), np.zeros(130)], axis=1).astype(np.int32)
    both = np.concatenate([big, np.array([[1, 1, 5, 1]], np.int32)])
    t2 = sa.SparseTensor((2, 2, 130, 2), both, np.ones(131, np.float32), sa.SA_FMT_CSF, device=-1)
    sub = sa.sa_tensor_worklist(t2.handle, 6)[1]
    main = sa.sa_tensor_worklist(t2.handle, 4)[1]
    assert [tuple(x[:2]) for x in sub.tolist()] == [(1, 2)] and set(main[:, 0].tolist()) == {0}
