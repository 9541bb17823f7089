"""Seeded synthetic inputs for the five contraction-chain workloads.

Each ``make_*`` function returns a :class:`Workload`: shuffled COO coordinates and
values of the sparse operand B, the dense row-major operands, and the shapes.  The
"full" presets have the sizes and distributions of the benchmark configurations; the
"mini" presets use the same recipes at sizes a CPU evaluation finishes in seconds.

Recipes (all deterministic given the seed; streams: 0 structure, 1 values, 2 dense
operands, 3 COO shuffle):

* slice sizes "Zipf(alpha) over i": n_r = N * r^-alpha / H for rank r = 1..I, rounded by
  largest remainder to sum to N exactly; ranks are assigned to slice ids by a seeded
  permutation.
* fibers per parent: count = min(dim, max(1, round(n / mean))); the parent's n entries
  are split over them as 1 + (integer parts of cumulative exponential spacings), i.e.
  every fiber holds at least one entry, lengths are geometric-like with the requested
  mean and sum to n exactly.  Where the count hits the dimension cap the mean rises.
* coordinates inside a fiber / row are distinct and pseudo-uniform: the c-th child of a
  parent gets the image of c under a bijection of [0, dim) keyed by the parent.
* the COO list is handed out in a seeded random order, never sorted.

This module only draws inputs; it contains none of the contraction arithmetic.
"""
from dataclasses import dataclass, field
from concurrent.futures import ThreadPoolExecutor
import numpy as np

from . import rng

BASE_SEED = 20231109

S_STRUCT, S_VALS, S_DENSE, S_SHUFFLE = 0, 1, 2, 3


@dataclass
class Workload:
    name: str
    expr: str                  # 'spttm_ttm3' | 'spttm_ttm4' | 'sddmm_spmm' | 'spmm_gemm' | 'ttmc3' | 'sddmm_spmm_gemm' | 'spmmh_gemm'
    fmt: str                   # 'csf' | 'csr'
    dims: tuple                # dimensions of B
    coords: np.ndarray         # int32 [nnz, order], shuffled
    vals: np.ndarray           # float32 [nnz]
    dense: list                # float32 row-major operands, in expression order
    out_shape: tuple
    seed: int
    notes: dict = field(default_factory=dict)

    @property
    def nnz(self):
        return int(self.vals.shape[0])


# --------------------------------------------------------------------------- helpers

def zipf_sizes(total, count, alpha):
    """Deterministic Zipf sizes by rank (largest first), summing to ``total``."""
    r = np.arange(1, count + 1, dtype=np.float64)
    w = r ** (-alpha)
    x = total * (w / w.sum())
    n = np.floor(x).astype(np.int64)
    rem = int(total - n.sum())
    if rem > 0:
        frac = x - n
        order = np.argsort(-frac, kind="stable")[:rem]
        n[order] += 1
    return n


def _segment_ids(counts):
    return np.repeat(np.arange(counts.shape[0], dtype=np.int64), counts)


def _index_in_segment(counts):
    starts = np.cumsum(counts) - counts
    return np.arange(int(counts.sum()), dtype=np.int64) - np.repeat(starts, counts)


def split_totals(seed, stream, totals, parts, cap):
    """Split each totals[s] over parts[s] children, every child >= 1, child <= cap.

    Children get 1 + the increments of floor(extra * cumulative exponential weight /
    total weight), extra = totals - parts.  Returns the flat child sizes (parent-major).
    """
    totals = np.asarray(totals, dtype=np.int64)
    parts = np.asarray(parts, dtype=np.int64)
    assert np.all(parts <= totals) and np.all((parts > 0) | (totals == 0))
    nchild = int(parts.sum())
    if nchild == 0:
        return np.zeros(0, dtype=np.int64)
    seg = _segment_ids(parts)
    u = rng.uniform01(seed, stream, np.arange(nchild, dtype=np.uint64))
    w = -np.log1p(-u) + 1e-300
    cw = np.cumsum(w)
    starts = np.cumsum(parts) - parts
    nz = parts > 0
    base = np.zeros(parts.shape[0], dtype=np.float64)
    base[nz] = cw[starts[nz]] - w[starts[nz]]
    tot = np.zeros(parts.shape[0], dtype=np.float64)
    tot[nz] = cw[(starts + parts - 1)[nz]] - base[nz]
    extra = (totals - parts).astype(np.float64)
    rel = (cw - base[seg]) / tot[seg]
    last = np.zeros(nchild, dtype=bool)
    last[(starts + parts - 1)[nz]] = True
    rel[last] = 1.0
    c = np.floor(extra[seg] * rel).astype(np.int64)
    prev = np.empty_like(c)
    prev[0] = 0
    prev[1:] = c[:-1]
    prev[starts[nz]] = 0
    sizes = 1 + (c - prev)
    # rare: a child above the cap; push the excess onto its siblings
    if cap is not None and np.any(sizes > cap):
        for s in np.unique(seg[sizes > cap]):
            a, b = int(starts[s]), int(starts[s] + parts[s])
            v = sizes[a:b]
            assert v.sum() <= cap * v.shape[0], "parent cannot fit under the cap"
            excess = int(np.maximum(v - cap, 0).sum())
            v = np.minimum(v, cap)
            i = 0
            while excess > 0:
                room = int(cap - v[i])
                take = min(room, excess)
                v[i] += take
                excess -= take
                i += 1
            sizes[a:b] = v
    return sizes


def _parent_keys(seed, stream, n_parents):
    return rng.u64(seed, stream, np.arange(n_parents, dtype=np.uint64))


def distinct_children(seed, stream, counts, dim):
    """For every parent p, counts[p] distinct pseudo-uniform values in [0, dim)."""
    counts = np.asarray(counts, dtype=np.int64)
    assert counts.size == 0 or counts.max() <= dim
    keys = _parent_keys(seed, stream, counts.shape[0])
    return rng.keyed_bijection(_index_in_segment(counts), dim, np.repeat(keys, counts))


def _threaded(fn, n, chunk=1 << 22):
    bounds = [(a, min(n, a + chunk)) for a in range(0, n, chunk)]
    if len(bounds) <= 1:
        return [fn(a, b) for a, b in bounds]
    with ThreadPoolExecutor(max_workers=8) as ex:
        return list(ex.map(lambda ab: fn(*ab), bounds))


def dense_uniform(seed, which, rows, cols, lo=-1.0, hi=1.0):
    n = rows * cols
    out = np.empty(n, dtype=np.float32)

    def fill(a, b):
        out[a:b] = rng.uniform_f32(seed, S_DENSE + 16 * which, np.arange(a, b, dtype=np.uint64), lo, hi)
    _threaded(fill, n)
    return out.reshape(rows, cols)


def dense_normal(seed, which, rows, cols):
    n = rows * cols
    out = np.empty(n, dtype=np.float32)

    def fill(a, b):
        out[a:b] = rng.normal_f32(seed, S_DENSE + 16 * which, np.arange(a, b, dtype=np.uint64))
    _threaded(fill, n)
    return out.reshape(rows, cols)


def sparse_values(seed, nnz, lo, hi):
    out = np.empty(nnz, dtype=np.float32)

    def fill(a, b):
        out[a:b] = rng.uniform_f32(seed, S_VALS, np.arange(a, b, dtype=np.uint64), lo, hi)
    _threaded(fill, nnz)
    return out


def shuffle_coo(seed, cols, vals):
    """Return the COO entries in a seeded random order as (int32 [nnz, order], vals)."""
    nnz = vals.shape[0]
    perm = rng.permutation(seed, S_SHUFFLE, nnz)
    coords = np.empty((nnz, len(cols)), dtype=np.int32)
    for d, c in enumerate(cols):
        coords[:, d] = c[perm]
    return coords, vals[perm]


# --------------------------------------------------------------------------- recipes

def make_ttm3_uniform(name, seed, I, J, K, nnz, L, M):
    """Order-3 B with ``nnz`` distinct uniform coordinates; U(-1,1) values and factors."""
    lin = rng.keyed_bijection(np.arange(nnz, dtype=np.uint64), I * J * K, rng._base(seed, S_STRUCT))
    i, rem = np.divmod(lin, J * K)
    j, k = np.divmod(rem, K)
    vals = sparse_values(seed, nnz, -1.0, 1.0)
    coords, vals = shuffle_coo(seed, [i, j, k], vals)
    C = dense_uniform(seed, 0, J, L)
    D = dense_uniform(seed, 1, K, M)
    return Workload(name, "spttm_ttm3", "csf", (I, J, K), coords, vals, [C, D], (I, L, M), seed)


def _zipf_slices(seed, I, nnz, alpha):
    by_rank = zipf_sizes(nnz, I, alpha)
    ids = rng.permutation(seed, S_STRUCT + 100, I)
    n = np.zeros(I, dtype=np.int64)
    n[ids] = by_rank
    return n


def _fiber_counts(n, mean, dim, child_cap):
    f = np.minimum(dim, np.maximum(1, np.rint(n / mean).astype(np.int64)))
    f = np.minimum(f, n)                       # a fiber holds at least one entry
    # a parent must fit: n <= f * child_cap
    need = -(-n // child_cap)
    return np.maximum(f, need)


def make_ttm3_zipf(name, seed, I, J, K, nnz, alpha, mean_fiber, L, M):
    """Order-3 CSF workload: Zipf slice sizes, geometric-like fiber lengths."""
    n_i = _zipf_slices(seed, I, nnz, alpha)
    f_i = _fiber_counts(n_i, mean_fiber, J, K)
    assert np.all(f_i <= J)
    flen = split_totals(seed, S_STRUCT + 1, n_i, f_i, K)
    j_f = distinct_children(seed, S_STRUCT + 2, f_i, J)
    i_f = _segment_ids(f_i)
    k_p = distinct_children(seed, S_STRUCT + 3, flen, K)
    i_p = np.repeat(i_f, flen)
    j_p = np.repeat(j_f, flen)
    vals = sparse_values(seed, nnz, -1.0, 1.0)
    coords, vals = shuffle_coo(seed, [i_p, j_p, k_p], vals)
    C = dense_uniform(seed, 0, J, L)
    D = dense_uniform(seed, 1, K, M)
    notes = {"fibers": int(f_i.sum()), "max_slice": int(n_i.max()), "nonempty_slices": int((n_i > 0).sum())}
    return Workload(name, "spttm_ttm3", "csf", (I, J, K), coords, vals, [C, D], (I, L, M), seed, notes)


def make_ttmc3_zipf(name, seed, I, J, K, nnz, alpha, mean_fiber, L, M, N):
    """Kernel 5 workload: the order-3 Zipf tensor of make_ttm3_zipf with a factor matrix per mode."""
    w = make_ttm3_zipf(name, seed, I, J, K, nnz, alpha, mean_fiber, M, N)      # D (J x M), E (K x N)
    C = dense_uniform(seed, 2, I, L)
    return Workload(name, "ttmc3", "csf", (I, J, K), w.coords, w.vals, [C] + w.dense, (L, M, N), seed, w.notes)


def make_ttm4_zipf(name, seed, I, J, K, O, nnz, alpha, mean_fiber, L, M, N):
    """Order-4 CSF workload: Zipf slices, geometric-like fan-out (mean ``mean_fiber``) per level."""
    n_i = _zipf_slices(seed, I, nnz, alpha)
    f2_i = _fiber_counts(n_i, mean_fiber * mean_fiber, J, K * O)
    assert np.all(f2_i <= J)
    n_ij = split_totals(seed, S_STRUCT + 1, n_i, f2_i, K * O)
    j_f = distinct_children(seed, S_STRUCT + 2, f2_i, J)
    i_f = _segment_ids(f2_i)
    f3_ij = _fiber_counts(n_ij, mean_fiber, K, O)
    assert np.all(f3_ij <= K)
    n_ijk = split_totals(seed, S_STRUCT + 3, n_ij, f3_ij, O)
    k_g = distinct_children(seed, S_STRUCT + 4, f3_ij, K)
    o_p = distinct_children(seed, S_STRUCT + 5, n_ijk, O)
    i_g = np.repeat(i_f, f3_ij)
    j_g = np.repeat(j_f, f3_ij)
    i_p = np.repeat(i_g, n_ijk)
    j_p = np.repeat(j_g, n_ijk)
    k_p = np.repeat(k_g, n_ijk)
    vals = sparse_values(seed, nnz, -1.0, 1.0)
    coords, vals = shuffle_coo(seed, [i_p, j_p, k_p, o_p], vals)
    C = dense_uniform(seed, 0, J, L)
    D = dense_uniform(seed, 1, K, M)
    E = dense_uniform(seed, 2, O, N)
    notes = {"fibers2": int(f2_i.sum()), "fibers3": int(f3_ij.sum()), "max_slice": int(n_i.max())}
    return Workload(name, "spttm_ttm4", "csf", (I, J, K, O), coords, vals, [C, D, E], (I, L, M, N), seed, notes)


def powerlaw_degrees(total, rows, alpha, cap):
    """Rank-Zipf degrees deg_r = min(cap, s * r^-alpha), s chosen so they sum to ``total``."""
    r = np.arange(1, rows + 1, dtype=np.float64) ** (-alpha)
    assert total <= cap * rows
    lo, hi = 0.0, float(cap) * float(rows) ** alpha + 1.0
    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if np.minimum(cap, mid * r).sum() < total:
            lo = mid
        else:
            hi = mid
    x = np.minimum(cap, hi * r)
    d = np.floor(x).astype(np.int64)
    rem = int(total - d.sum())
    if rem > 0:
        frac = np.where(d < cap, x - d, -1.0)
        d[np.argsort(-frac, kind="stable")[:rem]] += 1
    elif rem < 0:
        idx = np.nonzero(d > 0)[0][::-1][:(-rem)]
        d[idx] -= 1
    assert d.sum() == total and d.max() <= cap
    return d


def _csr_workload(name, expr, seed, I, J, deg, val_lo, val_hi):
    j_p = distinct_children(seed, S_STRUCT + 2, deg, J)
    i_p = _segment_ids(deg)
    vals = sparse_values(seed, int(deg.sum()), val_lo, val_hi)
    return shuffle_coo(seed, [i_p, j_p], vals)


def make_sddmm_spmm(name, seed, I, J, nnz, alpha, cap, K, L):
    """CSR B with rank-Zipf row degrees; U(0,1) values; N(0,1) dense operands."""
    by_rank = powerlaw_degrees(nnz, I, alpha, min(cap, J))
    ids = rng.permutation(seed, S_STRUCT + 100, I)
    deg = np.zeros(I, dtype=np.int64)
    deg[ids] = by_rank
    coords, vals = _csr_workload(name, "sddmm_spmm", seed, I, J, deg, 0.0, 1.0)
    C = dense_normal(seed, 0, I, K)
    D = dense_normal(seed, 1, J, K)
    E = dense_normal(seed, 2, J, L)
    notes = {"max_degree": int(deg.max()), "nonempty_rows": int((deg > 0).sum())}
    return Workload(name, "sddmm_spmm", "csr", (I, J), coords, vals, [C, D, E], (I, L), seed, notes)


def poisson_degrees(seed, rows, mean, total, cap):
    """Poisson(mean) degrees by inverse CDF, then +-1 adjustments on seeded rows to hit ``total``."""
    kmax = int(mean + 12.0 * np.sqrt(mean) + 20)
    k = np.arange(kmax + 1, dtype=np.float64)
    logp = -mean + k * np.log(mean) - np.cumsum(np.log(np.maximum(k, 1.0)))
    cdf = np.cumsum(np.exp(logp))
    u = rng.uniform01(seed, S_STRUCT + 1, np.arange(rows, dtype=np.uint64))
    d = np.minimum(np.searchsorted(cdf, u, side="right"), cap).astype(np.int64)
    diff = int(total - d.sum())
    order = rng.permutation(seed, S_STRUCT + 6, rows)
    step = 1 if diff > 0 else -1
    pos = 0
    while diff != 0:
        take = order[pos:pos + abs(diff)]
        pos += take.shape[0]
        if pos >= rows:
            pos = 0
        ok = take[(d[take] + step >= 0) & (d[take] + step <= cap)]
        d[ok] += step
        diff -= step * ok.shape[0]
    return d


def make_spmm_gemm(name, seed, I, J, nnz, L, M):
    """CSR B with Poisson row degrees, uniform distinct columns; N(0,1) dense operands."""
    deg = poisson_degrees(seed, I, nnz / I, nnz, J)
    coords, vals = _csr_workload(name, "spmm_gemm", seed, I, J, deg, -1.0, 1.0)
    C = dense_normal(seed, 0, J, L)
    D = dense_normal(seed, 1, L, M)
    notes = {"max_degree": int(deg.max())}
    return Workload(name, "spmm_gemm", "csr", (I, J), coords, vals, [C, D], (I, M), seed, notes)


# --------------------------------------------------------------------------- presets

def make(config, scale="full", seed=None):
    """Build workload ``config`` (1..5) at ``scale`` 'full' or 'mini' ('mid', a quarter-size profiling case, exists for configs 2, 4, 5 and 8)."""
    config = int(config)
    s = BASE_SEED + config if seed is None else int(seed)
    full = scale == "full"
    if config == 1:
        return make_ttm3_uniform("cfg1-ttm3-uniform", s, 200, 200, 200, 20000, 16, 16)
    if config == 2:
        if full:
            return make_ttm3_zipf("cfg2-ttm3-zipf", s, 100000, 80000, 80000, 50_000_000, 1.2, 8.0, 32, 32)
        if scale == "mid":      # a quarter of the slices and nonzeros, same factor tables (profiling case)
            return make_ttm3_zipf("cfg2-ttm3-zipf-mid", s, 25000, 80000, 80000, 12_500_000, 1.2, 8.0, 32, 32)
        return make_ttm3_zipf("cfg2-ttm3-zipf-mini", s, 3000, 700, 900, 250_000, 1.2, 8.0, 32, 32)
    if config == 3:
        if full:
            return make_sddmm_spmm("cfg3-sddmm-spmm", s, 1_000_000, 1_000_000, 30_000_000, 1.5, 50_000, 64, 64)
        return make_sddmm_spmm("cfg3-sddmm-spmm-mini", s, 20_000, 20_000, 300_000, 1.5, 3_000, 64, 64)
    if config == 4:
        if full:
            return make_spmm_gemm("cfg4-spmm-gemm", s, 4_000_000, 4_000_000, 100_000_000, 256, 64)
        if scale == "mid":      # a quarter of the full size: same row law, C still 8x larger than L2 (profiling case)
            return make_spmm_gemm("cfg4-spmm-gemm-mid", s, 1_000_000, 1_000_000, 25_000_000, 256, 64)
        return make_spmm_gemm("cfg4-spmm-gemm-mini", s, 12_000, 12_000, 300_000, 256, 64)
    if config == 5:
        if full:
            return make_ttm4_zipf("cfg5-ttm4-zipf", s, 50_000, 20_000, 20_000, 20_000, 100_000_000,
                                  1.2, 6.0, 16, 16, 16)
        if scale == "mid":      # a quarter of the slices and nonzeros, same factor tables (profiling case)
            return make_ttm4_zipf("cfg5-ttm4-zipf-mid", s, 12_500, 20_000, 20_000, 20_000, 25_000_000,
                                  1.2, 6.0, 16, 16, 16)
        return make_ttm4_zipf("cfg5-ttm4-zipf-mini", s, 600, 150, 120, 130, 200_000, 1.2, 6.0, 16, 16, 16)
    if config == 6:
        # kernel 5 (all-mode TTMC) on a tensor with the shape and size the paper quotes for nell-2
        if full:
            return make_ttmc3_zipf("cfg6-ttmc3-nell2-shaped", s, 12_000, 9_000, 288_000, 76_880_000, 1.2, 8.0, 16, 16, 16)
        return make_ttmc3_zipf("cfg6-ttmc3-mini", s, 300, 200, 250, 60_000, 1.2, 8.0, 16, 16, 16)
    if config == 11:
        # kernel 5 on a tensor with the shape and size the paper quotes for flickr-3d: many more slices than
        # nell-2, so the slice temporaries of the fissioned schedule (I x M x N floats) weigh as much as B itself
        if full:
            return make_ttmc3_zipf("cfg11-ttmc3-flickr-shaped", s, 320_000, 2_820_000, 1_600_000, 112_890_000, 1.2, 8.0, 16, 16, 16)
        return make_ttmc3_zipf("cfg11-ttmc3-mini", s, 3000, 2000, 1500, 60_000, 1.2, 8.0, 16, 16, 16)
    if config == 7:
        # kernel 2 (SDDMM, SpMM, GEMM) on the tensor of config 3 with a 64 x 64 weight matrix F
        if full:
            w = make(3, "full", seed=s)
            F = dense_normal(s, 3, 64, 64)
            return Workload("cfg7-sddmm-spmm-gemm", "sddmm_spmm_gemm", "csr", w.dims, w.coords, w.vals, w.dense + [F],
                            (w.dims[0], 64), s, w.notes)
        w = make_sddmm_spmm("tmp", s, 6_000, 6_000, 60_000, 1.5, 1_500, 32, 32)
        F = dense_normal(s, 3, 32, 32)
        return Workload("cfg7-sddmm-spmm-gemm-mini", "sddmm_spmm_gemm", "csr", w.dims, w.coords, w.vals, w.dense + [F],
                        (w.dims[0], 32), s, w.notes)
    if config == 8:
        # kernel 3 (SpMMH, GEMM): the tensor recipe of config 4 with a second J x L matrix for the Hadamard product
        if full:
            w = make_spmm_gemm("tmp", s, 4_000_000, 4_000_000, 100_000_000, 256, 64)
        elif scale == "mid":
            w = make_spmm_gemm("tmp", s, 1_000_000, 1_000_000, 25_000_000, 256, 64)
        else:
            w = make_spmm_gemm("tmp", s, 9_000, 9_000, 200_000, 128, 32)
        C, E = w.dense
        D = dense_normal(s, 2, C.shape[0], C.shape[1])
        return Workload("cfg8-spmmh-gemm" + ("" if full else "-" + scale), "spmmh_gemm", "csr", w.dims, w.coords, w.vals,
                        [C, D, E], w.out_shape, s, w.notes)
    if config == 9:
        # kernel 8 (MTTKRP, GEMM): the tensor of config 2 with rank-32 factors and a 32 x 32 weight matrix E
        if full:
            w = make_ttm3_zipf("tmp", s, 100000, 80000, 80000, 50_000_000, 1.2, 8.0, 32, 32)
        else:
            w = make_ttm3_zipf("tmp", s, 2500, 600, 800, 200_000, 1.2, 8.0, 32, 32)
        E = dense_uniform(s, 2, 32, 32)
        return Workload("cfg9-mttkrp-gemm" + ("" if full else "-mini"), "mttkrp_gemm", "csf", w.dims, w.coords, w.vals,
                        w.dense + [E], (w.dims[0], 32), s, w.notes)
    if config == 10:
        # kernel 7 (SpTTM, SpTTM): the tensor of config 2, C = 80000 x 32 (rows by k), D = 32 x 32; the output has
        # one row of 32 values per (i,j) fiber of B
        if full:
            w = make_ttm3_zipf("tmp", s, 100000, 80000, 80000, 50_000_000, 1.2, 8.0, 32, 32)
        else:
            w = make_ttm3_zipf("tmp", s, 2500, 600, 800, 200_000, 1.2, 8.0, 32, 32)
        D = dense_uniform(s, 2, 32, 32)
        key = w.coords[:, 0].astype(np.int64) * int(w.dims[1]) + w.coords[:, 1]
        f2 = int(np.unique(key).shape[0])
        return Workload("cfg10-spttm-spttm" + ("" if full else "-mini"), "spttm_spttm", "csf", w.dims, w.coords, w.vals,
                        [w.dense[1], D], (f2, 32), s, w.notes)
    raise ValueError("config must be 1..11")
