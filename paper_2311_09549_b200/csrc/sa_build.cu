// Host-side construction of the compressed levels (Section 2.1 of the paper: CSR / CSF as a
// tree of levels, arrays named pos / crd / vals as in Fig. 1b) and of the load-balancing work
// lists (nonzero-balanced pieces of slices, fibers and rows) the kernels consume.
#include <algorithm>
#include <cstring>
#include <omp.h>

#include "sa_internal.h"

namespace {

int bits_for(int64_t dim)
{
    int b = 1;
    while ((int64_t(1) << b) < dim) ++b;
    return b;
}

// Stable LSD radix sort of (key, idx) pairs on the low `total_bits` bits, 11 bits per pass.
void radix_sort(std::vector<uint64_t> &keys, std::vector<uint32_t> &idx, int total_bits)
{
    const size_t n = keys.size();
    if (n < 2) return;
    constexpr int DB = 11, NB = 1 << DB;
    const int passes = (total_bits + DB - 1) / DB;
    std::vector<uint64_t> k2(n);
    std::vector<uint32_t> i2(n);
    const int nt = std::max(1, omp_get_max_threads());
    std::vector<size_t> hist(size_t(nt) * NB);
    uint64_t *ks = keys.data(), *kd = k2.data();
    uint32_t *is = idx.data(), *id = i2.data();
    for (int pass = 0; pass < passes; ++pass) {
        const int shift = pass * DB;
#pragma omp parallel num_threads(nt)
        {
            const int tid = omp_get_thread_num();
            const size_t a = n * size_t(tid) / nt, b = n * size_t(tid + 1) / nt;
            size_t *h = hist.data() + size_t(tid) * NB;
            std::fill(h, h + NB, size_t(0));
            for (size_t p = a; p < b; ++p) ++h[(ks[p] >> shift) & (NB - 1)];
#pragma omp barrier
#pragma omp single
            {
                size_t run = 0;
                for (int d = 0; d < NB; ++d)
                    for (int t = 0; t < nt; ++t) {
                        size_t c = hist[size_t(t) * NB + d];
                        hist[size_t(t) * NB + d] = run;
                        run += c;
                    }
            }
            for (size_t p = a; p < b; ++p) {
                size_t q = h[(ks[p] >> shift) & (NB - 1)]++;
                kd[q] = ks[p];
                id[q] = is[p];
            }
        }
        std::swap(ks, kd);
        std::swap(is, id);
    }
    if (ks != keys.data()) {
        std::memcpy(keys.data(), ks, n * sizeof(uint64_t));
        std::memcpy(idx.data(), is, n * sizeof(uint32_t));
    }
}

}  // namespace

sa_status sa_build_levels(sa_tensor *t, const int32_t *coords, const float *vals)
{
    const int order = t->order;
    const int64_t nnz = t->nnz;
    int bits[SA_MAX_ORDER], shift[SA_MAX_ORDER];
    int total = 0;
    for (int d = 0; d < order; ++d) total += (bits[d] = bits_for(t->dims[d]));
    if (total > 64) return SA_E_UNSUPPORTED;
    for (int d = 0, s = total; d < order; ++d) { s -= bits[d]; shift[d] = s; }

    std::vector<uint64_t> keys;
    std::vector<uint32_t> idx;
    try {
        keys.resize(size_t(nnz));
        idx.resize(size_t(nnz));
    } catch (...) { return SA_E_ALLOC; }

    int bad = 0;
#pragma omp parallel for reduction(| : bad) schedule(static)
    for (int64_t p = 0; p < nnz; ++p) {
        uint64_t k = 0;
        for (int d = 0; d < order; ++d) {
            const int64_t c = coords[p * order + d];
            if (c < 0 || c >= t->dims[d]) bad |= 1;
            k |= uint64_t(uint32_t(c)) << shift[d];
        }
        keys[size_t(p)] = k;
        idx[size_t(p)] = uint32_t(p);
    }
    if (bad) return SA_E_COORD_RANGE;

    radix_sort(keys, idx, total);

    int dup = 0;
#pragma omp parallel for reduction(| : dup) schedule(static)
    for (int64_t p = 1; p < nnz; ++p)
        if (keys[size_t(p)] == keys[size_t(p - 1)]) dup |= 1;
    if (dup) return SA_E_COORD_DUP;

    try {
        t->vals.resize(size_t(nnz));
#pragma omp parallel for schedule(static)
        for (int64_t p = 0; p < nnz; ++p) t->vals[size_t(p)] = vals[idx[size_t(p)]];
        std::vector<uint32_t>().swap(idx);

        const int last = order - 1;
        auto coord_of = [&](uint64_t k, int d) { return int32_t((k >> shift[d]) & ((uint64_t(1) << bits[d]) - 1)); };

        if (t->fmt == SA_FMT_CSR) {
            const int64_t I = t->dims[0];
            t->count[0] = I;
            t->count[1] = nnz;
            t->pos[1].assign(size_t(I) + 1, 0);
            t->crd[1].resize(size_t(nnz));
            for (int64_t p = 0; p < nnz; ++p) {
                t->pos[1][size_t(coord_of(keys[size_t(p)], 0)) + 1]++;
                t->crd[1][size_t(p)] = coord_of(keys[size_t(p)], 1);
            }
            for (int64_t i = 0; i < I; ++i) t->pos[1][size_t(i) + 1] += t->pos[1][size_t(i)];
        } else {
            // prefix of level l = key >> shift[l]; a new node opens at every level >= the first
            // level whose prefix differs from the previous entry's
            for (int l = 0; l <= last; ++l) { t->crd[l].clear(); t->pos[l].clear(); }
            t->crd[last].resize(size_t(nnz));
            for (int64_t p = 0; p < nnz; ++p) {
                const uint64_t k = keys[size_t(p)];
                int first = 0;
                if (p > 0) {
                    const uint64_t diff = k ^ keys[size_t(p - 1)];
                    first = last;
                    for (int l = 0; l < last; ++l)
                        if ((diff >> shift[l]) != 0) { first = l; break; }
                }
                for (int l = first; l < last; ++l) {
                    t->pos[l + 1].push_back(int64_t(l + 1 == last ? p : int64_t(t->crd[l + 1].size())));
                    t->crd[l].push_back(coord_of(k, l));
                }
                t->crd[last][size_t(p)] = coord_of(k, last);
            }
            for (int l = 0; l <= last; ++l) t->count[l] = int64_t(t->crd[l].size());
            for (int l = 0; l < last; ++l) t->pos[l + 1].push_back(t->count[l + 1]);
            t->pos[0] = {0, t->count[0]};
        }
    } catch (...) { return SA_E_ALLOC; }
    return SA_OK;
}

// ------------------------------------------------------------------------------ work lists

namespace {

sa_item empty_item()
{
    sa_item it;
    it.out_row = 0; it.row_end = 0; it.f0 = 0; it.f1 = 0; it.p0 = 0; it.p1 = 0; it.dest = -1; it.pad = 0;
    return it;
}

struct group_rec { int64_t len; std::vector<sa_item> items; };

// Chunk of nonzeros one CTA reduces into a single tile: at least min_chunk, and large enough that
// a slice is cut into at most max_parts partial tiles.
int64_t chunk_for(int64_t n, int64_t min_chunk, int64_t max_parts)
{
    int64_t c = (n + max_parts - 1) / max_parts;
    c = ((c + min_chunk - 1) / min_chunk) * min_chunk;
    return std::max(c, min_chunk);
}

void append_empty_slices(sa_tensor *t, sa_worklist &wl)
{
    const int64_t I = t->dims[0];
    size_t s = 0;
    for (int64_t i = 0; i < I; ++i) {
        if (s < t->crd[0].size() && t->crd[0][s] == i) { ++s; continue; }
        wl.fix.push_back(sa_fix{int32_t(i), 0, 0, 0});
    }
}

// Order-3 CSF.  An item ("unit") is a piece [p0, p1) of one slice with the fibers [f0, f1) it touches (a
// fiber may be cut between two units, each adds its part).  Slices above SMALL_MAX nonzeros are cut into
// chunks; the SA_TTM3_WARPS warps of a thread block take equal pieces of a chunk and reduce their tiles on chip.
// Smaller slices are one unit each; a warp evaluates a task of up to MAX_UNITS such units, about
// SMALL_MAX nonzeros in total.  Inside a unit the warp's SA_STREAMS lane groups stream the parts given by
// sa_unit3_streams; stream_f0 holds the fiber in which each part starts.
// `n_slices` slices; slice s is output row row_of(s), owns the fibers [pos1[s], pos1[s + 1]) whose nonzeros are
// [pos2[f], pos2[f + 1]).  (Order 3: the slices of the tensor.  Order 4: the (i,j) subtrees, whose "fibers" are
// the (i,j,k) fibers; output row = index of the (i,j) fiber.)
template <typename RowOf, typename Skip>
void build_ttm3_lists(sa_worklist &wl, int64_t n_slices, RowOf row_of, Skip skip, const std::vector<int64_t> &pos1,
                      const std::vector<int64_t> &pos2)
{
    constexpr int64_t SMALL_MAX = 2048, MIN_CHUNK = 8192, MAX_PARTS = 192, MAX_UNITS = 16;
    std::vector<sa_item> small;
    std::vector<group_rec> groups;
    for (int64_t s = 0; s < n_slices; ++s) {
        if (skip(s)) continue;                    // evaluated by another kernel
        const int64_t fa = pos1[size_t(s)], fb = pos1[size_t(s) + 1];
        const int64_t pa = pos2[size_t(fa)], pb = pos2[size_t(fb)];
        const int64_t n = pb - pa;
        const int32_t row = row_of(s);
        if (n <= SMALL_MAX) {
            sa_item it = empty_item();
            it.out_row = row; it.row_end = row + 1; it.pad = int32_t(s);
            it.f0 = int32_t(fa); it.f1 = int32_t(fb); it.p0 = int32_t(pa); it.p1 = int32_t(pb);
            small.push_back(it);
            continue;
        }
        const int64_t chunk = chunk_for(n, MIN_CHUNK, MAX_PARTS);
        const int64_t ng = (n + chunk - 1) / chunk;
        int32_t slot0 = -1;
        if (ng > 1) {
            slot0 = int32_t(wl.n_slots);
            wl.fix.push_back(sa_fix{row, slot0, int32_t(ng), 0});
            wl.n_slots += ng;
        }
        for (int64_t g = 0; g < ng; ++g) {
            const int64_t ga = pa + g * chunk, gb = std::min(pb, ga + chunk);
            int64_t piece = (gb - ga + SA_TTM3_WARPS - 1) / SA_TTM3_WARPS;
            piece = (piece + 31) / 32 * 32;
            group_rec rec;
            rec.len = gb - ga;
            for (int w = 0; w < SA_TTM3_WARPS; ++w) {
                const int64_t qa = std::min(gb, ga + w * piece), qb = std::min(gb, qa + piece);
                if (qa >= qb) break;              // the remaining warps of this block have nothing to do
                sa_item it = empty_item();
                it.out_row = row; it.row_end = row + 1; it.pad = int32_t(s);
                it.dest = ng > 1 ? slot0 + int32_t(g) : -1;
                // fiber holding nonzero qa, and one past the fiber holding nonzero qb - 1
                const int64_t f0 = (std::upper_bound(pos2.begin() + fa, pos2.begin() + fb + 1, qa) - pos2.begin()) - 1;
                const int64_t f1 = (std::upper_bound(pos2.begin() + fa, pos2.begin() + fb + 1, qb - 1) - pos2.begin());
                it.f0 = int32_t(f0); it.f1 = int32_t(f1); it.p0 = int32_t(qa); it.p1 = int32_t(qb);
                rec.items.push_back(it);
            }
            groups.push_back(std::move(rec));
        }
    }
    std::stable_sort(groups.begin(), groups.end(), [](const group_rec &a, const group_rec &b) { return a.len > b.len; });
    std::stable_sort(small.begin(), small.end(),
                     [](const sa_item &a, const sa_item &b) { return (a.p1 - a.p0) > (b.p1 - b.p0); });
    wl.n_group_ctas = int64_t(groups.size());
    wl.task_start.clear();
    for (auto &g : groups)
        for (int w = 0; w < SA_TTM3_WARPS; ++w) {
            wl.task_start.push_back(int32_t(wl.items.size()));
            if (size_t(w) < g.items.size()) wl.items.push_back(g.items[size_t(w)]);
        }
    // a task strings several small slices together only when there are enough of them to fill the machine
    // (a few thousand warps) anyway
    const int64_t max_units = std::min<int64_t>(MAX_UNITS, std::max<int64_t>(1, int64_t(small.size()) / 4096));
    for (size_t x = 0; x < small.size();) {
        wl.task_start.push_back(int32_t(wl.items.size()));
        int64_t total = 0, cnt = 0;
        while (x < small.size() && cnt < max_units && (cnt == 0 || total + (small[x].p1 - small[x].p0) <= SMALL_MAX)) {
            total += small[x].p1 - small[x].p0;
            wl.items.push_back(small[x]);
            ++x; ++cnt;
        }
    }
    wl.task_start.push_back(int32_t(wl.items.size()));
    wl.stream_f0.resize(wl.items.size() * SA_STREAMS);
    for (size_t u = 0; u < wl.items.size(); ++u) {
        const sa_item &it = wl.items[u];
        int64_t lo[SA_STREAMS], hi[SA_STREAMS];
        sa_unit3_streams(it.p0, it.p1, lo, hi);
        for (int q = 0; q < SA_STREAMS; ++q) {
            int64_t f = it.f0;
            if (lo[q] < hi[q])
                f = (std::upper_bound(pos2.begin() + it.f0, pos2.begin() + it.f1 + 1, lo[q]) - pos2.begin()) - 1;
            wl.stream_f0[u * SA_STREAMS + size_t(q)] = int32_t(f);
        }
    }
}

void build_ttm3(sa_tensor *t, sa_worklist &wl)
{
    build_ttm3_lists(wl, t->count[0], [&](int64_t s) { return t->crd[0][size_t(s)]; }, [](int64_t) { return false; }, t->pos[1],
                     t->pos[2]);
    append_empty_slices(t, wl);
}


// A subtree (i,j) that the subtree kernel of pass 1 can take whole.
static bool subtree_is_small(const sa_tensor *t, int64_t f2)
{
    const auto &pos2 = t->pos[2], &pos3 = t->pos[3];
    const int64_t fa = pos2[size_t(f2)], fb = pos2[size_t(f2) + 1];
    return fb - fa <= SA_SUB_MAX_F3 && pos3[size_t(fb)] - pos3[size_t(fa)] <= SA_SUB_MAX_NNZ;
}

// Order-4 CSF, schedule SA_SCHED_FISSIONED: the chain is evaluated in two passes (see sa_ttm4_fis.cu).  Pass 1 runs the order-3 kernel with
// the large (i,j) subtrees as slices: `wl` gets the same lists as an order-3 tensor whose slices are those
// level-1 fibers (output row = fiber index); the small subtrees go to the subtree kernel's list.  Pass 2 contracts the per-fiber temporaries of each slice with rows of
// C: `wl2` holds one item per (piece of a slice, quarter of the 256 temporaries' columns); a slice with more
// than CHUNK_F fibers is cut into pieces whose partial tiles the fix-up kernel sums.
void build_ttm4_fissioned(sa_tensor *t, sa_worklist &wl, sa_worklist &wl2)
{
    build_ttm3_lists(wl, t->count[1], [](int64_t f) { return int32_t(f); }, [&](int64_t f) { return subtree_is_small(t, f); },
                     t->pos[2], t->pos[3]);
    constexpr int64_t CHUNK_F = 512;
    const auto &pos1 = t->pos[1];
    std::vector<sa_item> items;
    for (int64_t s = 0; s < t->count[0]; ++s) {
        const int64_t fa = pos1[size_t(s)], fb = pos1[size_t(s) + 1];
        const int32_t row = t->crd[0][size_t(s)];
        const int64_t nc = (fb - fa + CHUNK_F - 1) / CHUNK_F;
        int32_t slot0 = -1;
        if (nc > 1) {
            slot0 = int32_t(wl2.n_slots);
            wl2.fix.push_back(sa_fix{row, slot0, int32_t(nc), 0});
            wl2.n_slots += nc;
        }
        for (int64_t c = 0; c < nc; ++c) {
            const int64_t f0 = fa + c * CHUNK_F, f1 = std::min(fb, fa + (c + 1) * CHUNK_F);
            // a piece of at most eight fibers (one tensor-core group) is one item that takes the four quarters in turn
            const int nq = f1 - f0 <= 8 ? 1 : 4;
            for (int qc = 0; qc < nq; ++qc) {
                sa_item it = empty_item();
                it.out_row = row; it.row_end = row + 1;
                it.f0 = int32_t(f0); it.f1 = int32_t(f1);
                it.p0 = it.f0; it.p1 = it.f1;          // size key: fibers
                it.dest = nc > 1 ? slot0 + int32_t(c) : -1;
                it.pad = nq == 1 ? 4 : qc;
                items.push_back(it);
            }
        }
    }
    // largest first: the tail of the launch is then made of the cheapest items
    std::stable_sort(items.begin(), items.end(), [](const sa_item &a, const sa_item &b) { return (a.f1 - a.f0) > (b.f1 - b.f0); });
    wl2.items = std::move(items);
    wl2.n_group_ctas = 0;
    append_empty_slices(t, wl2);
}

// Order 4, pass 1 on whole (i,j) subtrees: items are ranges of consecutive small subtrees (subtree_is_small) with
// at most SA_SUB_MAX_F3 level-2 fibers, SA_SUB_MAX_ROWS subtrees and about 512 nonzeros (f0/f1 = the fibers,
// p0/p1 = the nonzeros).  No subtree is cut, so there are no partial tiles; the large subtrees are in the main list.
void build_ttm4_subtrees(sa_tensor *t, sa_worklist &wl)
{
    const auto &pos2 = t->pos[2], &pos3 = t->pos[3];
    const int64_t F2 = t->count[1];
    constexpr int64_t TARGET_NNZ = 512;
    auto nnz_at = [&](int64_t f2) { return pos3[size_t(pos2[size_t(f2)])]; };
    std::vector<sa_item> items;
    int64_t r0 = 0;
    auto flush = [&](int64_t r1) {
        if (r1 > r0) {
            sa_item it = empty_item();
            it.out_row = int32_t(r0); it.row_end = int32_t(r1);
            it.f0 = int32_t(pos2[size_t(r0)]); it.f1 = int32_t(pos2[size_t(r1)]);
            it.p0 = int32_t(nnz_at(r0)); it.p1 = int32_t(nnz_at(r1));
            items.push_back(it);
        }
        r0 = r1;
    };
    for (int64_t r = 0; r < F2; ++r) {
        if (!subtree_is_small(t, r)) {
            flush(r);
            r0 = r + 1;
            continue;
        }
        if (r > r0 && (pos2[size_t(r) + 1] - pos2[size_t(r0)] > SA_SUB_MAX_F3 || r - r0 >= SA_SUB_MAX_ROWS ||
                       nnz_at(r + 1) - nnz_at(r0) > TARGET_NNZ))
            flush(r);
    }
    flush(F2);
    for (const sa_item &it : items) wl.nnz += it.p1 - it.p0;
    wl.items = std::move(items);
    wl.n_group_ctas = 0;
}

// Order-4 CSF (see sa_ttm4.cu).  The chain runs as one fused kernel over *pieces*: contiguous ranges of (i,j)
// subtrees holding about PIECE_NNZ nonzeros, one thread block each.  A piece is a run of *super-items* (at most
// SA_F4_POOL subtrees: what the block's pool of 16 x 16 temporaries holds), a super-item a run of *items* that
// the block's warps take one at a time:
//   kind 0: at most 32 consecutive subtrees, about an eighth of the super-item's nonzeros (the kernel evaluates
//           their level-2 fibers in batches of at most SA_F4_ROWS);   f0/f1 = fibers, p0/p1 = nonzeros
//   kind 1: up to 8 consecutive *large* subtrees (more than SA_SUB_MAX_NNZ nonzeros), whose temporaries the
//           order-3 kernel has written beforehand; f0 = index of the first one among the large subtrees.
// Nothing is cut at a slice boundary: the block follows the slices through pos[1] while it consumes the
// temporaries.  A slice that lies in several pieces gets one partial tile per piece (consecutive slots) and a
// fix-up entry.  `wl` (main list): the order-3 lists over the large subtrees, output row = index among them.
static bool subtree_is_large(const sa_tensor *t, int64_t f2)
{
    const auto &pos2 = t->pos[2], &pos3 = t->pos[3];
    return pos3[size_t(pos2[size_t(f2) + 1])] - pos3[size_t(pos2[size_t(f2)])] > SA_SUB_MAX_NNZ;
}

void build_ttm4(sa_tensor *t, sa_worklist &wl, sa_worklist &wl_items, sa_worklist &wl_fix)
{
    const auto &pos1 = t->pos[1], &pos2 = t->pos[2], &pos3 = t->pos[3];
    const int64_t F2 = t->count[1], S = t->count[0];
    std::vector<int32_t> large_ord(size_t(F2), -1);
    int32_t n_large = 0;
    for (int64_t r = 0; r < F2; ++r)
        if (subtree_is_large(t, r)) large_ord[size_t(r)] = n_large++;
    t->f4_n_large = n_large;
    build_ttm3_lists(wl, F2, [&](int64_t r) { return large_ord[size_t(r)]; }, [&](int64_t r) { return large_ord[size_t(r)] < 0; },
                     pos2, pos3);
    wl.nnz = 0;
    for (const sa_item &it : wl.items) wl.nnz += it.p1 - it.p0;

    constexpr int64_t PIECE_NNZ = 16384, LARGE_WEIGHT = 64;
    auto nnz_at = [&](int64_t r) { return pos3[size_t(pos2[size_t(r)])]; };
    std::vector<sa_item> &items = wl_items.items;
    std::vector<int32_t> &supers = t->f4_supers, &pieces = t->f4_pieces;
    auto push_item = [&](int64_t r0, int64_t r1, int kind) {
        sa_item it = empty_item();
        it.out_row = int32_t(r0); it.row_end = int32_t(r1); it.pad = kind;
        if (kind == 0) {
            it.f0 = int32_t(pos2[size_t(r0)]); it.f1 = int32_t(pos2[size_t(r1)]);
            it.p0 = int32_t(nnz_at(r0)); it.p1 = int32_t(nnz_at(r1));
        } else {
            it.f0 = large_ord[size_t(r0)]; it.f1 = it.f0 + int32_t(r1 - r0);
        }
        items.push_back(it);
    };
    // One super-item = the subtrees [r0, r1), r1 - r0 <= SA_F4_POOL.  Its small subtrees are cut into at most SA_F4_WARPS
    // nonzero-balanced runs (one per warp of the block); a run also ends at a large subtree and after 32 subtrees.
    auto push_super = [&](int64_t r0, int64_t r1) {
        int64_t small_nnz = 0;
        for (int64_t r = r0; r < r1; ++r)
            if (large_ord[size_t(r)] < 0) small_nnz += nnz_at(r + 1) - nnz_at(r);
        const int64_t target = (small_nnz + SA_F4_WARPS - 1) / SA_F4_WARPS;
        const int32_t item0 = int32_t(items.size());
        int64_t run0 = r0, run_nnz = 0;
        int run_kind = -1;
        for (int64_t r = r0; r < r1; ++r) {
            const int kind = large_ord[size_t(r)] >= 0 ? 1 : 0;
            const bool full = run_kind >= 0 && (kind != run_kind || (kind == 1 ? r - run0 >= 8 : (run_nnz >= target || r - run0 >= 32)));
            if (full) { push_item(run0, r, run_kind); run_kind = -1; }
            if (run_kind < 0) { run_kind = kind; run0 = r; run_nnz = 0; }
            if (kind == 0) run_nnz += nnz_at(r + 1) - nnz_at(r);
        }
        if (run_kind >= 0) push_item(run0, r1, run_kind);
        supers.push_back(item0); supers.push_back(int32_t(items.size()));
        supers.push_back(int32_t(r0)); supers.push_back(int32_t(r1));
    };
    // slice that holds subtree r (r < F2)
    auto slice_of = [&](int64_t r) { return int64_t(std::upper_bound(pos1.begin(), pos1.end(), r) - pos1.begin()) - 1; };
    auto push_piece = [&](int64_t r0, int64_t r1) {
        const int32_t sup0 = int32_t(supers.size() / 4);
        for (int64_t r = r0; r < r1; r += SA_F4_POOL) push_super(r, std::min<int64_t>(r1, r + SA_F4_POOL));
        pieces.push_back(sup0); pieces.push_back(int32_t(supers.size() / 4));
        pieces.push_back(int32_t(slice_of(r0))); pieces.push_back(int32_t(slice_of(r1 - 1)));
        pieces.push_back(-1); pieces.push_back(-1);       // destinations of the first / last slice: set below
        pieces.push_back(int32_t(r0)); pieces.push_back(int32_t(r1));
    };
    {
        int64_t piece_r0 = 0, piece_w = 0;
        for (int64_t r = 0; r < F2; ++r) {
            if (piece_w >= PIECE_NNZ) { push_piece(piece_r0, r); piece_r0 = r; piece_w = 0; }
            piece_w += large_ord[size_t(r)] >= 0 ? LARGE_WEIGHT : nnz_at(r + 1) - nnz_at(r);
        }
        if (F2 > piece_r0) push_piece(piece_r0, F2);
    }
    wl_items.n_group_ctas = 0;
    // partial tiles: a slice that lies in more than one piece gets one slot per piece
    std::vector<int32_t> slice_slots(size_t(S), 0), slice_slot0(size_t(S), -1);
    const size_t n_pieces = pieces.size() / 8;
    for (size_t p = 0; p < n_pieces; ++p)
        for (int64_t s = pieces[8 * p + 2]; s <= pieces[8 * p + 3]; ++s) slice_slots[size_t(s)]++;
    for (int64_t s = 0; s < S; ++s)
        if (slice_slots[size_t(s)] > 1) {
            slice_slot0[size_t(s)] = int32_t(wl_fix.n_slots);
            wl_fix.fix.push_back(sa_fix{t->crd[0][size_t(s)], int32_t(wl_fix.n_slots), slice_slots[size_t(s)], 0});
            wl_fix.n_slots += slice_slots[size_t(s)];
        }
    std::vector<int32_t> next_slot(slice_slot0);
    for (size_t p = 0; p < n_pieces; ++p) {
        const int64_t sa = pieces[8 * p + 2], sb = pieces[8 * p + 3];
        if (slice_slot0[size_t(sa)] >= 0) pieces[8 * p + 4] = next_slot[size_t(sa)]++;
        if (sb != sa) { if (slice_slot0[size_t(sb)] >= 0) pieces[8 * p + 5] = next_slot[size_t(sb)]++; }
        else pieces[8 * p + 5] = pieces[8 * p + 4];
    }
    append_empty_slices(t, wl_fix);
}

// Rows of a sparse matrix given by its pos array: row ranges of about target_nnz nonzeros (at most max_rows rows); rows longer than
// long_thresh are cut into pieces of `piece` nonzeros whose partial rows the fix-up kernel sums.
// quarter_rows: a range item also records the rows that hold its nonzeros p0 + q ceil((p1 - p0) / 4), q = 1, 2, 3
// (fields f0, f1, pad), for kernels whose lane groups take equal counts of nonzeros rather than of rows.
void build_rows(const std::vector<int64_t> &pos, int64_t I, sa_worklist &wl, int64_t target_nnz, int64_t max_rows,
                int64_t long_thresh, int64_t piece, bool quarter_rows = false)
{
    std::vector<sa_item> longs, ranges;
    int64_t r0 = 0;
    auto flush = [&](int64_t r1) {
        if (r1 > r0) {
            sa_item it = empty_item();
            it.out_row = int32_t(r0); it.row_end = int32_t(r1);
            it.p0 = int32_t(pos[size_t(r0)]); it.p1 = int32_t(pos[size_t(r1)]);
            if (quarter_rows) {
                const int64_t share = (int64_t(it.p1) - it.p0 + 3) / 4;
                int32_t rows[3];
                for (int q = 1; q < 4; ++q) {
                    const int64_t at = std::min<int64_t>(int64_t(it.p0) + q * share, it.p1);
                    // the last row starting at or before `at`, inside the item
                    int64_t r = (std::upper_bound(pos.begin() + r0, pos.begin() + r1 + 1, at) - pos.begin()) - 1;
                    rows[q - 1] = int32_t(std::min<int64_t>(std::max<int64_t>(r, r0), r1 - 1));
                }
                it.f0 = rows[0]; it.f1 = rows[1]; it.pad = rows[2];
            }
            ranges.push_back(it);
        }
        r0 = r1;
    };
    for (int64_t r = 0; r < I; ++r) {
        const int64_t a = pos[size_t(r)], b = pos[size_t(r) + 1];
        if (b - a > long_thresh) {
            flush(r);
            const int64_t np = (b - a + piece - 1) / piece;
            const int32_t slot0 = int32_t(wl.n_slots);
            wl.fix.push_back(sa_fix{int32_t(r), slot0, int32_t(np), 0});
            wl.n_slots += np;
            for (int64_t q = 0; q < np; ++q) {
                sa_item it = empty_item();
                it.out_row = int32_t(r); it.row_end = int32_t(r + 1);
                it.p0 = int32_t(a + q * piece); it.p1 = int32_t(std::min(b, a + (q + 1) * piece));
                it.dest = slot0 + int32_t(q);
                longs.push_back(it);
            }
            r0 = r + 1;
            continue;
        }
        if (pos[size_t(r) + 1] - pos[size_t(r0)] > target_nnz && r > r0) flush(r);
        if (r + 1 - r0 >= max_rows) flush(r + 1);
    }
    flush(I);
    // longest first: the tail of the launch is then made of the cheapest items
    std::stable_sort(ranges.begin(), ranges.end(),
                     [](const sa_item &a, const sa_item &b) { return (a.p1 - a.p0) > (b.p1 - b.p0); });
    wl.n_group_ctas = 0;
    wl.items = std::move(longs);
    wl.items.insert(wl.items.end(), ranges.begin(), ranges.end());
}

}  // namespace

void sa_build_worklists(sa_tensor *t)
{
    if (t->fmt == SA_FMT_CSF && t->order == 3) {
        build_ttm3(t, t->wl_main);
        // kernel 7 walks the tensor as a sparse matrix whose rows are the (i,j) fibers
        build_rows(t->pos[2], t->count[1], t->wl_aux, 1024, 4096, 4096, 2048, true);
    }
    if (t->fmt == SA_FMT_CSF && t->order == 4) {
        build_ttm4(t, t->wl_main, t->wl_sub, t->wl_aux);
        build_ttm4_fissioned(t, t->wl4_main, t->wl4_aux);
        build_ttm4_subtrees(t, t->wl4_sub);
        t->wl4_main.nnz = t->nnz - t->wl4_sub.nnz;
    }
    if (t->fmt == SA_FMT_CSR) {
        build_rows(t->pos[1], t->dims[0], t->wl_main, 256, 32, 1024, 512);    // fused SDDMM -> SpMM
        build_rows(t->pos[1], t->dims[0], t->wl_aux, 256, 16, 4096, 2048);    // SpMM -> GEMM (both orders)
    }
}
