// C-ABI entry points (declared in include/sparseauto.h): handle lifetime, argument checks and
// the host table (expression, schedule) -> launcher that stands in for the run-time lookup from
// chosen schedules to compiled functions outlined in the paper's discussion of run-time overheads
// (Section 6).
#include <cstring>
#include <new>

#include "sa_internal.h"

namespace {

void *default_alloc(size_t bytes, void *)
{
    void *p = nullptr;
    if (cudaMalloc(&p, bytes) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return p;
}

void default_release(void *p, void *) { cudaFree(p); }

// Allocate device memory through the tensor's allocator and copy n elements of src into it.  The block
// ends with at least 64 zero bytes: kernels that read index and value arrays in aligned groups of eight
// elements may run past the last element and must find valid (zero) indices there.
template <typename T>
sa_status upload(sa_tensor *t, const T *src, size_t n, T **dst)
{
    *dst = nullptr;
    const size_t used = n * sizeof(T);
    const size_t bytes = sa_align256(used + 64);
    void *p = t->alloc.alloc(bytes, t->alloc.ctx);
    if (!p) return SA_E_ALLOC;
    t->dev_blocks.push_back(p);
    if (n && cudaMemcpy(p, src, used, cudaMemcpyHostToDevice) != cudaSuccess) return SA_E_CUDA;
    if (cudaMemset(static_cast<char *>(p) + used, 0, bytes - used) != cudaSuccess) return SA_E_CUDA;
    *dst = static_cast<T *>(p);
    return SA_OK;
}

sa_status upload_pos32(sa_tensor *t, const std::vector<int64_t> &pos, int32_t **dst)
{
    std::vector<int32_t> p32(pos.size());
    for (size_t i = 0; i < pos.size(); ++i) p32[i] = int32_t(pos[i]);
    return upload(t, p32.data(), p32.size(), dst);
}

sa_status upload_worklist(sa_tensor *t, sa_worklist &wl)
{
    sa_status s = upload(t, wl.fix.data(), wl.fix.size(), &wl.d_fix);
    if (s != SA_OK) return s;
    if (wl.task_start.empty()) return upload(t, wl.items.data(), wl.items.size(), &wl.d_items);
    // order-3 CSF: the kernel reads the compact per-unit records and the task list
    std::vector<sa_unit3> units(wl.items.size());
    for (size_t u = 0; u < units.size(); ++u) {
        const sa_item &it = wl.items[u];
        units[u].out_row = it.out_row; units[u].dest = it.dest; units[u].p0 = it.p0; units[u].p1 = it.p1;
        for (int q = 0; q < SA_STREAMS; ++q) units[u].sf[q] = wl.stream_f0[u * SA_STREAMS + size_t(q)];
    }
    s = upload(t, units.data(), units.size(), &wl.d_units3);
    if (s != SA_OK) return s;
    return upload(t, wl.task_start.data(), wl.task_start.size(), &wl.d_task_start);
}

struct device_guard {
    int prev = -1;
    bool ok = false;
    explicit device_guard(int dev)
    {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~device_guard() { if (prev >= 0) cudaSetDevice(prev); }
};

bool dense_ok(const sa_dense &d)
{
    return d.ptr != nullptr && d.rows > 0 && d.cols > 0 && d.ld >= d.cols && (d.ld % 4) == 0 &&
           (reinterpret_cast<uintptr_t>(d.ptr) % 16) == 0;
}

// Shape check of the operand list; fills the number of operands the expression takes.
sa_status check_ops(const sa_tensor *t, sa_expr expr, const sa_dense *ops, int n_ops, bool shapes_only)
{
    if (!ops) return SA_E_ARG;
    int want = 0;
    switch (expr) {
        case SA_EXPR_SPTTM_TTM3: want = 2; break;
        case SA_EXPR_SPTTM_TTM4: want = 3; break;
        case SA_EXPR_SDDMM_SPMM: want = 3; break;
        case SA_EXPR_SPMM_GEMM: want = 2; break;
        case SA_EXPR_TTMC3: want = 3; break;
        case SA_EXPR_SDDMM_SPMM_GEMM: want = 4; break;
        case SA_EXPR_SPMMH_GEMM: want = 3; break;
        case SA_EXPR_MTTKRP_GEMM: want = 3; break;
        case SA_EXPR_SPTTM_SPTTM: want = 2; break;
        default: return SA_E_ARG;
    }
    if (n_ops != want) return SA_E_ARG;
    for (int i = 0; i < n_ops; ++i) {
        if (ops[i].rows <= 0 || ops[i].cols <= 0) return SA_E_SHAPE;
        if (!shapes_only && !dense_ok(ops[i])) return ops[i].ptr ? SA_E_SHAPE : SA_E_ARG;
    }
    switch (expr) {
        case SA_EXPR_SPTTM_TTM3:
            if (t->fmt != SA_FMT_CSF || t->order != 3) return SA_E_FORMAT;
            if (ops[0].rows != t->dims[1] || ops[1].rows != t->dims[2]) return SA_E_SHAPE;
            if (!sa_ranks_ok_ttm3(ops[0].cols, ops[1].cols)) return SA_E_UNSUPPORTED;
            break;
        case SA_EXPR_SPTTM_TTM4:
            if (t->fmt != SA_FMT_CSF || t->order != 4) return SA_E_FORMAT;
            if (ops[0].rows != t->dims[1] || ops[1].rows != t->dims[2] || ops[2].rows != t->dims[3]) return SA_E_SHAPE;
            if (!sa_ranks_ok_ttm4(ops[0].cols, ops[1].cols, ops[2].cols)) return SA_E_UNSUPPORTED;
            break;
        case SA_EXPR_SDDMM_SPMM:
            if (t->fmt != SA_FMT_CSR) return SA_E_FORMAT;
            if (ops[0].rows != t->dims[0] || ops[1].rows != t->dims[1] || ops[2].rows != t->dims[1] ||
                ops[0].cols != ops[1].cols)
                return SA_E_SHAPE;
            if (!sa_ranks_ok_sddmm(ops[0].cols, ops[2].cols)) return SA_E_UNSUPPORTED;
            break;
        case SA_EXPR_SPMM_GEMM:
            if (t->fmt != SA_FMT_CSR) return SA_E_FORMAT;
            if (ops[0].rows != t->dims[1] || ops[1].rows != ops[0].cols) return SA_E_SHAPE;
            if (!sa_ranks_ok_spmm_gemm(ops[0].cols, ops[1].cols)) return SA_E_UNSUPPORTED;
            break;
        case SA_EXPR_SDDMM_SPMM_GEMM:
            if (t->fmt != SA_FMT_CSR) return SA_E_FORMAT;
            if (ops[0].rows != t->dims[0] || ops[1].rows != t->dims[1] || ops[2].rows != t->dims[1] ||
                ops[0].cols != ops[1].cols || ops[3].rows != ops[2].cols)
                return SA_E_SHAPE;
            if (!sa_ranks_ok_sddmm(ops[0].cols, ops[2].cols) || !sa_dense_gemm_ok(ops[2].cols, ops[3].cols)) return SA_E_UNSUPPORTED;
            break;
        case SA_EXPR_MTTKRP_GEMM:
            if (t->fmt != SA_FMT_CSF || t->order != 3) return SA_E_FORMAT;
            if (ops[0].rows != t->dims[1] || ops[1].rows != t->dims[2] || ops[1].cols != ops[0].cols ||
                ops[2].rows != ops[0].cols)
                return SA_E_SHAPE;
            if (!sa_ranks_ok_mttkrp_gemm(ops[0].cols, ops[2].cols)) return SA_E_UNSUPPORTED;
            break;
        case SA_EXPR_SPTTM_SPTTM:
            if (t->fmt != SA_FMT_CSF || t->order != 3) return SA_E_FORMAT;
            if (ops[0].rows != t->dims[2] || ops[1].rows != ops[0].cols) return SA_E_SHAPE;
            if (!sa_ranks_ok_spttm_spttm(ops[0].cols, ops[1].cols)) return SA_E_UNSUPPORTED;
            break;
        case SA_EXPR_SPMMH_GEMM:
            if (t->fmt != SA_FMT_CSR) return SA_E_FORMAT;
            if (ops[0].rows != t->dims[1] || ops[1].rows != t->dims[1] || ops[1].cols != ops[0].cols ||
                ops[2].rows != ops[0].cols)
                return SA_E_SHAPE;
            if (!sa_ranks_ok_spmm_gemm(ops[0].cols, ops[2].cols)) return SA_E_UNSUPPORTED;
            break;
        case SA_EXPR_TTMC3:
            if (t->fmt != SA_FMT_CSF || t->order != 3) return SA_E_FORMAT;
            if (ops[0].rows != t->dims[0] || ops[1].rows != t->dims[1] || ops[2].rows != t->dims[2]) return SA_E_SHAPE;
            if (!sa_ranks_ok_ttmc3(ops[0].cols, ops[1].cols, ops[2].cols)) return SA_E_UNSUPPORTED;
            break;
    }
    return SA_OK;
}

size_t workspace_bytes(const sa_tensor *t, sa_expr expr, sa_schedule sched, const sa_dense *ops);

// Bytes loaded for `uses` row reads of a dense table with `cols` columns: one row per use, whether the row comes
// from HBM or from the last-level cache (a gathered row occupies the load path either way; with the table
// counted once when it fits the cache, the model preferred (B.C).D on cache-resident C where B.(C.D) measured
// 1.2 to 1.8 times faster).
double table_bytes(const sa_tensor *, double, double cols, double uses) { return 4.0 * cols * uses; }

// Cost of one concrete schedule (not DEFAULT): see sa_schedule_cost in sparseauto.h.
void schedule_cost(const sa_tensor *t, sa_expr expr, sa_schedule sched, const sa_dense *ops, sa_cost *c)
{
    const double nnz = double(t->nnz), I = double(t->dims[0]);
    const double F2 = t->fmt == SA_FMT_CSF ? double(t->count[1]) : 0.0, F3 = t->order == 4 ? double(t->count[2]) : 0.0;
    const double S = t->fmt == SA_FMT_CSF ? double(t->count[0]) : I;
    double it = 0, by = 0, tmp = 0;
    switch (expr) {
        case SA_EXPR_SPTTM_TTM3: {      // i, j' < t(m); k': t += B D , l: A += t C >
            const double L = ops[0].cols, M = ops[1].cols;
            it = nnz * M + F2 * L * M;
            tmp = M;
            by = 8 * nnz + 8 * F2 + 8 * S + table_bytes(t, ops[0].rows, L, F2) + table_bytes(t, ops[1].rows, M, nnz) + 4 * I * L * M;
            break;
        }
        case SA_EXPR_SPTTM_TTM4: {      // i, j' < T2(m,n); k' < t(n); o': .. , m: .. > , l: .. >
            const double L = ops[0].cols, M = ops[1].cols, N = ops[2].cols;
            it = nnz * N + F3 * M * N + F2 * L * M * N;
            tmp = sched == SA_SCHED_FISSIONED ? N + F2 * M * N : N + M * N;
            by = 8 * nnz + 8 * F3 + 8 * F2 + 8 * S + table_bytes(t, ops[0].rows, L, F2) + table_bytes(t, ops[1].rows, M, F3) +
                 table_bytes(t, ops[2].rows, N, nnz) + 4 * I * L * M * N + (sched == SA_SCHED_FISSIONED ? 8 * F2 * M * N : 0.0);
            break;
        }
        case SA_EXPR_SDDMM_SPMM: {      // i, j' < t; k: t += B C D , l: A += t E >
            const double K = ops[0].cols, L = ops[2].cols;
            it = nnz * (K + L);
            tmp = 1;
            by = 8 * nnz + 4 * (I + 1) + 4 * I * K + table_bytes(t, ops[1].rows, K, nnz) + table_bytes(t, ops[2].rows, L, nnz) + 4 * I * L;
            break;
        }
        case SA_EXPR_SDDMM_SPMM_GEMM: { // i < T(l); j' < t; k: .. , l: T += t E > , m,l: A += T F >
            const double K = ops[0].cols, L = ops[2].cols, M = ops[3].cols;
            it = nnz * (K + L) + I * L * M;
            tmp = 1 + L;
            by = 8 * nnz + 4 * (I + 1) + 4 * I * K + table_bytes(t, ops[1].rows, K, nnz) + table_bytes(t, ops[2].rows, L, nnz) +
                 8 * I * L + 4 * L * M + 4 * I * M;
            break;
        }
        case SA_EXPR_SPMMH_GEMM: {      // i < T(l); j', l: T += B C D , m,l: A += T E >
            const double L = ops[0].cols, M = ops[2].cols;
            it = nnz * L + I * L * M;
            tmp = L;
            by = 8 * nnz + 4 * (I + 1) + table_bytes(t, ops[0].rows, L, nnz) + table_bytes(t, ops[1].rows, L, nnz) + 4 * L * M + 4 * I * M;
            break;
        }
        case SA_EXPR_SPMM_GEMM: {
            const double J = double(t->dims[1]), L = ops[0].cols, M = ops[1].cols;
            if (sched == SA_SCHED_ASSOC_RIGHT) {   // < E(j,m); j,l,m: E += C D , i,j',m: A += B E >
                it = J * L * M + nnz * M;
                tmp = J * M;
                by = 4 * J * (L + M) + 4 * L * M + 8 * nnz + 4 * (I + 1) + table_bytes(t, J, M, nnz) + 4 * I * M;
            } else {                               // i < T(l); j',l: T += B C , m,l: A += T D >
                it = nnz * L + I * L * M;
                tmp = L;
                by = 8 * nnz + 4 * (I + 1) + table_bytes(t, J, L, nnz) + 4 * L * M + 4 * I * M;
            }
            break;
        }
        case SA_EXPR_SPTTM_SPTTM: {
            const double K = double(t->dims[2]), L = ops[0].cols, M = ops[1].cols;
            if (sched == SA_SCHED_ASSOC_RIGHT) {   // < E(k,m); k,l,m: E += C D , (i,j'),k',m: A += B E >
                it = K * L * M + nnz * M;
                tmp = K * M;
                by = 4 * K * (L + M) + 4 * L * M + 8 * nnz + 4 * (F2 + 1) + table_bytes(t, K, M, nnz) + 4 * F2 * M;
            } else {                               // (i,j') < T(l); k',l: T += B C , m,l: A += T D >, T kept for the dense stage
                it = nnz * L + F2 * L * M;
                tmp = F2 * L;
                by = 8 * nnz + 4 * (F2 + 1) + table_bytes(t, K, L, nnz) + 8 * F2 * L + 4 * L * M + 4 * F2 * M;
            }
            break;
        }
        case SA_EXPR_TTMC3: {           // i < T(m,n); j' < t(n); k': .. , m: .. > , l: A += T C >, or the l loop fissioned off
            const double L = ops[0].cols, M = ops[1].cols, N = ops[2].cols;
            it = nnz * N + F2 * M * N + S * L * M * N;
            by = 8 * nnz + 8 * F2 + 8 * S + table_bytes(t, ops[1].rows, M, F2) + table_bytes(t, ops[2].rows, N, nnz) + 4 * S * L + 4 * L * M * N;
            if (sched == SA_SCHED_FISSIONED) {
                tmp = N + I * M * N;
                by += 8 * I * M * N;
            } else {
                tmp = N + M * N;
            }
            break;
        }
        case SA_EXPR_MTTKRP_GEMM: {     // i < T(r); j' < t(r); k': t += B D , r: T += t C > , m,r: A += T E >
            const double R = ops[0].cols, M = ops[2].cols;
            it = nnz * R + F2 * R + I * R * M;
            tmp = R + I * R;
            by = 8 * nnz + 8 * F2 + 8 * S + table_bytes(t, ops[0].rows, R, F2) + table_bytes(t, ops[1].rows, R, nnz) + 8 * I * R +
                 4 * R * M + 4 * I * M;
            break;
        }
    }
    c->iterations = it;
    c->moved_bytes = by;
    c->temp_elements = tmp;
    c->workspace_bytes = workspace_bytes(t, expr, sched, ops);
    c->resolved = int(sched);
}

// Host table: which concrete schedule runs for (expr, sched).  Returns false if the pair is not in the table.
// Where an expression has two schedules the default is chosen per tensor, in the spirit of the paper's run-time
// Stage 4 (Section 5.2: the schedules that survive compile-time pruning are compared with the concrete sizes
// plugged into their cost expressions, and one whose auxiliary memory is too large is passed over): among the
// candidates whose workspace is within the tensor's auxiliary-memory cap the one that moves fewer bytes runs;
// when none fits, the one with the smaller workspace.
bool resolve_schedule(const sa_tensor *t, sa_expr expr, sa_schedule sched, const sa_dense *ops, sa_schedule *resolved)
{
    switch (expr) {
        case SA_EXPR_TTMC3: {
            // Fused over i (the paper's shape, slice temporaries on chip) exists while the block accumulator fits
            // shared memory.  The fissioned schedule keeps 24 instead of 16 warps per SM resident and measured 1.45
            // to 1.5 times faster on both benchmark tensors although it moves the I x M x N temporaries through
            // HBM, so it is the default as long as its workspace is within the auxiliary-memory cap; above the cap
            // the fused one runs (its workspace, the block accumulators, does not grow with the tensor).
            const bool can_fuse = sa_ttmc3_fused_ok(ops[0].cols, ops[1].cols, ops[2].cols);
            if (sched == SA_SCHED_FISSIONED) { *resolved = sched; return true; }
            if (sched == SA_SCHED_FUSED) { *resolved = sched; return can_fuse; }
            if (sched != SA_SCHED_DEFAULT) return false;
            const uint64_t cap = t->aux_limit.load();
            const size_t wx = workspace_bytes(t, expr, SA_SCHED_FISSIONED, ops);
            *resolved = (can_fuse && wx > cap && workspace_bytes(t, expr, SA_SCHED_FUSED, ops) <= cap) ? SA_SCHED_FUSED : SA_SCHED_FISSIONED;
            return true;
        }
        case SA_EXPR_SPTTM_TTM4: {
            // Fused: the temporaries T2 of the (i,j) subtrees stay on chip.  Fissioned: they pass through the workspace
            // (1 KB per subtree); that schedule keeps twice as many warps resident and measured 15 % faster on the
            // benchmark tensor, so it is the default while its workspace is within the auxiliary-memory cap.
            if (sched == SA_SCHED_FUSED || sched == SA_SCHED_FISSIONED) { *resolved = sched; return true; }
            if (sched != SA_SCHED_DEFAULT) return false;
            const uint64_t cap = t->aux_limit.load();
            *resolved = (workspace_bytes(t, expr, SA_SCHED_FISSIONED, ops) > cap && workspace_bytes(t, expr, SA_SCHED_FUSED, ops) <= cap)
                            ? SA_SCHED_FUSED : SA_SCHED_FISSIONED;
            return true;
        }
        case SA_EXPR_SPTTM_TTM3:
        case SA_EXPR_SDDMM_SPMM_GEMM:
        case SA_EXPR_SPMMH_GEMM:
        case SA_EXPR_MTTKRP_GEMM:
            if (sched == SA_SCHED_DEFAULT || sched == SA_SCHED_FUSED) { *resolved = SA_SCHED_FUSED; return true; }
            return false;
        case SA_EXPR_SDDMM_SPMM:
            if (sched == SA_SCHED_DEFAULT || sched == SA_SCHED_FUSED) { *resolved = SA_SCHED_FUSED; return true; }
            if (sched == SA_SCHED_DEBUG_MATERIALIZE) { *resolved = sched; return true; }
            return false;
        case SA_EXPR_SPMM_GEMM:
        case SA_EXPR_SPTTM_SPTTM:
            if (sched == SA_SCHED_DEFAULT) {
                sa_cost left, right;
                schedule_cost(t, expr, SA_SCHED_ASSOC_LEFT, ops, &left);
                schedule_cost(t, expr, SA_SCHED_ASSOC_RIGHT, ops, &right);
                const uint64_t cap = t->aux_limit.load();
                const bool lf = left.workspace_bytes <= cap, rf = right.workspace_bytes <= cap;
                bool take_left;
                if (lf != rf) take_left = lf;
                else if (!lf) take_left = left.workspace_bytes <= right.workspace_bytes;
                else take_left = left.moved_bytes <= right.moved_bytes;
                *resolved = take_left ? SA_SCHED_ASSOC_LEFT : SA_SCHED_ASSOC_RIGHT;
                return true;
            }
            if (sched == SA_SCHED_FUSED || sched == SA_SCHED_ASSOC_LEFT) { *resolved = SA_SCHED_ASSOC_LEFT; return true; }
            if (sched == SA_SCHED_ASSOC_RIGHT) { *resolved = sched; return true; }
            return false;
    }
    return false;
}

size_t workspace_bytes(const sa_tensor *t, sa_expr expr, sa_schedule sched, const sa_dense *ops)
{
    switch (expr) {
        case SA_EXPR_SPTTM_TTM3: return sa_ws_ttm3(t, ops);
        case SA_EXPR_SPTTM_TTM4: return sched == SA_SCHED_FISSIONED ? sa_ws_ttm4_fissioned(t, ops) : sa_ws_ttm4(t, ops);
        case SA_EXPR_SDDMM_SPMM: return sa_ws_sddmm_spmm(t, ops, sched == SA_SCHED_DEBUG_MATERIALIZE);
        case SA_EXPR_SPMM_GEMM: return sa_ws_spmm_gemm(t, ops, sched == SA_SCHED_ASSOC_RIGHT);
        case SA_EXPR_TTMC3: return sa_ws_ttmc3(t, ops, sched == SA_SCHED_FISSIONED);
        case SA_EXPR_SDDMM_SPMM_GEMM: return sa_ws_sddmm_spmm_gemm(t, ops);
        case SA_EXPR_SPMMH_GEMM: return sa_ws_spmmh_gemm(t, ops);
        case SA_EXPR_MTTKRP_GEMM: return sa_ws_mttkrp_gemm(t, ops);
        case SA_EXPR_SPTTM_SPTTM: return sa_ws_spttm_spttm(t, ops, sched == SA_SCHED_ASSOC_RIGHT);
    }
    return 0;
}

}  // namespace

extern "C" {

sa_status sa_tensor_create(int order, const int64_t *dims, int64_t nnz, const int32_t *coords, const float *vals,
                           sa_format fmt, int device, const sa_allocator *dev_alloc, sa_tensor **out)
{
    if (!out) return SA_E_ARG;
    *out = nullptr;
    if (!dims || nnz < 0 || (nnz > 0 && (!coords || !vals)) || device < -1) return SA_E_ARG;
    if (fmt != SA_FMT_CSR && fmt != SA_FMT_CSF) return SA_E_ARG;
    if (order < 2 || order > SA_MAX_ORDER) return SA_E_FORMAT;
    if ((fmt == SA_FMT_CSR) != (order == 2)) return SA_E_FORMAT;
    if (nnz >= (int64_t(1) << 31) - 64) return SA_E_UNSUPPORTED;
    for (int d = 0; d < order; ++d)
        if (dims[d] < 1 || dims[d] >= (int64_t(1) << 31)) return SA_E_ARG;
    if (dev_alloc && (!dev_alloc->alloc || !dev_alloc->release)) return SA_E_ARG;

    sa_tensor *t = new (std::nothrow) sa_tensor();
    if (!t) return SA_E_ALLOC;
    t->order = order;
    t->fmt = fmt;
    t->nnz = nnz;
    t->device = device;
    for (int d = 0; d < order; ++d) t->dims[d] = dims[d];
    if (dev_alloc) t->alloc = *dev_alloc;
    else { t->alloc = sa_allocator{default_alloc, default_release, nullptr}; t->own_alloc = true; }

    sa_status s = sa_build_levels(t, coords, vals);
    if (s == SA_OK) {
        try { sa_build_worklists(t); } catch (...) { s = SA_E_ALLOC; }
    }
    if (s == SA_OK && device >= 0) try {
        device_guard g(device);
        if (!g.ok) s = SA_E_CUDA;
        // An order-4 tensor without subtrees for the order-3 kernel is read through the packed nonzero records
        // alone: its separate last-level index, value and end-of-fiber arrays stay on the host.
        const bool packed_only = fmt == SA_FMT_CSF && order == 4 && t->wl_main.items.empty() && t->wl4_main.items.empty();
        for (int l = 0; l < order && s == SA_OK; ++l) {
            if (fmt == SA_FMT_CSR && l == 0) continue;   // dense level: nothing stored
            s = upload_pos32(t, t->pos[l], &t->d_pos[l]);
            if (s == SA_OK && !(packed_only && l == order - 1)) s = upload(t, t->crd[l].data(), t->crd[l].size(), &t->d_crd[l]);
        }
        if (s == SA_OK && !packed_only) s = upload(t, t->vals.data(), t->vals.size(), &t->d_vals);
        if (s == SA_OK && fmt == SA_FMT_CSF) {
            // one bit per nonzero: set on the last nonzero of every last-level fiber
            const int last = order - 1;
            std::vector<uint32_t> bits(size_t(nnz / 32 + 1), 0u);
            for (int64_t f = 0; f < t->count[last - 1]; ++f) {
                const int64_t p = t->pos[last][size_t(f) + 1] - 1;
                bits[size_t(p >> 5)] |= 1u << (p & 31);
            }
            if (!packed_only) s = upload(t, bits.data(), bits.size(), &t->d_endbits);
            if (s == SA_OK) {
                std::vector<int2> pack(size_t(nnz) + 1);
                for (int64_t p = 0; p < nnz; ++p) {
                    const uint32_t end = (bits[size_t(p >> 5)] >> (p & 31)) & 1u;
                    int32_t vb;
                    std::memcpy(&vb, &t->vals[size_t(p)], sizeof(vb));
                    pack[size_t(p)] = make_int2(int32_t(uint32_t(t->crd[last][size_t(p)]) | (end << 31)), vb);
                }
                pack[size_t(nnz)] = make_int2(0, 0);
                s = upload(t, pack.data(), pack.size(), &t->d_nzpack);
            }
        }
        const int32_t zeros[4] = {0, 0, 0, 0};
        if (s == SA_OK) s = upload(t, zeros, 4, &t->d_status);
        if (s == SA_OK) s = upload_worklist(t, t->wl_main);
        if (s == SA_OK) s = upload_worklist(t, t->wl_aux);
        if (s == SA_OK) s = upload_worklist(t, t->wl_sub);
        if (s == SA_OK && fmt == SA_FMT_CSF && order == 4) {
            s = upload_worklist(t, t->wl4_main);
            if (s == SA_OK) s = upload_worklist(t, t->wl4_aux);
            if (s == SA_OK) s = upload_worklist(t, t->wl4_sub);
            if (s == SA_OK) s = upload(t, t->f4_supers.data(), t->f4_supers.size(), &t->d_f4_supers);
            if (s == SA_OK) s = upload(t, t->f4_pieces.data(), t->f4_pieces.size(), &t->d_f4_pieces);
        }
        if (s == SA_OK && cudaDeviceSynchronize() != cudaSuccess) s = SA_E_CUDA;
        if (s == SA_E_CUDA) cudaGetLastError();
    } catch (...) { s = SA_E_ALLOC; }      // a host vector of the upload section could not be allocated
    if (s != SA_OK) { sa_destroy(t); return s; }
    *out = t;
    return SA_OK;
}

sa_status sa_tensor_info(const sa_tensor *t, int64_t *nnz, int64_t *level_counts, int64_t *n_chunks)
{
    if (!t) return SA_E_ARG;
    if (nnz) *nnz = t->nnz;
    if (level_counts)
        for (int l = 0; l < t->order; ++l) level_counts[l] = t->count[l];
    if (n_chunks) *n_chunks = int64_t(t->wl_main.items.size());
    return SA_OK;
}

sa_status sa_tensor_export(const sa_tensor *t, int level, int64_t *pos, int32_t *crd, float *vals)
{
    if (!t || level < 0 || level >= t->order) return SA_E_ARG;
    const bool dense_level = (t->fmt == SA_FMT_CSR && level == 0);
    if (dense_level && (pos || crd)) return SA_E_ARG;
    if (vals && level != t->order - 1) return SA_E_ARG;
    if (pos) std::memcpy(pos, t->pos[level].data(), t->pos[level].size() * sizeof(int64_t));
    if (crd) std::memcpy(crd, t->crd[level].data(), t->crd[level].size() * sizeof(int32_t));
    if (vals) std::memcpy(vals, t->vals.data(), t->vals.size() * sizeof(float));
    return SA_OK;
}

sa_status sa_tensor_worklist(const sa_tensor *t, int which, int64_t *counts, int32_t *items, int32_t *fix)
{
    if (!t || which < 0 || which > 6) return SA_E_ARG;
    if (which == 3) {
        // order-4 CSF: the pieces (8 integers each, returned as items) and super-items (4 integers each, returned
        // as fix-up entries) of the fused kernel
        if (counts) {
            counts[0] = int64_t(t->f4_pieces.size() / 8);
            counts[1] = t->f4_n_large;
            counts[2] = int64_t(t->f4_supers.size() / 4);
            counts[3] = 0;
        }
        if (items) std::memcpy(items, t->f4_pieces.data(), t->f4_pieces.size() * sizeof(int32_t));
        if (fix) std::memcpy(fix, t->f4_supers.data(), t->f4_supers.size() * sizeof(int32_t));
        return SA_OK;
    }
    const sa_worklist &wl = which == 0 ? t->wl_main : which == 1 ? t->wl_aux : which == 2 ? t->wl_sub
                          : which == 4 ? t->wl4_main : which == 5 ? t->wl4_aux : t->wl4_sub;
    if (counts) {
        counts[0] = int64_t(wl.items.size());
        counts[1] = wl.n_group_ctas;
        counts[2] = int64_t(wl.fix.size());
        counts[3] = wl.n_slots;
    }
    if (items) std::memcpy(items, wl.items.data(), wl.items.size() * sizeof(sa_item));
    if (fix) std::memcpy(fix, wl.fix.data(), wl.fix.size() * sizeof(sa_fix));
    return SA_OK;
}

sa_status sa_tensor_tasks(const sa_tensor *t, int64_t *n_tasks, int32_t *task_start, int32_t *stream_f0)
{
    if (!t) return SA_E_ARG;
    if (t->fmt != SA_FMT_CSF) return SA_E_FORMAT;
    const sa_worklist &wl = t->wl_main;
    if (n_tasks) *n_tasks = int64_t(wl.task_start.size()) - 1;
    if (task_start) std::memcpy(task_start, wl.task_start.data(), wl.task_start.size() * sizeof(int32_t));
    if (stream_f0) std::memcpy(stream_f0, wl.stream_f0.data(), wl.stream_f0.size() * sizeof(int32_t));
    return SA_OK;
}

sa_status sa_workspace_size(const sa_tensor *t, sa_expr expr, sa_schedule sched, const sa_dense *ops, int n_ops,
                            size_t *bytes)
{
    if (!t || !bytes) return SA_E_ARG;
    sa_status s = check_ops(t, expr, ops, n_ops, true);
    if (s != SA_OK) return s;
    sa_schedule r;
    if (!resolve_schedule(t, expr, sched, ops, &r)) return SA_E_UNSUPPORTED;
    *bytes = workspace_bytes(t, expr, r, ops);
    return SA_OK;
}

sa_status sa_schedule_cost(const sa_tensor *t, sa_expr expr, sa_schedule sched, const sa_dense *ops, int n_ops, sa_cost *cost)
{
    if (!t || !cost) return SA_E_ARG;
    sa_status s = check_ops(t, expr, ops, n_ops, true);
    if (s != SA_OK) return s;
    sa_schedule r;
    if (!resolve_schedule(t, expr, sched, ops, &r)) return SA_E_UNSUPPORTED;
    schedule_cost(t, expr, r, ops, cost);
    return SA_OK;
}

sa_status sa_tensor_set_aux_limit(sa_tensor *t, size_t bytes)
{
    if (!t) return SA_E_ARG;
    t->aux_limit = uint64_t(bytes);
    return SA_OK;
}

sa_status sa_run(const sa_tensor *t, sa_expr expr, sa_schedule sched, const sa_dense *ops, int n_ops, float *out,
                 void *workspace, size_t ws_bytes, void *cuda_stream)
{
    if (!t || t->device < 0) return SA_E_ARG;
    const bool empty_out = expr == SA_EXPR_SPTTM_SPTTM && t->count[1] == 0;    // a sparse output without rows
    if ((!out && !empty_out) || reinterpret_cast<uintptr_t>(out) % 16) return SA_E_ARG;
    sa_status s = check_ops(t, expr, ops, n_ops, false);
    if (s != SA_OK) return s;
    sa_schedule r;
    if (!resolve_schedule(t, expr, sched, ops, &r)) return SA_E_UNSUPPORTED;
    const size_t need = workspace_bytes(t, expr, r, ops);
    if (need > 0 && (!workspace || ws_bytes < need || reinterpret_cast<uintptr_t>(workspace) % 256))
        return SA_E_WORKSPACE;
    device_guard g(t->device);
    if (!g.ok) return SA_E_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int launches = 0;
    switch (expr) {
        case SA_EXPR_SPTTM_TTM3: s = sa_launch_ttm3(t, ops, out, workspace, ws_bytes, stream, &launches); break;
        case SA_EXPR_SPTTM_TTM4:
            s = r == SA_SCHED_FISSIONED ? sa_launch_ttm4_fissioned(t, ops, out, workspace, ws_bytes, stream, &launches)
                                        : sa_launch_ttm4(t, ops, out, workspace, ws_bytes, stream, &launches);
            break;
        case SA_EXPR_SDDMM_SPMM:
            s = sa_launch_sddmm_spmm(t, ops, out, workspace, ws_bytes, r == SA_SCHED_DEBUG_MATERIALIZE, stream, &launches);
            break;
        case SA_EXPR_SPMM_GEMM:
            s = sa_launch_spmm_gemm(t, ops, out, workspace, ws_bytes, r == SA_SCHED_ASSOC_RIGHT, stream, &launches);
            break;
        case SA_EXPR_TTMC3: s = sa_launch_ttmc3(t, ops, out, workspace, ws_bytes, r == SA_SCHED_FISSIONED, stream, &launches); break;
        case SA_EXPR_SDDMM_SPMM_GEMM: s = sa_launch_sddmm_spmm_gemm(t, ops, out, workspace, ws_bytes, stream, &launches); break;
        case SA_EXPR_SPMMH_GEMM: s = sa_launch_spmmh_gemm(t, ops, out, workspace, ws_bytes, stream, &launches); break;
        case SA_EXPR_MTTKRP_GEMM: s = sa_launch_mttkrp_gemm(t, ops, out, workspace, ws_bytes, stream, &launches); break;
        case SA_EXPR_SPTTM_SPTTM:
            s = sa_launch_spttm_spttm(t, ops, out, workspace, ws_bytes, r == SA_SCHED_ASSOC_RIGHT, stream, &launches);
            break;
    }
    if (s == SA_E_CUDA) cudaGetLastError();
    if (s == SA_OK) t->last_launches = launches;
    return s;
}

sa_status sa_last_launch_count(const sa_tensor *t, int *launches)
{
    if (!t || !launches) return SA_E_ARG;
    *launches = t->last_launches;
    return SA_OK;
}

sa_status sa_device_status_words(const sa_tensor *t, void *cuda_stream, int32_t *words)
{
    if (!t || t->device < 0 || !words) return SA_E_ARG;
    device_guard g(t->device);
    if (!g.ok) return SA_E_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(words, t->d_status, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return SA_E_CUDA;
    }
    return SA_OK;
}

sa_status sa_last_device_status(const sa_tensor *t, void *cuda_stream)
{
    if (!t || t->device < 0) return SA_E_ARG;
    device_guard g(t->device);
    if (!g.ok) return SA_E_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    int32_t word[4] = {0, 0, 0, 0};
    if (cudaMemcpyAsync(word, t->d_status, sizeof(word), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return SA_E_CUDA;
    }
    if (word[0] != 0) {
        cudaMemsetAsync(t->d_status, 0, sizeof(word), stream);
        cudaStreamSynchronize(stream);
        return word[0] == SA_E_TIMEOUT ? SA_E_TIMEOUT : SA_E_BOUNDS;
    }
    return SA_OK;
}

#ifdef SA_TEST_HOOKS
// Test library only (not declared in sparseauto.h): write one of the four device status words.
sa_status sa_test_set_status_word(const sa_tensor *t, int index, int32_t value, void *cuda_stream)
{
    if (!t || t->device < 0 || index < 0 || index > 3) return SA_E_ARG;
    device_guard g(t->device);
    if (!g.ok) return SA_E_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(t->d_status + index, &value, sizeof(value), cudaMemcpyHostToDevice, stream) != cudaSuccess ||
        cudaStreamSynchronize(stream) != cudaSuccess) {
        cudaGetLastError();
        return SA_E_CUDA;
    }
    return SA_OK;
}
#endif

void sa_destroy(sa_tensor *t)
{
    if (!t) return;
    if (t->device >= 0) {
        device_guard g(t->device);
        for (void *p : t->dev_blocks) t->alloc.release(p, t->alloc.ctx);
    }
    delete t;
}

const char *sa_status_string(sa_status s)
{
    switch (s) {
        case SA_OK: return "ok";
        case SA_E_ARG: return "invalid argument";
        case SA_E_COORD_RANGE: return "coordinate out of range";
        case SA_E_COORD_DUP: return "duplicate coordinate";
        case SA_E_FORMAT: return "format does not fit the order or the expression";
        case SA_E_SHAPE: return "dense operand shape, leading dimension or alignment mismatch";
        case SA_E_UNSUPPORTED: return "not in the compiled kernel table";
        case SA_E_ALLOC: return "allocation failed";
        case SA_E_WORKSPACE: return "workspace missing, misaligned or too small";
        case SA_E_CUDA: return "CUDA runtime error";
        case SA_E_BOUNDS: return "device-side index check failed";
        case SA_E_TIMEOUT: return "device-side wait ran out";
    }
    return "unknown status";
}

}  // extern "C"
