// Internal declarations shared by the host builder, the API layer and the kernel launchers.
#pragma once

#include <cuda_runtime.h>
#include <atomic>
#include <cstdint>
#include <vector>

#include "sparseauto.h"

constexpr int SA_MAX_ORDER = 4;
constexpr int SA_WARPS_PER_CTA = 8;
constexpr int SA_TTM3_WARPS = 4;     // warps per thread block of the order-3 kernel (they share one chunk of a large slice)

// One unit of work for one warp.  32 bytes, read once per warp.
//   CSF tensors: a contiguous range of level-1 fibers [f0, f1) inside ONE slice, clipped to the
//   nonzero range [p0, p1) (order 3; a fiber may be cut between two items, each adds its part).
//   CSR tensors: either whole rows [out_row, row_end) or, for a long row, the nonzeros [p0, p1)
//   of row out_row (row_end == out_row + 1).
//   dest < 0: the result is stored to `out`; dest >= 0: it is a partial result written to slot
//   `dest` of the workspace and summed by the fix-up kernel.
struct sa_item {
    int32_t out_row;
    int32_t row_end;
    int32_t f0, f1;
    int32_t p0, p1;
    int32_t dest;
    int32_t pad;      // order-4 CSF: which half of the last dense index n this item covers (0 / 1)
};

// Fix-up entry: out[out_row] = sum of `count` partial tiles starting at slot0 (count == 0: zeros).
struct sa_fix {
    int32_t out_row;
    int32_t slot0;
    int32_t count;
    int32_t pad;
};

// Order-3 CSF only: what the kernel reads per item (a piece of one slice, "unit").  The warp's 32 lanes
// form SA_STREAMS groups of 8 lanes; each group streams one contiguous part of [p0, p1) whose start is a
// multiple of SA_ROUND nonzeros (see sa_unit3_streams); sf[q] is the level-1 fiber that holds the first
// nonzero of part q.
constexpr int SA_STREAMS = 4;
constexpr int SA_ROUND = 16;         // nonzeros a stream takes per round of the order-3 kernel
struct sa_unit3 {
    int32_t out_row;
    int32_t dest;
    int32_t p0, p1;
    int32_t sf[SA_STREAMS];
};
static_assert(sizeof(sa_unit3) == 32, "sa_unit3 is read as two 16-byte pieces");

// Nonzero ranges of the SA_STREAMS parts of a unit [p0, p1): part q = [lo[q], hi[q]) (empty if lo >= hi);
// every part starts at base + q * slen with base = p0 rounded down to a multiple of SA_ROUND and slen a
// multiple of SA_ROUND, clipped to [p0, p1).  The same arithmetic runs in the kernel.
static inline void sa_unit3_streams(int64_t p0, int64_t p1, int64_t *lo, int64_t *hi)
{
    const int64_t base = p0 & ~int64_t(SA_ROUND - 1), span = p1 - base;
    const int64_t slen = ((span + SA_STREAMS - 1) / SA_STREAMS + SA_ROUND - 1) & ~int64_t(SA_ROUND - 1);
    for (int q = 0; q < SA_STREAMS; ++q) {
        const int64_t a = base + q * slen;
        lo[q] = a > p0 ? a : p0;
        hi[q] = a + slen < p1 ? a + slen : p1;
    }
}

struct sa_worklist {
    std::vector<sa_item> items;   // [n_group_ctas * SA_WARPS_PER_CTA group items][warp items]
    std::vector<sa_fix> fix;
    int64_t n_group_ctas = 0;     // leading CTAs whose 8 warps reduce into one tile
    int64_t n_slots = 0;          // partial tiles in the workspace
    int64_t nnz = 0;              // nonzeros the list covers (set for the order-4 lists of pass 1)
    sa_item *d_items = nullptr;
    sa_fix *d_fix = nullptr;
    // order-3 CSF: warp w evaluates items [task_start[w], task_start[w + 1]); the first
    // n_group_ctas * SA_TTM3_WARPS tasks hold at most one item each
    std::vector<int32_t> task_start;
    std::vector<int32_t> stream_f0;   // [items * SA_STREAMS]
    int32_t *d_task_start = nullptr;
    sa_unit3 *d_units3 = nullptr;
};

struct sa_tensor {
    int order = 0;
    sa_format fmt = SA_FMT_CSF;
    int64_t dims[SA_MAX_ORDER] = {0, 0, 0, 0};
    int64_t nnz = 0;
    int device = 0;
    sa_allocator alloc{nullptr, nullptr, nullptr};
    bool own_alloc = false;

    // host copies (export + partitioning)
    std::vector<int64_t> pos[SA_MAX_ORDER];   // pos[l]: count(l-1)+1 entries; empty for a dense level
    std::vector<int32_t> crd[SA_MAX_ORDER];   // crd[l]: count(l) entries; empty for a dense level
    std::vector<float> vals;
    int64_t count[SA_MAX_ORDER] = {0, 0, 0, 0};

    // device copies (pos as int32: nnz < 2^31)
    int32_t *d_pos[SA_MAX_ORDER] = {nullptr, nullptr, nullptr, nullptr};
    int32_t *d_crd[SA_MAX_ORDER] = {nullptr, nullptr, nullptr, nullptr};
    float *d_vals = nullptr;
    uint32_t *d_endbits = nullptr;            // CSF: bit (p & 31) of word p / 32 is set when nonzero p is the last of
                                              // its last-level fiber ((i,j) for order 3, (i,j,k) for order 4)
    int2 *d_nzpack = nullptr;                 // CSF: per nonzero (last-level index | end-of-fiber bit << 31, value bits): what the
                                              // group-per-fiber kernels (kernel 7, order-4 subtree kernel) stream, one 8-byte load
    int32_t *d_status = nullptr;              // [4] device status word

    sa_worklist wl_main;                      // TTM3 / SDDMM-SpMM; order-4 CSF: the order-3 lists over the large (i,j) subtrees
    sa_worklist wl_aux;                       // CSR: SpMM-GEMM row items; order-3 CSF: fiber rows (kernel 7); order-4 CSF: partial
                                              // slice tiles and fix-up entries of the fused kernel
    sa_worklist wl_sub;                       // order-4 CSF: items of the fused kernel (runs of (i,j) subtrees)
    // order-4 CSF, schedule SA_SCHED_FISSIONED (sa_ttm4_fis.cu): order-3 lists over the (i,j) subtrees the subtree kernel
    // does not take, pass-2 items (piece of a slice x quarter of the columns) with their fix-up entries, and ranges of
    // whole small subtrees for the subtree kernel
    sa_worklist wl4_main, wl4_aux, wl4_sub;
    // order-4 CSF: super-items (item0, item1, r0, r1) and pieces (sup0, sup1, first slice, last slice, destination of
    // the first slice, of the last slice, r0, r1) of the fused kernel, see build_ttm4; subtrees above SA_SUB_MAX_NNZ
    std::vector<int32_t> f4_supers, f4_pieces;
    int32_t *d_f4_supers = nullptr, *d_f4_pieces = nullptr;
    int32_t f4_n_large = 0;

    mutable std::atomic<int> last_launches{0};   // concurrent sa_run calls may write it
    std::atomic<uint64_t> aux_limit{~uint64_t(0)};   // caller's cap on a default schedule's workspace (sa_tensor_set_aux_limit)
    std::vector<void *> dev_blocks;           // everything obtained from the allocator
};

// Limits of the fused order-4 kernel: level-2 fiber rows a warp parks per batch, temporaries in a thread block's
// pool (= subtrees per super-item), nonzeros of a subtree the kernel evaluates itself (larger ones go through the
// order-3 kernel first).
#ifndef SA_F4_ROWS_N
#define SA_F4_ROWS_N 32
#endif
#ifndef SA_F4_POOL_N
#define SA_F4_POOL_N 64
#endif
#ifndef SA_F4_WARPS_N
#define SA_F4_WARPS_N 8
#endif
#ifndef SA_F4_CTAS_N
#define SA_F4_CTAS_N 2
#endif
constexpr int SA_F4_ROWS = SA_F4_ROWS_N;
constexpr int SA_F4_POOL = SA_F4_POOL_N;
constexpr int SA_F4_WARPS = SA_F4_WARPS_N;    // warps per thread block of the fused kernel
constexpr int SA_F4_CTAS = SA_F4_CTAS_N;      // thread blocks per SM the fused kernel's register budget is set for
constexpr int SA_SUB_MAX_NNZ = 4096;
// Limits of the subtree kernel of the fissioned order-4 schedule: level-2 fibers an item parks in shared memory and
// rows (subtrees) per item.
constexpr int SA_SUB_MAX_F3 = 64;
constexpr int SA_SUB_MAX_ROWS = 32;

// ---- host builder (sa_build.cu)
sa_status sa_build_levels(sa_tensor *t, const int32_t *coords, const float *vals);
void sa_build_worklists(sa_tensor *t);

// What the order-3 kernel needs to know about the tensor it walks: an order-3 CSF tensor, or an order-4 one
// seen as a collection of (i,j) subtrees (slices = level-1 fibers, fibers = level-2 nodes).
struct sa_ttm3_view {
    const sa_worklist *wl;        // units, tasks, fix-up entries
    const int32_t *crd_fiber;     // per fiber: row of the first factor
    const int32_t *crd_nz;        // per nonzero: row of the second factor
    const float *vals;
    const uint32_t *endbits;      // bit p set: nonzero p is the last of its fiber
    int64_t n_fibers, n_out_rows;
    int64_t nnz;                  // nonzeros the lists cover (chooses the register budget)
    int64_t nnz_total;            // length of the index / value arrays (bounds of the self-checking build)
    int32_t *status;              // the tensor's device status word
};
sa_status sa_launch_ttm3_view(const sa_ttm3_view &v, const sa_dense &first, const sa_dense &second, float *out,
                              float *partial, cudaStream_t stream, int *launches);

// ---- launchers (one per chain); all asynchronous on `stream`, return SA_OK or SA_E_*.
sa_status sa_launch_ttm3(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                         cudaStream_t stream, int *launches);
size_t sa_ws_ttm3(const sa_tensor *t, const sa_dense *ops);
sa_status sa_launch_ttm4(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                         cudaStream_t stream, int *launches);
size_t sa_ws_ttm4(const sa_tensor *t, const sa_dense *ops);
sa_status sa_launch_ttm4_fissioned(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                                   cudaStream_t stream, int *launches);
size_t sa_ws_ttm4_fissioned(const sa_tensor *t, const sa_dense *ops);
sa_status sa_launch_sddmm_spmm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                               bool materialize, cudaStream_t stream, int *launches);
size_t sa_ws_sddmm_spmm(const sa_tensor *t, const sa_dense *ops, bool materialize);
sa_status sa_launch_spmm_gemm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                              bool assoc_right, cudaStream_t stream, int *launches);
size_t sa_ws_spmm_gemm(const sa_tensor *t, const sa_dense *ops, bool assoc_right);
// Kernel 3 <SpMMH,GEMM>: the row kernel of (B.C).D with the Hadamard product C(j,:) * D(j,:) as the gathered row.
sa_status sa_launch_spmmh_gemm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                               cudaStream_t stream, int *launches);
size_t sa_ws_spmmh_gemm(const sa_tensor *t, const sa_dense *ops);

sa_status sa_launch_ttmc3(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes, bool fissioned,
                          cudaStream_t stream, int *launches);
size_t sa_ws_ttmc3(const sa_tensor *t, const sa_dense *ops, bool fissioned);
// Kernel 5 with the loop over i kept fused (sa_ttm3.cu): available while the block accumulator fits shared memory
bool sa_ttmc3_fused_ok(int64_t L3, int64_t M, int64_t N);
size_t sa_ws_ttmc3_fused(int64_t L3, int64_t M, int64_t N);
sa_status sa_launch_ttmc3_fused_stage(const sa_tensor *t, const sa_dense &C3, const sa_dense &D, const sa_dense &E, float *partials,
                                      cudaStream_t stream, int *n_blocks);

// Kernel 2 <SDDMM,SpMM,GEMM>: the fused SDDMM->SpMM kernel into a row temporary, then the dense stage.
sa_status sa_launch_sddmm_spmm_gemm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                                    cudaStream_t stream, int *launches);
size_t sa_ws_sddmm_spmm_gemm(const sa_tensor *t, const sa_dense *ops);
bool sa_dense_gemm_ok(int64_t L, int64_t M);
// out (rows x M) = A (rows x L) . B (L x M); `status` is the tensor's device status word (a wait that runs out
// inside the tcgen05 kernel records SA_E_TIMEOUT there).  L >= 64 runs on tcgen05, L = 32 on mma.sync.
sa_status sa_launch_dense_gemm(int64_t rows, const float *A, int64_t lda, const float *B, int64_t ldb, int64_t L,
                               int64_t M, float *out, int32_t *status, cudaStream_t stream);
bool sa_dense_gemm_tc_ok(int64_t L, int64_t M);
sa_status sa_launch_dense_gemm_tc(int64_t rows, const float *A, int64_t lda, const float *B, int64_t ldb, int64_t L,
                                  int64_t M, float *out, int32_t *status, cudaStream_t stream);

// Kernel 7 <SpTTM,SpTTM>: out = one row of M values per (i,j) fiber, in CSF order
bool sa_ranks_ok_spttm_spttm(int64_t L, int64_t M);
size_t sa_ws_spttm_spttm(const sa_tensor *t, const sa_dense *ops, bool right);
sa_status sa_launch_spttm_spttm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes, bool right,
                                cudaStream_t stream, int *launches);

// Kernel 8 <MTTKRP,GEMM>
sa_status sa_launch_mttkrp_gemm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                                cudaStream_t stream, int *launches);
size_t sa_ws_mttkrp_gemm(const sa_tensor *t, const sa_dense *ops);
bool sa_ranks_ok_mttkrp_gemm(int64_t R, int64_t M);

// Supported-rank predicates (shared by sa_workspace_size and sa_run).
bool sa_ranks_ok_ttm3(int64_t L, int64_t M);
bool sa_ranks_ok_ttm4(int64_t L, int64_t M, int64_t N);
bool sa_ranks_ok_ttmc3(int64_t L, int64_t M, int64_t N);
bool sa_ranks_ok_sddmm(int64_t K, int64_t L);
bool sa_ranks_ok_spmm_gemm(int64_t L, int64_t M);

static inline size_t sa_align256(size_t x) { return (x + 255) & ~size_t(255); }
