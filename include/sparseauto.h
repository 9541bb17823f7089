/*
 * sparseauto.h -- C ABI of the B200 executor for fissioned / fused sparse contraction chains.
 *
 * The library evaluates chains O(idx_out) = sum_contract I_1(idx_1) * ... * I_n(idx_n) with
 * one sparse operand B (first) and dense row-major operands (problem statement of Section 4.1;
 * storage as in Section 2.1 and the pos/crd/vals arrays of Fig. 1b) under the branched loop
 * nests that kernel fission and fusion produce (Section 4.2; chosen schedules in the Table
 * of kernels, Section 6).  A fixed host table maps (expression, schedule) to ahead-of-time
 * compiled CUDA kernels; it stands in for the run-time lookup from chosen schedules to compiled
 * functions that the paper outlines in its discussion of run-time overheads (Section 6).
 *
 * Conventions
 *   - Pointers marked HOST are ordinary host memory, DEVICE are device memory of the device the
 *     tensor was created on.  No call takes or returns a C++ or framework type.
 *   - All calls return an sa_status; nothing throws or aborts.  When a call fails before a
 *     launch, nothing is enqueued and `out` is untouched.
 *   - A tensor handle is immutable after creation; sa_run calls on different streams with
 *     distinct `out` / `workspace` buffers may run concurrently.
 *   - Requires a CUDA device of compute capability 10.0 (sm_100a); there is no CPU path.
 */
#ifndef SPARSEAUTO_H
#define SPARSEAUTO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sa_tensor sa_tensor; /* opaque */

typedef enum {
    SA_OK = 0,
    SA_E_ARG = 1,          /* null pointer, negative size, bad enum value                      */
    SA_E_COORD_RANGE = 2,  /* a coordinate lies outside dims                                   */
    SA_E_COORD_DUP = 3,    /* the same coordinate is stored twice                              */
    SA_E_FORMAT = 4,       /* format / order combination not representable                     */
    SA_E_SHAPE = 5,        /* dense operand shapes do not match the expression                 */
    SA_E_UNSUPPORTED = 6,  /* valid request outside the compiled kernel table                  */
    SA_E_ALLOC = 7,        /* host or device allocation failed                                 */
    SA_E_WORKSPACE = 8,    /* workspace missing, misaligned or too small                       */
    SA_E_CUDA = 9,         /* a CUDA runtime call or launch failed                             */
    SA_E_BOUNDS = 10,      /* device-side index check failed (status word)                     */
    SA_E_TIMEOUT = 11      /* a bounded device-side wait ran out (status word)                 */
} sa_status;

/* Level formats of Section 2.1.  CSR: dense row level + compressed column level (order 2).
 * CSF: every level compressed (order 3 and 4); level 0 lists the non-empty slices. */
typedef enum { SA_FMT_CSR = 1, SA_FMT_CSF = 2 } sa_format;

/* Expressions (Table of kernels, Section 6; index letters as used in this library). */
typedef enum {
    /* kernel 6 <SpTTM,TTM>:  A(i,l,m) = sum_{j,k} B(i,j,k) C(j,l) D(k,m); ops = {C, D}          */
    SA_EXPR_SPTTM_TTM3 = 1,
    /* order-4 analogue:      A(i,l,m,n) = sum_{j,k,o} B(i,j,k,o) C(j,l) D(k,m) E(o,n);
     * ops = {C, D, E}; the two-level nesting of kernel 5's second schedule.  SA_SCHED_FUSED: one
     * kernel, the 16 x 16 temporaries T2(m,n) of the (i,j) subtrees stay in shared memory (only
     * subtrees above 4096 nonzeros pass theirs through the workspace).  SA_SCHED_FISSIONED: two
     * passes with all temporaries in the workspace (1 KB per subtree), faster on this device while
     * memory allows.  SA_SCHED_DEFAULT: fissioned unless its workspace is above the auxiliary-memory
     * cap and the fused one's is not                                                             */
    SA_EXPR_SPTTM_TTM4 = 2,
    /* kernel 1 <SDDMM,SpMM>: A(i,l) = sum_j B(i,j) (sum_k C(i,k) D(j,k)) E(j,l); ops = {C,D,E}  */
    SA_EXPR_SDDMM_SPMM = 3,
    /* kernel 4 <SpMM,GEMM>:  A(i,m) = sum_{j,l} B(i,j) C(j,l) D(l,m); ops = {C, D}             */
    SA_EXPR_SPMM_GEMM = 4,
    /* kernel 5 <3D TTMC>:    A(l,m,n) = sum_{i,j,k} B(i,j,k) C(i,l) D(j,m) E(k,n); ops = {C, D, E};
     * B order-3 CSF.  SA_SCHED_FUSED (L M N <= 8192): the slice temporaries T(i; m,n) stay on chip,
     * every thread block accumulates into its own L x M x N tile; SA_SCHED_FISSIONED: they pass
     * through the workspace (faster on this device: more resident warps); SA_SCHED_DEFAULT: fissioned
     * unless its workspace is above the auxiliary-memory cap and the fused one's is not          */
    SA_EXPR_TTMC3 = 5,
    /* kernel 2 <SDDMM,SpMM,GEMM>: A(i,m) = sum_{j,k,l} B(i,j) C(i,k) D(j,k) E(j,l) F(l,m);
     * ops = {C, D, E, F}; B CSR; two-level schedule with the row temporary T(l) in the workspace */
    SA_EXPR_SDDMM_SPMM_GEMM = 6,
    /* kernel 3 <SpMMH,GEMM>: A(i,m) = sum_{j,l} B(i,j) C(j,l) D(j,l) E(l,m); ops = {C, D, E}; B CSR;
     * the Description column of the Table of kernels (SpMM with a Hadamard product, then GEMM),
     * evaluated per row as T(l) = sum_j B(i,j) C(j,l) D(j,l) followed by T . E                   */
    SA_EXPR_SPMMH_GEMM = 7,
    /* kernel 8 <MTTKRP,GEMM>: A(i,m) = sum_{j,k,r} B(i,j,k) C(j,r) D(k,r) E(r,m); ops = {C, D, E};
     * B order-3 CSF; the MTTKRP rows T(i,:) (R floats per slice) live in the workspace              */
    SA_EXPR_MTTKRP_GEMM = 8,
    /* kernel 7 <SpTTM,SpTTM>: A(i,j,m) = sum_{k,l} B(i,j,k) C(k,l) D(l,m); ops = {C (dims[2] x L), D (L x M)};
     * B order-3 CSF.  The output is sparse with B's (i,j) pattern: `out` receives one row of M values per
     * level-1 node (fiber (i,j)) of B, F2 x M floats in CSF order, F2 = level_counts[1] of sa_tensor_info;
     * the coordinates of row f are those sa_tensor_export returns for levels 0 and 1.
     * SA_SCHED_FUSED / ASSOC_LEFT: the nest of the Table of kernels, fiber temporaries T(f, 0:L) in the
     * workspace, then T . D; SA_SCHED_ASSOC_RIGHT: (C . D) first, then one gathered row per nonzero;
     * SA_SCHED_DEFAULT: the one that moves fewer bytes.  L, M in {32, 64}.  A tensor without nonzeros has
     * no output rows; `out` may then be NULL.                                                            */
    SA_EXPR_SPTTM_SPTTM = 9
} sa_expr;

typedef enum {
    SA_SCHED_DEFAULT = 0,      /* the host table's choice for the expression; where two schedules exist
                                  (SPMM_GEMM, SPTTM_SPTTM) the one that moves fewer bytes for this
                                  tensor among those within the auxiliary-memory cap, see sa_schedule_cost */
    SA_SCHED_FUSED = 1,        /* the fissioned / fused branched nest of the Table of kernels   */
    SA_SCHED_ASSOC_LEFT = 2,   /* SA_EXPR_SPMM_GEMM (and SPTTM_SPTTM): (B.C).D, row temporary of L floats    */
    SA_SCHED_ASSOC_RIGHT = 3,  /* SA_EXPR_SPMM_GEMM (and SPTTM_SPTTM): B.(C.D), J x M temporary in workspace */
    SA_SCHED_FISSIONED = 4,    /* one more level of kernel fission: the temporaries of the outermost producer /
                                  consumer pair pass through the workspace.  SA_EXPR_TTMC3: T(i,m,n) per slice
                                  (bitwise reproducible, which SA_SCHED_FUSED is not there: its block
                                  accumulators take shared-memory atomic adds); SA_EXPR_SPTTM_TTM4: T2(m,n) per
                                  (i,j) subtree                                                    */
    SA_SCHED_DEBUG_MATERIALIZE = 9 /* SA_EXPR_SDDMM_SPMM only, for tests: additionally writes the
                                      sampled values B(i,j) * sum_k C(i,k) D(j,k), aligned with
                                      the exported last-level crd array, to the workspace       */
} sa_schedule;

/* Device allocator used for the tensor's device arrays.  alloc returns a DEVICE pointer aligned
 * to at least 256 bytes or NULL; release frees it.  NULL allocator: cudaMalloc / cudaFree. */
typedef struct {
    void *(*alloc)(size_t bytes, void *ctx);
    void (*release)(void *ptr, void *ctx);
    void *ctx;
} sa_allocator;

/* Dense fp32 operand, DEVICE, row-major: element (r, c) at ptr[r * ld + c], ld >= cols
 * (layout of the dense operands in Fig. 1b).  ptr must be 16-byte aligned and ld a multiple
 * of 4.  Caller-owned; only read. */
typedef struct {
    const float *ptr;
    int64_t rows, cols, ld;
} sa_dense;

/*
 * Build the compressed representation of B from coordinate form (Section 2.1).
 *   order   2 (with SA_FMT_CSR) or 3, 4 (with SA_FMT_CSF)
 *   dims    HOST [order], each in [1, 2^31)
 *   nnz     number of stored entries, 0 <= nnz < 2^31
 *   coords  HOST [nnz * order], entry p at coords[p*order .. p*order+order-1], any order;
 *           explicit zeros in vals stay part of the pattern
 *   vals    HOST [nnz] fp32
 *   device  CUDA device ordinal; becomes the tensor's device.  -1 builds a host-only handle
 *           (levels and work lists, no device arrays) that serves sa_tensor_info / _export /
 *           _worklist only; sa_run on it is SA_E_ARG.
 *   dev_alloc  optional allocator for the device arrays (see sa_allocator)
 *   out     receives the handle
 * The entries are sorted lexicographically, the per-level pos / crd arrays and the
 * load-balancing work lists (nonzero-balanced pieces of slices / rows, with their fiber and
 * nonzero ranges) are built on the host and copied to the device.  coords / vals are copied;
 * the caller may free them on return.  Synchronous.
 * Errors: SA_E_ARG, SA_E_FORMAT, SA_E_COORD_RANGE, SA_E_COORD_DUP, SA_E_UNSUPPORTED (the
 * packed coordinate needs more than 64 bits), SA_E_ALLOC, SA_E_CUDA.
 */
sa_status sa_tensor_create(int order, const int64_t *dims, int64_t nnz, const int32_t *coords,
                           const float *vals, sa_format fmt, int device,
                           const sa_allocator *dev_alloc, sa_tensor **out);

/* Sizes of the level structure of Section 2.1.  level_counts HOST [order]: number of stored nodes per level
 * (CSR level 0: rows; last level: nnz; level 1 of a CSF tensor is the paper's nnz(B_ij), the quantity its cost
 * expressions in Section 3 use).  n_chunks: number of work items in the tensor's main work list.  Any
 * output pointer may be NULL. */
sa_status sa_tensor_info(const sa_tensor *t, int64_t *nnz, int64_t *level_counts, int64_t *n_chunks);

/*
 * Copy one level of the compressed structure back to HOST arrays (names as in Fig. 1b).
 *   level 0..order-1.  pos: [count(level-1) + 1] entries (count(-1) = 1); crd: [count(level)];
 *   vals: [nnz], only for the last level.  NULL outputs are skipped.  A CSR tensor has no
 *   pos / crd at level 0 (dense level): asking for them is SA_E_ARG.
 * The arrays are unique for a given input (lexicographic order), so they can be compared
 * bit for bit with an independent construction.
 */
sa_status sa_tensor_export(const sa_tensor *t, int level, int64_t *pos, int32_t *crd, float *vals);

/*
 * Copy a load-balancing work list to HOST arrays: the slice / fiber / nonzero partition arrays the kernels
 * walk (housekeeping for tests and tools; the lists realise the parallel outer loops of the schedules in the
 * Table of kernels, Section 6).  which:
 *   0  main list (order-3 CSF: units of kernel 6, grouped into tasks, see sa_tensor_tasks; CSR: rows for
 *      SA_EXPR_SDDMM_SPMM; order-4 CSF: the same kind of list over the (i,j) subtrees above 4096 nonzeros,
 *      out_row = index among those subtrees, [f0,f1) level-2 nodes)
 *   1  second list (CSR: rows for SA_EXPR_SPMM_GEMM; order-3 CSF: fiber rows for SA_EXPR_SPTTM_SPTTM, rows =
 *      level-1 fibers; order-4 CSF: no items, only the fix-up entries and partial-tile slots of the fused kernel)
 *   2  order-4 CSF: the items of the fused kernel, runs of (i,j) subtrees: out_row / row_end = first subtree /
 *      one past the last (at most 32), last field = kind.  Kind 0: the kernel evaluates them, [f0,f1) their
 *      level-2 fibers, [p0,p1) their nonzeros.  Kind 1: subtrees above 4096 nonzeros (at most 8), whose
 *      temporaries the main list's kernel writes first; f0 = index of the first among those subtrees.
 *   3  order-4 CSF: `items` receives the pieces (one thread block each), 8 int32 per piece: first super-item,
 *      one past the last, first slice, last slice (positions in the level-0 crd array), partial-tile slot of
 *      the first slice or -1, of the last slice or -1, first subtree, one past the last; `fix` receives the
 *      super-items, 4 int32 each: first item, one past the last, first subtree, one past the last (at most 64
 *      subtrees).  counts = {pieces, subtrees above 4096 nonzeros, super-items, 0}.
 *   4, 5, 6  order-4 CSF, the lists of SA_SCHED_FISSIONED: 4 = like list 0 over the (i,j) subtrees with more than 64
 *      level-2 fibers or 4096 nonzeros (out_row = index of the level-1 fiber); 5 = second pass, one item per (piece
 *      of at most 512 level-1 fibers [f0,f1) of slice out_row, quarter of the 256 columns (m,n) in the last field;
 *      a piece of at most eight fibers is a single item with 4 there: all quarters),
 *      with the fix-up entries of slices cut into pieces; 6 = first pass on whole small subtrees: rows
 *      [out_row,row_end) = level-1 fibers, [f0,f1) their level-2 fibers (at most 64), [p0,p1) their nonzeros
 * For which = 0..2 and 4..6:
 *   counts [4]: number of items, number of leading groups that one thread block reduces into a
 *               single tile (8 items each; order-3 tensors: 4 tasks each, see sa_tensor_tasks),
 *               number of fix-up entries, number of partial-tile slots
 *   items  [n_items * 8] int32 per item: out_row, row_end, f0, f1, p0, p1, dest, last --
 *               fibers [f0,f1) (CSF) clipped to nonzeros [p0,p1) of slice out_row, or rows
 *               [out_row,row_end) / nonzeros [p0,p1) of a long row (CSR); dest = partial slot or -1;
 *               the last field is the position of the item's slice in the level-0 crd array (list 0)
 *   fix    [n_fix * 4] int32 per entry: out_row, slot0, count, 0 -- out[out_row] = sum of `count`
 *               partial tiles from slot0 (count 0: the slice / row is empty and is zero-filled)
 * NULL outputs are skipped.
 */
sa_status sa_tensor_worklist(const sa_tensor *t, int which, int64_t *counts, int32_t *items, int32_t *fix);

/*
 * CSF tensors: how the items of the main work list are handed to warps (the warp-level
 * partition arrays of the fiber stage; housekeeping, no passage of the paper).
 *   n_tasks     number of tasks; warp w of the launch evaluates task w
 *   task_start  HOST [n_tasks + 1]: task w holds the items [task_start[w], task_start[w + 1]).  The first
 *               4 * counts[1] tasks (counts of sa_tensor_worklist) hold one item or none: four
 *               consecutive ones are the pieces of one chunk of a large slice, summed by one thread
 *               block.  Every later task holds up to 16 whole small slices.
 *   stream_f0   HOST [n_items * 4]: inside an item the warp's four groups of eight lanes each stream a
 *               contiguous part of the nonzeros [p0, p1).  With b = p0 rounded down to a multiple of 8
 *               and s = ceil((p1 - b) / 4) rounded up to a multiple of 8, part q is
 *               [b + q s, b + (q + 1) s) clipped to [p0, p1); stream_f0[4 n + q] is the level-1 fiber
 *               that holds the first nonzero of part q of item n (f0 of the item if the part is empty).
 * NULL outputs are skipped.  Errors: SA_E_ARG, SA_E_FORMAT (not a CSF tensor).
 */
sa_status sa_tensor_tasks(const sa_tensor *t, int64_t *n_tasks, int32_t *task_start, int32_t *stream_f0);

/* Bytes of DEVICE workspace sa_run needs for this tensor / expression / schedule / operand
 * shapes (may be 0): the schedule's auxiliary memory in the sense of Section 5 (the dense temporaries
 * of the chosen nest that do not fit on chip, plus the partial tiles of split slices / rows).  Only the
 * shapes in ops are read. */
sa_status sa_workspace_size(const sa_tensor *t, sa_expr expr, sa_schedule sched, const sa_dense *ops,
                            int n_ops, size_t *bytes);

/*
 * What a schedule costs for this tensor and these operand shapes: the quantities the paper's run-time Stage 4
 * (Section 5.2) compares -- a time term and the auxiliary memory -- with concrete sizes plugged in.
 *   iterations      iteration complexity of the branched loop nest that runs, i.e. its total number of loop
 *                   iterations in the sense of Section 3 (the caption formulas of the figure with the five
 *                   schedules of kernel 5 are of this kind); sparse loops count stored nodes of their level
 *   moved_bytes     bytes the schedule's kernels load and store: streams of B once, the output once, dense
 *                   operands that are read in order once, gathered rows once per use (a row served by the
 *                   last-level cache still occupies the load path), temporaries in the workspace written and
 *                   read.  This is the time term the default schedule is chosen by (the chains are bound by
 *                   memory traffic here, not by loop iterations).
 *   temp_elements   dense temporaries that pass values from producer to consumer nests, in elements: the
 *                   paper's auxiliary memory (Section 4.2; table of auxiliary memory requirements, Section 6),
 *                   whether they live in registers, shared memory or the workspace
 *   workspace_bytes what sa_workspace_size returns for the schedule
 *   resolved        the schedule that runs (differs from `sched` for SA_SCHED_DEFAULT)
 * Only the shapes in ops are read.  Errors: SA_E_ARG, SA_E_FORMAT, SA_E_SHAPE, SA_E_UNSUPPORTED.
 */
typedef struct {
    double iterations, moved_bytes, temp_elements;
    size_t workspace_bytes;
    int resolved;
} sa_cost;
sa_status sa_schedule_cost(const sa_tensor *t, sa_expr expr, sa_schedule sched, const sa_dense *ops, int n_ops,
                           sa_cost *cost);

/*
 * Cap, in bytes, on the workspace a schedule picked by SA_SCHED_DEFAULT may need (the user-given upper bound on
 * auxiliary memory that Section 5.2 mentions for its memory pruning; the paper's own Stage 4 uses half of the
 * last-level cache).  Among the expression's schedules whose workspace fits, the default takes the one with the
 * smallest moved_bytes; if none fits, the one with the smallest workspace.  Explicitly named schedules are not
 * affected.  Default: no cap.  Set it before sizing workspaces; not synchronised with concurrent sa_run calls.
 */
sa_status sa_tensor_set_aux_limit(sa_tensor *t, size_t bytes);

/*
 * Evaluate the chain: out = expr(B, ops...), asynchronously on cuda_stream.
 *   ops        HOST array of n_ops descriptors of DEVICE operands, in the order listed at sa_expr
 *   out        DEVICE fp32, dense row-major, contiguous, 16-byte aligned; FULLY OVERWRITTEN
 *              (the statement is an assignment; empty slices / rows become +0.0)
 *   workspace  DEVICE scratch of at least sa_workspace_size bytes, 256-byte aligned; may be
 *              NULL when that size is 0.  Contents on entry are ignored.
 *   cuda_stream  a cudaStream_t (NULL = default stream)
 * Compiled dense ranks (anything else is SA_E_UNSUPPORTED): SPTTM_TTM3 L, M in {16, 32};
 * SPTTM_TTM4 L = M = N = 16; SDDMM_SPMM K, L in {32, 64, 128}; SPMM_GEMM L in {128, 256},
 * M in {32, 64}; TTMC3 L, M, N in {16, 32}; SDDMM_SPMM_GEMM K, L in {32, 64, 128}, M in {32, 64};
 * SPMMH_GEMM L in {128, 256}, M in {32, 64}; MTTKRP_GEMM R = 32, M in {32, 64};
 * SPTTM_SPTTM L, M in {32, 64} (out: level_counts[1] x M, see sa_expr).
 * Arithmetic: fp32 throughout; stages on tensor cores split every fp32 operand into two parts and
 * add three partial products (TF32 parts in the per-slice contractions, BF16 parts in the dense GEMM
 * stage), so every output element stays within 1e-4 of the sum of the absolute values of its terms.
 * The dense GEMM stage (SPMM_GEMM as B.(C.D), SDDMM_SPMM_GEMM) waits on on-chip hand-offs with a
 * 2-second limit; if one runs out the kernel returns and sa_last_device_status reports SA_E_TIMEOUT.
 * Returns launch errors only; completion is observed by synchronising the stream.
 * Errors: SA_E_ARG, SA_E_SHAPE, SA_E_UNSUPPORTED, SA_E_WORKSPACE, SA_E_CUDA.
 */
sa_status sa_run(const sa_tensor *B, sa_expr expr, sa_schedule sched, const sa_dense *ops, int n_ops,
                 float *out, void *workspace, size_t workspace_bytes, void *cuda_stream);

/*
 * (No counterpart in the paper: an addition for callers of this library that must not allocate.)
 *
 * sa_run for SA_EXPR_SPTTM_TTM3 without a caller-supplied workspace and without any allocation.
 * Some callers cannot hand sa_run a workspace because they are not in a position to obtain
 * device memory when they call: code that runs after start-up under a fixed memory plan in
 * which every byte is already assigned, plug-ins whose host application owns all allocation,
 * and latency-critical loops that must stay clear of cudaMalloc / cudaFree because those calls
 * may synchronise the whole device.  For them the partial tiles of split slices go to a scratch
 * array of 4 MiB that is built into the library (a file-scope __device__
 * array: every device that loads the library holds these 4 MiB until the process exits).
 *
 *   B, ops, out, cuda_stream   as for sa_run with SA_EXPR_SPTTM_TTM3 (ops = {C, D}, n_ops = 2)
 *
 * The call itself makes no cudaMalloc, cudaFree or other allocating call.  The first call on a
 * device looks up the scratch array's device address (cudaGetSymbolAddress, with that device
 * current) and caches it; make that first call before starting any stream capture.
 * Limit: sa_workspace_size(B, SA_EXPR_SPTTM_TTM3, ...) must not exceed 4 MiB (1024 partial
 * tiles at L = M = 32); beyond that the call returns SA_E_WORKSPACE and enqueues nothing --
 * use sa_run with a workspace instead.
 * All calls in a process share the one array per device.  Nothing in it has to start at zero
 * (every slot that is read was written earlier in the same call), so it is not cleared, and it
 * keeps the previous call's partial tiles.  Two calls that overlap on the device -- different
 * streams, or different handles on the same device -- race on it and give wrong results: keep
 * calls of this entry point ordered on one stream, or use sa_run with separate workspaces.
 * Errors: SA_E_ARG, SA_E_FORMAT, SA_E_SHAPE, SA_E_UNSUPPORTED, SA_E_WORKSPACE, SA_E_CUDA.
 */
sa_status sa_run_ttm3_static_scratch(const sa_tensor *B, const sa_dense *ops, int n_ops, float *out,
                                     void *cuda_stream);

/* Number of kernel launches the last successful sa_run on this handle enqueued. */
sa_status sa_last_launch_count(const sa_tensor *t, int *launches);

/* Synchronise cuda_stream and report the device-side status word of the tensor (SA_OK,
 * SA_E_BOUNDS, SA_E_TIMEOUT), clearing it. */
sa_status sa_last_device_status(const sa_tensor *t, void *cuda_stream);

/* Synchronise cuda_stream and copy the raw status word to HOST words[4] without clearing it: words[0] is
 * 0 or the status above; for SA_E_BOUNDS (set only by a library built with -DSA_DEBUG_BOUNDS) words[1] is
 * the number of the check that failed, words[2] the offending index, words[3] the global thread. */
sa_status sa_device_status_words(const sa_tensor *t, void *cuda_stream, int32_t *words);

/* Release device and host memory of the handle.  NULL is accepted. */
void sa_destroy(sa_tensor *t);

const char *sa_status_string(sa_status s);

#ifdef __cplusplus
}
#endif
#endif /* SPARSEAUTO_H */
