// Order-4 chain A(i,l,m,n) = sum_{j,k,o} B(i,j,k,o) C(j,l) D(k,m) E(o,n), schedule SA_SCHED_FISSIONED: the two-level
// nest of sa_ttm4.cu with its outer producer/consumer pair fissioned at the j' loop,
//   pass 1:  T2(f; m,n) = sum_{k,o} B(f; k,o) D(k,m) E(o,n)   for every level-1 fiber f = (i,j)   -> workspace
//   pass 2:  A(i, l, (m,n)) = sum_{f in slice i} C(j_f, l) T2(f; (m,n))                              per slice
// The temporaries T2 (1 KB per (i,j) subtree) are written and read once through HBM: about three times the bytes
// of the fused schedule, and a workspace that grows with the tensor.  In exchange pass 1 needs neither a pool of
// temporaries nor the slice accumulators in registers, keeps twice as many warps per SM resident, and the two
// passes together are faster on the benchmark tensor; the default schedule takes it while the workspace fits the
// caller's cap (sa_tensor_set_aux_limit).
// Pass 1 is kernel 6 on the (i,j) subtrees: the small ones (at most 64 level-2 fibers and 4096 nonzeros) by the
// subtree kernel below, the others by the order-3 kernel (sa_ttm3.cu) with the level-1 fibers as slices, D and E as
// factors.  Pass 2 contracts, per slice, the temporaries with the rows C(j,:) on tensor cores.
#include <algorithm>

#include "sa_device.cuh"

namespace {

constexpr int R = 16;                  // L = M = N = 16
constexpr int TILE4 = R * R * R;       // floats per output slice
constexpr int T2F = R * R;             // floats per temporary
constexpr int QC = 64;                 // temporary columns per item (a quarter)
constexpr int NT4 = QC / 8;            // n8 tiles per item

// Limits for the checks of the self-checking build (SA_CHK, sa_device.cuh).
struct fis_limits {
    int32_t *status;
    uint32_t c_rows, d_rows, e_rows, n_slices;
    int32_t n_subtrees, n_fibers, n_slots, nnz;
};

// Pass 2.  One warp per item (fibers [f0, f1) of one slice, quarter `pad` of the temporaries' columns; `pad` = 4:
// all four quarters, one after the other, for pieces of at most eight fibers); warps take items in a grid-wide
// stride, largest items first.  Seen from a warp, its items are one sequence of groups (item, quarter, eight fibers).
// The temporaries of a group (8 rows of 64 floats) are copied to shared memory with cp.async three groups ahead of
// their use, across quarter and item boundaries, so that the stream of 1 KB tiles out of HBM never stops at the many
// short items; the C values of a group (a few gathered words out of L2) are loaded one group ahead into registers.
constexpr int SL_DEPTH = 4;                        // stages of the shared-memory ring (groups in flight + 1)
constexpr int SL_RS = QC + 8;                      // row stride in floats: rows t and t + 1 land 8 banks apart
constexpr int SL_STAGE = 8 * SL_RS;                // floats per stage
constexpr int SL_SMEM = SA_WARPS_PER_CTA * SL_DEPTH * SL_STAGE * int(sizeof(float));   // 72 KB

// Position in a warp's sequence of groups.
struct sl_cursor {
    int64_t n;              // item
    int row, dest;          // its output slice and partial slot (< 0: none)
    int f0, f1, f;          // its fibers, and the first fiber of the current group
    int qc, q_last;         // current and last quarter
    bool live;
};

__device__ __forceinline__ void sl_load_item(sl_cursor &c, const sa_item *__restrict__ items, int64_t n_items, int64_t stride,
                                             const fis_limits &lim)
{
    for (;;) {
        c.live = c.n < n_items;
        if (!c.live) return;
        const int4 ia = __ldg(reinterpret_cast<const int4 *>(items + c.n));          // out_row, row_end, f0, f1
        const int4 ib = __ldg(reinterpret_cast<const int4 *>(items + c.n) + 1);      // p0, p1, dest, quarter
        if (SA_CHK(lim.status, ia.z >= 0 && ia.z <= ia.w && ia.w <= lim.n_subtrees && uint32_t(ib.w) <= 4u && uint32_t(ia.x) < lim.n_slices &&
                                   ib.z < lim.n_slots, 72, c.n)) {
            c.row = ia.x; c.dest = ib.z;
            c.f0 = c.f = ia.z; c.f1 = ia.w;
            c.qc = ib.w == 4 ? 0 : ib.w;
            c.q_last = ib.w == 4 ? 3 : ib.w;
            return;
        }
        c.n += stride;          // a record that fails its check is skipped
    }
}

// To the next group: eight fibers on, else the next quarter of the item, else the next item of the warp.
__device__ __forceinline__ void sl_advance(sl_cursor &c, const sa_item *__restrict__ items, int64_t n_items, int64_t stride,
                                           const fis_limits &lim)
{
    c.f += 8;
    if (c.f < c.f1) return;
    c.f = c.f0;
    if (++c.qc <= c.q_last) return;
    c.n += stride;
    sl_load_item(c, items, n_items, stride, lim);
}

// The C entries of a group for a lane's A fragments: fibers t and t + 4 of the group, columns g and g + 8; fibers
// past the end of the item read as zero.  Two dependent gathers (the fiber's j, then C(j,:)), taken in two steps one
// group apart so that neither latency lies between two groups' products.
__device__ __forceinline__ void sl_load_j(uint32_t (&j)[2], const sl_cursor &cur, int lane, const int32_t *__restrict__ crd_j,
                                          const fis_limits &lim)
{
    const int t = lane & 3;
    const int fa = cur.f + t, fb = cur.f + t + 4;
    const bool va = cur.live && fa < cur.f1, vb = cur.live && fb < cur.f1;
    j[0] = uint32_t(va ? __ldg(crd_j + fa) : 0);
    j[1] = uint32_t(vb ? __ldg(crd_j + fb) : 0);
    if (!SA_CHK(lim.status, j[0] < lim.c_rows, 71, j[0])) j[0] = 0u;
    if (!SA_CHK(lim.status, j[1] < lim.c_rows, 71, j[1])) j[1] = 0u;
}
__device__ __forceinline__ void sl_load_c(float (&c)[4], const uint32_t (&j)[2], const sl_cursor &cur, int lane,
                                          const float *__restrict__ C, uint32_t ldc)
{
    const int g = lane >> 2, t = lane & 3;
    const bool va = cur.live && cur.f + t < cur.f1, vb = cur.live && cur.f + t + 4 < cur.f1;
    const float *ca = C + j[0] * ldc + g;
    const float *cb = C + j[1] * ldc + g;
    c[0] = va ? __ldg(ca) : 0.f;
    c[1] = va ? __ldg(ca + 8) : 0.f;
    c[2] = vb ? __ldg(cb) : 0.f;
    c[3] = vb ? __ldg(cb + 8) : 0.f;
}

// Copies of the group's eight quarter rows into a stage: 128 pieces of 16 bytes, four per lane; rows past the end of
// the item are filled with zeros (their C entries are zero too, but what the stage held before need not be finite).
__device__ __forceinline__ void sl_issue(const sl_cursor &cur, uint32_t stage, int lane, const float *__restrict__ T2)
{
    if (cur.live) {
        const int piece = lane & 15;
        const float *src = T2 + int64_t(cur.f) * T2F + cur.qc * QC + 4 * piece;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = (lane >> 4) + 2 * i;
            const uint32_t dst = stage + uint32_t(r * SL_RS + 4 * piece) * 4u;
            if (cur.f + r < cur.f1) cp_async16_raw(dst, src + int64_t(r) * T2F);
            else asm volatile("st.shared.v4.f32 [%0], {%1,%1,%1,%1};" ::"r"(dst), "f"(0.f) : "memory");
        }
    }
    cp_async_commit();
}

__global__ void __launch_bounds__(256, 2)
ttm4_slice_kernel(const sa_item *__restrict__ items, int64_t n_items, const int32_t *__restrict__ crd_j,
                  const float *__restrict__ T2, const float *__restrict__ C, uint32_t ldc, float *__restrict__ out,
                  float *__restrict__ partial, const fis_limits lim)
{
    extern __shared__ __align__(16) float sl_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, g = lane >> 2, t = lane & 3;
    const int64_t stride = int64_t(gridDim.x) * SA_WARPS_PER_CTA;
    const uint32_t ring = smem_u32(sl_smem) + uint32_t(warp) * uint32_t(SL_DEPTH * SL_STAGE * 4);
    sl_cursor prod, cons, next, next2;               // groups i + 3, i, i + 1, i + 2
    prod.n = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    sl_load_item(prod, items, n_items, stride, lim);
    cons = next = prod;
    if (!cons.live) return;
    // the first SL_DEPTH - 1 groups go out before anything is consumed
#pragma unroll
    for (int s = 0; s < SL_DEPTH - 1; ++s) {
        sl_issue(prod, ring + uint32_t(s * SL_STAGE * 4), lane, T2);
        if (prod.live) sl_advance(prod, items, n_items, stride, lim);
    }
    float cc[4], cn[4];
    uint32_t jc[2], jn[2], jn2[2];
    sl_load_j(jc, cons, lane, crd_j, lim);
    sl_advance(next, items, n_items, stride, lim);
    sl_load_j(jn, next, lane, crd_j, lim);
    sl_load_c(cc, jc, cons, lane, C, ldc);
    next2 = next;
    if (next2.live) sl_advance(next2, items, n_items, stride, lim);
    float acc[NT4][4];
#pragma unroll
    for (int nt = 0; nt < NT4; ++nt)
#pragma unroll
        for (int x = 0; x < 4; ++x) acc[nt][x] = 0.f;
    int sc = 0;                                       // stage of the group being consumed
    while (cons.live) {
        __syncwarp();                                 // every lane is done with the stage that is filled next
        sl_issue(prod, ring + uint32_t((sc == 0 ? SL_DEPTH - 1 : sc - 1) * SL_STAGE * 4), lane, T2);
        if (prod.live) sl_advance(prod, items, n_items, stride, lim);
        sl_load_j(jn2, next2, lane, crd_j, lim);                  // both in flight during the products below
        sl_load_c(cn, jn, next, lane, C, ldc);
        cp_async_wait<SL_DEPTH - 1>();
        __syncwarp();
        const float *st = sl_smem + (warp * SL_DEPTH + sc) * SL_STAGE;
        uint32_t ah[4], al[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) split_tf32(cc[x], ah[x], al[x]);
#pragma unroll
        for (int nt = 0; nt < NT4; ++nt) {
            uint32_t bh[2], bl[2];
            split_tf32(st[t * SL_RS + 8 * nt + g], bh[0], bl[0]);
            split_tf32(st[(t + 4) * SL_RS + 8 * nt + g], bh[1], bl[1]);
            mma_m16n8k8_tf32(acc[nt], al, bh);
            mma_m16n8k8_tf32(acc[nt], ah, bl);
            mma_m16n8k8_tf32(acc[nt], ah, bh);
        }
        if (cons.f + 8 >= cons.f1) {
            // the quarter's last group: element (l, column 64 qc + 8 nt + 2 t (+1)) of the slice tile, l = g and g + 8
            float *dst = (cons.dest >= 0 ? partial + int64_t(cons.dest) * TILE4 : out + int64_t(cons.row) * TILE4) + cons.qc * QC + 2 * t;
#pragma unroll
            for (int nt = 0; nt < NT4; ++nt) {
                const float2 lo = make_float2(acc[nt][0], acc[nt][1]), hi = make_float2(acc[nt][2], acc[nt][3]);
                if (cons.dest >= 0) {
                    *reinterpret_cast<float2 *>(dst + g * T2F + 8 * nt) = lo;
                    *reinterpret_cast<float2 *>(dst + (g + 8) * T2F + 8 * nt) = hi;
                } else {
                    sa_st_cs2(dst + g * T2F + 8 * nt, lo);
                    sa_st_cs2(dst + (g + 8) * T2F + 8 * nt, hi);
                }
#pragma unroll
                for (int x = 0; x < 4; ++x) acc[nt][x] = 0.f;
            }
        }
        cons = next;
        next = next2;
        if (next2.live) sl_advance(next2, items, n_items, stride, lim);
#pragma unroll
        for (int x = 0; x < 4; ++x) cc[x] = cn[x];
        jn[0] = jn2[0]; jn[1] = jn2[1];
        sc = sc == SL_DEPTH - 1 ? 0 : sc + 1;
    }
    cp_async_wait<0>();
}

// Pass 1 on whole (i,j) subtrees (tensors whose subtrees are all small: the usual case, a subtree holds a few
// dozen nonzeros).  One warp per item = a range of consecutive subtrees with at most SA_SUB_MAX_F3 level-2 fibers.
//   Phase A (Q1):  t(f; n) = sum_o B(f; o) E(o,n) for every level-2 fiber f = (i,j,k) of the item.  Four lanes own a
//     row of E as one float4 each, so the warp's eight lane groups walk equal shares of the item's nonzeros, one
//     nonzero per group and step (index/value pairs eight per load and one load ahead, eight row gathers in
//     flight); the end-of-fiber bit travels in the sign bit of the index and parks t(f; :) in the fiber's own slot
//     of the warp's shared-memory tile, so the parked rows end up in fiber order without any bookkeeping.
//   Phase B (Q2):  T2(m,n) += D(k_f, m) t(f; n) over the fibers of each subtree, eight fibers at a time as
//     T2 += Dg^T (16 x 8) . t (8 x 16) on tensor cores (m16n8k8 TF32, both operands split into a high and a low part,
//     three products): a lane loads four values of D and four of the parked rows per group, where one fiber per step
//     on the ALUs cost it six values per fiber, and the load/store pipe is what bounds this kernel.  Fibers past
//     the end of a subtree enter as zero rows.  The 1 KB tile is stored when the subtree's last group is in.
// Against the order-3 kernel on the same subtrees this drops the per-unit pipeline drains, the cross-stream
// bookkeeping of parked rows and the slice-wide accumulator tile.
constexpr int SUB_RS = R + 8;          // floats per parked row: t(16), the fiber's k, pad; rows t and t + 1 land 8 banks apart
constexpr int SUB_SMEM = SA_WARPS_PER_CTA * SA_SUB_MAX_F3 * SUB_RS * int(sizeof(float));   // 48 KB

// CONTIG: both factor matrices are stored without padding (leading dimension 16), so a row offset is a shift.
template <bool CONTIG>
__global__ void __launch_bounds__(256, 4)
ttm4_subtree_kernel(const sa_item *__restrict__ items, int64_t n_items, const int32_t *__restrict__ pos2,
                    const int32_t *__restrict__ pos3, const int32_t *__restrict__ crd_k, const int2 *__restrict__ nz,
                    const float *__restrict__ D, int64_t ldd, const float *__restrict__ E, int64_t lde, float *__restrict__ T2,
                    const fis_limits lim)
{
    extern __shared__ __align__(16) float sub_smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    if (idx >= n_items) return;
    const sa_item it = items[idx];
    if (!SA_CHK(lim.status, it.f0 >= 0 && it.f1 - it.f0 <= SA_SUB_MAX_F3 && it.f1 <= lim.n_fibers && it.out_row >= 0 &&
                                it.row_end - it.out_row <= SA_SUB_MAX_ROWS && it.row_end <= lim.n_subtrees && it.p0 >= 0 && it.p1 <= lim.nnz,
                73, idx))
        return;
    float *pk = sub_smem + warp * (SA_SUB_MAX_F3 * SUB_RS);
    // row offsets in 32-bit arithmetic (the launcher checks rows * ld < 2^31)
    const uint32_t ld_d = CONTIG ? uint32_t(R) : uint32_t(ldd), ld_e = CONTIG ? uint32_t(R) : uint32_t(lde);
    const int nf3 = it.f1 - it.f0;
    // the k of the item's fibers (requested now; their D row offsets are parked beside the rows of t)
    static_assert(SA_SUB_MAX_F3 <= 64, "two index registers per lane");
    int kk0 = lane < nf3 ? __ldg(crd_k + it.f0 + lane) : 0;
    int kk1 = lane + 32 < nf3 ? __ldg(crd_k + it.f0 + 32 + lane) : 0;
    if (!SA_CHK(lim.status, uint32_t(kk0) < lim.d_rows && uint32_t(kk1) < lim.d_rows, 74, kk0)) kk0 = kk1 = 0;
    // word 16 of a fiber's parked row: the element offset of its row of D
    pk[lane * SUB_RS + R] = __uint_as_float(uint32_t(kk0) * ld_d);
    pk[(lane + 32) * SUB_RS + R] = __uint_as_float(uint32_t(kk1) * ld_d);
    {   // ---- phase A
        const int g = lane >> 2, l = lane & 3;
        // shares of the eight groups: equal counts of nonzeros, whatever the fiber boundaries (whole-fiber shares left
        // the longest group 1.6 times the mean, and every group runs as many steps as the longest).  A fiber cut by
        // a share boundary gets its parts added together after the loop.
        const int s0 = lane < nf3 ? __ldg(pos3 + it.f0 + lane) : 0x7fffffff;
        const int s1 = lane + 32 < nf3 ? __ldg(pos3 + it.f0 + 32 + lane) : 0x7fffffff;
        const int share = (it.p1 - it.p0 + 7) >> 3;
        const int ga = min(it.p0 + g * share, it.p1), gb = min(ga + share, it.p1);
        const int mylen = gb - ga;
        const int maxlen = share;
        int slot = 0;                                   // the fiber that holds nonzero ga: the last one starting at or before it
#pragma unroll
        for (int q = 0; q < 8; ++q) {
            const int target = min(it.p0 + q * share, it.p1);
            const int cnt = __popc(__ballot_sync(SA_FULL_MASK, s0 <= target)) + __popc(__ballot_sync(SA_FULL_MASK, s1 <= target));
            if (g == q) slot = cnt - 1;
        }
        auto fetch1 = [&](int q, int &x, float &v) {
            x = 0;
            v = 0.f;
            if (q < mylen && SA_CHK(lim.status, ga + q >= 0 && ga + q < lim.nnz, 75, ga + q)) {
                const int2 w = __ldg(nz + ga + q);                   // (index o | end-of-fiber bit << 31, value bits)
                x = w.x;
                v = __int_as_float(w.y);
            }
        };
        // lane l of the group holds nonzeros c + l and c + 4 + l of the group's stream
        auto fetch = [&](int c, int (&x)[2], float (&v)[2]) {
            fetch1(c + l, x[0], v[0]);
            fetch1(c + 4 + l, x[1], v[1]);
        };
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        int xn[2];
        float vn[2];
        fetch(0, xn, vn);
        for (int c = 0; c < maxlen; c += 8) {
            const int x[2] = {xn[0], xn[1]};
            const float v[2] = {vn[0], vn[1]};
            fetch(c + 8, xn, vn);
#pragma unroll
            for (int h = 0; h < 2; ++h) {               // two batches of four row gathers
                int xs[4];
                float vs[4];
                float4 e[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    xs[u] = __shfl_sync(SA_FULL_MASK, x[h], u, 4);
                    vs[u] = __shfl_sync(SA_FULL_MASK, v[h], u, 4);
                    uint32_t o = uint32_t(xs[u]) & 0x7fffffffu;
                    if (!SA_CHK(lim.status, o < lim.e_rows, 76, o)) o = 0u;
                    e[u] = sa_ldg4(E + (o * ld_e + 4u * l));
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (c + 4 * h + u < mylen) {
                        acc.x = fmaf(vs[u], e[u].x, acc.x);
                        acc.y = fmaf(vs[u], e[u].y, acc.y);
                        acc.z = fmaf(vs[u], e[u].z, acc.z);
                        acc.w = fmaf(vs[u], e[u].w, acc.w);
                    }
                    if (xs[u] < 0) {                                  // last nonzero of fiber it.f0 + slot
                        if (SA_CHK(lim.status, slot >= 0 && slot < nf3, 77, slot)) *reinterpret_cast<float4 *>(pk + slot * SUB_RS + 4 * l) = acc;
                        acc = make_float4(0.f, 0.f, 0.f, 0.f);
                        ++slot;
                    }
                }
            }
        }
        // the open part of a cut fiber is added to the fiber's row once every group has stored the rows it closed
        __syncwarp();
        // (a sum left open is what the accumulator holds; after a fiber's last nonzero it is zero and nothing is added)
        if ((acc.x != 0.f || acc.y != 0.f || acc.z != 0.f || acc.w != 0.f) && SA_CHK(lim.status, slot >= 0 && slot < nf3, 77, slot)) {
            float *row = pk + slot * SUB_RS + 4 * l;
            atomicAdd(row, acc.x);
            atomicAdd(row + 1, acc.y);
            atomicAdd(row + 2, acc.z);
            atomicAdd(row + 3, acc.w);
        }
    }
    __syncwarp();
    {   // ---- phase B: per subtree, eight fibers at a time, T2 += D(k_f, :)^T (16 x 8) . t (8 x 16) on tensor cores
        const int g = lane >> 2, t = lane & 3;
        const int nr = it.row_end - it.out_row;
        const int my_end = lane < nr ? __ldg(pos2 + it.out_row + lane + 1) - it.f0 : 0x7fffffff;   // local end of subtree `lane`
        int fbeg = 0;
        for (int r = 0; r < nr; ++r) {
            const int fend = min(__shfl_sync(SA_FULL_MASK, my_end, r), nf3);
            float acc[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int x = 0; x < 4; ++x) acc[nt][x] = 0.f;
            for (int fg = fbeg; fg < fend; fg += 8) {
                // fibers fg + t and fg + t + 4 of the group; past the subtree's end they count as zero rows
                const bool va = fg + t < fend, vb = fg + t + 4 < fend;
                const float *ra = pk + (va ? fg + t : fbeg) * SUB_RS;
                const float *rb = pk + (vb ? fg + t + 4 : fbeg) * SUB_RS;
                const float *da = D + __float_as_uint(ra[R]) + g;
                const float *db = D + __float_as_uint(rb[R]) + g;
                float av[4];
                av[0] = va ? __ldg(da) : 0.f;
                av[1] = va ? __ldg(da + 8) : 0.f;
                av[2] = vb ? __ldg(db) : 0.f;
                av[3] = vb ? __ldg(db + 8) : 0.f;
                uint32_t ah[4], al[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) split_tf32(av[x], ah[x], al[x]);
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    uint32_t bh[2], bl[2];
                    split_tf32(va ? ra[8 * nt + g] : 0.f, bh[0], bl[0]);
                    split_tf32(vb ? rb[8 * nt + g] : 0.f, bh[1], bl[1]);
                    mma_m16n8k8_tf32(acc[nt], al, bh);
                    mma_m16n8k8_tf32(acc[nt], ah, bl);
                    mma_m16n8k8_tf32(acc[nt], ah, bh);
                }
            }
            // element (m, n) of the subtree's temporary: m = g and g + 8, n = 8 nt + 2 t (+ 1)
            float *dst = T2 + int64_t(it.out_row + r) * T2F + 2 * t;
#pragma unroll
            for (int nt = 0; nt < 2; ++nt) {
                *reinterpret_cast<float2 *>(dst + g * R + 8 * nt) = make_float2(acc[nt][0], acc[nt][1]);
                *reinterpret_cast<float2 *>(dst + (g + 8) * R + 8 * nt) = make_float2(acc[nt][2], acc[nt][3]);
            }
            fbeg = fend;
        }
    }
}

struct ttm4_plan {
    size_t t2_bytes, p1_bytes, p2_bytes;
};

ttm4_plan plan(const sa_tensor *t)
{
    ttm4_plan p;
    p.t2_bytes = sa_align256(size_t(t->count[1]) * T2F * sizeof(float));
    p.p1_bytes = sa_align256(size_t(t->wl4_main.n_slots) * T2F * sizeof(float));
    p.p2_bytes = sa_align256(size_t(t->wl4_aux.n_slots) * TILE4 * sizeof(float));
    return p;
}

}  // namespace

// workspace: [T2: one 16 x 16 temporary per level-1 fiber][partial temporaries of pass 1][partial tiles of pass 2]
size_t sa_ws_ttm4_fissioned(const sa_tensor *t, const sa_dense *)
{
    const ttm4_plan p = plan(t);
    return p.t2_bytes + p.p1_bytes + p.p2_bytes;
}

sa_status sa_launch_ttm4_fissioned(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t, cudaStream_t stream,
                         int *launches)
{
    const ttm4_plan p = plan(t);
    *launches = 0;
    for (int i = 0; i < 3; ++i)                     // every range check comes before the first launch
        if (ops[i].rows * ops[i].ld >= (int64_t(1) << 30)) return SA_E_UNSUPPORTED;   // 32-bit element offsets of factor rows
    char *base = static_cast<char *>(ws);
    float *T2 = reinterpret_cast<float *>(base);
    float *part1 = reinterpret_cast<float *>(base + p.t2_bytes);
    float *part2 = reinterpret_cast<float *>(base + p.t2_bytes + p.p1_bytes);
    // the large subtrees: kernel 6 with the (i,j) subtrees as slices, factors D (rows by k) and E (rows by o)
    sa_ttm3_view v;
    v.wl = &t->wl4_main;
    v.crd_fiber = t->d_crd[2];
    v.crd_nz = t->d_crd[3];
    v.vals = t->d_vals;
    v.endbits = t->d_endbits;
    v.n_fibers = t->count[2];
    v.n_out_rows = t->count[1];
    v.nnz = t->wl4_main.nnz;
    v.nnz_total = t->nnz;
    v.status = t->d_status;
    fis_limits lim;
    lim.status = t->d_status;
    lim.c_rows = uint32_t(ops[0].rows); lim.d_rows = uint32_t(ops[1].rows); lim.e_rows = uint32_t(ops[2].rows);
    lim.n_slices = uint32_t(t->dims[0]);
    lim.n_subtrees = int32_t(t->count[1]); lim.n_fibers = int32_t(t->count[2]);
    lim.n_slots = int32_t(t->wl4_aux.n_slots); lim.nnz = int32_t(t->nnz);
    // pass 1: the small subtrees whole (subtree kernel), the large ones as slices of the order-3 kernel
    const int64_t n_sub = int64_t(t->wl4_sub.items.size());
    *launches = 0;
    if (n_sub > 0) {
        const bool contig = ops[1].ld == R && ops[2].ld == R;
        auto kern = contig ? ttm4_subtree_kernel<true> : ttm4_subtree_kernel<false>;
        static bool attr_contig[SA_MAX_DEVICE_FLAGS], attr_strided[SA_MAX_DEVICE_FLAGS];
        if (!sa_set_smem_once(kern, SUB_SMEM, contig ? attr_contig : attr_strided)) return SA_E_CUDA;
        const int64_t ctas = (n_sub + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
        kern<<<(unsigned)ctas, 256, SUB_SMEM, stream>>>(t->wl4_sub.d_items, n_sub, t->d_pos[2], t->d_pos[3], t->d_crd[2],
                                                                       t->d_nzpack, ops[1].ptr, ops[1].ld, ops[2].ptr, ops[2].ld, T2, lim);
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    if (!t->wl4_main.items.empty()) {
        int n1 = 0;
        const sa_status s = sa_launch_ttm3_view(v, ops[1], ops[2], T2, part1, stream, &n1);
        if (s != SA_OK) return s;
        *launches += n1;
    }
    // pass 2
    const sa_worklist &wl = t->wl4_aux;
    const int64_t n_items = int64_t(wl.items.size());
    if (n_items > 0) {
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        const int64_t ctas = std::min<int64_t>((n_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA, int64_t(sms) * 2);
        static bool attr_slice[SA_MAX_DEVICE_FLAGS];
        if (!sa_set_smem_once(ttm4_slice_kernel, SL_SMEM, attr_slice)) return SA_E_CUDA;
        ttm4_slice_kernel<<<(unsigned)ctas, 256, SL_SMEM, stream>>>(wl.d_items, n_items, t->d_crd[1], T2, ops[0].ptr, uint32_t(ops[0].ld),
                                                                  out, part2, lim);
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    if (!wl.fix.empty()) {
        if (sa_launch_fixup(wl, part2, out, TILE4, stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}
