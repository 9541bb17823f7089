// Order-4 analogue of kernel 6:  A(i,l,m,n) = sum_{j,k,o} B(i,j,k,o) C(j,l) D(k,m) E(o,n),
// scheduled with the two-level branched nesting the paper uses for the second schedule of its
// 3-D TTMC kernel (Table of kernels, Section 6; recursive producer/consumer split of Section 4.2):
//   i, j' < T2(m,n) ;  k' < t(n) ; o': t(n) += B E(o,n) , m: T2(m,n) += t(n) D(k,m) > ,
//                      l: A(i,l,m,n) += T2(m,n) C(j,l) >
// One fused kernel; no temporary leaves the chip.  A thread block of eight warps owns a *piece*, a
// contiguous run of (i,j) subtrees of about 16 K nonzeros, and walks it in *super-items* of at most
// SA_F4_POOL subtrees:
//   produce.  The warps take the super-item's items from a shared counter.  An item is a run of
//     subtrees with at most SA_F4_ROWS level-2 fibers (a larger subtree is one item evaluated in
//     batches of that many fibers).  Per batch:
//       stage A (fp32 ALU):  t(f; n) = sum_o B(f; o) E(o,n) for every fiber f = (i,j,k).  Four lanes own a row
//         of E as one float4 each, so the warp's eight lane groups walk nonzero-balanced shares of the batch's
//         fibers, one nonzero per group and step (8-byte nonzero records eight per group and one load ahead,
//         eight row gathers in flight); the end-of-fiber bit travels in the sign bit of the index and parks
//         t(f; :) in the fiber's row of the warp's shared-memory region, next to the row D(k_f, :) that a
//         cp.async fetched meanwhile.
//       stage B (tensor cores):  T2(m,n) += sum_f D(k_f, m) t(f; n) over the fibers of a subtree, eight fibers
//         per m16n8k8 TF32 product (both operands split into a high and a low TF32 part: three products,
//         fp32-level accuracy).  When a subtree's last fiber is in, its 16 x 16 temporary goes to the block's
//         pool in shared memory.
//     Subtrees above SA_SUB_MAX_NNZ nonzeros are not evaluated here: the order-3 kernel (sa_ttm3.cu, the (i,j)
//     subtrees as slices, D and E as factors) has written their temporaries to the workspace, and an item of
//     kind 1 copies them into the pool.
//   consume (tensor cores).  After a block-wide barrier every warp updates its 32 of the 256 columns (m,n)
//     of the slice tile,  A(i, :, (m,n)) += C(j,:)^T (16 x 8) . T2 (8 x 32), eight subtrees per product, again
//     TF32 x 3, with the accumulators in registers across super-items.  When the block passes the end of a
//     slice (pos of level 1) the warps store their columns of the tile -- to the output, or, for a slice that
//     lies in several pieces, to a partial tile that the deterministic fix-up kernel sums.
// The only traffic besides B, the factor rows and A is the partial tiles (16 KB per piece boundary inside a
// slice) and the temporaries of the large subtrees.
#include <algorithm>

#include "sa_device.cuh"

namespace {

constexpr int R = 16;                  // L = M = N = 16
constexpr int TILE4 = R * R * R;       // floats per output slice
constexpr int T2F = R * R;             // floats per temporary
constexpr int F4_WARPS = SA_F4_WARPS;   // warps that produce; the first F4_CWARPS of them also consume
constexpr int F4_CWARPS = 8;           // 256 columns (m,n) / 32 per warp
constexpr int F4_RS = 32;              // floats per parked fiber row: t(f; 0..15) | D(k_f, 0..15), rotated by 8 (row & 3) floats
constexpr int F4_TS = T2F + 8;         // floats per pooled temporary: consecutive temporaries 8 banks apart
constexpr int F4_CS = 24;              // floats per staged row of C
constexpr int F4_PARK = SA_F4_ROWS * F4_RS;
constexpr int F4_SMEM = (F4_WARPS * F4_PARK + SA_F4_POOL * F4_TS + SA_F4_POOL * F4_CS) * int(sizeof(float)) + 16;

struct f4_limits {
    int32_t *status;
    uint32_t c_rows, d_rows, e_rows, n_slices;
    int32_t n_subtrees, n_fibers, n_large, n_slots, nnz;
};

// Position of element (m, n) inside a pooled temporary: bit 3 of n is flipped on every other pair of rows, so that
// neither the accumulator-fragment stores of stage B nor the operand-fragment loads of the consumer collide.
__device__ __forceinline__ int f4_pos(int m, int n) { return m * R + (n ^ (((m >> 1) & 1) << 3)); }

// Where float `pos` (0..15: t(f; pos), 16..31: D(k_f, pos - 16)) of parked row r lives: every row is rotated by a
// quarter more than the one before, so that the operand-fragment loads of stage B (four consecutive rows x eight
// consecutive floats) fall into 32 different banks without padding.
__device__ __forceinline__ int f4_rowpos(int r, int pos) { return r * F4_RS + ((pos + 8 * (r & 3)) & 31); }

// Stage A on a batch of nf <= SA_F4_ROWS fibers: row r of pk gets t(f_r; :).  s3 = pos3[first fiber + lane] (INT_MAX
// past the batch), pe = pos3[one past the last fiber].  A lane group keeps ONE running sum over its whole share and
// parks it at every end-of-fiber bit (no reset: a predicated store and a pointer bump per step); the rows are
// turned into per-fiber sums afterwards by subtracting the previous row inside each group's share.
__device__ __forceinline__ void f4_stage_a(float *pk, uint32_t pk_s, int nf, int s3, int pe, const int2 *__restrict__ nz,
                                           const float *__restrict__ E, uint32_t ld_e, int lane, const f4_limits &lim)
{
    const int g = lane >> 2, l = lane & 3;
    const int pb0 = __shfl_sync(SA_FULL_MASK, s3, 0);
    // shares of the eight groups: whole fibers, cut where the nonzero count passes the next eighth of the batch
    int fa = 0, fb = nf;
    uint32_t first = 1u;                                      // bit r: row r is the first of some group's share
#pragma unroll
    for (int q = 1; q < 8; ++q) {
        const int target = pb0 + int(int64_t(pe - pb0) * q / 8);
        const int cnt = __popc(__ballot_sync(SA_FULL_MASK, s3 < target));
        if (g == q) fa = cnt;
        if (g + 1 == q) fb = cnt;
        first |= 1u << (cnt & 31);
    }
    const int sa = __shfl_sync(SA_FULL_MASK, s3, fa & 31), sb = __shfl_sync(SA_FULL_MASK, s3, fb & 31);
    const int ga = fa < nf ? sa : pe, gb = fb < nf ? sb : pe;
    const int mylen = gb - ga;
    const int maxlen = __reduce_max_sync(SA_FULL_MASK, mylen);
    int slot = fa;                                            // row the group parks next
    auto fetch1 = [&](int q, int &x, float &v) {
        x = 0;
        v = 0.f;
        if (q < mylen && SA_CHK(lim.status, ga + q >= 0 && ga + q < lim.nnz, 21, ga + q)) {
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
        int xs[8];
        float vs[8];
        float4 e[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            xs[u] = __shfl_sync(SA_FULL_MASK, x[u >> 2], u & 3, 4);
            vs[u] = __shfl_sync(SA_FULL_MASK, v[u >> 2], u & 3, 4);
            uint32_t o = uint32_t(xs[u]) & 0x7fffffffu;
            if (!SA_CHK(lim.status, o < lim.e_rows, 22, o)) o = 0u;
            e[u] = sa_ldg4(E + (o * ld_e + 4u * l));
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (c + u < mylen) {
                acc.x = fmaf(vs[u], e[u].x, acc.x);
                acc.y = fmaf(vs[u], e[u].y, acc.y);
                acc.z = fmaf(vs[u], e[u].z, acc.z);
                acc.w = fmaf(vs[u], e[u].w, acc.w);
            }
            if (xs[u] < 0) {                                      // last nonzero of a fiber: park the running sum
                if (!SA_CHK(lim.status, slot < nf, 23, slot)) slot = 0;
                *reinterpret_cast<float4 *>(pk + f4_rowpos(slot, 4 * l)) = acc;
                ++slot;
            }
        }
    }
    __syncwarp();
    // running sums -> per-fiber sums: row r -= row r - 1 unless r opens a group's share (eight rows per pass, lane =
    // (row, float4 of the row); everything is read before anything is written)
    float4 cur[SA_F4_ROWS / 8], prev[SA_F4_ROWS / 8];
#pragma unroll
    for (int i = 0; i < SA_F4_ROWS / 8; ++i) {
        const int row = g + 8 * i;
        cur[i] = prev[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row < nf) {
            cur[i] = *reinterpret_cast<const float4 *>(pk + f4_rowpos(row, 4 * l));
            if (!((first >> row) & 1u)) prev[i] = *reinterpret_cast<const float4 *>(pk + f4_rowpos(row - 1, 4 * l));
        }
    }
    __syncwarp();
#pragma unroll
    for (int i = 0; i < SA_F4_ROWS / 8; ++i) {
        const int row = g + 8 * i;
        if (row < nf)
            *reinterpret_cast<float4 *>(pk + f4_rowpos(row, 4 * l)) =
                make_float4(cur[i].x - prev[i].x, cur[i].y - prev[i].y, cur[i].z - prev[i].z, cur[i].w - prev[i].w);
    }
}

// One item of kind 0: subtrees [it.out_row, it.row_end), fibers [it.f0, it.f1).  Temporaries go to pool slots
// slot0 + (subtree - it.out_row).
__device__ __forceinline__ void f4_small_item(const sa_item &it, float *pk, float *pool_slot0, const int32_t *__restrict__ pos2,
                                              const int32_t *__restrict__ pos3, const int32_t *__restrict__ crd_k,
                                              const int2 *__restrict__ nz, const float *__restrict__ D, uint32_t ld_d,
                                              const float *__restrict__ E, uint32_t ld_e, int lane, const f4_limits &lim)
{
    const int g = lane >> 2, t = lane & 3;
    const int nsub = it.row_end - it.out_row;
    const int my_end = lane < nsub ? __ldg(pos2 + it.out_row + lane + 1) : 0x7fffffff;   // fiber at which subtree `lane` ends
    float tacc[2][4];
#pragma unroll
    for (int nt = 0; nt < 2; ++nt)
#pragma unroll
        for (int x = 0; x < 4; ++x) tacc[nt][x] = 0.f;
    const int nft = it.f1 - it.f0;
    const int nbat = (nft + SA_F4_ROWS - 1) / SA_F4_ROWS, bsz = (nft + nbat - 1) / nbat;
    const uint32_t pk_s = smem_u32(pk);
    // per-batch arrays: start of every fiber, its row of D, end of the last fiber -- read one batch ahead
    struct meta { int s3, kk, pe; };
    auto load_meta = [&](int fb0) {
        meta m;
        const int nf = min(bsz, it.f1 - fb0);
        const bool mine = lane < nf && SA_CHK(lim.status, fb0 + lane >= 0 && fb0 + lane < lim.n_fibers, 24, fb0 + lane);
        m.s3 = mine ? __ldg(pos3 + fb0 + lane) : 0x7fffffff;
        m.kk = mine ? __ldg(crd_k + fb0 + lane) : 0;
        m.pe = __ldg(pos3 + fb0 + nf);
        return m;
    };
    meta cm = load_meta(it.f0);
    int cur = 0, cur_end = __shfl_sync(SA_FULL_MASK, my_end, 0);
    for (int fb0 = it.f0; fb0 < it.f1; fb0 += bsz) {
        const int nf = min(bsz, it.f1 - fb0);
        const meta m = cm;
        if (fb0 + bsz < it.f1) cm = load_meta(fb0 + bsz);
        int kk = m.kk;
        if (!SA_CHK(lim.status, uint32_t(kk) < lim.d_rows, 25, kk)) kk = 0;
        // rows of D the batch's fibers need in stage B: fetched while stage A runs
#pragma unroll
        for (int i = 0; i < SA_F4_ROWS / 8; ++i) {
            const int row = g + 8 * i;
            const int k = __shfl_sync(SA_FULL_MASK, kk, row);
            if (row < nf) cp_async16_raw(pk_s + uint32_t(f4_rowpos(row, R + 4 * t)) * 4u, D + (uint32_t(k) * ld_d + 4u * t));
        }
        cp_async_commit();
        f4_stage_a(pk, pk_s, nf, m.s3, m.pe, nz, E, ld_e, lane, lim);
        cp_async_wait<0>();
        __syncwarp();
        // ---- stage B: the batch's fibers, subtree by subtree, eight per product
        int f = fb0;
        const int fb1 = fb0 + nf;
        while (f < fb1) {
            const int e = max(f, min(cur_end, fb1));
            for (int g8 = f; g8 < e; g8 += 8) {
                const bool va = g8 + t < e, vb = g8 + t + 4 < e;
                const int qa = min(g8 - fb0 + t, SA_F4_ROWS - 1), qb = min(g8 - fb0 + t + 4, SA_F4_ROWS - 1);
                const float *ra = pk + qa * F4_RS, *rb = pk + qb * F4_RS;
                const int oa = 8 * (qa & 3), ob = 8 * (qb & 3);          // rotation of the two rows
                // A operand: D(k_f, m), m = g and g + 8, fibers t and t + 4;  B operand: t(f; n), n = 8 nt + g
                uint32_t ah[4], al[4];
                split_tf32(va ? ra[(R + g + oa) & 31] : 0.f, ah[0], al[0]);
                split_tf32(va ? ra[(R + g + 8 + oa) & 31] : 0.f, ah[1], al[1]);
                split_tf32(vb ? rb[(R + g + ob) & 31] : 0.f, ah[2], al[2]);
                split_tf32(vb ? rb[(R + g + 8 + ob) & 31] : 0.f, ah[3], al[3]);
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    uint32_t bh[2], bl[2];
                    split_tf32(va ? ra[(8 * nt + g + oa) & 31] : 0.f, bh[0], bl[0]);
                    split_tf32(vb ? rb[(8 * nt + g + ob) & 31] : 0.f, bh[1], bl[1]);
                    mma_m16n8k8_tf32(tacc[nt], al, bh);
                    mma_m16n8k8_tf32(tacc[nt], ah, bl);
                    mma_m16n8k8_tf32(tacc[nt], ah, bh);
                }
            }
            f = e;
            if (e >= cur_end) {
                // the subtree is complete: T2(m, 8 nt + 2 t (+1)) for m = g and g + 8 goes to the pool
                float *dst = pool_slot0 + cur * F4_TS;
#pragma unroll
                for (int nt = 0; nt < 2; ++nt) {
                    *reinterpret_cast<float2 *>(dst + f4_pos(g, 8 * nt + 2 * t)) = make_float2(tacc[nt][0], tacc[nt][1]);
                    *reinterpret_cast<float2 *>(dst + f4_pos(g + 8, 8 * nt + 2 * t)) = make_float2(tacc[nt][2], tacc[nt][3]);
#pragma unroll
                    for (int x = 0; x < 4; ++x) tacc[nt][x] = 0.f;
                }
                ++cur;
                cur_end = __shfl_sync(SA_FULL_MASK, my_end, cur & 31);
                if (cur >= nsub) cur_end = 0x7fffffff;
            }
        }
        __syncwarp();           // the next batch overwrites the parked rows
    }
}

// One item of kind 1: the temporaries of the large subtrees [it.out_row, it.row_end) were written by the order-3
// kernel to T2L[it.f0 ...]; copy them into the pool.
__device__ __forceinline__ void f4_large_item(const sa_item &it, float *pool_slot0, const float *__restrict__ T2L, int lane,
                                              const f4_limits &lim)
{
    for (int r = 0; r < it.row_end - it.out_row; ++r) {
        if (!SA_CHK(lim.status, it.f0 + r >= 0 && it.f0 + r < lim.n_large, 26, it.f0 + r)) continue;
        const float *src = T2L + int64_t(it.f0 + r) * T2F;
        float *dst = pool_slot0 + r * F4_TS;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            const int e = 4 * (lane + 32 * i);
            const float4 v = __ldcs(reinterpret_cast<const float4 *>(src + e));
            *reinterpret_cast<float4 *>(dst + f4_pos(e >> 4, e & 15)) = v;
        }
    }
}

// acc += C(j,:)^T (16 x n) . T2 (n x 32) for the n <= 8 pooled temporaries at tp (rows of C at cp), columns
// 32 warp .. 32 warp + 31 of (m,n).
__device__ __forceinline__ void f4_consume(float (&acc)[4][4], const float *tp, const float *cp, int n, int warp, int lane)
{
    const int g = lane >> 2, t = lane & 3;
    const bool va = t < n, vb = t + 4 < n;
    const float *ca = cp + (va ? t : 0) * F4_CS, *cb = cp + (vb ? t + 4 : 0) * F4_CS;
    const float *ta = tp + (va ? t : 0) * F4_TS, *tb = tp + (vb ? t + 4 : 0) * F4_TS;
    uint32_t ah[4], al[4];
    split_tf32(va ? ca[g] : 0.f, ah[0], al[0]);
    split_tf32(va ? ca[g + 8] : 0.f, ah[1], al[1]);
    split_tf32(vb ? cb[g] : 0.f, ah[2], al[2]);
    split_tf32(vb ? cb[g + 8] : 0.f, ah[3], al[3]);
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        const int col = (32 * warp + 8 * nt + g) ^ ((warp & 1) << 3);       // f4_pos of column (m,n) = 32 warp + 8 nt + g
        uint32_t bh[2], bl[2];
        split_tf32(va ? ta[col] : 0.f, bh[0], bl[0]);
        split_tf32(vb ? tb[col] : 0.f, bh[1], bl[1]);
        mma_m16n8k8_tf32(acc[nt], al, bh);
        mma_m16n8k8_tf32(acc[nt], ah, bl);
        mma_m16n8k8_tf32(acc[nt], ah, bh);
    }
}

// A warp's columns of a slice tile: element (l, 32 warp + 8 nt + 2 t (+1)), l = g and g + 8.
__device__ __forceinline__ void f4_store(const float (&acc)[4][4], float *dst, bool streaming, int warp, int lane)
{
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int nt = 0; nt < 4; ++nt) {
        float *p = dst + g * T2F + 32 * warp + 8 * nt + 2 * t;
        const float2 lo = make_float2(acc[nt][0], acc[nt][1]), hi = make_float2(acc[nt][2], acc[nt][3]);
        if (streaming) {
            sa_st_cs2(p, lo);
            sa_st_cs2(p + 8 * T2F, hi);
        } else {
            *reinterpret_cast<float2 *>(p) = lo;
            *reinterpret_cast<float2 *>(p + 8 * T2F) = hi;
        }
    }
}

// CONTIG: D and E are stored without padding (leading dimension 16), so a row offset is a shift.
template <bool CONTIG>
__global__ void __launch_bounds__(32 * F4_WARPS, SA_F4_CTAS)
ttm4_fused_kernel(const int4 *__restrict__ pieces, const int4 *__restrict__ supers, const sa_item *__restrict__ items,
                  const int32_t *__restrict__ pos1, const int32_t *__restrict__ crd0, const int32_t *__restrict__ crd_j,
                  const int32_t *__restrict__ pos2, const int32_t *__restrict__ pos3, const int32_t *__restrict__ crd_k,
                  const int2 *__restrict__ nz, const float *__restrict__ C, uint32_t ldc, const float *__restrict__ D, uint32_t ldd,
                  const float *__restrict__ E, uint32_t lde, const float *__restrict__ T2L, float *__restrict__ out,
                  float *__restrict__ partial, const f4_limits lim)
{
    extern __shared__ __align__(16) unsigned char f4_smem[];
    float *park = reinterpret_cast<float *>(f4_smem);
    float *pool = park + F4_WARPS * F4_PARK;
    float *cs = pool + SA_F4_POOL * F4_TS;
    int *ctr = reinterpret_cast<int *>(cs + SA_F4_POOL * F4_CS);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float *pk = park + warp * F4_PARK;
    const uint32_t ld_d = CONTIG ? uint32_t(R) : ldd, ld_e = CONTIG ? uint32_t(R) : lde;

    const int4 pa = __ldg(pieces + 2 * blockIdx.x);        // first super-item, one past the last, first slice, last slice
    const int4 pb = __ldg(pieces + 2 * blockIdx.x + 1);    // partial slot of the first slice, of the last slice, first subtree, one past the last
    int s = pa.z;
    int bound = __ldg(pos1 + s + 1);                       // subtree at which slice s ends
    float acc[4][4];
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
        for (int x = 0; x < 4; ++x) acc[nt][x] = 0.f;
    if (threadIdx.x == 0) ctr[pa.x & 1] = __ldg(supers + pa.x).x;
    __syncthreads();
    for (int sup = pa.x; sup < pa.y; ++sup) {
        const int4 S = __ldg(supers + sup);                // first item, one past the last, first subtree, one past the last
        {   // rows of C the consumer needs, one float4 per thread
            const int slot = threadIdx.x >> 2, part = threadIdx.x & 3;
            if (slot < S.w - S.z) {
                uint32_t j = uint32_t(__ldg(crd_j + S.z + slot));
                if (!SA_CHK(lim.status, j < lim.c_rows, 27, j)) j = 0u;
                *reinterpret_cast<float4 *>(cs + slot * F4_CS + 4 * part) = sa_ldg4(C + (j * ldc + 4u * part));
            }
        }
        // ---- produce
        for (;;) {
            int k = 0;
            if (lane == 0) k = atomicAdd(ctr + (sup & 1), 1);
            k = __shfl_sync(SA_FULL_MASK, k, 0);
            if (k >= S.y) break;
            sa_item it;
            {
                const int4 ia = __ldg(reinterpret_cast<const int4 *>(items + k));          // first subtree, one past the last, f0, f1
                const int4 ib = __ldg(reinterpret_cast<const int4 *>(items + k) + 1);      // p0, p1, -, kind
                it.out_row = ia.x; it.row_end = ia.y; it.f0 = ia.z; it.f1 = ia.w;
                it.p0 = ib.x; it.p1 = ib.y; it.dest = ib.z; it.pad = ib.w;
            }
            if (!SA_CHK(lim.status, it.out_row >= S.z && it.row_end <= S.w && it.row_end - it.out_row <= 32, 28, k)) continue;
            float *slot0 = pool + (it.out_row - S.z) * F4_TS;
            if (it.pad == 0) f4_small_item(it, pk, slot0, pos2, pos3, crd_k, nz, D, ld_d, E, ld_e, lane, lim);
            else f4_large_item(it, slot0, T2L, lane, lim);
        }
        __syncthreads();
        if (threadIdx.x == 0 && sup + 1 < pa.y) ctr[(sup + 1) & 1] = __ldg(supers + sup + 1).x;
        // ---- consume
        int r = S.z;
        while (r < S.w) {
            const int n = min(8, min(S.w, bound) - r);
            if (n < 1) {                                      // cannot happen with consistent lists; never spin
                SA_CHK(lim.status, false, 29, r);
                break;
            }
            if (warp < F4_CWARPS) f4_consume(acc, pool + (r - S.z) * F4_TS, cs + (r - S.z) * F4_CS, n, warp, lane);
            r += n;
            if (r == bound) {
                // slice s is complete (as far as this piece holds it)
                const bool part = s == pa.z && pb.x >= 0;
                const uint32_t row = uint32_t(__ldg(crd0 + s));
                if (warp < F4_CWARPS && (part ? SA_CHK(lim.status, pb.x < lim.n_slots, 30, pb.x) : SA_CHK(lim.status, row < lim.n_slices, 31, row)))
                    f4_store(acc, part ? partial + int64_t(pb.x) * TILE4 : out + int64_t(row) * TILE4, !part, warp, lane);
#pragma unroll
                for (int nt = 0; nt < 4; ++nt)
#pragma unroll
                    for (int x = 0; x < 4; ++x) acc[nt][x] = 0.f;
                ++s;
                bound = s <= pa.w ? __ldg(pos1 + s + 1) : 0x7fffffff;
            }
        }
        __syncthreads();
    }
    // the piece ends inside slice s: what it holds of that slice is a partial tile
    if (warp < F4_CWARPS && s <= pa.w && SA_CHK(lim.status, pb.y >= 0 && pb.y < lim.n_slots, 32, pb.y))
        f4_store(acc, partial + int64_t(pb.y) * TILE4, false, warp, lane);
}

struct ttm4_plan {
    size_t t2l_bytes, p1_bytes, p2_bytes;
};

ttm4_plan plan(const sa_tensor *t)
{
    ttm4_plan p;
    p.t2l_bytes = sa_align256(size_t(t->f4_n_large) * T2F * sizeof(float));
    p.p1_bytes = sa_align256(size_t(t->wl_main.n_slots) * T2F * sizeof(float));
    p.p2_bytes = sa_align256(size_t(t->wl_aux.n_slots) * TILE4 * sizeof(float));
    return p;
}

}  // namespace

bool sa_ranks_ok_ttm4(int64_t L, int64_t M, int64_t N) { return L == R && M == R && N == R; }

// workspace: [temporaries of the large subtrees][their partial temporaries (order-3 kernel)][partial slice tiles]
size_t sa_ws_ttm4(const sa_tensor *t, const sa_dense *)
{
    const ttm4_plan p = plan(t);
    return p.t2l_bytes + p.p1_bytes + p.p2_bytes;
}

sa_status sa_launch_ttm4(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t, cudaStream_t stream,
                         int *launches)
{
    const ttm4_plan p = plan(t);
    *launches = 0;
    // every range check comes before the first launch: 32-bit element offsets of factor rows
    for (int i = 0; i < 3; ++i)
        if (ops[i].rows * ops[i].ld >= (int64_t(1) << 30)) return SA_E_UNSUPPORTED;
    if (t->count[1] > 0 && (!t->d_f4_pieces || !t->d_f4_supers || !t->d_nzpack)) return SA_E_UNSUPPORTED;
    char *base = static_cast<char *>(ws);
    float *T2L = reinterpret_cast<float *>(base);
    float *part1 = reinterpret_cast<float *>(base + p.t2l_bytes);
    float *part2 = reinterpret_cast<float *>(base + p.t2l_bytes + p.p1_bytes);
    if (!t->wl_main.items.empty()) {
        // the large subtrees: kernel 6 with the (i,j) subtrees as slices, factors D (rows by k) and E (rows by o)
        sa_ttm3_view v;
        v.wl = &t->wl_main;
        v.crd_fiber = t->d_crd[2];
        v.crd_nz = t->d_crd[3];
        v.vals = t->d_vals;
        v.endbits = t->d_endbits;
        v.n_fibers = t->count[2];
        v.n_out_rows = t->f4_n_large;
        v.nnz = t->wl_main.nnz;
        v.nnz_total = t->nnz;
        v.status = t->d_status;
        int n1 = 0;
        const sa_status s = sa_launch_ttm3_view(v, ops[1], ops[2], T2L, part1, stream, &n1);
        if (s != SA_OK) return s;
        *launches += n1;
    }
    const int64_t n_pieces = int64_t(t->f4_pieces.size() / 8);
    if (n_pieces > 0) {
        const bool contig = ops[1].ld == R && ops[2].ld == R;
        auto kern = contig ? ttm4_fused_kernel<true> : ttm4_fused_kernel<false>;
        static bool attr_contig[SA_MAX_DEVICE_FLAGS], attr_strided[SA_MAX_DEVICE_FLAGS];
        if (!sa_set_smem_once(kern, F4_SMEM, contig ? attr_contig : attr_strided)) return SA_E_CUDA;
        f4_limits lim;
        lim.status = t->d_status;
        lim.c_rows = uint32_t(ops[0].rows); lim.d_rows = uint32_t(ops[1].rows); lim.e_rows = uint32_t(ops[2].rows);
        lim.n_slices = uint32_t(t->dims[0]);
        lim.n_subtrees = int32_t(t->count[1]); lim.n_fibers = int32_t(t->count[2]); lim.n_large = t->f4_n_large;
        lim.n_slots = int32_t(t->wl_aux.n_slots); lim.nnz = int32_t(t->nnz);
        kern<<<(unsigned)n_pieces, 32 * F4_WARPS, F4_SMEM, stream>>>(
            reinterpret_cast<const int4 *>(t->d_f4_pieces), reinterpret_cast<const int4 *>(t->d_f4_supers), t->wl_sub.d_items,
            t->d_pos[1], t->d_crd[0], t->d_crd[1], t->d_pos[2], t->d_pos[3], t->d_crd[2], t->d_nzpack, ops[0].ptr,
            uint32_t(ops[0].ld), ops[1].ptr, uint32_t(ops[1].ld), ops[2].ptr, uint32_t(ops[2].ld), T2L, out, part2, lim);
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    if (!t->wl_aux.fix.empty()) {
        if (sa_launch_fixup(t->wl_aux, part2, out, TILE4, stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}
