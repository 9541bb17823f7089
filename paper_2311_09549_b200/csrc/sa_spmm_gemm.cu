// Kernel 4 <SpMM,GEMM>:  A(i,m) = sum_{j,l} B(i,j) C(j,l) D(l,m)  in both association orders.
//
// ASSOC_LEFT  (B.C).D : the row-fused nest of the paper's Table of kernels (Section 6) with the
//   producer/consumer roles per row: T(l) = sum_j' B(i,j) C(j,l) is a row temporary of L floats
//   (registers -> shared memory), immediately consumed by A(i,:) = T . D with D resident in shared
//   memory.  (The paper's own pick keeps a scalar and loops k outermost per row; the 1-D temporary
//   is the SparseLNR variant it discusses in "Effect of transpositions".)
// ASSOC_RIGHT B.(C.D) : E = C.D first (J x M temporary in the workspace, memory depth 2, which
//   the paper's Stage-1 pruning still admits), then the SpMM loop nest of Fig. 1b, A = B.E.
#include "sa_device.cuh"

constexpr int LEFT_UNROLL = 4;     // gathered rows in flight per warp in the (B.C).D row kernel (8 was slower)

namespace {


// Row (L floats in shared memory) times D (L x M in shared memory); lane owns m = lane + 32*q.
template <int L, int M>
__device__ __forceinline__ void row_times_D(const float *__restrict__ Ts, const float *__restrict__ Ds, int lane,
                                            float (&o)[M / 32])
{
    constexpr int MV = M / 32;
#pragma unroll
    for (int q = 0; q < MV; ++q) o[q] = 0.f;
#pragma unroll 4
    for (int l = 0; l < L; l += 4) {
        const float4 t = *reinterpret_cast<const float4 *>(Ts + l);
#pragma unroll
        for (int q = 0; q < MV; ++q) {
            const float *d = Ds + l * M + q * 32 + lane;
            o[q] = fmaf(t.x, d[0], o[q]);
            o[q] = fmaf(t.y, d[M], o[q]);
            o[q] = fmaf(t.z, d[2 * M], o[q]);
            o[q] = fmaf(t.w, d[3 * M], o[q]);
        }
    }
}

template <int L, int M>
__device__ __forceinline__ void load_D(float *Ds, const float *__restrict__ D, int64_t ldd)
{
    for (int x = threadIdx.x * 4; x < L * M; x += blockDim.x * 4) {
        const int l = x / M, m = x % M;
        *reinterpret_cast<float4 *>(Ds + x) = sa_ldg4(D + int64_t(l) * ldd + m);
    }
}

template <int L, int M, bool HAD>
__global__ void __launch_bounds__(256, 3)
spmm_gemm_left_kernel(const sa_item *__restrict__ items, int64_t n_items, const int32_t *__restrict__ pos,
                      const int32_t *__restrict__ crd, const float *__restrict__ vals, const float *__restrict__ C,
                      int64_t ldc, const float *__restrict__ H, int64_t ldh, const float *__restrict__ D, int64_t ldd,
                      float *__restrict__ out, float *__restrict__ partial, const sa_limits lim)
{
    constexpr int LV4 = L / 128, MV = M / 32;
    extern __shared__ __align__(16) float smem[];
    float *Ds = smem;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float *Ts = smem + L * M + warp * L;
    load_D<L, M>(Ds, D, ldd);
    __syncthreads();
    for (int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp; idx < n_items;
         idx += int64_t(gridDim.x) * SA_WARPS_PER_CTA) {
        const sa_item it = items[idx];
        for (int r = it.out_row; r < it.row_end; ++r) {
            if (!SA_CHK(lim.status, uint32_t(r) < lim.out_rows && it.dest < lim.n_slots, 51, r)) continue;
            const int a = it.dest >= 0 ? it.p0 : pos[r];
            const int b = it.dest >= 0 ? it.p1 : pos[r + 1];
            if (!SA_CHK(lim.status, a >= 0 && a <= b && b <= lim.nnz, 52, b)) continue;
            float4 t[LV4];
#pragma unroll
            for (int q = 0; q < LV4; ++q) t[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int base = a; base < b; base += 32) {
                const int n = min(32, b - base);
                int jj = 0;
                float vv = 0.f;
                if (lane < n) { jj = crd[base + lane]; vv = vals[base + lane]; }
                if (!SA_CHK(lim.status, uint32_t(jj) < lim.gather_rows, 53, jj)) jj = 0;
#pragma unroll LEFT_UNROLL
                for (int s = 0; s < n; ++s) {
                    const int j = __shfl_sync(SA_FULL_MASK, jj, s);
                    const float v = __shfl_sync(SA_FULL_MASK, vv, s);
                    const float *crow = C + int64_t(j) * ldc + lane * 4;
                    const float *hrow = H + int64_t(j) * ldh + lane * 4;     // HAD: the row of the Hadamard partner
#pragma unroll
                    for (int q = 0; q < LV4; ++q) {
                        float4 c = sa_ldg4(crow + q * 128);
                        if (HAD) {
                            const float4 h = sa_ldg4(hrow + q * 128);
                            c.x *= h.x; c.y *= h.y; c.z *= h.z; c.w *= h.w;
                        }
                        t[q].x = fmaf(v, c.x, t[q].x); t[q].y = fmaf(v, c.y, t[q].y);
                        t[q].z = fmaf(v, c.z, t[q].z); t[q].w = fmaf(v, c.w, t[q].w);
                    }
                }
            }
            float *dst = it.dest >= 0 ? partial + int64_t(it.dest) * M : out + int64_t(r) * M;
            if (b > a) {
#pragma unroll
                for (int q = 0; q < LV4; ++q) *reinterpret_cast<float4 *>(Ts + q * 128 + lane * 4) = t[q];
                __syncwarp();
                float o[MV];
                row_times_D<L, M>(Ts, Ds, lane, o);
                __syncwarp();
#pragma unroll
                for (int q = 0; q < MV; ++q) sa_st_cs(dst + q * 32 + lane, o[q]);
            } else {
#pragma unroll
                for (int q = 0; q < MV; ++q) sa_st_cs(dst + q * 32 + lane, 0.f);
            }
        }
    }
}

// ---- E = C . D on tensor cores (dense stage of ASSOC_RIGHT) -----------------------------------
// Thread block: 128 rows of C x all M columns, 8 warps as 4 (rows) x 2 (columns), warp tile
// 32 x M/2.  D stays in shared memory for the whole (persistent) block, already split into its
// high and low BF16 parts; C streams through a 3-stage cp.async ring in chunks of 32 columns.
__device__ __forceinline__ void g_cp_async16(float *dst_smem, const float *src)
{
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
}

// BF16x3 products: x = b1 + b2 with b1 = bf16(x), b2 = bf16(x - b1) represents x to 2^-18 relative;
// b1.b1 + b1.b2 + b2.b1 then misses the fp32 product by about 1e-5 relative (inside the 1e-4 tolerance), and one
// m16n8k16 BF16 MMA does the work of two m16n8k8 TF32 MMAs: three of them cost half the tensor-pipe time of a
// three-product TF32 scheme, which was what bound this kernel (tensor pipe 56 % busy, DRAM 23 %).  D is kept as
// packed pairs (D(2p,m), D(2p+1,m)).
__device__ __forceinline__ uint32_t bf16x2_rn(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
// (b1, b2) of the pair (x0, x1): h = packed b1 parts, l = packed b2 parts
__device__ __forceinline__ void bf16_split2(float x0, float x1, uint32_t &h, uint32_t &l)
{
    h = bf16x2_rn(x0, x1);
    l = bf16x2_rn(x0 - __uint_as_float(h << 16), x1 - __uint_as_float(h & 0xffff0000u));
}
__device__ __forceinline__ void g_mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int L, int M>
struct gemm_bf16_cfg {
    static constexpr int BM = 128, KC = 32, NS = 3;
    static constexpr int CS = KC + 8;                 // row stride of a C chunk (conflict-free 64-bit A reads)
    static constexpr int DS = M + 8;                  // row stride of the packed D pairs (conflict-free B reads)
    static constexpr int NT = M / 16;                 // n8 tiles per warp (warp covers M/2 columns)
    static constexpr int D_WORDS = (L / 2) * DS * 2;  // high and low parts
    static constexpr int STAGE = BM * CS;
    static constexpr size_t SMEM = size_t(D_WORDS + NS * STAGE) * sizeof(float);
};

template <int L, int M>
__global__ void __launch_bounds__(256, 1)
gemm_bf16x3_kernel(int64_t J, const float *__restrict__ C, int64_t ldc, const float *__restrict__ D, int64_t ldd,
                   float *__restrict__ Eout)
{
    using G = gemm_bf16_cfg<L, M>;
    extern __shared__ __align__(16) float smem[];
    uint32_t *Dh = reinterpret_cast<uint32_t *>(smem);
    uint32_t *Dl = Dh + (L / 2) * G::DS;
    float *Cs = smem + G::D_WORDS;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int wr = warp >> 1, wc = warp & 1;           // warp tile: rows 32*wr.., columns (M/2)*wc..
    for (int x = threadIdx.x; x < (L / 2) * M; x += 256) {
        const int p = x / M, m = x % M;
        uint32_t h, l;
        bf16_split2(__ldg(D + int64_t(2 * p) * ldd + m), __ldg(D + int64_t(2 * p + 1) * ldd + m), h, l);
        Dh[p * G::DS + m] = h;
        Dl[p * G::DS + m] = l;
    }
    const int64_t n_tiles = (J + G::BM - 1) / G::BM;
    const int64_t my_tiles = blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    constexpr int KCH = L / G::KC;                     // chunks per row tile
    const int64_t n_chunks = my_tiles * KCH;
    auto issue = [&](int64_t q) {
        if (q < n_chunks) {
            const int64_t row0 = (int64_t(blockIdx.x) + (q / KCH) * gridDim.x) * G::BM;
            const int k0 = int(q % KCH) * G::KC;
            float *dst = Cs + int(q % G::NS) * G::STAGE;
#pragma unroll
            for (int x = threadIdx.x; x < G::BM * (G::KC / 4); x += 256) {
                const int r = x / (G::KC / 4), c4 = x % (G::KC / 4);
                const int64_t row = min(row0 + r, J - 1);            // rows past the end re-read the last row
                g_cp_async16(dst + r * G::CS + c4 * 4, C + row * ldc + k0 + c4 * 4);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    issue(0);
    issue(1);
    __syncthreads();                                   // D is in place
    float acc[2][G::NT][4];
    for (int64_t q = 0; q < n_chunks; ++q) {
        const int kc = int(q % KCH);
        if (kc == 0) {
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nt = 0; nt < G::NT; ++nt)
#pragma unroll
                    for (int z = 0; z < 4; ++z) acc[mt][nt][z] = 0.f;
        }
        asm volatile("cp.async.wait_group 1;" ::: "memory");
        __syncthreads();                               // chunk q landed for everyone; chunk q-1 fully consumed
        issue(q + 2);
        const float *cs = Cs + int(q % G::NS) * G::STAGE + (32 * wr) * G::CS;
        const uint32_t *dh = Dh + (kc * (G::KC / 2)) * G::DS + (M / 2) * wc;
        const uint32_t *dl = Dl + (kc * (G::KC / 2)) * G::DS + (M / 2) * wc;
#pragma unroll
        for (int kt = 0; kt < G::KC / 16; ++kt) {
            uint32_t ah[2][4], al[2][4];
#pragma unroll
            for (int mt = 0; mt < 2; ++mt) {
                const float *p = cs + (16 * mt + g) * G::CS + 16 * kt + 2 * t;
                const float2 x0 = *reinterpret_cast<const float2 *>(p);                   // (row g,     k 2t, 2t+1)
                const float2 x1 = *reinterpret_cast<const float2 *>(p + 8 * G::CS);       // (row g + 8, k 2t, 2t+1)
                const float2 x2 = *reinterpret_cast<const float2 *>(p + 8);               // (row g,     k 2t+8, 2t+9)
                const float2 x3 = *reinterpret_cast<const float2 *>(p + 8 * G::CS + 8);   // (row g + 8, k 2t+8, 2t+9)
                bf16_split2(x0.x, x0.y, ah[mt][0], al[mt][0]);
                bf16_split2(x1.x, x1.y, ah[mt][1], al[mt][1]);
                bf16_split2(x2.x, x2.y, ah[mt][2], al[mt][2]);
                bf16_split2(x3.x, x3.y, ah[mt][3], al[mt][3]);
            }
#pragma unroll
            for (int nt = 0; nt < G::NT; ++nt) {
                const int off = (8 * kt + t) * G::DS + 8 * nt + g;          // pair row (16 kt + 2 t) / 2
                const uint32_t bh0 = dh[off], bh1 = dh[off + 4 * G::DS];
                const uint32_t bl0 = dl[off], bl1 = dl[off + 4 * G::DS];
#pragma unroll
                for (int mt = 0; mt < 2; ++mt) {
                    g_mma_bf16(acc[mt][nt], al[mt], bh0, bh1);
                    g_mma_bf16(acc[mt][nt], ah[mt], bl0, bl1);
                    g_mma_bf16(acc[mt][nt], ah[mt], bh0, bh1);
                }
            }
        }
        if (kc == KCH - 1) {
            const int64_t row0 = (int64_t(blockIdx.x) + (q / KCH) * gridDim.x) * G::BM + 32 * wr;
#pragma unroll
            for (int mt = 0; mt < 2; ++mt)
#pragma unroll
                for (int nt = 0; nt < G::NT; ++nt) {
                    const int64_t r = row0 + 16 * mt + g;
                    const int col = (M / 2) * wc + 8 * nt + 2 * t;
                    if (r < J) *reinterpret_cast<float2 *>(Eout + r * M + col) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
                    if (r + 8 < J) *reinterpret_cast<float2 *>(Eout + (r + 8) * M + col) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
                }
        }
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// A = B . E (the CSR SpMM nest of Fig. 1b); lane owns MV = M/32 consecutive columns.
template <int MV>
__global__ void __launch_bounds__(256)
spmm_kernel(const sa_item *__restrict__ items, int64_t n_items, const int32_t *__restrict__ pos,
            const int32_t *__restrict__ crd, const float *__restrict__ vals, const float *__restrict__ E,
            float *__restrict__ out, float *__restrict__ partial, const sa_limits lim)
{
    constexpr int M = MV * 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    if (idx >= n_items) return;
    const sa_item it = items[idx];
    for (int r = it.out_row; r < it.row_end; ++r) {
        if (!SA_CHK(lim.status, uint32_t(r) < lim.out_rows && it.dest < lim.n_slots, 54, r)) continue;
        const int a = it.dest >= 0 ? it.p0 : pos[r];
        const int b = it.dest >= 0 ? it.p1 : pos[r + 1];
        if (!SA_CHK(lim.status, a >= 0 && a <= b && b <= lim.nnz, 55, b)) continue;
        float acc[MV];
#pragma unroll
        for (int q = 0; q < MV; ++q) acc[q] = 0.f;
        for (int base = a; base < b; base += 32) {
            const int n = min(32, b - base);
            int jj = 0;
            float vv = 0.f;
            if (lane < n) { jj = crd[base + lane]; vv = vals[base + lane]; }
            if (!SA_CHK(lim.status, uint32_t(jj) < lim.gather_rows, 56, jj)) jj = 0;
#pragma unroll 8
            for (int s = 0; s < n; ++s) {
                const int j = __shfl_sync(SA_FULL_MASK, jj, s);
                const float v = __shfl_sync(SA_FULL_MASK, vv, s);
                const float *erow = E + int64_t(j) * M + lane * MV;
                if (MV == 2) {
                    const float2 e = sa_ldg2(erow);
                    acc[0] = fmaf(v, e.x, acc[0]);
                    acc[1 % MV] = fmaf(v, e.y, acc[1 % MV]);
                } else {
                    acc[0] = fmaf(v, __ldg(erow), acc[0]);
                }
            }
        }
        float *dst = it.dest >= 0 ? partial + int64_t(it.dest) * M : out + int64_t(r) * M;
#pragma unroll
        for (int q = 0; q < MV; ++q) dst[lane * MV + q] = acc[q];
    }
}

// The same product over the (i,j) fibers of an order-3 CSF tensor (kernel 7; eight to twelve nonzeros per
// fiber): M/4 lanes own a row of E as one float4 each, so a warp works on 128/M fibers' streams at once, one
// nonzero per group and step.  A group takes a contiguous share of the item's fibers and walks their nonzeros
// as one stream, eight index/value pairs per load (the next eight already requested), eight row gathers in
// flight; index, end-of-fiber bit (sign bit) and value of a nonzero come as one 8-byte record (half the load
// wavefronts of separate index, value and bit arrays, and the L1 pipe is what this kernel saturates first); the
// bit closes the output row.
// A piece of a long fiber (dest >= 0) is split over the groups by nonzeros and summed across them at the end; a range
// of whole fibers is split by nonzeros as well, and the parts of a fiber cut between two groups are added in order.
template <int M>
__global__ void __launch_bounds__(256)
fiber_spmm_kernel(const sa_item *__restrict__ items, int64_t n_items, const int32_t *__restrict__ pos,
                  const int2 *__restrict__ nz, const float *__restrict__ E, int64_t lde, float *__restrict__ out,
                  float *__restrict__ partial, const sa_limits lim)
{
    constexpr int LPR = M / 4, NG = 32 / LPR;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    if (idx >= n_items) return;
    const sa_item it = items[idx];
    const int g = lane / LPR, l = lane % LPR;
    const bool piece = it.dest >= 0;
    int ga, gb, row = 0;
    if (piece) {
        const int64_t len = it.p1 - it.p0;
        ga = it.p0 + int(len * g / NG);
        gb = it.p0 + int(len * (g + 1) / NG);
    } else {
        // equal counts of nonzeros per group, whatever the row boundaries: quarters of the item (the work list names
        // the row each quarter starts in), two of them per group when there are two groups.  With equal counts of
        // rows the longest group had 1.2 times the mean length, and a range of one long row was all one group's.
        static_assert(NG == 4 || NG == 2, "quarter rows of the work list");
        const int quarter = (it.p1 - it.p0 + 3) >> 2, share = quarter * (4 / NG), first = g * (4 / NG);
        ga = min(it.p0 + g * share, it.p1);
        gb = min(ga + share, it.p1);
        row = first == 0 ? it.out_row : first == 1 ? it.f0 : first == 2 ? it.f1 : it.pad;
    }
    const int mylen = gb - ga;
    const int maxlen = __reduce_max_sync(SA_FULL_MASK, mylen);
    bool open = false;                      // the group's last nonzero did not end its row
    auto fetch = [&](int c, int &x, float &v) {                      // lanes 0..7 of the group: nonzero ga + c + lane
        const int p = ga + c + (l & 7);
        x = 0;
        v = 0.f;
        if (c + (l & 7) < mylen && SA_CHK(lim.status, p >= 0 && p < lim.nnz, 61, p)) {
            const int2 w = __ldg(nz + p);                            // (index | end-of-fiber bit << 31, value bits)
            x = piece ? (w.x & 0x7fffffff) : w.x;
            v = __int_as_float(w.y);
        }
    };
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    int xn;
    float vn;
    fetch(0, xn, vn);
    for (int c = 0; c < maxlen; c += 8) {
        const int x = xn;
        const float v = vn;
        fetch(c + 8, xn, vn);
        int xs[8];
        float vs[8];
        float4 e[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {                                 // positions past the group's end: row 0, value 0
            xs[u] = __shfl_sync(SA_FULL_MASK, x, u, LPR);
            vs[u] = __shfl_sync(SA_FULL_MASK, v, u, LPR);
            uint32_t k = uint32_t(xs[u]) & 0x7fffffffu;
            if (!SA_CHK(lim.status, k < lim.gather_rows, 62, k)) k = 0u;
            e[u] = sa_ldg4(E + int64_t(k) * lde + 4 * l);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (c + u < mylen) {
                acc.x = fmaf(vs[u], e[u].x, acc.x);
                acc.y = fmaf(vs[u], e[u].y, acc.y);
                acc.z = fmaf(vs[u], e[u].z, acc.z);
                acc.w = fmaf(vs[u], e[u].w, acc.w);
            }
            if (c + u < mylen) open = xs[u] >= 0;
            if (xs[u] < 0) {                                          // last nonzero of its fiber
                if (SA_CHK(lim.status, uint32_t(row) < lim.out_rows, 63, row)) *reinterpret_cast<float4 *>(out + int64_t(row) * M + 4 * l) = acc;
                acc = make_float4(0.f, 0.f, 0.f, 0.f);
                ++row;
            }
        }
    }
    if (!piece) {
        // A row cut by a share boundary was stored by the group that met its end; the groups before it add their
        // parts now, one group after the other (a long row may have several), so that the sum has a fixed order.
#pragma unroll
        for (int s = 0; s < NG - 1; ++s) {
            __syncwarp();
            if (g == s && open && SA_CHK(lim.status, uint32_t(row) < lim.out_rows, 63, row)) {
                float4 *dst = reinterpret_cast<float4 *>(out + int64_t(row) * M + 4 * l);
                float4 o = __ldcg(dst);
                o.x += acc.x; o.y += acc.y; o.z += acc.z; o.w += acc.w;
                *dst = o;
            }
        }
    }
    if (piece) {
#pragma unroll
        for (int off = LPR; off < 32; off <<= 1) {
            acc.x += __shfl_xor_sync(SA_FULL_MASK, acc.x, off);
            acc.y += __shfl_xor_sync(SA_FULL_MASK, acc.y, off);
            acc.z += __shfl_xor_sync(SA_FULL_MASK, acc.z, off);
            acc.w += __shfl_xor_sync(SA_FULL_MASK, acc.w, off);
        }
        if (g == 0 && SA_CHK(lim.status, it.dest < lim.n_slots, 64, it.dest)) *reinterpret_cast<float4 *>(partial + int64_t(it.dest) * M + 4 * l) = acc;
    }
}

int resident_ctas(const void *kernel, size_t smem)
{
    int dev = 0, sms = 148, per_sm = 1;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, 256, smem) != cudaSuccess || per_sm < 1) per_sm = 1;
    return sms * per_sm;
}

template <int L, int M>
sa_status run(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, bool right, cudaStream_t stream, int *launches)
{
    const sa_worklist &wl = t->wl_aux;
    const int64_t n_items = int64_t(wl.items.size());
    const size_t smem = size_t(L * M + SA_WARPS_PER_CTA * L) * sizeof(float);
    *launches = 0;
    if (!right) {
        float *partial = static_cast<float *>(ws);
        auto kern = spmm_gemm_left_kernel<L, M, false>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) return SA_E_CUDA;
        const int64_t want = (n_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
        const int64_t ctas = std::min<int64_t>(want, resident_ctas(reinterpret_cast<const void *>(kern), smem));
        if (ctas > 0) {
            kern<<<(unsigned)ctas, 256, smem, stream>>>(wl.d_items, n_items, t->d_pos[1], t->d_crd[1], t->d_vals, ops[0].ptr,
                                                       ops[0].ld, ops[0].ptr, ops[0].ld, ops[1].ptr, ops[1].ld, out, partial,
                                                       sa_make_limits(t, t->dims[1], t->dims[0], wl.n_slots));
            if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
            *launches += 1;
        }
        if (!wl.fix.empty()) {
            if (sa_launch_fixup(wl, partial, out, M, stream) != cudaSuccess) return SA_E_CUDA;
            *launches += 1;
        }
        return SA_OK;
    }
    const int64_t J = t->dims[1];
    float *E = static_cast<float *>(ws);
    float *partial = reinterpret_cast<float *>(static_cast<char *>(ws) + sa_align256(size_t(J) * M * sizeof(float)));
    const sa_status gs = sa_launch_dense_gemm(J, ops[0].ptr, ops[0].ld, ops[1].ptr, ops[1].ld, L, M, E, t->d_status, stream);
    if (gs != SA_OK) return gs;
    *launches += 1;
    const int64_t ctas = (n_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
    if (ctas > 0) {
        spmm_kernel<M / 32><<<(unsigned)ctas, 256, 0, stream>>>(wl.d_items, n_items, t->d_pos[1], t->d_crd[1], t->d_vals, E,
                                                               out, partial, sa_make_limits(t, J, t->dims[0], wl.n_slots));
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    if (!wl.fix.empty()) {
        if (sa_launch_fixup(wl, partial, out, M, stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}

// Kernel 3 <SpMMH,GEMM>: ops = {C, D, E}; the gathered row is C(j,:) * D(j,:), the resident matrix is E.
template <int L, int M>
sa_status run_hadamard(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, cudaStream_t stream, int *launches)
{
    const sa_worklist &wl = t->wl_aux;
    const int64_t n_items = int64_t(wl.items.size());
    const size_t smem = size_t(L * M + SA_WARPS_PER_CTA * L) * sizeof(float);
    *launches = 0;
    float *partial = static_cast<float *>(ws);
    auto kern = spmm_gemm_left_kernel<L, M, true>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) return SA_E_CUDA;
    const int64_t want = (n_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
    const int64_t ctas = std::min<int64_t>(want, resident_ctas(reinterpret_cast<const void *>(kern), smem));
    if (ctas > 0) {
        kern<<<(unsigned)ctas, 256, smem, stream>>>(wl.d_items, n_items, t->d_pos[1], t->d_crd[1], t->d_vals, ops[0].ptr,
                                                   ops[0].ld, ops[1].ptr, ops[1].ld, ops[2].ptr, ops[2].ld, out, partial,
                                                   sa_make_limits(t, t->dims[1], t->dims[0], wl.n_slots));
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    if (!wl.fix.empty()) {
        if (sa_launch_fixup(wl, partial, out, M, stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}

// Kernel 7 <SpTTM,SpTTM>: A(i,j,m) = sum_{k,l} B(i,j,k) C(k,l) D(l,m), one row of M values per (i,j) fiber of B
// (the output has B's level-2 pattern).  Seen from the fibers, B is a sparse matrix B' with one row per fiber
// and the chain is <SpMM,GEMM> on it: `right` = B'.(C.D), else (B'.C).D with the fiber temporaries T(f,:)
// (the t of the paper's nest, widened to a vector and kept for the dense stage) in the workspace.
template <int L, int M>
sa_status run_fibers(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, bool right, cudaStream_t stream, int *launches)
{
    const sa_worklist &wl = t->wl_aux;
    const int64_t n_items = int64_t(wl.items.size());
    const int64_t F2 = t->count[1], K = t->dims[2];
    const int64_t ctas = (n_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
    *launches = 0;
    if (right) {
        float *E = static_cast<float *>(ws);
        float *partial = reinterpret_cast<float *>(static_cast<char *>(ws) + sa_align256(size_t(K) * M * sizeof(float)));
        const sa_status gs = sa_launch_dense_gemm(K, ops[0].ptr, ops[0].ld, ops[1].ptr, ops[1].ld, L, M, E, t->d_status, stream);
        if (gs != SA_OK) return gs;
        *launches += 1;
        if (ctas > 0) {
            fiber_spmm_kernel<M><<<(unsigned)ctas, 256, 0, stream>>>(wl.d_items, n_items, t->d_pos[2], t->d_nzpack, E, M, out, partial,
                                                                     sa_make_limits(t, K, F2, wl.n_slots));
            if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
            *launches += 1;
        }
        if (!wl.fix.empty()) {
            if (sa_launch_fixup(wl, partial, out, M, stream) != cudaSuccess) return SA_E_CUDA;
            *launches += 1;
        }
        return SA_OK;
    }
    float *T = static_cast<float *>(ws);
    float *partial = reinterpret_cast<float *>(static_cast<char *>(ws) + sa_align256(size_t(F2) * L * sizeof(float)));
    if (ctas > 0) {
        fiber_spmm_kernel<L><<<(unsigned)ctas, 256, 0, stream>>>(wl.d_items, n_items, t->d_pos[2], t->d_nzpack, ops[0].ptr, ops[0].ld,
                                                                T, partial, sa_make_limits(t, K, F2, wl.n_slots));
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    if (!wl.fix.empty()) {
        if (sa_launch_fixup(wl, partial, T, L, stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    const sa_status gs = sa_launch_dense_gemm(F2, T, L, ops[1].ptr, ops[1].ld, L, M, out, t->d_status, stream);
    if (gs != SA_OK) return gs;
    *launches += 1;
    return SA_OK;
}

}  // namespace

// out (rows x M) = A (rows x L, leading dimension lda) . B (L x M), BF16x3 on tensor cores; used as the
// dense stage of other chains.  L in {32, 64, 128, 256}, M in {32, 64}.
template <int L, int M>
static sa_status dense_gemm(int64_t rows, const float *A, int64_t lda, const float *B, int64_t ldb, float *out,
                            cudaStream_t stream)
{
    using GC = gemm_bf16_cfg<L, M>;
    auto gk = gemm_bf16x3_kernel<L, M>;
    if (cudaFuncSetAttribute(gk, cudaFuncAttributeMaxDynamicSharedMemorySize, int(GC::SMEM)) != cudaSuccess) return SA_E_CUDA;
    const int64_t ctas = std::min<int64_t>((rows + GC::BM - 1) / GC::BM, resident_ctas(reinterpret_cast<const void *>(gk), GC::SMEM));
    if (ctas > 0) gk<<<(unsigned)ctas, 256, GC::SMEM, stream>>>(rows, A, lda, B, ldb, out);
    return cudaGetLastError() == cudaSuccess ? SA_OK : SA_E_CUDA;
}

bool sa_dense_gemm_ok(int64_t L, int64_t M) { return (L == 32 || L == 64 || L == 128 || L == 256) && (M == 32 || M == 64); }

sa_status sa_launch_dense_gemm(int64_t rows, const float *A, int64_t lda, const float *B, int64_t ldb, int64_t L,
                               int64_t M, float *out, int32_t *status, cudaStream_t stream)
{
    if (sa_dense_gemm_tc_ok(L, M)) return sa_launch_dense_gemm_tc(rows, A, lda, B, ldb, L, M, out, status, stream);
#define SA_CASE(l, m) if (L == l && M == m) return dense_gemm<l, m>(rows, A, lda, B, ldb, out, stream);
    SA_CASE(32, 32) SA_CASE(32, 64)
#undef SA_CASE
    return SA_E_UNSUPPORTED;
}

bool sa_ranks_ok_spmm_gemm(int64_t L, int64_t M) { return (L == 128 || L == 256) && (M == 32 || M == 64); }

// workspace: ASSOC_RIGHT [E = C.D, J x M][partial rows]; ASSOC_LEFT [partial rows]
size_t sa_ws_spmm_gemm(const sa_tensor *t, const sa_dense *ops, bool right)
{
    const size_t M = size_t(ops[1].cols);
    size_t b = sa_align256(size_t(t->wl_aux.n_slots) * M * sizeof(float));
    if (right) b += sa_align256(size_t(t->dims[1]) * M * sizeof(float));
    return b;
}

sa_status sa_launch_spmm_gemm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t, bool right,
                              cudaStream_t stream, int *launches)
{
    const int64_t L = ops[0].cols, M = ops[1].cols;
    if (L == 128 && M == 32) return run<128, 32>(t, ops, out, ws, right, stream, launches);
    if (L == 128 && M == 64) return run<128, 64>(t, ops, out, ws, right, stream, launches);
    if (L == 256 && M == 32) return run<256, 32>(t, ops, out, ws, right, stream, launches);
    if (L == 256 && M == 64) return run<256, 64>(t, ops, out, ws, right, stream, launches);
    return SA_E_UNSUPPORTED;
}

size_t sa_ws_spmmh_gemm(const sa_tensor *t, const sa_dense *ops)
{
    return sa_align256(size_t(t->wl_aux.n_slots) * size_t(ops[2].cols) * sizeof(float));
}

sa_status sa_launch_spmmh_gemm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t, cudaStream_t stream,
                               int *launches)
{
    const int64_t L = ops[0].cols, M = ops[2].cols;
    if (L == 128 && M == 32) return run_hadamard<128, 32>(t, ops, out, ws, stream, launches);
    if (L == 128 && M == 64) return run_hadamard<128, 64>(t, ops, out, ws, stream, launches);
    if (L == 256 && M == 32) return run_hadamard<256, 32>(t, ops, out, ws, stream, launches);
    if (L == 256 && M == 64) return run_hadamard<256, 64>(t, ops, out, ws, stream, launches);
    return SA_E_UNSUPPORTED;
}

bool sa_ranks_ok_spttm_spttm(int64_t L, int64_t M) { return (L == 32 || L == 64) && (M == 32 || M == 64); }

// workspace: right [E = C.D, K x M][partial rows of M]; else [T, one row of L per fiber][partial rows of L]
size_t sa_ws_spttm_spttm(const sa_tensor *t, const sa_dense *ops, bool right)
{
    const size_t L = size_t(ops[0].cols), M = size_t(ops[1].cols);
    if (right) return sa_align256(size_t(t->dims[2]) * M * sizeof(float)) + sa_align256(size_t(t->wl_aux.n_slots) * M * sizeof(float));
    return sa_align256(size_t(t->count[1]) * L * sizeof(float)) + sa_align256(size_t(t->wl_aux.n_slots) * L * sizeof(float));
}

sa_status sa_launch_spttm_spttm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t, bool right,
                                cudaStream_t stream, int *launches)
{
    const int64_t L = ops[0].cols, M = ops[1].cols;
    if (L == 32 && M == 32) return run_fibers<32, 32>(t, ops, out, ws, right, stream, launches);
    if (L == 32 && M == 64) return run_fibers<32, 64>(t, ops, out, ws, right, stream, launches);
    if (L == 64 && M == 32) return run_fibers<64, 32>(t, ops, out, ws, right, stream, launches);
    if (L == 64 && M == 64) return run_fibers<64, 64>(t, ops, out, ws, right, stream, launches);
    return SA_E_UNSUPPORTED;
}
