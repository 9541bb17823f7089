// Kernel 6 <SpTTM,TTM>:  A(i,l,m) = sum_{j,k} B(i,j,k) C(j,l) D(k,m), scheduled as the branched
// nest  i, j' < t ; k': t += B(i,j,k) D(k,m) , l: A(i,l,m) += t C(j,l) >  of the paper's Table of
// kernels (Section 6).  Producer (SpTTM, fp32 ALU): the nonzeros of a work item are streamed in
// flat batches of 32; the D rows of a batch are gathered with cp.async into a per-warp ring of
// shared-memory stages (several batches in flight per warp, no registers tied up); the fiber
// temporary t(m) lives in one register per lane (lane = m) and is closed by an end-of-fiber flag
// carried in the index stream.  Consumer (TTM, tensor cores): closed temporaries are staged eight
// at a time in shared memory and the slice tile is updated as A(i,:,:) += Cg^T (L x 8) . T (8 x M)
// with m16n8k8 TF32 MMAs, each operand split into a high and a low TF32 part (three products) so
// the stage keeps fp32-level accuracy.  The order-3 intermediate T(i,j,m) is never stored.
#include "sa_device.cuh"

namespace {

__device__ __forceinline__ uint32_t tf32_rna(float x)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}

__device__ __forceinline__ void split_tf32(float x, uint32_t &hi, uint32_t &lo)
{
    hi = tf32_rna(x);
    lo = tf32_rna(x - __uint_as_float(hi));
}

__device__ __forceinline__ void mma_m16n8k8_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

__device__ __forceinline__ void cp_async16(float *dst_smem, const float *src)
{
    const uint32_t d = static_cast<uint32_t>(__cvta_generic_to_shared(dst_smem));
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

template <int L, int M>
struct cfg {
    static constexpr int MT = L / 16;       // m16 tiles over l
    static constexpr int NT = M / 8;        // n8 tiles over m
    static constexpr int TS = M;            // row stride of the staged temporaries (unpadded: two CTAs of
                                            // 8 warps x (3 stages + ring) must fit one SM's shared memory)
    static constexpr int RS = M + 8;        // row stride of a warp's tile in the CTA reduction
    static constexpr int NS = 3;            // cp.async stages (batches of 32 factor rows) per warp
    static constexpr int STAGE = 32 * M;    // floats per stage
    static constexpr int WORK = NS * STAGE + 16 * TS + 32;                 // stages + ring of temporaries + values of a batch
    static constexpr int WARP_SMEM = (L * RS > WORK ? L * RS : WORK);      // floats per warp
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void cp_async16_raw(uint32_t dst_smem, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}

// Gather the 32 rows D(k_s, :) of one batch into a stage: LPR lanes copy one row in 16-byte pieces.
// dst_lane: shared address of the stage plus this lane's (row-in-group, piece) offset; src_lane: D plus
// the lane's piece offset; row_bytes = 4 * ld(D) (byte offsets fit 32 bits, checked by the launcher).
template <int M>
__device__ __forceinline__ void stage_rows(uint32_t dst_lane, int kbatch, const char *__restrict__ src_lane,
                                           uint32_t row_bytes, int r)
{
    constexpr int LPR = M / 4, RPI = 32 / LPR;
#pragma unroll
    for (int q = 0; q < 32 / RPI; ++q) {
        const uint32_t k = uint32_t(__shfl_sync(SA_FULL_MASK, kbatch, q * RPI + r)) & 0x3fffffffu;
        cp_async16_raw(dst_lane + q * RPI * M * 4, src_lane + k * row_bytes);
    }
}

// The values of C one flush needs: rows of the fibers x = t and x = t + 4 of the next group of eight,
// columns 16 mt + g and 16 mt + g + 8.  Loaded right after the previous flush so that the L2 latency
// is covered by the producer work in between.
template <int L, int M>
__device__ __forceinline__ void load_cfrag(float (&cf)[cfg<L, M>::MT][4], const float *__restrict__ crow_a,
                                           const float *__restrict__ crow_b, int lane)
{
    const int g = lane >> 2;
#pragma unroll
    for (int mt = 0; mt < cfg<L, M>::MT; ++mt) {
        cf[mt][0] = __ldg(crow_a + 16 * mt + g);
        cf[mt][1] = __ldg(crow_a + 16 * mt + g + 8);
        cf[mt][2] = __ldg(crow_b + 16 * mt + g);
        cf[mt][3] = __ldg(crow_b + 16 * mt + g + 8);
    }
}

// acc += Cg^T . T for eight staged fibers: rows (row0 + x) & 15, x = 0..7, of the 16-row ring.
template <int L, int M>
__device__ __forceinline__ void ttm3_flush(float (&acc)[cfg<L, M>::MT][cfg<L, M>::NT][4], const float *__restrict__ Tbuf,
                                           int row0, const float (&cf)[cfg<L, M>::MT][4], int lane)
{
    using K = cfg<L, M>;
    const int g = lane >> 2, t = lane & 3;
    const float *ta = Tbuf + ((row0 + t) & 15) * K::TS + g;
    const float *tb = Tbuf + ((row0 + t + 4) & 15) * K::TS + g;
    uint32_t bh[K::NT][2], bl[K::NT][2];
#pragma unroll
    for (int nt = 0; nt < K::NT; ++nt) {
        split_tf32(ta[8 * nt], bh[nt][0], bl[nt][0]);
        split_tf32(tb[8 * nt], bh[nt][1], bl[nt][1]);
    }
#pragma unroll
    for (int mt = 0; mt < K::MT; ++mt) {
        uint32_t ah[4], al[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) split_tf32(cf[mt][x], ah[x], al[x]);
#pragma unroll
        for (int nt = 0; nt < K::NT; ++nt) {
            mma_m16n8k8_tf32(acc[mt][nt], al, bh[nt]);
            mma_m16n8k8_tf32(acc[mt][nt], ah, bl[nt]);
            mma_m16n8k8_tf32(acc[mt][nt], ah, bh[nt]);
        }
    }
}

// Store a slice tile held as MMA accumulator fragments (streaming stores: the output is written once).
template <int L, int M>
__device__ __forceinline__ void store_tile(const float (&acc)[cfg<L, M>::MT][cfg<L, M>::NT][4], float *__restrict__ dst, int lane)
{
    using K = cfg<L, M>;
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int mt = 0; mt < K::MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < K::NT; ++nt) {
            const int l = 16 * mt + g, mm = 8 * nt + 2 * t;
            sa_st_cs2(dst + l * M + mm, make_float2(acc[mt][nt][0], acc[mt][nt][1]));
            sa_st_cs2(dst + (l + 8) * M + mm, make_float2(acc[mt][nt][2], acc[mt][nt][3]));
        }
}

// One warp evaluates one work item: nonzeros [p0,p1) starting inside fiber f0.  MULTI: the item is a run
// of whole small slices (positions it.pad .. it.row_end - 1 in crd_i); the warp streams through all of
// them and stores each slice's tile to `out` when the slice-end flag (bit 30 of the index stream) comes
// by.  Otherwise the item is a piece of one slice and the tile is left in acc for the caller.
template <int L, int M>
__device__ __forceinline__ void ttm3_warp_item(const sa_item &it, const int32_t *__restrict__ crd_j,
                                               const int32_t *__restrict__ kflag, const float *__restrict__ vals,
                                               const float *__restrict__ C, uint32_t ldc, const float *__restrict__ D,
                                               uint32_t ldd, float *__restrict__ wsm,
                                               float (&acc)[cfg<L, M>::MT][cfg<L, M>::NT][4], const bool multi,
                                               const int32_t *__restrict__ crd_i, float *__restrict__ out)
{
    using K = cfg<L, M>;
    static_assert(K::NS == 3, "the register ring below is written for three stages");
    const int lane = threadIdx.x & 31;
    const int m = lane & (M - 1);
    const int t4 = lane & 3;
    float *Tbuf = wsm + K::NS * K::STAGE;
    float *vs = Tbuf + 16 * K::TS;                  // values of the batch being consumed
#pragma unroll
    for (int mt = 0; mt < K::MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < K::NT; ++nt)
#pragma unroll
            for (int q = 0; q < 4; ++q) acc[mt][nt][q] = 0.f;
    if (it.p0 >= it.p1) return;
    const int p0 = it.p0, p1 = it.p1, f0 = it.f0, fmax = it.f1 - 1;
    const int nb = (p1 - p0 + 31) >> 5;
    // per-lane constants of the row gather
    constexpr int LPR = M / 4;
    const int gr = lane / LPR, gc = lane % LPR;
    const uint32_t dst_lane = smem_u32(wsm) + uint32_t(gr * M + gc * 4) * 4u;
    const char *src_lane = reinterpret_cast<const char *>(D + gc * 4);
    const uint32_t row_bytes = ldd * 4u;
    int pn = p0 + lane;                              // position this lane loads next
    auto load_kv = [&](int &k, float &v) {
        k = 0;
        v = 0.f;
        if (pn < p1) { k = kflag[pn]; v = vals[pn]; }
        pn += 32;
    };
    // index/value registers of batches B .. B+6: the index of a batch is needed two rounds before its
    // values (to request its rows), and a streaming load takes several rounds to arrive; row gathers
    // of batches B+1, B+2 are in flight while B is consumed
    int k0, k1, k2, k3, k4, k5, k6;
    float v0, v1, v2, v3, v4, v5, v6;
    load_kv(k0, v0);
    load_kv(k1, v1);
    load_kv(k2, v2);
    load_kv(k3, v3);
    load_kv(k4, v4);
    load_kv(k5, v5);
    load_kv(k6, v6);
    stage_rows<M>(dst_lane, k0, src_lane, row_bytes, gr);
    cp_async_commit();
    if (1 < nb) stage_rows<M>(dst_lane + K::STAGE * 4, k1, src_lane, row_bytes, gr);
    cp_async_commit();
    int nclosed = 0, nflushed = 0;          // fibers closed / handed to the tensor cores so far
    float cf[K::MT][4];                     // C values of the next flush
    load_cfrag<L, M>(cf, C + uint32_t(crd_j[min(f0 + t4, fmax)]) * ldc, C + uint32_t(crd_j[min(f0 + t4 + 4, fmax)]) * ldc, lane);
    float T = 0.f, U = 0.f;                 // two partial sums of the open fiber (shorter dependency chains)
    int s_cur = 0, s_issue = 2;
    int slice = it.pad;                     // MULTI: position of the slice being accumulated
    // hand the n (<= 8) oldest closed fibers to the tensor cores and fetch the C values of the next group
    auto flush_group = [&](int n) {
        for (int x = n; x < 8; ++x) Tbuf[((nflushed + x) & 15) * K::TS + m] = 0.f;   // unused rows
        __syncwarp();
        ttm3_flush<L, M>(acc, Tbuf, nflushed, cf, lane);
        __syncwarp();
        nflushed += n;
        load_cfrag<L, M>(cf, C + uint32_t(crd_j[min(f0 + nflushed + t4, fmax)]) * ldc,
                         C + uint32_t(crd_j[min(f0 + nflushed + t4 + 4, fmax)]) * ldc, lane);
    };
    // T += v * d for one nonzero; `end` (warp-uniform) closes the fiber into the ring of temporaries
#define SA_TTM3_STEP(v, d, end)                                   \
    T = fmaf(v, d, T);                                            \
    if (end) {                                                    \
        Tbuf[(nclosed & 15) * K::TS + m] = T + U;                 \
        T = 0.f;                                                  \
        U = 0.f;                                                  \
        ++nclosed;                                                \
    }
#pragma unroll 1
    for (int b = 0; b < nb; ++b) {
        if (b + 2 < nb) stage_rows<M>(dst_lane + s_issue * (K::STAGE * 4), k2, src_lane, row_bytes, gr);
        cp_async_commit();
        vs[lane] = v0;
        cp_async_wait<2>();
        __syncwarp();
        const float *st = wsm + s_cur * K::STAGE + m;
        unsigned ends = __ballot_sync(SA_FULL_MASK, k0 < 0);
        const unsigned sends = multi ? __ballot_sync(SA_FULL_MASK, (k0 & 0x40000000) != 0) : 0u;
        const int rem = p1 - p0 - 32 * b;
        if (rem <= 32) ends |= 1u << (rem - 1);         // the item's last nonzero closes its (possibly cut) fiber
        const int nchunks = rem >= 32 ? 4 : (rem + 7) >> 3;
#pragma unroll 1
        for (int c = 0; c < nchunks; ++c) {
            const unsigned e8 = (ends >> (8 * c)) & 0xffu;
            const float *sc = st + 8 * c * M;
            const float4 va = *reinterpret_cast<const float4 *>(vs + 8 * c);
            const float4 vb = *reinterpret_cast<const float4 *>(vs + 8 * c + 4);
            if (((sends >> (8 * c)) & 0xffu) != 0) {
                // a slice ends inside this chunk: one nonzero at a time, the tile leaves at the slice end
                const unsigned s8 = (sends >> (8 * c)) & 0xffu;
                T += U;
                U = 0.f;
#pragma unroll 1
                for (int u = 0; u < 8; ++u) {
                    T = fmaf(vs[8 * c + u], sc[u * M], T);
                    if (e8 & (1u << u)) {
                        Tbuf[(nclosed & 15) * K::TS + m] = T;
                        T = 0.f;
                        ++nclosed;
                        const bool slice_end = (s8 & (1u << u)) != 0;
                        if (slice_end || nclosed - nflushed >= 8) flush_group(min(8, nclosed - nflushed));
                        if (slice_end) {
                            store_tile<L, M>(acc, out + int64_t(crd_i[slice]) * (L * M), lane);
                            ++slice;
#pragma unroll
                            for (int mt = 0; mt < K::MT; ++mt)
#pragma unroll
                                for (int nt = 0; nt < K::NT; ++nt)
#pragma unroll
                                    for (int q = 0; q < 4; ++q) acc[mt][nt][q] = 0.f;
                        }
                    }
                }
                continue;
            }
            if ((e8 & 0xfu) == 0) {
                T = fmaf(va.x, sc[0], T);
                U = fmaf(va.y, sc[M], U);
                T = fmaf(va.z, sc[2 * M], T);
                U = fmaf(va.w, sc[3 * M], U);
            } else {
                SA_TTM3_STEP(va.x, sc[0], e8 & 1u)
                SA_TTM3_STEP(va.y, sc[M], e8 & 2u)
                SA_TTM3_STEP(va.z, sc[2 * M], e8 & 4u)
                SA_TTM3_STEP(va.w, sc[3 * M], e8 & 8u)
            }
            if ((e8 & 0xf0u) == 0) {
                T = fmaf(vb.x, sc[4 * M], T);
                U = fmaf(vb.y, sc[5 * M], U);
                T = fmaf(vb.z, sc[6 * M], T);
                U = fmaf(vb.w, sc[7 * M], U);
            } else {
                SA_TTM3_STEP(vb.x, sc[4 * M], e8 & 16u)
                SA_TTM3_STEP(vb.y, sc[5 * M], e8 & 32u)
                SA_TTM3_STEP(vb.z, sc[6 * M], e8 & 64u)
                SA_TTM3_STEP(vb.w, sc[7 * M], e8 & 128u)
            }
            if (nclosed - nflushed >= 8) flush_group(8);
        }
        __syncwarp();                                   // stage s_cur and vs are free for the next round
        k0 = k1; k1 = k2; k2 = k3; k3 = k4; k4 = k5; k5 = k6;
        v0 = v1; v1 = v2; v2 = v3; v3 = v4; v4 = v5; v5 = v6;
        load_kv(k6, v6);
        s_issue = s_cur;
        s_cur = s_cur == 2 ? 0 : s_cur + 1;
    }
#undef SA_TTM3_STEP
    cp_async_wait<0>();
    if (nclosed - nflushed > 0) flush_group(nclosed - nflushed);      // pieces of one slice: the open group
}

template <int L, int M>
__global__ void __launch_bounds__(256, 2)
ttm3_kernel(const sa_item *__restrict__ items, int64_t n_items, int n_group_ctas, const int32_t *__restrict__ crd_i,
            const int32_t *__restrict__ crd_j, const int32_t *__restrict__ kflag, const float *__restrict__ vals, const float *__restrict__ C, uint32_t ldc,
            const float *__restrict__ D, uint32_t ldd, float *__restrict__ out, float *__restrict__ partial)
{
    using K = cfg<L, M>;
    constexpr int TILE = L * M;
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    float *wsm = smem + warp * K::WARP_SMEM;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    const bool group = int(blockIdx.x) < n_group_ctas;
    float acc[K::MT][K::NT][4];
    sa_item it;
    it.f0 = it.f1 = it.p0 = it.p1 = 0;
    it.dest = -1;
    it.out_row = 0;
    it.pad = it.row_end = 0;
    if (idx < n_items) it = items[idx];
    if (idx < n_items || group)
        ttm3_warp_item<L, M>(it, crd_j, kflag, vals, C, ldc, D, ldd, wsm, acc, !group, crd_i, out);
    if (!group) return;                 // runs of small slices: every tile was stored at its slice end
    // the CTA's eight warps hold partial tiles of the same slice: sum them in a fixed order
#pragma unroll
    for (int mt = 0; mt < K::MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < K::NT; ++nt) {
            const int l = 16 * mt + g, mm = 8 * nt + 2 * t;
            *reinterpret_cast<float2 *>(wsm + l * K::RS + mm) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
            *reinterpret_cast<float2 *>(wsm + (l + 8) * K::RS + mm) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
        }
    __syncthreads();
    const sa_item lead = items[int64_t(blockIdx.x) * SA_WARPS_PER_CTA];
    float *dst = lead.dest >= 0 ? partial + int64_t(lead.dest) * TILE : out + int64_t(lead.out_row) * TILE;
    for (int x = threadIdx.x * 4; x < TILE; x += 256 * 4) {
        const int off = (x / M) * K::RS + (x % M);
        float4 s = *reinterpret_cast<const float4 *>(smem + off);
#pragma unroll
        for (int w = 1; w < SA_WARPS_PER_CTA; ++w) {
            const float4 v = *reinterpret_cast<const float4 *>(smem + w * K::WARP_SMEM + off);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        if (lead.dest >= 0) *reinterpret_cast<float4 *>(dst + x) = s;
        else sa_st_cs4(dst + x, s);
    }
}

template <int L, int M>
cudaError_t launch(const sa_tensor *t, const sa_dense *ops, float *out, float *partial, cudaStream_t stream)
{
    const sa_worklist &wl = t->wl_main;
    const int64_t n_items = int64_t(wl.items.size());
    const int64_t n_warp_items = n_items - wl.n_group_ctas * SA_WARPS_PER_CTA;
    const int64_t ctas = wl.n_group_ctas + (n_warp_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
    if (ctas == 0) return cudaSuccess;
    constexpr size_t smem = size_t(SA_WARPS_PER_CTA) * cfg<L, M>::WARP_SMEM * sizeof(float);
    auto kern = ttm3_kernel<L, M>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess)
        return cudaGetLastError();
    kern<<<(unsigned)ctas, 256, smem, stream>>>(wl.d_items, n_items, int(wl.n_group_ctas), t->d_crd[0], t->d_crd[1], t->d_crd_endflag,
                                               t->d_vals, ops[0].ptr, uint32_t(ops[0].ld), ops[1].ptr, uint32_t(ops[1].ld), out, partial);
    return cudaGetLastError();
}

}  // namespace

bool sa_ranks_ok_ttm3(int64_t L, int64_t M) { return (L == 16 || L == 32) && (M == 16 || M == 32); }

size_t sa_ws_ttm3(const sa_tensor *t, const sa_dense *ops)
{
    return sa_align256(size_t(t->wl_main.n_slots) * size_t(ops[0].cols * ops[1].cols) * sizeof(float));
}

sa_status sa_launch_ttm3(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                         cudaStream_t stream, int *launches)
{
    const int64_t L = ops[0].cols, M = ops[1].cols;
    (void)ws_bytes;
    // the kernel addresses factor rows with 32-bit byte offsets
    for (int i = 0; i < 2; ++i)
        if (ops[i].rows * ops[i].ld >= (int64_t(1) << 30)) return SA_E_UNSUPPORTED;
    if (!t->d_crd_endflag) return SA_E_UNSUPPORTED;      // last dimension >= 2^30: no room for the flag bits
    float *partial = static_cast<float *>(ws);
    cudaError_t e;
    if (L == 16 && M == 16) e = launch<16, 16>(t, ops, out, partial, stream);
    else if (L == 32 && M == 16) e = launch<32, 16>(t, ops, out, partial, stream);
    else if (L == 16 && M == 32) e = launch<16, 32>(t, ops, out, partial, stream);
    else if (L == 32 && M == 32) e = launch<32, 32>(t, ops, out, partial, stream);
    else return SA_E_UNSUPPORTED;
    if (e != cudaSuccess) return SA_E_CUDA;
    *launches = t->wl_main.items.empty() ? 0 : 1;
    if (!t->wl_main.fix.empty()) {
        if (sa_launch_fixup(t->wl_main, partial, out, int(L * M), stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}

// ------------------------------------------------------------------ entry point without allocation

// Scratch for sa_run_ttm3_static_scratch: part of the library image, so every device that loads the
// library carries these 4 MiB until the process exits.
constexpr size_t SA_STATIC_SCRATCH_BYTES = size_t(4) << 20;
static __device__ __align__(256) float sa_static_scratch[SA_STATIC_SCRATCH_BYTES / sizeof(float)];

namespace {

constexpr int SA_MAX_DEVICES = 64;
float *g_static_scratch_addr[SA_MAX_DEVICES];   // device address of sa_static_scratch, per device; set once

// In host code `sa_static_scratch` only names the symbol; the address a kernel can use has to be
// asked for, with the owning device current.
sa_status static_scratch_address(int device, float **addr)
{
    if (device < 0 || device >= SA_MAX_DEVICES) return SA_E_ARG;
    if (!g_static_scratch_addr[device]) {
        float *p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&p), sa_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return SA_E_CUDA;
        }
        g_static_scratch_addr[device] = p;
    }
    *addr = g_static_scratch_addr[device];
    return SA_OK;
}

}  // namespace

extern "C" sa_status sa_run_ttm3_static_scratch(const sa_tensor *t, const sa_dense *ops, int n_ops, float *out,
                                                void *cuda_stream)
{
    if (!t || !ops || !out || n_ops != 2 || t->device < 0) return SA_E_ARG;
    if (reinterpret_cast<uintptr_t>(out) % 16) return SA_E_ARG;
    if (t->fmt != SA_FMT_CSF || t->order != 3) return SA_E_FORMAT;
    for (int i = 0; i < 2; ++i) {
        if (!ops[i].ptr) return SA_E_ARG;
        if (ops[i].rows != t->dims[i + 1] || ops[i].cols <= 0 || ops[i].ld < ops[i].cols || ops[i].ld % 4 ||
            reinterpret_cast<uintptr_t>(ops[i].ptr) % 16)
            return SA_E_SHAPE;
    }
    if (!sa_ranks_ok_ttm3(ops[0].cols, ops[1].cols)) return SA_E_UNSUPPORTED;
    const size_t need = sa_ws_ttm3(t, ops);
    if (need > SA_STATIC_SCRATCH_BYTES) return SA_E_WORKSPACE;   // the partial tiles do not fit the built-in scratch
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return SA_E_CUDA; }
    if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) { cudaGetLastError(); return SA_E_CUDA; }
    float *scratch = nullptr;
    sa_status s = static_scratch_address(t->device, &scratch);
    int launches = 0;
    if (s == SA_OK)
        s = sa_launch_ttm3(t, ops, out, scratch, SA_STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(cuda_stream), &launches);
    if (s == SA_E_CUDA) cudaGetLastError();
    if (s == SA_OK) t->last_launches = launches;
    if (prev != t->device) cudaSetDevice(prev);
    return s;
}
