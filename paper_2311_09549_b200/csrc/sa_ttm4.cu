// Order-4 analogue of kernel 6:  A(i,l,m,n) = sum_{j,k,o} B(i,j,k,o) C(j,l) D(k,m) E(o,n),
// scheduled with the two-level branched nesting the paper uses for the second schedule of its
// 3-D TTMC kernel (Table of kernels, Section 6; recursive producer/consumer split of Section 4.2):
//   i, j' < T2(m,n) ;  k' < t(n) ; o': t(n) += B E(o,n) , m: T2(m,n) += t(n) D(k,m) > ,
//                      l: A(i,l,m,n) += T2(m,n) C(j,l) >
// Both temporaries and the slice tile live in registers.  To keep the 16 x 16 x 16 tile within a
// warp's registers the n range is halved: every work item is evaluated by two independent warps,
// one per half of n (8 columns), each streaming the item's nonzeros once.  Lane (q, n8): q = lane/8
// is one of four nonzeros taken per step, n8 the column; t is reduced over q when a level-3 fiber
// (i,j,k) closes, T2(m = 4q..4q+3, n8) and the tile A(i, l, 4q..4q+3, n8) stay distributed.
// The nonzeros are streamed in flat batches of 32; rows E(o,:) of a batch and the rows D(k,:) of
// the level-3 fibers that close in it are gathered with cp.async into a three-stage per-warp ring.
#include "sa_device.cuh"

namespace {

constexpr int R = 16;                  // L = M = N = 16
constexpr int TILE4 = R * R * R;       // floats per output slice
constexpr int NH = 8;                  // columns n per warp
constexpr int NS4 = 3;                 // stages
constexpr int E_STAGE = 32 * NH;       // floats: 32 half rows of E
constexpr int D_STAGE = 32 * R;        // floats: up to 32 rows of D
constexpr int STAGE4 = E_STAGE + D_STAGE;
constexpr int WARP4 = NS4 * STAGE4 + 32;                 // + values of the batch being consumed
constexpr int HALF_TILE = R * R * NH;                    // floats a warp accumulates
static_assert(SA_WARPS_PER_CTA * WARP4 >= SA_WARPS_PER_CTA * HALF_TILE, "the CTA reduction reuses the stage memory");

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void cp_async16_raw(uint32_t dst_smem, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

struct ttm4_args {
    const int32_t *pos2;      // level-1 fiber (i,j) -> first level-2 node
    const int32_t *crd_j;     // per level-1 fiber
    const int32_t *crd_k;     // per level-2 node
    const int32_t *oflag;     // per nonzero: o, bit 31 = last of its (i,j,k) fiber, bit 30 = last of its (i,j) fiber
    const float *vals;
    const float *C, *D, *E;
    uint32_t ldc, ldd, lde;
};

// One warp, one work item (level-1 fibers [f0,f1) of a slice = nonzeros [p0,p1)), one half of n.
__device__ __forceinline__ void ttm4_warp_item(const sa_item &it, const ttm4_args &a, float *__restrict__ wsm,
                                               float (&acc)[R][4])
{
    const int lane = threadIdx.x & 31;
    const int q = lane >> 3, n8 = lane & 7;
    const int nh = it.pad;
#pragma unroll
    for (int l = 0; l < R; ++l)
#pragma unroll
        for (int x = 0; x < 4; ++x) acc[l][x] = 0.f;
    if (it.p0 >= it.p1) return;
    const int p0 = it.p0, p1 = it.p1;
    const int nb = (p1 - p0 + 31) >> 5;
    float *vs = wsm + NS4 * STAGE4;

    // ---- streams: nonzeros (o + flags, value) seven batches deep, level-2 coordinates k 64 deep
    int pn = p0 + lane;
    auto load_ov = [&](int &o, float &v) {
        o = 0;
        v = 0.f;
        if (pn < p1) { o = a.oflag[pn]; v = a.vals[pn]; }
        pn += 32;
    };
    int o0, o1, o2, o3, o4, o5, o6;
    float v0, v1, v2, v3, v4, v5, v6;
    load_ov(o0, v0); load_ov(o1, v1); load_ov(o2, v2); load_ov(o3, v3);
    load_ov(o4, v4); load_ov(o5, v5); load_ov(o6, v6);
    const int g_first = a.pos2[it.f0], g_last = a.pos2[it.f1] - 1;     // level-2 nodes of the item
    int gk_base = g_first;                                            // kk0: k of nodes gk_base .. +31, kk1 / kk2: the next 32 + 32
    auto load_k = [&](int base) { return a.crd_k[min(base + lane, g_last)]; };
    int kk0 = load_k(gk_base), kk1 = load_k(gk_base + 32), kk2 = load_k(gk_base + 64);   // kk2: prefetch only
    int g_staged = g_first;                                           // first node whose D row is not yet requested

    // ---- row gathers of one batch: E half rows of its 32 nonzeros, D rows of the fibers closing in it
    const uint32_t ws_addr = smem_u32(wsm);
    const char *e_lane = reinterpret_cast<const char *>(a.E + nh * NH + (lane & 1) * 4);
    const char *d_lane = reinterpret_cast<const char *>(a.D + (lane & 3) * 4);
    const uint32_t e_row_bytes = a.lde * 4u, d_row_bytes = a.ldd * 4u;
    auto stage_batch = [&](int stage, int obatch) {
        const uint32_t base = ws_addr + uint32_t(stage * STAGE4) * 4u;
        // E: two lanes per row, 16 rows per instruction
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int row = h * 16 + (lane >> 1);
            const uint32_t o = uint32_t(__shfl_sync(SA_FULL_MASK, obatch, row)) & 0x3fffffffu;
            cp_async16_raw(base + uint32_t(row * NH + (lane & 1) * 4) * 4u, e_lane + o * e_row_bytes);
        }
        // D: the c level-3 fibers that close in this batch are nodes g_staged .. g_staged + c - 1
        const int c = __popc(__ballot_sync(SA_FULL_MASK, obatch < 0));
        // g_staged - gk_base < 32 on entry and c <= 32: every node needed lies in kk0 / kk1
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int row = h * 8 + (lane >> 2);     // row-th closing fiber of the batch
            if (h * 8 < c) {
                const int rel = min(g_staged + row, g_last) - gk_base;       // 0 .. 63
                const int ka = __shfl_sync(SA_FULL_MASK, kk0, rel & 31);
                const int kb = __shfl_sync(SA_FULL_MASK, kk1, rel & 31);
                const uint32_t k = uint32_t(rel < 32 ? ka : kb);
                cp_async16_raw(base + uint32_t(E_STAGE + row * R + (lane & 3) * 4) * 4u, d_lane + k * d_row_bytes);
            }
        }
        g_staged += c;
        if (g_staged - gk_base >= 32) {              // the first 32 coordinates are used up
            kk0 = kk1;
            kk1 = kk2;
            gk_base += 32;
            kk2 = load_k(gk_base + 64);
        }
    };
    stage_batch(0, o0);
    cp_async_commit();
    if (1 < nb) stage_batch(1, o1);
    cp_async_commit();

    // ---- consumer state
    int f = it.f0;                                   // current level-1 fiber
    float4 crow[4];                                  // C(j, 0..15) of the current level-1 fiber, loaded at its start
    auto load_crow = [&](int fiber) {
        const float *p = a.C + uint32_t(a.crd_j[min(fiber, it.f1 - 1)]) * a.ldc;
#pragma unroll
        for (int x = 0; x < 4; ++x) crow[x] = sa_ldg4(p + 4 * x);
    };
    load_crow(f);
    float t = 0.f;                                   // partial t(n8) of the open level-3 fiber, this lane's nonzeros
    float t2[4] = {0.f, 0.f, 0.f, 0.f};              // T2(4q .. 4q+3, n8) of the open level-1 fiber
    int s_cur = 0, s_issue = 2;
#pragma unroll 1
    for (int b = 0; b < nb; ++b) {
        if (b + 2 < nb) stage_batch(s_issue, o2);
        cp_async_commit();
        vs[lane] = v0;
        cp_async_wait<2>();
        __syncwarp();
        const float *est = wsm + s_cur * STAGE4 + n8;             // E_half(o_s, n8) at est[s * NH]
        const float *dst = wsm + s_cur * STAGE4 + E_STAGE + 4 * q; // D(k_e, 4q..4q+3) at dst[e * R]
        unsigned ends3 = __ballot_sync(SA_FULL_MASK, o0 < 0);
        unsigned ends2 = __ballot_sync(SA_FULL_MASK, (o0 & 0x40000000) != 0);
        const int rem = p1 - p0 - 32 * b;
        const int nsteps = rem >= 32 ? 8 : (rem + 3) >> 2;
        int dcount = 0;                              // level-3 fibers closed so far in this batch
#pragma unroll 1
        for (int s = 0; s < nsteps; ++s) {
            const float prod = vs[4 * s + q] * est[(4 * s + q) * NH];
            unsigned e4 = (ends3 >> (4 * s)) & 0xfu;
            if (e4 == 0) {
                t += prod;
                continue;
            }
            const unsigned f4 = (ends2 >> (4 * s)) & 0xfu;
            int prev = -1;
            while (e4) {
                const int e = __ffs(e4) - 1;
                e4 &= e4 - 1;
                float tf = t + ((q > prev && q <= e) ? prod : 0.f);
                tf += __shfl_xor_sync(SA_FULL_MASK, tf, 8);
                tf += __shfl_xor_sync(SA_FULL_MASK, tf, 16);
                const float4 d4 = *reinterpret_cast<const float4 *>(dst + dcount * R);
                t2[0] = fmaf(d4.x, tf, t2[0]);
                t2[1] = fmaf(d4.y, tf, t2[1]);
                t2[2] = fmaf(d4.z, tf, t2[2]);
                t2[3] = fmaf(d4.w, tf, t2[3]);
                ++dcount;
                t = 0.f;
                prev = e;
                if (f4 & (1u << e)) {                // the level-1 fiber (i,j) closes too
#pragma unroll
                    for (int x = 0; x < 4; ++x) {
                        const float4 c = crow[x];
#pragma unroll
                        for (int y = 0; y < 4; ++y) {
                            acc[4 * x + 0][y] = fmaf(c.x, t2[y], acc[4 * x + 0][y]);
                            acc[4 * x + 1][y] = fmaf(c.y, t2[y], acc[4 * x + 1][y]);
                            acc[4 * x + 2][y] = fmaf(c.z, t2[y], acc[4 * x + 2][y]);
                            acc[4 * x + 3][y] = fmaf(c.w, t2[y], acc[4 * x + 3][y]);
                        }
                    }
                    t2[0] = t2[1] = t2[2] = t2[3] = 0.f;
                    ++f;
                    load_crow(f);
                }
            }
            t = q > prev ? prod : 0.f;
        }
        __syncwarp();                                // stage s_cur and vs are free for the next round
        o0 = o1; o1 = o2; o2 = o3; o3 = o4; o4 = o5; o5 = o6;
        v0 = v1; v1 = v2; v2 = v3; v3 = v4; v4 = v5; v5 = v6;
        load_ov(o6, v6);
        s_issue = s_cur;
        s_cur = s_cur == 2 ? 0 : s_cur + 1;
    }
    cp_async_wait<0>();
}

__global__ void __launch_bounds__(256, 2)
ttm4_kernel(const sa_item *__restrict__ items, int64_t n_items, int n_group_ctas, ttm4_args a, float *__restrict__ out,
            float *__restrict__ partial)
{
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q = lane >> 3, n8 = lane & 7;
    float *wsm = smem + warp * WARP4;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    const bool group = int(blockIdx.x) < n_group_ctas;
    float acc[R][4];
    sa_item it;
    it.f0 = it.f1 = it.p0 = it.p1 = 0;
    it.dest = -1;
    it.out_row = 0;
    it.pad = 0;
    if (idx < n_items) it = items[idx];
    if (idx < n_items || group) ttm4_warp_item(it, a, wsm, acc);
    // element (l, m = 4q + y, n = 8 nh + n8) of the slice tile
    if (!group) {
        if (idx >= n_items) return;
        float *dst = out + int64_t(it.out_row) * TILE4 + (4 * q) * R + it.pad * NH + n8;
#pragma unroll
        for (int l = 0; l < R; ++l)
#pragma unroll
            for (int y = 0; y < 4; ++y) sa_st_cs(dst + (l * R + y) * R, acc[l][y]);
        return;
    }
    // the CTA's eight warps hold partial half tiles of one slice and one half of n: sum them in a fixed order
    __syncthreads();                                 // every warp is done with its stages
    float *red = smem + warp * HALF_TILE;            // [l][m][n8]
#pragma unroll
    for (int l = 0; l < R; ++l)
#pragma unroll
        for (int y = 0; y < 4; ++y) red[(l * R + 4 * q + y) * NH + n8] = acc[l][y];
    __syncthreads();
    const sa_item lead = items[int64_t(blockIdx.x) * SA_WARPS_PER_CTA];
    float *dst = (lead.dest >= 0 ? partial + int64_t(lead.dest) * TILE4 : out + int64_t(lead.out_row) * TILE4) + lead.pad * NH;
    for (int x = threadIdx.x * 4; x < HALF_TILE; x += 256 * 4) {
        float4 s = *reinterpret_cast<const float4 *>(smem + x);
#pragma unroll
        for (int w = 1; w < SA_WARPS_PER_CTA; ++w) {
            const float4 v = *reinterpret_cast<const float4 *>(smem + w * HALF_TILE + x);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        float *p = dst + (x / NH) * R + (x % NH);    // (l, m) row of 16 floats, this half's 8 columns
        if (lead.dest >= 0) *reinterpret_cast<float4 *>(p) = s;
        else sa_st_cs4(p, s);
    }
}

}  // namespace

bool sa_ranks_ok_ttm4(int64_t L, int64_t M, int64_t N) { return L == R && M == R && N == R; }

size_t sa_ws_ttm4(const sa_tensor *t, const sa_dense *) { return sa_align256(size_t(t->wl_main.n_slots) * TILE4 * sizeof(float)); }

sa_status sa_launch_ttm4(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t, cudaStream_t stream,
                         int *launches)
{
    const sa_worklist &wl = t->wl_main;
    float *partial = static_cast<float *>(ws);
    const int64_t n_items = int64_t(wl.items.size());
    const int64_t n_warp_items = n_items - wl.n_group_ctas * SA_WARPS_PER_CTA;
    const int64_t ctas = wl.n_group_ctas + (n_warp_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
    *launches = 0;
    if (!t->d_crd_endflag) return SA_E_UNSUPPORTED;                  // last dimension >= 2^30
    for (int i = 0; i < 3; ++i)
        if (ops[i].rows * ops[i].ld >= (int64_t(1) << 30)) return SA_E_UNSUPPORTED;   // 32-bit byte offsets of factor rows
    if (ctas > 0) {
        ttm4_args a;
        a.pos2 = t->d_pos[2]; a.crd_j = t->d_crd[1]; a.crd_k = t->d_crd[2]; a.oflag = t->d_crd_endflag; a.vals = t->d_vals;
        a.C = ops[0].ptr; a.D = ops[1].ptr; a.E = ops[2].ptr;
        a.ldc = uint32_t(ops[0].ld); a.ldd = uint32_t(ops[1].ld); a.lde = uint32_t(ops[2].ld);
        constexpr size_t smem = size_t(SA_WARPS_PER_CTA) * WARP4 * sizeof(float);
        if (cudaFuncSetAttribute(ttm4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) return SA_E_CUDA;
        ttm4_kernel<<<(unsigned)ctas, 256, smem, stream>>>(wl.d_items, n_items, int(wl.n_group_ctas), a, out, partial);
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    if (!wl.fix.empty()) {
        if (sa_launch_fixup(wl, partial, out, TILE4, stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}
