// Kernel 6 <SpTTM,TTM>:  A(i,l,m) = sum_{j,k} B(i,j,k) C(j,l) D(k,m), scheduled as the branched
// nest  i, j' < t ; k': t += B(i,j,k) D(k,m) , l: A(i,l,m) += t C(j,l) >  of the paper's Table of
// kernels (Section 6): per fiber (i,j) the SpTTM producer fills a temporary of M floats held in
// registers (one lane per m), then the consumer adds the rank-1 update C(j,:)^T x temporary into
// the slice's L x M tile, also held in registers.  The sampled order-3 intermediate
// T(i,j,m) is never stored.
#include "sa_device.cuh"

namespace {

// One warp evaluates one work item: fibers [f0,f1) of a slice clipped to nonzeros [p0,p1).
// Lane layout: G = 32/M lane groups; group h takes every G-th nonzero of a fiber and, in the
// consumer stage, the l range [h*L/G, (h+1)*L/G).  acc[ll] = A(i, h*L/G + ll, m).
template <int L, int M>
__device__ __forceinline__ void ttm3_warp_item(const sa_item &it, const int32_t *__restrict__ pos2,
                                               const int32_t *__restrict__ crd_j, const int32_t *__restrict__ crd_k,
                                               const float *__restrict__ vals, const float *__restrict__ C, int64_t ldc,
                                               const float *__restrict__ D, int64_t ldd, float (&acc)[L * M / 32])
{
    constexpr int G = 32 / M;
    constexpr int LPG = L / G;
    const int lane = threadIdx.x & 31;
    const int h = lane / M, m = lane % M;
#pragma unroll
    for (int q = 0; q < LPG; ++q) acc[q] = 0.f;
    for (int f = it.f0; f < it.f1; ++f) {
        const int a = max(pos2[f], it.p0), b = min(pos2[f + 1], it.p1);
        float t = 0.f;
        for (int base = a; base < b; base += 32) {
            const int n = min(32, b - base);
            int kk = 0;
            float vv = 0.f;
            if (lane < n) { kk = crd_k[base + lane]; vv = vals[base + lane]; }
#pragma unroll 4
            for (int s = 0; s < n; s += G) {
                const int src = (s + h) & 31;
                const int k = __shfl_sync(SA_FULL_MASK, kk, src);
                const float v = __shfl_sync(SA_FULL_MASK, vv, src);
                t = fmaf(v, __ldg(D + int64_t(k) * ldd + m), t);
            }
        }
        if (G == 2) t += __shfl_xor_sync(SA_FULL_MASK, t, 16);
        const float *crow = C + int64_t(crd_j[f]) * ldc + h * LPG;
#pragma unroll
        for (int q = 0; q < LPG; q += 4) {
            const float4 c = sa_ldg4(crow + q);
            acc[q + 0] = fmaf(c.x, t, acc[q + 0]);
            acc[q + 1] = fmaf(c.y, t, acc[q + 1]);
            acc[q + 2] = fmaf(c.z, t, acc[q + 2]);
            acc[q + 3] = fmaf(c.w, t, acc[q + 3]);
        }
    }
}

template <int L, int M>
__global__ void __launch_bounds__(256)
ttm3_kernel(const sa_item *__restrict__ items, int64_t n_items, int n_group_ctas, const int32_t *__restrict__ pos2,
            const int32_t *__restrict__ crd_j, const int32_t *__restrict__ crd_k, const float *__restrict__ vals,
            const float *__restrict__ C, int64_t ldc, const float *__restrict__ D, int64_t ldd,
            float *__restrict__ out, float *__restrict__ partial)
{
    constexpr int G = 32 / M;
    constexpr int LPG = L / G;
    constexpr int TILE = L * M;
    __shared__ float red[SA_WARPS_PER_CTA * TILE];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int h = lane / M, m = lane % M;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    const bool group = int(blockIdx.x) < n_group_ctas;
    float acc[LPG];
    sa_item it;
    it.f0 = it.f1 = 0;
    it.dest = -1;
    it.out_row = 0;
    if (idx < n_items) it = items[idx];
    if (idx < n_items || group) ttm3_warp_item<L, M>(it, pos2, crd_j, crd_k, vals, C, ldc, D, ldd, acc);
    if (!group) {
        if (idx >= n_items) return;
        float *dst = out + int64_t(it.out_row) * TILE + h * LPG * M + m;
#pragma unroll
        for (int q = 0; q < LPG; ++q) sa_st_cs(dst + q * M, acc[q]);
        return;
    }
    // the CTA's eight warps hold partial tiles of the same slice: sum them in a fixed order
#pragma unroll
    for (int q = 0; q < LPG; ++q) red[warp * TILE + (h * LPG + q) * M + m] = acc[q];
    __syncthreads();
    const sa_item lead = items[int64_t(blockIdx.x) * SA_WARPS_PER_CTA];
    float *dst = lead.dest >= 0 ? partial + int64_t(lead.dest) * TILE : out + int64_t(lead.out_row) * TILE;
    for (int x = threadIdx.x * 4; x < TILE; x += 256 * 4) {
        float4 s = *reinterpret_cast<const float4 *>(red + x);
#pragma unroll
        for (int w = 1; w < SA_WARPS_PER_CTA; ++w) {
            const float4 v = *reinterpret_cast<const float4 *>(red + w * TILE + x);
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
    ttm3_kernel<L, M><<<(unsigned)ctas, 256, 0, stream>>>(wl.d_items, n_items, int(wl.n_group_ctas), t->d_pos[2],
                                                         t->d_crd[1], t->d_crd[2], t->d_vals, ops[0].ptr, ops[0].ld,
                                                         ops[1].ptr, ops[1].ld, out, partial);
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
