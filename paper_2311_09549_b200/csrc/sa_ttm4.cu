// Order-4 analogue of kernel 6:  A(i,l,m,n) = sum_{j,k,o} B(i,j,k,o) C(j,l) D(k,m) E(o,n),
// scheduled with the two-level branched nesting the paper uses for the second schedule of its
// 3-D TTMC kernel (Table of kernels, Section 6; recursive producer/consumer split of Section 4.2):
//   i, j' < T2(m,n) ;  k' < t(n) ; o': t(n) += B E(o,n) , m: T2(m,n) += t(n) D(k,m) > ,
//                      l: A(i,l,m,n) += T2(m,n) C(j,l) >
// Both temporaries (N and M x N floats) and the slice tile live in registers.
#include "sa_device.cuh"

namespace {

constexpr int R = 16;                 // L = M = N = 16
constexpr int TILE4 = R * R * R;      // floats per output slice

// Lane (h, n): h = lane / 16, n = lane % 16.  Half h takes every second nonzero in the producer
// of t, owns m in [8h, 8h+8) of T2 and of the slice tile: acc[l][mm] = A(i, l, 8h+mm, n).
__device__ __forceinline__ void ttm4_warp_item(const sa_item &it, const int32_t *__restrict__ pos2,
                                               const int32_t *__restrict__ pos3, const int32_t *__restrict__ crd_j,
                                               const int32_t *__restrict__ crd_k, const int32_t *__restrict__ crd_o,
                                               const float *__restrict__ vals, const float *__restrict__ C, int64_t ldc,
                                               const float *__restrict__ D, int64_t ldd, const float *__restrict__ E,
                                               int64_t lde, float (&acc)[R][8])
{
    const int lane = threadIdx.x & 31;
    const int h = lane >> 4, n = lane & 15;
#pragma unroll
    for (int l = 0; l < R; ++l)
#pragma unroll
        for (int q = 0; q < 8; ++q) acc[l][q] = 0.f;
    for (int f = it.f0; f < it.f1; ++f) {
        float t2[8];
#pragma unroll
        for (int q = 0; q < 8; ++q) t2[q] = 0.f;
        const int ga = pos2[f], gb = pos2[f + 1];
        for (int g = ga; g < gb; ++g) {
            const int a = pos3[g], b = pos3[g + 1];
            float t = 0.f;
            for (int base = a; base < b; base += 32) {
                const int cnt = min(32, b - base);
                int oo = 0;
                float vv = 0.f;
                if (lane < cnt) { oo = crd_o[base + lane]; vv = vals[base + lane]; }
#pragma unroll 4
                for (int s = 0; s < cnt; s += 2) {
                    const int src = (s + h) & 31;
                    const int o = __shfl_sync(SA_FULL_MASK, oo, src);
                    const float v = __shfl_sync(SA_FULL_MASK, vv, src);
                    t = fmaf(v, __ldg(E + int64_t(o) * lde + n), t);
                }
            }
            t += __shfl_xor_sync(SA_FULL_MASK, t, 16);
            const float *drow = D + int64_t(crd_k[g]) * ldd + h * 8;
            const float4 d0 = sa_ldg4(drow), d1 = sa_ldg4(drow + 4);
            t2[0] = fmaf(d0.x, t, t2[0]); t2[1] = fmaf(d0.y, t, t2[1]);
            t2[2] = fmaf(d0.z, t, t2[2]); t2[3] = fmaf(d0.w, t, t2[3]);
            t2[4] = fmaf(d1.x, t, t2[4]); t2[5] = fmaf(d1.y, t, t2[5]);
            t2[6] = fmaf(d1.z, t, t2[6]); t2[7] = fmaf(d1.w, t, t2[7]);
        }
        const float *crow = C + int64_t(crd_j[f]) * ldc;
#pragma unroll
        for (int l4 = 0; l4 < R; l4 += 4) {
            const float4 c = sa_ldg4(crow + l4);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                acc[l4 + 0][q] = fmaf(c.x, t2[q], acc[l4 + 0][q]);
                acc[l4 + 1][q] = fmaf(c.y, t2[q], acc[l4 + 1][q]);
                acc[l4 + 2][q] = fmaf(c.z, t2[q], acc[l4 + 2][q]);
                acc[l4 + 3][q] = fmaf(c.w, t2[q], acc[l4 + 3][q]);
            }
        }
    }
}

__global__ void __launch_bounds__(256, 1)
ttm4_kernel(const sa_item *__restrict__ items, int64_t n_items, int n_group_ctas, const int32_t *__restrict__ pos2,
            const int32_t *__restrict__ pos3, const int32_t *__restrict__ crd_j, const int32_t *__restrict__ crd_k,
            const int32_t *__restrict__ crd_o, const float *__restrict__ vals, const float *__restrict__ C, int64_t ldc,
            const float *__restrict__ D, int64_t ldd, const float *__restrict__ E, int64_t lde,
            float *__restrict__ out, float *__restrict__ partial)
{
    __shared__ float red[TILE4];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int h = lane >> 4, n = lane & 15;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    const bool group = int(blockIdx.x) < n_group_ctas;
    float acc[R][8];
    sa_item it;
    it.f0 = it.f1 = 0;
    it.dest = -1;
    it.out_row = 0;
    if (idx < n_items) it = items[idx];
    if (idx < n_items || group) ttm4_warp_item(it, pos2, pos3, crd_j, crd_k, crd_o, vals, C, ldc, D, ldd, E, lde, acc);
    // element (l, m = 8h+q, n) of the tile
    const int lane_off = (h * 8) * R + n;
    if (!group) {
        if (idx >= n_items) return;
        float *dst = out + int64_t(it.out_row) * TILE4 + lane_off;
#pragma unroll
        for (int l = 0; l < R; ++l)
#pragma unroll
            for (int q = 0; q < 8; ++q) sa_st_cs(dst + (l * R + q) * R, acc[l][q]);
        return;
    }
    // eight partial tiles of one slice: accumulate warp after warp through one shared tile
    for (int w = 0; w < SA_WARPS_PER_CTA; ++w) {
        if (warp == w) {
#pragma unroll
            for (int l = 0; l < R; ++l)
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    float *p = red + lane_off + (l * R + q) * R;
                    *p = (w == 0 ? 0.f : *p) + acc[l][q];
                }
        }
        __syncthreads();
    }
    const sa_item lead = items[int64_t(blockIdx.x) * SA_WARPS_PER_CTA];
    float *dst = lead.dest >= 0 ? partial + int64_t(lead.dest) * TILE4 : out + int64_t(lead.out_row) * TILE4;
    for (int x = threadIdx.x * 4; x < TILE4; x += 256 * 4) {
        const float4 s = *reinterpret_cast<const float4 *>(red + x);
        if (lead.dest >= 0) *reinterpret_cast<float4 *>(dst + x) = s;
        else sa_st_cs4(dst + x, s);
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
    if (ctas > 0) {
        ttm4_kernel<<<(unsigned)ctas, 256, 0, stream>>>(wl.d_items, n_items, int(wl.n_group_ctas), t->d_pos[2], t->d_pos[3],
                                                        t->d_crd[1], t->d_crd[2], t->d_crd[3], t->d_vals, ops[0].ptr,
                                                        ops[0].ld, ops[1].ptr, ops[1].ld, ops[2].ptr, ops[2].ld, out,
                                                        partial);
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    if (!wl.fix.empty()) {
        if (sa_launch_fixup(wl, partial, out, TILE4, stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}
