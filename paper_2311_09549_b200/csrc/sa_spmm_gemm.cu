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

template <int L, int M>
__global__ void __launch_bounds__(256)
spmm_gemm_left_kernel(const sa_item *__restrict__ items, int64_t n_items, const int32_t *__restrict__ pos,
                      const int32_t *__restrict__ crd, const float *__restrict__ vals, const float *__restrict__ C,
                      int64_t ldc, const float *__restrict__ D, int64_t ldd, float *__restrict__ out,
                      float *__restrict__ partial)
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
            const int a = it.dest >= 0 ? it.p0 : pos[r];
            const int b = it.dest >= 0 ? it.p1 : pos[r + 1];
            float4 t[LV4];
#pragma unroll
            for (int q = 0; q < LV4; ++q) t[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            for (int base = a; base < b; base += 32) {
                const int n = min(32, b - base);
                int jj = 0;
                float vv = 0.f;
                if (lane < n) { jj = crd[base + lane]; vv = vals[base + lane]; }
#pragma unroll 4
                for (int s = 0; s < n; ++s) {
                    const int j = __shfl_sync(SA_FULL_MASK, jj, s);
                    const float v = __shfl_sync(SA_FULL_MASK, vv, s);
                    const float *crow = C + int64_t(j) * ldc + lane * 4;
#pragma unroll
                    for (int q = 0; q < LV4; ++q) {
                        const float4 c = sa_ldg4(crow + q * 128);
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

// E(j,:) = C(j,:) . D for all J rows; one warp per row, grid-stride.
template <int L, int M>
__global__ void __launch_bounds__(256)
gemm_rows_kernel(int64_t J, const float *__restrict__ C, int64_t ldc, const float *__restrict__ D, int64_t ldd,
                 float *__restrict__ Eout)
{
    constexpr int LV4 = L / 128, MV = M / 32;
    extern __shared__ __align__(16) float smem[];
    float *Ds = smem;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float *Ts = smem + L * M + warp * L;
    load_D<L, M>(Ds, D, ldd);
    __syncthreads();
    for (int64_t j = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp; j < J; j += int64_t(gridDim.x) * SA_WARPS_PER_CTA) {
        const float *crow = C + j * ldc + lane * 4;
#pragma unroll
        for (int q = 0; q < LV4; ++q)
            *reinterpret_cast<float4 *>(Ts + q * 128 + lane * 4) = __ldcs(reinterpret_cast<const float4 *>(crow + q * 128));
        __syncwarp();
        float o[MV];
        row_times_D<L, M>(Ts, Ds, lane, o);
        __syncwarp();
#pragma unroll
        for (int q = 0; q < MV; ++q) Eout[j * M + q * 32 + lane] = o[q];
    }
}

// A = B . E (the CSR SpMM nest of Fig. 1b); lane owns MV = M/32 consecutive columns.
template <int MV>
__global__ void __launch_bounds__(256)
spmm_kernel(const sa_item *__restrict__ items, int64_t n_items, const int32_t *__restrict__ pos,
            const int32_t *__restrict__ crd, const float *__restrict__ vals, const float *__restrict__ E,
            float *__restrict__ out, float *__restrict__ partial)
{
    constexpr int M = MV * 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    if (idx >= n_items) return;
    const sa_item it = items[idx];
    for (int r = it.out_row; r < it.row_end; ++r) {
        const int a = it.dest >= 0 ? it.p0 : pos[r];
        const int b = it.dest >= 0 ? it.p1 : pos[r + 1];
        float acc[MV];
#pragma unroll
        for (int q = 0; q < MV; ++q) acc[q] = 0.f;
        for (int base = a; base < b; base += 32) {
            const int n = min(32, b - base);
            int jj = 0;
            float vv = 0.f;
            if (lane < n) { jj = crd[base + lane]; vv = vals[base + lane]; }
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
        auto kern = spmm_gemm_left_kernel<L, M>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) return SA_E_CUDA;
        const int64_t want = (n_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
        const int64_t ctas = std::min<int64_t>(want, resident_ctas(reinterpret_cast<const void *>(kern), smem));
        if (ctas > 0) {
            kern<<<(unsigned)ctas, 256, smem, stream>>>(wl.d_items, n_items, t->d_pos[1], t->d_crd[1], t->d_vals, ops[0].ptr,
                                                       ops[0].ld, ops[1].ptr, ops[1].ld, out, partial);
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
    auto gk = gemm_rows_kernel<L, M>;
    if (cudaFuncSetAttribute(gk, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) return SA_E_CUDA;
    const int64_t gctas = std::min<int64_t>((J + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA,
                                            resident_ctas(reinterpret_cast<const void *>(gk), smem));
    gk<<<(unsigned)gctas, 256, smem, stream>>>(J, ops[0].ptr, ops[0].ld, ops[1].ptr, ops[1].ld, E);
    if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
    *launches += 1;
    const int64_t ctas = (n_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
    if (ctas > 0) {
        spmm_kernel<M / 32><<<(unsigned)ctas, 256, 0, stream>>>(wl.d_items, n_items, t->d_pos[1], t->d_crd[1], t->d_vals, E,
                                                               out, partial);
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    if (!wl.fix.empty()) {
        if (sa_launch_fixup(wl, partial, out, M, stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}

}  // namespace

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
