// Kernel 1 <SDDMM,SpMM>:  A(i,l) = sum_j B(i,j) (sum_k C(i,k) D(j,k)) E(j,l), scheduled as the
// fused nest  i, j' < t ; k: t += B(i,j) C(i,k) D(j,k) , l: A(i,l) += t E(j,l) >  of the paper's
// Table of kernels (Section 6): the sampled value is a scalar temporary that is consumed at once,
// the sampled matrix is never written (auxiliary memory 1 in the paper's memory table).
#include "sa_device.cuh"

namespace {

// One warp per work item; a lane owns KV = K/32 consecutive k and LV = L/32 consecutive l.
template <int KV, int LV>
__global__ void __launch_bounds__(256)
sddmm_spmm_kernel(const sa_item *__restrict__ items, int64_t n_items, const int32_t *__restrict__ pos,
                  const int32_t *__restrict__ crd, const float *__restrict__ vals, const float *__restrict__ C,
                  int64_t ldc, const float *__restrict__ D, int64_t ldd, const float *__restrict__ E, int64_t lde,
                  float *__restrict__ out, float *__restrict__ partial, float *__restrict__ sampled)
{
    constexpr int L = LV * 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    if (idx >= n_items) return;
    const sa_item it = items[idx];
    for (int r = it.out_row; r < it.row_end; ++r) {
        const int a = it.dest >= 0 ? it.p0 : pos[r];
        const int b = it.dest >= 0 ? it.p1 : pos[r + 1];
        float c[KV], acc[LV];
#pragma unroll
        for (int q = 0; q < LV; ++q) acc[q] = 0.f;
        if (b > a) {
#pragma unroll
            for (int q = 0; q < KV; ++q) c[q] = __ldg(C + int64_t(r) * ldc + lane * KV + q);
        }
        for (int base = a; base < b; base += 32) {
            const int n = min(32, b - base);
            int jj = 0;
            float vv = 0.f;
            if (lane < n) { jj = crd[base + lane]; vv = vals[base + lane]; }
#pragma unroll 4
            for (int s = 0; s < n; ++s) {
                const int j = __shfl_sync(SA_FULL_MASK, jj, s);
                const float v = __shfl_sync(SA_FULL_MASK, vv, s);
                const float *drow = D + int64_t(j) * ldd + lane * KV;
                const float *erow = E + int64_t(j) * lde + lane * LV;
                float d[KV], e[LV];
                if (KV == 4) { const float4 x = sa_ldg4(drow); d[0] = x.x; d[1] = x.y; d[2 % KV] = x.z; d[3 % KV] = x.w; }
                else if (KV == 2) { const float2 x = sa_ldg2(drow); d[0] = x.x; d[1 % KV] = x.y; }
                else d[0] = __ldg(drow);
                if (LV == 4) { const float4 x = sa_ldg4(erow); e[0] = x.x; e[1] = x.y; e[2 % LV] = x.z; e[3 % LV] = x.w; }
                else if (LV == 2) { const float2 x = sa_ldg2(erow); e[0] = x.x; e[1 % LV] = x.y; }
                else e[0] = __ldg(erow);
                float dot = 0.f;
#pragma unroll
                for (int q = 0; q < KV; ++q) dot = fmaf(c[q], d[q], dot);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(SA_FULL_MASK, dot, o);
                const float sc = v * dot;
                if (sampled != nullptr && lane == 0) sampled[base + s] = sc;
#pragma unroll
                for (int q = 0; q < LV; ++q) acc[q] = fmaf(sc, e[q], acc[q]);
            }
        }
        float *dst = it.dest >= 0 ? partial + int64_t(it.dest) * L : out + int64_t(r) * L;
#pragma unroll
        for (int q = 0; q < LV; ++q) dst[lane * LV + q] = acc[q];
    }
}

template <int KV, int LV>
cudaError_t launch(const sa_tensor *t, const sa_dense *ops, float *out, float *partial, float *sampled,
                   cudaStream_t stream)
{
    const sa_worklist &wl = t->wl_main;
    const int64_t n_items = int64_t(wl.items.size());
    const int64_t ctas = (n_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
    if (ctas == 0) return cudaSuccess;
    sddmm_spmm_kernel<KV, LV><<<(unsigned)ctas, 256, 0, stream>>>(wl.d_items, n_items, t->d_pos[1], t->d_crd[1], t->d_vals,
                                                                 ops[0].ptr, ops[0].ld, ops[1].ptr, ops[1].ld, ops[2].ptr,
                                                                 ops[2].ld, out, partial, sampled);
    return cudaGetLastError();
}

bool rank_ok(int64_t r) { return r == 32 || r == 64 || r == 128; }

}  // namespace

bool sa_ranks_ok_sddmm(int64_t K, int64_t L) { return rank_ok(K) && rank_ok(L); }

// workspace: [partial rows of long-row pieces][sampled values, nnz floats, debug schedule only]
size_t sa_ws_sddmm_spmm(const sa_tensor *t, const sa_dense *ops, bool materialize)
{
    size_t b = sa_align256(size_t(t->wl_main.n_slots) * size_t(ops[2].cols) * sizeof(float));
    if (materialize) b += sa_align256(size_t(t->nnz) * sizeof(float));
    return b;
}

sa_status sa_launch_sddmm_spmm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t, bool materialize,
                               cudaStream_t stream, int *launches)
{
    const int64_t K = ops[0].cols, L = ops[2].cols;
    float *partial = static_cast<float *>(ws);
    float *sampled = nullptr;
    if (materialize)
        sampled = reinterpret_cast<float *>(static_cast<char *>(ws) + sa_align256(size_t(t->wl_main.n_slots) * size_t(L) * sizeof(float)));
    cudaError_t e = cudaErrorInvalidValue;
    const int kv = int(K / 32), lv = int(L / 32);
#define SA_CASE(a, b) if (kv == a && lv == b) e = launch<a, b>(t, ops, out, partial, sampled, stream);
    SA_CASE(1, 1) SA_CASE(1, 2) SA_CASE(1, 4) SA_CASE(2, 1) SA_CASE(2, 2) SA_CASE(2, 4) SA_CASE(4, 1) SA_CASE(4, 2) SA_CASE(4, 4)
#undef SA_CASE
    if (e != cudaSuccess) return SA_E_CUDA;
    *launches = t->wl_main.items.empty() ? 0 : 1;
    if (!t->wl_main.fix.empty()) {
        if (sa_launch_fixup(t->wl_main, partial, out, int(L), stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}
