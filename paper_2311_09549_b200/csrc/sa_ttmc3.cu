// Kernel 5 <3D TTMC>:  A(l,m,n) = sum_{i,j,k} B(i,j,k) C(i,l) D(j,m) E(k,n)  (the running example of
// the paper, Sections 1 and 3; chosen schedules in the Table of kernels, Section 6).  Evaluated as
//   T(i,m,n) = sum_j D(j,m) ( sum_k B(i,j,k) E(k,n) )        per slice, the branched nest of kernel 6
//   A(l,m,n) = sum_i C(i,l) T(i,m,n)                         contraction over the slices
// in two schedules:
//   SA_SCHED_FUSED      the paper's second schedule for this kernel with its temporaries widened to
//     vectors: i < T(m,n) ; j' < t(n) ; k': t += B E , m: T += t D > , l: A += T C >.  The slice
//     temporary stays on chip; every thread block keeps its own L x M x N accumulator in shared
//     memory (sa_ttm3.cu, ttmc3_fused_kernel) and the blocks' accumulators are added in block order.
//     Additions inside a block are shared-memory atomics: their order, and with it the last bits of
//     the result, may differ from run to run.
//   SA_SCHED_FISSIONED  the loop over i is fissioned from the l loop: the slice temporaries T(i,:,:)
//     (I x M x N floats, in the workspace) are written by the slice kernel of kernel 6 and reduced
//     over i by a small dense kernel (fixed chunks of slices, partial sums added in chunk order:
//     bitwise reproducible).  A temporary of three dimensions is what Stage 1 of the paper's
//     auto-scheduler prunes; it is kept as the reproducible alternative and for rank combinations
//     whose accumulator does not fit shared memory.
#include <algorithm>

#include "sa_device.cuh"

namespace {

constexpr int TTMC_MAX_CHUNKS = 512;

// P(c, l, col) = sum over the slices i of chunk c of C(i,l) * T(i,col).  One thread per column.
template <int L>
__global__ void __launch_bounds__(256)
ttmc3_partial_kernel(int64_t I, int chunk, int cols, const float *__restrict__ T, const float *__restrict__ C,
                     uint32_t ldc, float *__restrict__ P)
{
    const int col = blockIdx.x * 256 + threadIdx.x;
    const int64_t i0 = int64_t(blockIdx.y) * chunk, i1 = min(I, i0 + chunk);
    float acc[L];
#pragma unroll
    for (int l = 0; l < L; ++l) acc[l] = 0.f;
    if (col < cols) {
        for (int64_t i = i0; i < i1; ++i) {
            const float t = __ldcs(T + i * cols + col);
            const float *crow = C + i * ldc;
#pragma unroll
            for (int l = 0; l < L; l += 4) {
                const float4 c = sa_ldg4(crow + l);
                acc[l + 0] = fmaf(c.x, t, acc[l + 0]);
                acc[l + 1] = fmaf(c.y, t, acc[l + 1]);
                acc[l + 2] = fmaf(c.z, t, acc[l + 2]);
                acc[l + 3] = fmaf(c.w, t, acc[l + 3]);
            }
        }
        float *dst = P + (int64_t(blockIdx.y) * L) * cols + col;
#pragma unroll
        for (int l = 0; l < L; ++l) dst[int64_t(l) * cols] = acc[l];
    }
}

// A(x) = sum over chunks c of P(c, x), x = l * cols + col, in chunk order.
__global__ void __launch_bounds__(256)
ttmc3_final_kernel(int n_chunks, int64_t n_out, const float *__restrict__ P, float *__restrict__ A)
{
    const int64_t x = int64_t(blockIdx.x) * 256 + threadIdx.x;
    if (x >= n_out) return;
    float s = 0.f;
    for (int c = 0; c < n_chunks; ++c) s += P[int64_t(c) * n_out + x];
    A[x] = s;
}

struct ttmc3_plan {
    int chunk, n_chunks;
    size_t t_bytes, ttm3_bytes, p_bytes;
};

ttmc3_plan plan(const sa_tensor *t, const sa_dense *ops)
{
    ttmc3_plan p;
    const int64_t I = t->dims[0], L = ops[0].cols, cols = ops[1].cols * ops[2].cols;
    p.chunk = int(std::max<int64_t>(64, (I + TTMC_MAX_CHUNKS - 1) / TTMC_MAX_CHUNKS));
    p.n_chunks = int((I + p.chunk - 1) / p.chunk);
    p.t_bytes = sa_align256(size_t(I) * size_t(cols) * sizeof(float));
    p.ttm3_bytes = sa_ws_ttm3(t, ops + 1);
    p.p_bytes = sa_align256(size_t(p.n_chunks) * size_t(L) * size_t(cols) * sizeof(float));
    return p;
}

}  // namespace

bool sa_ranks_ok_ttmc3(int64_t L, int64_t M, int64_t N) { return (L == 16 || L == 32) && sa_ranks_ok_ttm3(M, N); }

// workspace, fissioned: [T: I x M x N][partial tiles of the slice kernel][P: chunks x L x M x N]
//            fused:     [accumulators of the blocks: blocks x L x M x N]
size_t sa_ws_ttmc3(const sa_tensor *t, const sa_dense *ops, bool fissioned)
{
    if (!fissioned) return sa_ws_ttmc3_fused(ops[0].cols, ops[1].cols, ops[2].cols);
    const ttmc3_plan p = plan(t, ops);
    return p.t_bytes + p.ttm3_bytes + p.p_bytes;
}

sa_status sa_launch_ttmc3(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t, bool fissioned,
                          cudaStream_t stream, int *launches)
{
    const int64_t I = t->dims[0], L = ops[0].cols;
    const int cols = int(ops[1].cols * ops[2].cols);
    if (ops[0].rows * ops[0].ld >= (int64_t(1) << 30)) return SA_E_UNSUPPORTED;
    if (!fissioned) {
        float *partials = static_cast<float *>(ws);
        int n_blocks = 0;
        const sa_status s = sa_launch_ttmc3_fused_stage(t, ops[0], ops[1], ops[2], partials, stream, &n_blocks);
        if (s != SA_OK) return s;
        const int64_t n_out = L * cols;
        // n_blocks == 0 (a tensor without nonzeros): the sum over no accumulators writes zeros
        ttmc3_final_kernel<<<(unsigned)((n_out + 255) / 256), 256, 0, stream>>>(n_blocks, n_out, partials, out);
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
        *launches = (n_blocks > 0 ? 1 : 0) + 1;
        return SA_OK;
    }
    const ttmc3_plan p = plan(t, ops);
    char *base = static_cast<char *>(ws);
    float *T = reinterpret_cast<float *>(base);
    void *ws3 = base + p.t_bytes;
    float *P = reinterpret_cast<float *>(base + p.t_bytes + p.ttm3_bytes);
    int n3 = 0;
    const sa_status s = sa_launch_ttm3(t, ops + 1, T, ws3, p.ttm3_bytes, stream, &n3);   // T(i,m,n), empty slices zero
    if (s != SA_OK) return s;
    *launches = n3;
    dim3 grid((unsigned)((cols + 255) / 256), (unsigned)p.n_chunks);
    if (L == 16) ttmc3_partial_kernel<16><<<grid, 256, 0, stream>>>(I, p.chunk, cols, T, ops[0].ptr, uint32_t(ops[0].ld), P);
    else ttmc3_partial_kernel<32><<<grid, 256, 0, stream>>>(I, p.chunk, cols, T, ops[0].ptr, uint32_t(ops[0].ld), P);
    if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
    const int64_t n_out = L * cols;
    ttmc3_final_kernel<<<(unsigned)((n_out + 255) / 256), 256, 0, stream>>>(p.n_chunks, n_out, P, out);
    if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
    *launches += 2;
    return SA_OK;
}
