// Measurement aid (no counterpart in the paper): how fast can this GPU gather whole rows of a small dense
// table through L2?  The order-3 / order-4 chains read one factor row per nonzero from tables of a few MB
// that stay L2-resident; this kernel issues the same loads (eight lanes per row, one 16-byte read-only load
// per lane, eight rows in flight per lane) with nothing else around them, which gives the ceiling the
// producer stage of those chains can be compared with.
#include "sa_device.cuh"

namespace {

template <int VEC>
__global__ void __launch_bounds__(256)
row_gather_kernel(const float *__restrict__ table, uint32_t ld, const int32_t *__restrict__ idx, int64_t n,
                  float *__restrict__ sink)
{
    const int lane8 = threadIdx.x & 7;
    const int64_t group = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) >> 3;
    const int64_t n_groups = (int64_t(gridDim.x) * blockDim.x) >> 3;
    const float *base = table + lane8 * VEC;
    float acc = 0.f;
    // every 8-lane group walks its own contiguous share of idx, eight rows per iteration
    const int64_t per = (n / n_groups) & ~int64_t(7);
    const int32_t *my = idx + group * per;
    for (int64_t p = 0; p < per; p += 8) {
        const int4 ka = __ldg(reinterpret_cast<const int4 *>(my + p));
        const int4 kb = __ldg(reinterpret_cast<const int4 *>(my + p + 4));
        const int k[8] = {ka.x, ka.y, ka.z, ka.w, kb.x, kb.y, kb.z, kb.w};
#pragma unroll
        for (int s = 0; s < 8; ++s) {
            const float *row = base + uint32_t(k[s]) * ld;
            if (VEC == 4) {
                const float4 v = __ldg(reinterpret_cast<const float4 *>(row));
                acc += v.x + v.y + v.z + v.w;
            } else {
                const float2 v = __ldg(reinterpret_cast<const float2 *>(row));
                acc += v.x + v.y;
            }
        }
    }
    if (acc == 123456.789f) sink[0] = acc;      // keeps the loads alive; practically never true
}

}  // namespace

extern "C" sa_status sa_probe_row_gather(const float *table, int64_t rows, int64_t ld, int row_floats, const int32_t *idx,
                                         int64_t n, float *sink, void *cuda_stream)
{
    if (!table || !idx || !sink || rows <= 0 || n < 0 || ld < row_floats || ld % 4 || rows * ld >= (int64_t(1) << 30)) return SA_E_ARG;
    if (row_floats != 32 && row_floats != 16) return SA_E_UNSUPPORTED;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return SA_E_CUDA; }
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const unsigned grid = unsigned(sms) * 8;     // 8 blocks of 8 warps per SM
    if (row_floats == 32) row_gather_kernel<4><<<grid, 256, 0, stream>>>(table, uint32_t(ld), idx, n, sink);
    else row_gather_kernel<2><<<grid, 256, 0, stream>>>(table, uint32_t(ld), idx, n, sink);
    if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;
    return SA_OK;
}
