// Measurement aid for bench.py (no counterpart in the paper, not part of libsparseauto.so): how fast can this GPU
// gather whole rows of a small dense table through L2?  The order-3 / order-4 chains read one factor row per
// nonzero from tables of a few MB that stay L2-resident; these kernels issue the same kind of loads with nothing
// else around them, in several shapes, so that the producer stage of those chains can be compared with the best
// bare gather:
//   lanes per row    4 or 8  (a row of 32 floats is 8 lanes x 16 bytes or 4 lanes x 32 bytes)
//   rows in flight   4, 8 or 16 per lane group (independent loads issued before the first is used)
//   blocks per SM    chosen by the caller through the grid size
// Every lane group walks its own contiguous share of the index array, like a stream of the real kernels.
#include <cuda_runtime.h>
#include <cstdint>

namespace {

template <int ROWF, int LPR, int INFLIGHT>
__global__ void __launch_bounds__(256)
row_gather_kernel(const float *__restrict__ table, uint32_t ld, const int32_t *__restrict__ idx, int64_t n,
                  float *__restrict__ sink)
{
    constexpr int FPL = ROWF / LPR;                 // floats per lane: 2, 4 or 8
    const int sub = threadIdx.x % LPR;
    const int64_t group = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) / LPR;
    const int64_t n_groups = (int64_t(gridDim.x) * blockDim.x) / LPR;
    const float *base = table + sub * FPL;
    float acc = 0.f;
    const int64_t per = (n / n_groups) / INFLIGHT * INFLIGHT;
    const int32_t *my = idx + group * per;
    for (int64_t p = 0; p < per; p += INFLIGHT) {
        int k[INFLIGHT];
#pragma unroll
        for (int s = 0; s < INFLIGHT; s += 4) {
            const int4 w = __ldg(reinterpret_cast<const int4 *>(my + p + s));
            k[s] = w.x; k[s + 1] = w.y; k[s + 2] = w.z; k[s + 3] = w.w;
        }
        float4 v[INFLIGHT][FPL >= 4 ? FPL / 4 : 1];
#pragma unroll
        for (int s = 0; s < INFLIGHT; ++s) {
            const float *row = base + uint32_t(k[s]) * ld;
            if (FPL >= 4) {
#pragma unroll
                for (int x = 0; x < FPL / 4; ++x) v[s][x] = __ldg(reinterpret_cast<const float4 *>(row) + x);
            } else {
                const float2 t = __ldg(reinterpret_cast<const float2 *>(row));
                v[s][0] = make_float4(t.x, t.y, 0.f, 0.f);
            }
        }
#pragma unroll
        for (int s = 0; s < INFLIGHT; ++s)
#pragma unroll
            for (int x = 0; x < (FPL >= 4 ? FPL / 4 : 1); ++x) acc += v[s][x].x + v[s][x].y + v[s][x].z + v[s][x].w;
    }
    if (acc == 123456.789f) sink[0] = acc;      // keeps the loads alive; practically never true
}

template <int ROWF, int LPR>
cudaError_t launch(int inflight, unsigned grid, const float *table, uint32_t ld, const int32_t *idx, int64_t n, float *sink,
                   cudaStream_t stream)
{
    if (inflight == 4) row_gather_kernel<ROWF, LPR, 4><<<grid, 256, 0, stream>>>(table, ld, idx, n, sink);
    else if (inflight == 8) row_gather_kernel<ROWF, LPR, 8><<<grid, 256, 0, stream>>>(table, ld, idx, n, sink);
    else if (inflight == 16) row_gather_kernel<ROWF, LPR, 16><<<grid, 256, 0, stream>>>(table, ld, idx, n, sink);
    else return cudaErrorInvalidValue;
    return cudaGetLastError();
}

}  // namespace

// Gather `n` rows of `row_floats` (16 or 32) floats of the device table (rows x ld, row-major) named by the device
// index array idx (values in [0, rows)), with `lanes_per_row` (4 or 8) lanes per row, `inflight` (4, 8, 16) rows in
// flight per lane group and `blocks_per_sm` blocks of 256 threads per SM.  Asynchronous on `cuda_stream`.
// Returns 0, or a non-zero code for an unsupported shape or a launch error.
extern "C" int sa_probe_row_gather(const float *table, int64_t rows, int64_t ld, int row_floats, const int32_t *idx, int64_t n,
                                   float *sink, int lanes_per_row, int inflight, int blocks_per_sm, void *cuda_stream)
{
    if (!table || !idx || !sink || rows <= 0 || n < 0 || ld < row_floats || ld % 4 || rows * ld >= (int64_t(1) << 30)) return 1;
    if (blocks_per_sm < 1 || blocks_per_sm > 32) return 1;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 2; }
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const unsigned grid = unsigned(sms) * unsigned(blocks_per_sm);
    cudaError_t e = cudaErrorInvalidValue;
    if (row_floats == 32 && lanes_per_row == 8) e = launch<32, 8>(inflight, grid, table, uint32_t(ld), idx, n, sink, stream);
    else if (row_floats == 32 && lanes_per_row == 4) e = launch<32, 4>(inflight, grid, table, uint32_t(ld), idx, n, sink, stream);
    else if (row_floats == 16 && lanes_per_row == 8) e = launch<16, 8>(inflight, grid, table, uint32_t(ld), idx, n, sink, stream);
    else if (row_floats == 16 && lanes_per_row == 4) e = launch<16, 4>(inflight, grid, table, uint32_t(ld), idx, n, sink, stream);
    if (e != cudaSuccess) { cudaGetLastError(); return 2; }
    return 0;
}
