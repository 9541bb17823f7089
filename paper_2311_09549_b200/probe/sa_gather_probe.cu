// Measurement aid for bench.py (no counterpart in the paper, not part of libsparseauto.so): how fast can this GPU
// gather whole rows of a small dense table through L2?  The order-3 / order-4 chains read one factor row per
// nonzero from tables of a few MB that stay L2-resident; these kernels issue the same kind of loads with nothing
// else around them, in several shapes, so that the producer stage of those chains can be compared with the best
// bare gather:
//   lanes per row    4 or 8  (a row of 32 floats is 8 lanes x 16 bytes or 4 lanes x 32 bytes)
//   rows in flight   4, 8 or 16 per lane group (independent loads issued before the first is used)
//   blocks per SM    chosen by the caller through the grid size
// Every lane group walks its own contiguous share of the index array, like a stream of the real kernels.
//
// A second family fetches the same rows with the copy engine instead of the load/store units: one
// cp.async.bulk.tensor (tile::gather4) instruction names four row indices and lands the four rows in shared memory,
// completion is counted by an mbarrier.  A warp keeps `stages` groups of sixteen rows in flight (four issuing lanes
// x four rows) and reads every landed row back with 16-byte shared-memory loads, as a consumer would.
#include <cuda.h>
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

// ---------------------------------------------------------------- rows fetched by the copy engine

__device__ __forceinline__ uint32_t smem_addr(const void *p) { return uint32_t(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Waits for the phase with the given parity, for at most 20 ms; on giving up writes `code` to *status (first writer
// wins) and returns false, so that a copy that never completes ends the kernel instead of hanging it.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, int32_t *status, int32_t code)
{
    unsigned long long t0 = 0;
    for (uint32_t tries = 0;; ++tries) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((tries & 63u) == 63u) {
            unsigned long long now;
            asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(now));
            if (t0 == 0) t0 = now;
            else if (now - t0 > 20000000ull) break;
        }
    }
    atomicCAS(status, 0, code);
    return false;
}
// Four rows r0 .. r3 of the 2-D tensor behind `tm`, from column 0, to 4 x (box width) contiguous bytes at dst.
__device__ __forceinline__ void tma_gather4(uint32_t dst, const CUtensorMap *tm, int r0, int r1, int r2, int r3, uint32_t bar)
{
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(dst), "l"(tm), "r"(0), "r"(r0), "r"(r1), "r"(r2), "r"(r3), "r"(bar) : "memory");
}

constexpr int TMA_WARPS = 4;           // warps per block, each with its own ring and barriers
constexpr int TMA_MAX_STAGES = 8;

template <int ROWF>
__global__ void __launch_bounds__(32 * TMA_WARPS)
tma_gather_kernel(const __grid_constant__ CUtensorMap tm, const int32_t *__restrict__ idx, int64_t n, int stages,
                  float *__restrict__ sink, int32_t *__restrict__ status)
{
    constexpr uint32_t ROW_BYTES = ROWF * 4, STAGE_BYTES = 16 * ROW_BYTES;      // sixteen rows per stage
    extern __shared__ __align__(1024) unsigned char smem[];
    __shared__ __align__(8) unsigned long long bars[TMA_WARPS][TMA_MAX_STAGES];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, q = lane >> 3;
    const bool issuer = (lane & 7) == 0;
    const uint32_t ring = smem_addr(smem) + uint32_t(warp) * uint32_t(stages) * STAGE_BYTES;
    const uint32_t bar0 = smem_addr(&bars[warp][0]);
    if (lane == 0)
        for (int s = 0; s < stages; ++s) mbar_init(bar0 + 8 * s, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    __syncthreads();
    const int64_t n_warps = int64_t(gridDim.x) * TMA_WARPS, gw = int64_t(blockIdx.x) * TMA_WARPS + warp;
    const int64_t iters = (n / n_warps) / 16;
    const int32_t *my = idx + gw * iters * 16;
    // The four indices an issuing lane needs per group are loaded a chunk of eight groups ahead, so that their
    // latency (they stream from HBM) is not part of the loop.
    constexpr int PF = 8;
    int4 kc[PF], kn[PF];
    auto load_chunk = [&](int4 (&k)[PF], int64_t chunk) {
#pragma unroll
        for (int j = 0; j < PF; ++j) {
            k[j] = make_int4(0, 0, 0, 0);
            if (issuer && chunk * PF + j < iters) k[j] = __ldg(reinterpret_cast<const int4 *>(my + (chunk * PF + j) * 16 + 4 * q));
        }
    };
    load_chunk(kc, 0);
    int64_t issued = 0, waited = 0;
    float acc = 0.f;
    bool ok = true;
    for (int64_t chunk = 0; ok && chunk * PF < iters + stages; ++chunk) {
        load_chunk(kn, chunk + 1);
#pragma unroll
        for (int j = 0; j < PF; ++j) {
            const int64_t it = chunk * PF + j, c = it - stages;      // group to issue, group to consume (same ring slot)
            const int s = int(it % stages);
            const uint32_t bar = bar0 + 8 * s;
            if (ok && c >= 0 && c < iters) {
                ok = mbar_wait_bounded(bar, uint32_t(c / stages) & 1u, status, 1);
                ok = __all_sync(0xffffffffu, ok);
                ++waited;
                if (ok) {
#pragma unroll
                    for (uint32_t off = 0; off < STAGE_BYTES; off += 512) {
                        float4 v;
                        asm volatile("ld.shared.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                                     : "r"(ring + s * STAGE_BYTES + off + 16 * lane) : "memory");
                        acc += v.x + v.y + v.z + v.w;
                    }
                }
                __syncwarp();           // every lane has read the slot before it is filled again
            }
            if (ok && it < iters) {
                if (lane == 0) mbar_arrive_expect_tx(bar, STAGE_BYTES);
                __syncwarp();
                if (issuer) tma_gather4(ring + s * STAGE_BYTES + q * 4 * ROW_BYTES, &tm, kc[j].x, kc[j].y, kc[j].z, kc[j].w, bar);
                ++issued;
            }
        }
#pragma unroll
        for (int j = 0; j < PF; ++j) kc[j] = kn[j];
    }
    // after a wait that gave up: give the copies still in flight the same bounded time before the block ends
    for (; waited < issued; ++waited) mbar_wait_bounded(bar0 + 8 * int(waited % stages), uint32_t(waited / stages) & 1u, status, 2);
    // the sum of everything read goes to sink[1], so that the caller can check that the right rows arrived
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) atomicAdd(sink + 1, acc);
}

typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                    const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                    CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

// The same gather through the copy engine: `stages` (1 .. 8) groups of sixteen rows in flight per warp, blocks of four
// warps, `blocks_per_sm` blocks per SM.  `status` is a device int32 that must be zero on entry; the kernel sets it to a
// non-zero code if a wait for landed rows gave up (after 20 ms), and ends.  The sum of all elements of the rows read (the
// first 16 * floor(n / (16 * warps)) * warps indices) is added to sink[1].  Returns 0, 1 (argument), 2 (CUDA error) or
// 3 (the driver has no tensor-map encoder or refused the map).
extern "C" int sa_probe_tma_gather(const float *table, int64_t rows, int64_t ld, int row_floats, const int32_t *idx, int64_t n,
                                   float *sink, int stages, int blocks_per_sm, int32_t *status, void *cuda_stream)
{
    if (!table || !idx || !sink || !status || rows <= 0 || n < 0 || ld < row_floats || ld % 4 || (row_floats != 32 && row_floats != 16)) return 1;
    if (reinterpret_cast<uintptr_t>(table) % 16 || reinterpret_cast<uintptr_t>(idx) % 16) return 1;
    if (stages < 1 || stages > TMA_MAX_STAGES || blocks_per_sm < 1 || blocks_per_sm > 16) return 1;
    static encode_tiled_fn encode = nullptr;
    if (!encode) {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &res) != cudaSuccess || !fn ||
            res != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            return 3;
        }
        encode = reinterpret_cast<encode_tiled_fn>(fn);
    }
    CUtensorMap tm;
    const cuuint64_t gdim[2] = {cuuint64_t(row_floats), cuuint64_t(rows)};
    const cuuint64_t gstride[1] = {cuuint64_t(ld) * 4};
    const cuuint32_t box[2] = {cuuint32_t(row_floats), 1};
    const cuuint32_t estride[2] = {1, 1};
    if (encode(&tm, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float *>(table), gdim, gstride, box, estride,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return 3;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return 2; }
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const size_t smem = size_t(TMA_WARPS) * size_t(stages) * 16 * size_t(row_floats) * 4;
    auto kern = row_floats == 32 ? tma_gather_kernel<32> : tma_gather_kernel<16>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess) { cudaGetLastError(); return 2; }
    kern<<<unsigned(sms) * unsigned(blocks_per_sm), 32 * TMA_WARPS, smem, static_cast<cudaStream_t>(cuda_stream)>>>(tm, idx, n, stages, sink, status);
    if (cudaGetLastError() != cudaSuccess) return 2;
    return 0;
}

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
