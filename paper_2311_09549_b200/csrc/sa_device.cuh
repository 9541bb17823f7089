// Small device helpers shared by the kernels.
#pragma once

#include <cuda_runtime.h>
#include <cstdint>

#include "sa_internal.h"

#define SA_FULL_MASK 0xffffffffu

__device__ __forceinline__ float4 sa_ldg4(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }
__device__ __forceinline__ float2 sa_ldg2(const float *p) { return __ldg(reinterpret_cast<const float2 *>(p)); }

// Streaming (evict-first) stores for output tiles that are written once and never re-read, so
// they do not displace the factor matrices held in L2.
__device__ __forceinline__ void sa_st_cs(float *p, float v) { __stcs(p, v); }
__device__ __forceinline__ void sa_st_cs4(float *p, float4 v) { __stcs(reinterpret_cast<float4 *>(p), v); }
__device__ __forceinline__ void sa_st_cs2(float *p, float2 v) { __stcs(reinterpret_cast<float2 *>(p), v); }

// Sum `count` partial tiles into out rows (count == 0: zero fill).  Tile size in floats is a
// power of two >= 16.  Block = 256 threads = W float4 columns x P phases over the partials;
// grid = (entries, tile_f4 / W).  Fixed summation order: deterministic.
static __global__ void __launch_bounds__(256)
sa_fixup_kernel(const sa_fix *__restrict__ fix, const float *__restrict__ partial, float *__restrict__ out,
                int tile_floats, int W)
{
    __shared__ float4 red[256];
    const sa_fix e = fix[blockIdx.x];
    const int P = 256 / W;
    const int col = threadIdx.x % W, phase = threadIdx.x / W;
    const int64_t f4 = int64_t(blockIdx.y) * W + col;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    const float *base = partial + int64_t(e.slot0) * tile_floats + f4 * 4;
#pragma unroll 4
    for (int q = phase; q < e.count; q += P) {
        const float4 v = *reinterpret_cast<const float4 *>(base + int64_t(q) * tile_floats);
        s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
    }
    red[threadIdx.x] = s;
    __syncthreads();
    if (phase == 0) {
        for (int q = 1; q < P; ++q) {
            const float4 v = red[q * W + col];
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        sa_st_cs4(out + int64_t(e.out_row) * tile_floats + f4 * 4, s);
    }
}

static inline cudaError_t sa_launch_fixup(const sa_worklist &wl, const float *partial, float *out, int tile_floats,
                                          cudaStream_t stream)
{
    if (wl.fix.empty()) return cudaSuccess;
    const int nf4 = tile_floats / 4;
    const int W = nf4 < 64 ? nf4 : 64;
    dim3 grid((unsigned)wl.fix.size(), (unsigned)(nf4 / W));
    sa_fixup_kernel<<<grid, 256, 0, stream>>>(wl.d_fix, partial, out, tile_floats, W);
    return cudaGetLastError();
}
