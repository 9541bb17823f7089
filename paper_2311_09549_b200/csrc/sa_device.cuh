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

// Self-checking build (-DSA_DEBUG_BOUNDS): every index that comes out of the tensor's arrays is checked before it
// is turned into an address; the first violation is recorded in the tensor's status word (check number, offending
// value, thread; read back by sa_last_device_status / sa_device_status_words) and the caller redirects the access to
// a valid element.  Nothing traps.  In the normal build SA_CHK is the constant true.
#ifdef SA_DEBUG_BOUNDS
__device__ __forceinline__ bool sa_dbg_ok(int32_t *status, bool ok, int code, int64_t value)
{
    if (!ok && atomicCAS(status, 0, int(SA_E_BOUNDS)) == 0) {
        status[1] = code;
        status[2] = int32_t(value);
        status[3] = int32_t(blockIdx.x * blockDim.x + threadIdx.x);
    }
    return ok;
}
#define SA_CHK(status, cond, code, value) sa_dbg_ok(status, cond, code, int64_t(value))
#else
#define SA_CHK(status, cond, code, value) true
#endif

// What the checks of the row / fiber kernels compare against: rows of the gathered dense operand(s), output rows,
// partial slots, nonzeros (items come from the work lists, indices from crd).
struct sa_limits {
    int32_t *status;
    uint32_t gather_rows, out_rows;
    int32_t n_slots, nnz;
};

static inline sa_limits sa_make_limits(const sa_tensor *t, int64_t gather_rows, int64_t out_rows, int64_t n_slots)
{
    sa_limits lim;
    lim.status = t->d_status;
    lim.gather_rows = uint32_t(gather_rows);
    lim.out_rows = uint32_t(out_rows);
    lim.n_slots = int32_t(n_slots);
    lim.nnz = int32_t(t->nnz);
    return lim;
}

// Opt a kernel into `bytes` of dynamic shared memory once per device instead of once per launch (the attribute is
// per device; `done` is the caller's flag array, one entry per device ordinal).
constexpr int SA_MAX_DEVICE_FLAGS = 64;
template <typename Kernel>
static inline bool sa_set_smem_once(Kernel kernel, int bytes, bool (&done)[SA_MAX_DEVICE_FLAGS])
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (dev >= 0 && dev < SA_MAX_DEVICE_FLAGS && done[dev]) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) != cudaSuccess) return false;
    if (dev >= 0 && dev < SA_MAX_DEVICE_FLAGS) done[dev] = true;
    return true;
}

// ---- PTX helpers shared by the kernels

// x = hi + lo with hi the upper 19 bits of x (a TF32 number) and lo = x - hi (exact in fp32), itself cut to
// TF32.  hi.hi + hi.lo + lo.hi then misses the true product by about 2^-20 relative.  (cvt.rna.tf32 costs
// several instructions per value on this target; plain masking is one.)
__device__ __forceinline__ void split_tf32(float x, uint32_t &hi, uint32_t &lo)
{
    hi = __float_as_uint(x) & 0xffffe000u;
    lo = __float_as_uint(x - __uint_as_float(hi)) & 0xffffe000u;
}

__device__ __forceinline__ void mma_m16n8k8_tf32(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void cp_async16_raw(uint32_t dst_smem, const void *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

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
