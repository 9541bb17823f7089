// Dense stage  E = C . D  (rows x L times L x M, fp32 in and out) on the fifth-generation tensor cores.
// It is the GEMM of the <SpMM,GEMM> chain in the order B.(C.D) and the trailing GEMM of the chains
// <SDDMM,SpMM,GEMM> and <MTTKRP,GEMM> (Table of kernels, Section 6).
//
// The stage is bound by reading C once from HBM, so the arithmetic only has to stay out of the way while
// keeping fp32 accuracy: every fp32 number x is split as x = b1 + b2 with b1 = bf16(x), b2 = bf16(x - b1),
// and a product is formed as b1.b1 + b1.b2 + b2.b1 (error about 1e-5 relative, inside the 1e-4 bound).
//
// One persistent thread block per SM, 128-row tiles, roles by warp:
//   warps 5..12  load 64-column chunks of C straight into registers (coalesced 128-bit loads, two chunks in
//                flight per thread while a third is converted), split them into the two BF16 parts and write
//                both as K-major 128-byte-swizzled operand tiles (four stages);
//   warp 4       one lane issues tcgen05.mma (M = 128, K = 16) from those tiles and from D^T, which sits in
//                shared memory for the life of the block with the low parts stacked under the high parts:
//                b1(C) . [b1(D) | b2(D)] is one product of N = 2M, b2(C) . b1(D) one of N = M onto the first
//                M columns; the accumulator (2M columns) lives in tensor memory, two of them so that a
//                tile's epilogue overlaps the next tile's products;
//   warps 0..3   read a finished accumulator with tcgen05.ld (warp w owns TMEM lanes 32w..32w+31 = tile rows),
//                add its two halves, transpose through a swizzled shared-memory tile and store E in
//                512-byte runs.
// What limits this kernel next to HBM is the shared-memory data pipe (operand writes, tensor-core operand
// reads, epilogue), which is why C never passes through a shared-memory fp32 stage and why the two products
// that share b1(C) are merged.
// Hand-offs are mbarriers; tcgen05.commit signals the completion of the products.  Every wait is bounded by a
// timer: on expiry the block raises its abort flag, all roles leave their loops, the status word is set to
// SA_E_TIMEOUT and tensor memory is released as on the normal path.
#include <algorithm>

#include "sa_device.cuh"

namespace {

constexpr int TC_BM = 128;                  // rows per tile = MMA M = TMEM lanes
constexpr int TC_KC = 64;                   // columns of C per chunk: one 128-byte swizzled BF16 row
constexpr int TC_OPS = 4;                   // operand stages
constexpr int TC_PF = 4;                    // chunks requested into L2 ahead of the loads into registers
constexpr int TC_EPI_WARPS = 4;
constexpr int TC_MMA_WARP = 4;
constexpr int TC_CONV_WARPS = 8;
constexpr int TC_CONV_T = TC_CONV_WARPS * 32;
constexpr int TC_THREADS = (TC_EPI_WARPS + 1 + TC_CONV_WARPS) * 32;
#ifndef SA_TC_WAIT_NS
#define SA_TC_WAIT_NS 2000000000ull
#endif
constexpr uint64_t TC_WAIT_NS = SA_TC_WAIT_NS;   // longest a hand-off may take before the block gives up (the test
                                                  // library that exercises the time-out path is built with 2 ms)
// Library built with -DSA_TEST_HOOKS only: when word 3 of the status words holds this value at launch, one
// conversion thread of every block withholds its first arrival, so that the first operand hand-off never
// completes and the bounded waits have to run out (tests/test_gpu_bounded_wait.py).
constexpr int TC_TEST_WITHHOLD = 0x7e57;

template <int L, int M>
struct tc_cfg {
    static constexpr int KCH = L / TC_KC;
    static constexpr uint32_t D_TILE = 2 * M * 128;                    // one chunk of D^T: M rows of b1, then M rows of b2
    static constexpr uint32_t OP_PART = TC_BM * 128;                   // one BF16 part of a chunk of C
    static constexpr uint32_t EPI_WARP = 32 * M * 4;                   // transposition tile of one epilogue warp
    static constexpr uint32_t OFF_D = 0, OFF_OP = uint32_t(KCH) * D_TILE;
    static constexpr uint32_t OFF_EPI = OFF_OP + TC_OPS * 2 * OP_PART;
    static constexpr uint32_t OFF_BAR = OFF_EPI + TC_EPI_WARPS * EPI_WARP;
    static constexpr size_t SMEM = size_t(OFF_BAR) + 128 + 1024;       // barriers + slack to align the base to 1 KB
    static constexpr uint32_t TMEM_COLS = 4 * M;                       // two fp32 accumulators of 2M columns
    static_assert(L % TC_KC == 0 && (M == 32 || M == 64), "unsupported shape");
    static_assert(D_TILE % 1024 == 0, "swizzle atoms must stay 1 KB aligned");
};

// barrier slots (8 bytes each) behind the ring
enum { B_FULL = 0, B_EMPTY = TC_OPS, B_ACC_FULL = 2 * TC_OPS, B_ACC_EMPTY = 2 * TC_OPS + 2, B_DRAIN = 2 * TC_OPS + 4, B_COUNT = 2 * TC_OPS + 5 };

__device__ __forceinline__ uint32_t tc_smem_u32(const void *p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t tc_timer()
{
    uint64_t t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Wait for the phase of `bar` with the given parity; false when the block is aborting or the timer ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try(bar, parity)) return true;
    const uint64_t t0 = tc_timer();
    for (uint32_t it = 1;; ++it) {
        if (mbar_try(bar, parity)) return true;
        if ((it & 63u) == 0) {
            if (*abort_flag) return false;
            if (tc_timer() - t0 > TC_WAIT_NS) {
                *abort_flag = 1;
                return false;
            }
        }
    }
}

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major operand tile stored in 128-byte rows with the 128-byte swizzle:
// start address and the 1024-byte distance between groups of eight rows, both in units of 16 bytes; bits 46-47
// hold the descriptor version of this architecture, bits 61-63 the swizzle mode (2 = 128 bytes).  The leading
// byte offset is not used by swizzled K-major tiles.
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr)
{
    return uint64_t((saddr & 0x3ffffu) >> 4) | (uint64_t(1) << 16) | (uint64_t(1024 >> 4) << 32) | (uint64_t(1) << 46) |
           (uint64_t(2) << 61);
}

// D[tmem] (+)= A[smem] . B[smem]^T, BF16 operands, fp32 accumulator, issued by one thread.
__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        :
        : "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The barrier receives one arrival when every tcgen05 operation this thread issued so far has completed.
__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// 16 consecutive accumulator columns of this thread's TMEM lane
__device__ __forceinline__ void tc_ld16(uint32_t taddr, float (&v)[16])
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
#pragma unroll
    for (int x = 0; x < 16; ++x) v[x] = __uint_as_float(r[x]);
}

__device__ __forceinline__ float4 tc_ldg4(const float *p)
{
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

// packed BF16 pair, element `lo` in the low half
__device__ __forceinline__ uint32_t tc_bf16x2(float lo, float hi)
{
    uint32_t d;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
    return d;
}
__device__ __forceinline__ void tc_split2(float x0, float x1, uint32_t &h, uint32_t &l)
{
    h = tc_bf16x2(x0, x1);
    l = tc_bf16x2(x0 - __uint_as_float(h << 16), x1 - __uint_as_float(h & 0xffff0000u));
}

// Byte offset of element (row, k) inside a K-major tile of 128-byte rows with the 128-byte swizzle: the
// 16-byte unit index is XORed with the row index modulo 8.
__device__ __forceinline__ uint32_t tc_sw128(uint32_t row, uint32_t k)
{
    return row * 128u + ((((k >> 3) ^ row) & 7u) << 4) + ((k & 7u) << 1);
}

template <int L, int M>
__global__ void __launch_bounds__(TC_THREADS, 1)
gemm_tc_kernel(int64_t J, const float *__restrict__ C, int64_t ldc, const float *__restrict__ D, int64_t ldd,
               float *__restrict__ Eout, int32_t *__restrict__ status)
{
    using G = tc_cfg<L, M>;
    extern __shared__ uint8_t tc_smem_raw[];
    uint8_t *smem = tc_smem_raw + ((1024u - (tc_smem_u32(tc_smem_raw) & 1023u)) & 1023u);
    const uint32_t sbase = tc_smem_u32(smem);
    const uint32_t bars = sbase + G::OFF_BAR;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(smem + G::OFF_BAR + 8 * B_COUNT);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(smem + G::OFF_BAR + 8 * B_COUNT + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // D^T as KCH operand tiles of 2M rows x 64 columns (k): rows n < M hold b1(D(k,n)), rows M + n hold b2
    for (int x = threadIdx.x; x < L * M; x += TC_THREADS) {
        const int k = x / M, n = x % M;
        const float v = __ldg(D + int64_t(k) * ldd + n);
        const uint32_t h = tc_bf16x2(v, 0.f) & 0xffffu;
        const uint32_t l = tc_bf16x2(v - __uint_as_float(h << 16), 0.f) & 0xffffu;
        const uint32_t off = G::OFF_D + uint32_t(k / TC_KC) * G::D_TILE + tc_sw128(n, k % TC_KC);
        *reinterpret_cast<uint16_t *>(smem + off) = uint16_t(h);
        *reinterpret_cast<uint16_t *>(smem + off + M * 128) = uint16_t(l);     // row n + M: same swizzle phase
    }
    fence_async_smem();
    if (threadIdx.x == 0) {
        for (int x = 0; x < TC_OPS; ++x) {
            mbar_init(bars + 8 * (B_FULL + x), TC_CONV_T);
            mbar_init(bars + 8 * (B_EMPTY + x), 1);
        }
        for (int x = 0; x < 2; ++x) {
            mbar_init(bars + 8 * (B_ACC_FULL + x), 1);
            mbar_init(bars + 8 * (B_ACC_EMPTY + x), TC_EPI_WARPS * 32);
        }
        mbar_init(bars + 8 * B_DRAIN, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == TC_MMA_WARP) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc_smem_u32(tmem_slot)),
                     "r"(G::TMEM_COLS)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int64_t n_tiles = (J + TC_BM - 1) / TC_BM;
    const int64_t my_tiles = blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int64_t n_chunks = my_tiles * G::KCH;

    if (warp < TC_EPI_WARPS) {
        // ---- epilogue: accumulator halves -> sum -> transposition tile -> rows of E
        constexpr int RC = M / 4;                                   // 16-byte units per row of E
        uint8_t *stage = smem + G::OFF_EPI + warp * G::EPI_WARP;
        for (int64_t tl = 0; tl < my_tiles; ++tl) {
            const uint32_t a = uint32_t(tl) & 1u, v = uint32_t(tl >> 1);
            const bool ok = mbar_wait(bars + 8 * (B_ACC_FULL + a), v & 1u, abort_flag);
            if (!__all_sync(SA_FULL_MASK, ok)) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + (uint32_t(32 * warp) << 16) + a * (2 * M);
#pragma unroll
            for (int c = 0; c < M / 16; ++c) {
                float p[16], r[16];
                tc_ld16(taddr + 16 * c, p);
                tc_ld16(taddr + M + 16 * c, r);
#pragma unroll
                for (int x = 0; x < 4; ++x)                         // unit 4c + x of row `lane`, XOR-swizzled by the row
                    *reinterpret_cast<float4 *>(stage + lane * (M * 4) + (((4 * c + x) ^ (lane & 7)) << 4)) =
                        make_float4(p[4 * x] + r[4 * x], p[4 * x + 1] + r[4 * x + 1], p[4 * x + 2] + r[4 * x + 2],
                                    p[4 * x + 3] + r[4 * x + 3]);
            }
            tc_fence_before();
            mbar_arrive(bars + 8 * (B_ACC_EMPTY + a));               // the accumulator is free again
            __syncwarp();
            const int64_t row0 = (int64_t(blockIdx.x) + tl * gridDim.x) * TC_BM + 32 * warp;
            float4 *dst = reinterpret_cast<float4 *>(Eout + row0 * M);
#pragma unroll
            for (int i = 0; i < RC; ++i) {
                const int idx = i * 32 + lane, r = idx / RC, j = idx % RC;
                const float4 val = *reinterpret_cast<const float4 *>(stage + r * (M * 4) + ((j ^ (r & 7)) << 4));
                if (row0 + r < J) dst[idx] = val;
            }
            __syncwarp();
        }
    } else if (warp == TC_MMA_WARP) {
        // ---- products: one lane issues, the whole warp follows the hand-offs
        constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(TC_BM >> 4) << 24);   // fp32 += bf16 . bf16, K-major
        constexpr uint32_t IDESC_2M = IDESC | (uint32_t((2 * M) >> 3) << 17), IDESC_M = IDESC | (uint32_t(M >> 3) << 17);
        for (int64_t q = 0; q < n_chunks; ++q) {
            const int kc = int(q % G::KCH);
            const int64_t tl = q / G::KCH;
            const uint32_t a = uint32_t(tl) & 1u, v = uint32_t(tl >> 1);
            const uint32_t s = uint32_t(q) % TC_OPS, u = uint32_t(q / TC_OPS);
            bool ok = true;
            if (kc == 0) ok = mbar_wait(bars + 8 * (B_ACC_EMPTY + a), (v & 1u) ^ 1u, abort_flag);
            if (ok) ok = mbar_wait(bars + 8 * (B_FULL + s), u & 1u, abort_flag);
            if (!__all_sync(SA_FULL_MASK, ok)) break;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t d_tmem = tmem_base + a * (2 * M);
                const uint32_t a_hi = sbase + G::OFF_OP + s * (2 * G::OP_PART), a_lo = a_hi + G::OP_PART;
                const uint32_t b = sbase + G::OFF_D + uint32_t(kc) * G::D_TILE;
#pragma unroll
                for (int k = 0; k < TC_KC / 16; ++k) {
                    const uint32_t adv = 32u * k;                        // 16 BF16 along K inside the swizzled row
                    tc_mma(d_tmem, tc_desc(a_hi + adv), tc_desc(b + adv), IDESC_2M, (kc | k) != 0);
                    tc_mma(d_tmem, tc_desc(a_lo + adv), tc_desc(b + adv), IDESC_M, 1u);
                }
                tc_commit(bars + 8 * (B_EMPTY + s));
                if (kc == G::KCH - 1) tc_commit(bars + 8 * (B_ACC_FULL + a));
            }
            __syncwarp();
        }
    } else {
        // ---- load and conversion: thread owns float4 column qf of rows r0, r0 + 16, ...
        const int t = threadIdx.x - (TC_EPI_WARPS + 1) * 32;
        const uint32_t qf = uint32_t(t) & 15u, r0 = uint32_t(t) >> 4, sw = r0 & 7u;
        const uint32_t op_off = G::OFF_OP + r0 * 128u + (((qf >> 1) ^ sw) << 4) + ((qf & 1u) << 3);
        constexpr int NR = TC_BM / 16;
        auto load = [&](float4 (&b)[NR], int64_t q) {
            if (q + TC_PF < n_chunks) {                            // one 128-byte line per thread: HBM latency is paid by L2
                const int64_t pq = q + TC_PF;
                const int64_t row = min((int64_t(blockIdx.x) + (pq / G::KCH) * gridDim.x) * TC_BM + (t >> 1), J - 1);
                asm volatile("prefetch.global.L2 [%0];" ::"l"(C + row * ldc + int(pq % G::KCH) * TC_KC + 32 * (t & 1)));
            }
            if (q < n_chunks) {
                const int64_t row0 = (int64_t(blockIdx.x) + (q / G::KCH) * gridDim.x) * TC_BM + r0;
                const float *src = C + int(q % G::KCH) * TC_KC + 4 * qf;
#pragma unroll
                for (int i = 0; i < NR; ++i) b[i] = tc_ldg4(src + min(row0 + 16 * i, J - 1) * ldc);   // rows past the end re-read the last row
            }
        };
#ifdef SA_TEST_HOOKS
        const bool withhold = t == 0 && status != nullptr && status[3] == TC_TEST_WITHHOLD;
#endif
        auto convert = [&](const float4 (&b)[NR], int64_t q) -> bool {
            const uint32_t s = uint32_t(q) % TC_OPS, u = uint32_t(q / TC_OPS);
            if (!mbar_wait(bars + 8 * (B_EMPTY + s), (u & 1u) ^ 1u, abort_flag)) return false;
            uint8_t *hi = smem + op_off + s * (2 * G::OP_PART), *lo = hi + G::OP_PART;
#pragma unroll
            for (int i = 0; i < NR; ++i) {
                uint2 h, l;
                tc_split2(b[i].x, b[i].y, h.x, l.x);
                tc_split2(b[i].z, b[i].w, h.y, l.y);
                *reinterpret_cast<uint2 *>(hi + i * (16 * 128)) = h;
                *reinterpret_cast<uint2 *>(lo + i * (16 * 128)) = l;
            }
            fence_async_smem();
#ifdef SA_TEST_HOOKS
            if (withhold && q == 0) return true;
#endif
            mbar_arrive(bars + 8 * (B_FULL + s));
            return true;
        };
        float4 b0[NR], b1[NR], b2[NR];
        load(b0, 0);
        load(b1, 1);
        for (int64_t q = 0; q < n_chunks; q += 3) {
            load(b2, q + 2);
            if (!convert(b0, q)) break;
            if (q + 1 >= n_chunks) break;
            load(b0, q + 3);
            if (!convert(b1, q + 1)) break;
            if (q + 2 >= n_chunks) break;
            load(b1, q + 4);
            if (!convert(b2, q + 2)) break;
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == TC_MMA_WARP) {
        if (*abort_flag) {
            // products may still be in flight: wait for them (bounded) before tensor memory goes back
            if (lane == 0) tc_commit(bars + 8 * B_DRAIN);
            __syncwarp();
            const uint64_t t0 = tc_timer();
            while (!mbar_try(bars + 8 * B_DRAIN, 0u) && tc_timer() - t0 < TC_WAIT_NS) {}
            __syncwarp();
        }
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(G::TMEM_COLS) : "memory");
    }
    if (threadIdx.x == 0 && *abort_flag && status != nullptr) atomicCAS(status, 0, int(SA_E_TIMEOUT));
}

template <int L, int M>
sa_status launch_tc(int64_t rows, const float *A, int64_t lda, const float *B, int64_t ldb, float *out, int32_t *status,
                    cudaStream_t stream)
{
    using G = tc_cfg<L, M>;
    auto k = gemm_tc_kernel<L, M>;
    if (cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, int(G::SMEM)) != cudaSuccess) return SA_E_CUDA;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const int64_t ctas = std::min<int64_t>((rows + TC_BM - 1) / TC_BM, sms);
    if (ctas > 0) k<<<(unsigned)ctas, TC_THREADS, G::SMEM, stream>>>(rows, A, lda, B, ldb, out, status);
    return cudaGetLastError() == cudaSuccess ? SA_OK : SA_E_CUDA;
}

}  // namespace

bool sa_dense_gemm_tc_ok(int64_t L, int64_t M) { return (L == 64 || L == 128 || L == 256) && (M == 32 || M == 64); }

sa_status sa_launch_dense_gemm_tc(int64_t rows, const float *A, int64_t lda, const float *B, int64_t ldb, int64_t L,
                                  int64_t M, float *out, int32_t *status, cudaStream_t stream)
{
#define SA_CASE(l, m) if (L == l && M == m) return launch_tc<l, m>(rows, A, lda, B, ldb, out, status, stream);
    SA_CASE(64, 32) SA_CASE(64, 64) SA_CASE(128, 32) SA_CASE(128, 64) SA_CASE(256, 32) SA_CASE(256, 64)
#undef SA_CASE
    return SA_E_UNSUPPORTED;
}
