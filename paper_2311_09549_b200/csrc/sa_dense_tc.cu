// Dense stage  E = C . D  (rows x L times L x M, fp32 in and out) on the fifth-generation tensor cores.
// It is the GEMM of the <SpMM,GEMM> chain in the order B.(C.D) and the trailing GEMM of the chains
// <SDDMM,SpMM,GEMM> and <MTTKRP,GEMM> (Table of kernels, Section 6).
//
// The stage is bound by reading C once from HBM, so the arithmetic only has to stay out of the way while
// keeping fp32 accuracy: every fp32 number x is split as x = b1 + b2 with b1 = bf16(x), b2 = bf16(x - b1),
// and a product is formed as b1.b1 + b1.b2 + b2.b1 (error about 1e-5 relative, inside the 1e-4 bound).
//
// One persistent thread block per SM, 128-row tiles, roles by warp:
//   warps 5..12  cp.async 64-column chunks of C into a private fp32 ring (every thread converts exactly the
//                bytes it copied itself, so the ring needs no barrier), split them into the two BF16 parts
//                and write both as K-major 128-byte-swizzled operand tiles;
//   warp 4       one lane issues tcgen05.mma (M = 128, N = M, K = 16; three per K step) from those tiles and
//                from D^T, which sits in shared memory (both BF16 parts) for the life of the block; the
//                accumulator lives in tensor memory, two of them so that a tile's epilogue overlaps the next
//                tile's products;
//   warps 0..3   read a finished accumulator with tcgen05.ld (warp w owns TMEM lanes 32w..32w+31 = tile rows)
//                and store the rows of E.
// Hand-offs are mbarriers; tcgen05.commit signals the completion of the products.  Every wait is bounded by a
// timer: on expiry the block raises its abort flag, all roles leave their loops, the status word is set to
// SA_E_TIMEOUT and tensor memory is released as on the normal path.
#include <algorithm>

#include "sa_device.cuh"

namespace {

constexpr int TC_BM = 128;                  // rows per tile = MMA M = TMEM lanes
constexpr int TC_KC = 64;                   // columns of C per chunk: one 128-byte swizzled BF16 row
constexpr int TC_NS = 3;                    // fp32 ring stages (two chunks in flight while one is converted)
constexpr int TC_EPI_WARPS = 4;
constexpr int TC_MMA_WARP = 4;
constexpr int TC_CONV_WARPS = 8;
constexpr int TC_CONV_T = TC_CONV_WARPS * 32;
constexpr int TC_THREADS = (TC_EPI_WARPS + 1 + TC_CONV_WARPS) * 32;
constexpr uint64_t TC_WAIT_NS = 2000000000ull;   // longest a hand-off may take before the block gives up

template <int L, int M>
struct tc_cfg {
    static constexpr int KCH = L / TC_KC;
    static constexpr uint32_t D_PART = uint32_t(KCH) * M * 128;        // one BF16 part of D^T (KCH tiles of M x 64)
    static constexpr uint32_t OP_PART = TC_BM * 128;                   // one BF16 part of a chunk of C
    static constexpr uint32_t RING_STAGE = TC_BM * TC_KC * 4;
    static constexpr uint32_t OFF_DH = 0, OFF_DL = D_PART, OFF_OP = 2 * D_PART;
    static constexpr uint32_t OFF_RING = OFF_OP + 4 * OP_PART;         // two operand stages x (high, low)
    static constexpr uint32_t OFF_BAR = OFF_RING + TC_NS * RING_STAGE;
    static constexpr size_t SMEM = size_t(OFF_BAR) + 128 + 1024;       // barriers + slack to align the base to 1 KB
    static constexpr uint32_t TMEM_COLS = 2 * M;                       // two fp32 accumulators of M columns
    static_assert(L % TC_KC == 0 && (M == 32 || M == 64), "unsupported shape");
    static_assert(D_PART % 1024 == 0, "swizzle atoms must stay 1 KB aligned");
};

// barrier slots (8 bytes each) behind the ring
enum { B_FULL = 0, B_EMPTY = 2, B_ACC_FULL = 4, B_ACC_EMPTY = 6, B_DRAIN = 8, B_COUNT = 9 };

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

__device__ __forceinline__ void tc_cp_async16(uint32_t dst, const float *src)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
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

    // D^T, both BF16 parts, as KCH operand tiles of M rows (n) x 64 columns (k)
    for (int x = threadIdx.x; x < L * M; x += TC_THREADS) {
        const int k = x / M, n = x % M;
        const float v = __ldg(D + int64_t(k) * ldd + n);
        const uint32_t h = tc_bf16x2(v, 0.f) & 0xffffu;
        const uint32_t l = tc_bf16x2(v - __uint_as_float(h << 16), 0.f) & 0xffffu;
        const uint32_t off = uint32_t(k / TC_KC) * (M * 128) + tc_sw128(n, k % TC_KC);
        *reinterpret_cast<uint16_t *>(smem + G::OFF_DH + off) = uint16_t(h);
        *reinterpret_cast<uint16_t *>(smem + G::OFF_DL + off) = uint16_t(l);
    }
    fence_async_smem();
    if (threadIdx.x == 0) {
        mbar_init(bars + 8 * (B_FULL + 0), TC_CONV_T);
        mbar_init(bars + 8 * (B_FULL + 1), TC_CONV_T);
        mbar_init(bars + 8 * (B_EMPTY + 0), 1);
        mbar_init(bars + 8 * (B_EMPTY + 1), 1);
        mbar_init(bars + 8 * (B_ACC_FULL + 0), 1);
        mbar_init(bars + 8 * (B_ACC_FULL + 1), 1);
        mbar_init(bars + 8 * (B_ACC_EMPTY + 0), TC_EPI_WARPS * 32);
        mbar_init(bars + 8 * (B_ACC_EMPTY + 1), TC_EPI_WARPS * 32);
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
        // ---- epilogue: accumulator -> rows of E
        for (int64_t tl = 0; tl < my_tiles; ++tl) {
            const uint32_t a = uint32_t(tl) & 1u, v = uint32_t(tl >> 1);
            const bool ok = mbar_wait(bars + 8 * (B_ACC_FULL + a), v & 1u, abort_flag);
            if (!__all_sync(SA_FULL_MASK, ok)) break;
            tc_fence_after();
            const int64_t row = (int64_t(blockIdx.x) + tl * gridDim.x) * TC_BM + 32 * warp + lane;
            const uint32_t taddr = tmem_base + (uint32_t(32 * warp) << 16) + a * M;
#pragma unroll
            for (int c = 0; c < M / 16; ++c) {
                float v16[16];
                tc_ld16(taddr + 16 * c, v16);
                if (row < J) {
                    float4 *dst = reinterpret_cast<float4 *>(Eout + row * M + 16 * c);
#pragma unroll
                    for (int x = 0; x < 4; ++x) dst[x] = make_float4(v16[4 * x], v16[4 * x + 1], v16[4 * x + 2], v16[4 * x + 3]);
                }
            }
            tc_fence_before();
            mbar_arrive(bars + 8 * (B_ACC_EMPTY + a));
        }
    } else if (warp == TC_MMA_WARP) {
        // ---- products: one lane issues, the whole warp follows the hand-offs
        constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | (uint32_t(M >> 3) << 17) | (uint32_t(TC_BM >> 4) << 24);
        for (int64_t q = 0; q < n_chunks; ++q) {
            const int kc = int(q % G::KCH);
            const int64_t tl = q / G::KCH;
            const uint32_t a = uint32_t(tl) & 1u, v = uint32_t(tl >> 1);
            const uint32_t s = uint32_t(q) & 1u, u = uint32_t(q >> 1);
            bool ok = true;
            if (kc == 0) ok = mbar_wait(bars + 8 * (B_ACC_EMPTY + a), (v & 1u) ^ 1u, abort_flag);
            if (ok) ok = mbar_wait(bars + 8 * (B_FULL + s), u & 1u, abort_flag);
            if (!__all_sync(SA_FULL_MASK, ok)) break;
            tc_fence_after();
            if (lane == 0) {
                const uint32_t d_tmem = tmem_base + a * M;
                const uint32_t a_hi = sbase + G::OFF_OP + s * (2 * G::OP_PART), a_lo = a_hi + G::OP_PART;
                const uint32_t b_hi = sbase + G::OFF_DH + uint32_t(kc) * (M * 128), b_lo = b_hi + G::D_PART;
#pragma unroll
                for (int k = 0; k < TC_KC / 16; ++k) {
                    const uint32_t adv = 32u * k;                        // 16 BF16 along K inside the swizzled row
                    tc_mma(d_tmem, tc_desc(a_lo + adv), tc_desc(b_hi + adv), IDESC, (kc | k) != 0);
                    tc_mma(d_tmem, tc_desc(a_hi + adv), tc_desc(b_lo + adv), IDESC, 1u);
                    tc_mma(d_tmem, tc_desc(a_hi + adv), tc_desc(b_hi + adv), IDESC, 1u);
                }
                tc_commit(bars + 8 * (B_EMPTY + s));
                if (kc == G::KCH - 1) tc_commit(bars + 8 * (B_ACC_FULL + a));
            }
            __syncwarp();
        }
    } else {
        // ---- copy and conversion: thread owns float4 column qf of rows r0, r0 + 16, ...
        const int t = threadIdx.x - (TC_EPI_WARPS + 1) * 32;
        const uint32_t qf = uint32_t(t) & 15u, r0 = uint32_t(t) >> 4, sw = r0 & 7u;
        const uint32_t ring = sbase + G::OFF_RING + r0 * 256u + ((qf ^ sw) << 4);
        const uint32_t op_off = r0 * 128u + (((qf >> 1) ^ sw) << 4) + ((qf & 1u) << 3);
        auto issue = [&](int64_t q) {
            if (q < n_chunks) {
                const int64_t row0 = (int64_t(blockIdx.x) + (q / G::KCH) * gridDim.x) * TC_BM + r0;
                const float *src = C + int(q % G::KCH) * TC_KC + 4 * qf;
                const uint32_t dst = ring + uint32_t(q % TC_NS) * G::RING_STAGE;
#pragma unroll
                for (int i = 0; i < TC_BM / 16; ++i) {
                    const int64_t row = min(row0 + 16 * i, J - 1);       // rows past the end re-read the last row
                    tc_cp_async16(dst + uint32_t(i) * (16u * 256u), src + row * ldc);
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
        };
#pragma unroll
        for (int q = 0; q < TC_NS - 1; ++q) issue(q);
        for (int64_t q = 0; q < n_chunks; ++q) {
            issue(q + TC_NS - 1);
            asm volatile("cp.async.wait_group %0;" ::"n"(TC_NS - 1) : "memory");
            const uint32_t s = uint32_t(q) & 1u, u = uint32_t(q >> 1);
            if (!mbar_wait(bars + 8 * (B_EMPTY + s), (u & 1u) ^ 1u, abort_flag)) break;
            const uint8_t *src = smem + (ring - sbase) + uint32_t(q % TC_NS) * G::RING_STAGE;
            uint8_t *hi = smem + G::OFF_OP + s * (2 * G::OP_PART) + op_off, *lo = hi + G::OP_PART;
#pragma unroll
            for (int i = 0; i < TC_BM / 16; ++i) {
                const float4 x = *reinterpret_cast<const float4 *>(src + i * (16 * 256));
                uint2 h, l;
                tc_split2(x.x, x.y, h.x, l.x);
                tc_split2(x.z, x.w, h.y, l.y);
                *reinterpret_cast<uint2 *>(hi + i * (16 * 128)) = h;
                *reinterpret_cast<uint2 *>(lo + i * (16 * 128)) = l;
            }
            fence_async_smem();
            mbar_arrive(bars + 8 * (B_FULL + s));
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
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
