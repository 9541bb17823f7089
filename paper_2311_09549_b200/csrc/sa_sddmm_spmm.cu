// Kernel 1 <SDDMM,SpMM>:  A(i,l) = sum_j B(i,j) (sum_k C(i,k) D(j,k)) E(j,l), scheduled as the
// fused nest  i, j' < t ; k: t += B(i,j) C(i,k) D(j,k) , l: A(i,l) += t E(j,l) >  of the paper's
// Table of kernels (Section 6): the sampled value is a scalar temporary that is consumed at once,
// the sampled matrix is never written (auxiliary memory 1 in the paper's memory table).
//
// One warp per work item (a range of short rows, or a piece of a long row).  The rows D(j,:) and
// E(j,:) of the item's nonzeros are gathered with cp.async into a per-warp ring of shared-memory
// stages that runs ahead of the arithmetic, so that the random row reads (the HBM-bound part: D
// and E exceed L2) stay in flight while earlier nonzeros are consumed.  K/4 lanes share one
// nonzero (a float4 of D each, shuffle reduction of the dot product), 32/(K/4) nonzeros per step.
#include "sa_device.cuh"

namespace {

template <int K, int L>
struct sd_cfg {
    static constexpr int LPN = K / 4;                 // lanes per nonzero
    static constexpr int NPS = 32 / LPN;              // nonzeros per step
    static constexpr int EV = L / LPN;                // floats of E(j,:) and of the output row per lane
    static constexpr int ROWF = K + L;                // floats staged per nonzero: D(j,:) then E(j,:)
    static constexpr int R = ROWF <= 128 ? 8 : 4;     // nonzeros per stage
    static constexpr int NS = 3;                      // stages per warp: one being consumed, two in flight
    static constexpr int STAGE = R * ROWF;            // floats per stage
    static constexpr int CPL = STAGE / 4 / 32;        // 16-byte copies per lane per stage
    static_assert(STAGE % 128 == 0 && R % NPS == 0 && 32 % R == 0, "stage shape");
};

template <int K, int L>
__global__ void __launch_bounds__(256, 2)
sddmm_spmm_kernel(const sa_item *__restrict__ items, int64_t n_items, const int32_t *__restrict__ pos,
                  const int32_t *__restrict__ crd, const float *__restrict__ vals, const float *__restrict__ C,
                  uint32_t ldc, const float *__restrict__ D, uint32_t ldd, const float *__restrict__ E, uint32_t lde,
                  float *__restrict__ out, float *__restrict__ partial, float *__restrict__ sampled, const sa_limits lim)
{
    using G = sd_cfg<K, L>;
    extern __shared__ __align__(16) float smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t idx = int64_t(blockIdx.x) * SA_WARPS_PER_CTA + warp;
    if (idx >= n_items) return;
    float *ring = smem + warp * (G::NS * G::STAGE);
    const sa_item it = items[idx];
    const int P0 = it.p0, total = it.p1 - it.p0;      // the item's nonzeros are contiguous
    const int li = lane % G::LPN, grp = lane / G::LPN;

    // column indices / values of the consumer's batch of 32 nonzeros (j0, v0) and the two after it
    int j0, j1, j2;
    float v0, v1, v2;
    auto load_jv = [&](int b, int &j, float &v) {
        const int p = 32 * b + lane;
        j = 0;
        v = 0.f;
        if (p < total && SA_CHK(lim.status, P0 + p >= 0 && P0 + p < lim.nnz, 41, P0 + p)) { j = crd[P0 + p]; v = vals[P0 + p]; }
        if (!SA_CHK(lim.status, uint32_t(j) < lim.gather_rows, 42, j)) j = 0;
    };
    int cb = 0;                                       // batch the consumer is in
    // per-lane constants of the gather: copy q of a stage moves 16-byte piece x = 32 q + lane, i.e. piece
    // cc = x % (ROWF/4) of nonzero r = x / (ROWF/4); pieces lie in the stage in the same order (byte 16 x)
    const char *src_q[G::CPL];                        // D or E plus the piece offset
    uint32_t rowb_q[G::CPL];                          // bytes between rows of that operand
    int r_q[G::CPL];
#pragma unroll
    for (int q = 0; q < G::CPL; ++q) {
        const int x = q * 32 + lane;
        const int cc = x % (G::ROWF / 4);
        r_q[q] = x / (G::ROWF / 4);
        src_q[q] = reinterpret_cast<const char *>(cc < K / 4 ? D + cc * 4 : E + (cc - K / 4) * 4);
        rowb_q[q] = (cc < K / 4 ? ldd : lde) * 4u;
    }
    const uint32_t ring_lane = smem_u32(ring) + uint32_t(lane) * 16u;
    int issue_slot = 0;                               // ring slot the next issued stage goes to
    auto issue_stage = [&](int s) {
        if (s * G::R < total) {
            const uint32_t dst = ring_lane + uint32_t(issue_slot * G::STAGE) * 4u;
            const int b = (s * G::R) >> 5;            // the stage lies inside one batch: cb or cb + 1
            const int jsrc = b == cb ? j0 : j1;
            const int lane0 = (s * G::R) & 31;
#pragma unroll
            for (int q = 0; q < G::CPL; ++q) {
                const uint32_t j = uint32_t(__shfl_sync(SA_FULL_MASK, jsrc, lane0 + r_q[q]));   // 0 beyond the item: row 0
                cp_async16_raw(dst + q * 512u, src_q[q] + j * rowb_q[q]);
            }
        }
        issue_slot = issue_slot == G::NS - 1 ? 0 : issue_slot + 1;
        cp_async_commit();
    };
    load_jv(0, j0, v0);
    load_jv(1, j1, v1);
    load_jv(2, j2, v2);
#pragma unroll
    for (int s = 0; s < G::NS - 1; ++s) issue_stage(s);
    int cur_stage = -1;
    int cur_off = -G::STAGE;                          // float offset of the consumer's stage in the ring
    // called when the consumer first touches stage s: refill the stage it left, wait for s
    auto enter = [&](int s) {
        __syncwarp();
        cur_off = cur_off == (G::NS - 1) * G::STAGE ? 0 : cur_off + G::STAGE;
        if (s > 0 && ((s * G::R) & 31) == 0) {
            j0 = j1; j1 = j2;
            v0 = v1; v1 = v2;
            ++cb;
            load_jv(cb + 2, j2, v2);
        }
        issue_stage(s + G::NS - 1);
        cp_async_wait<G::NS - 1>();
        __syncwarp();
        cur_stage = s;
    };

    const bool piece = it.dest >= 0;
    for (int r = it.out_row; r < it.row_end; ++r) {
        if (!SA_CHK(lim.status, uint32_t(r) < lim.out_rows && (!piece || it.dest < lim.n_slots), 43, r)) continue;
        const int a = piece ? 0 : pos[r] - P0;
        const int b = piece ? total : pos[r + 1] - P0;
        float acc[G::EV];
#pragma unroll
        for (int q = 0; q < G::EV; ++q) acc[q] = 0.f;
        if (b > a) {
            const float4 c4 = sa_ldg4(C + uint32_t(r) * ldc + 4 * li);
            for (int base = (a / G::NPS) * G::NPS; base < b; base += G::NPS) {
                const int st = base / G::R;
                if (st != cur_stage) enter(st);
                const int prel = base + grp;
                const bool active = prel >= a && prel < b;
                const float v = __shfl_sync(SA_FULL_MASK, v0, prel & 31);
                const float *slot = ring + cur_off + (prel & (G::R - 1)) * G::ROWF;
                const float4 d4 = *reinterpret_cast<const float4 *>(slot + 4 * li);
                float dot = fmaf(c4.x, d4.x, fmaf(c4.y, d4.y, fmaf(c4.z, d4.z, c4.w * d4.w)));
#pragma unroll
                for (int o = G::LPN / 2; o > 0; o >>= 1) dot += __shfl_xor_sync(SA_FULL_MASK, dot, o);
                if (active) {
                    const float sc = v * dot;
                    if (sampled != nullptr && li == 0) sampled[P0 + prel] = sc;
                    const float *e = slot + K + li * G::EV;
                    if (G::EV >= 4) {
#pragma unroll
                        for (int q = 0; q < G::EV; q += 4) {
                            const float4 e4 = *reinterpret_cast<const float4 *>(e + q);
                            acc[q] = fmaf(sc, e4.x, acc[q]);
                            acc[(q + 1) % G::EV] = fmaf(sc, e4.y, acc[(q + 1) % G::EV]);
                            acc[(q + 2) % G::EV] = fmaf(sc, e4.z, acc[(q + 2) % G::EV]);
                            acc[(q + 3) % G::EV] = fmaf(sc, e4.w, acc[(q + 3) % G::EV]);
                        }
                    } else if (G::EV == 2) {
                        const float2 e2 = *reinterpret_cast<const float2 *>(e);
                        acc[0] = fmaf(sc, e2.x, acc[0]);
                        acc[1 % G::EV] = fmaf(sc, e2.y, acc[1 % G::EV]);
                    } else {
                        acc[0] = fmaf(sc, e[0], acc[0]);
                    }
                }
            }
            // the NPS groups of lanes hold partial rows: add them up
#pragma unroll
            for (int o = 16; o >= G::LPN; o >>= 1)
#pragma unroll
                for (int q = 0; q < G::EV; ++q) acc[q] += __shfl_xor_sync(SA_FULL_MASK, acc[q], o);
        }
        if (grp == 0) {
            float *dst = (piece ? partial + int64_t(it.dest) * L : out + int64_t(r) * L) + li * G::EV;
            if (G::EV >= 4) {
#pragma unroll
                for (int q = 0; q < G::EV; q += 4)
                    *reinterpret_cast<float4 *>(dst + q) =
                        make_float4(acc[q], acc[(q + 1) % G::EV], acc[(q + 2) % G::EV], acc[(q + 3) % G::EV]);
            } else if (G::EV == 2) {
                *reinterpret_cast<float2 *>(dst) = make_float2(acc[0], acc[1 % G::EV]);
            } else {
                dst[0] = acc[0];
            }
        }
    }
    cp_async_wait<0>();
}

template <int K, int L>
cudaError_t launch(const sa_tensor *t, const sa_dense *ops, float *out, float *partial, float *sampled,
                   cudaStream_t stream)
{
    using G = sd_cfg<K, L>;
    const sa_worklist &wl = t->wl_main;
    const int64_t n_items = int64_t(wl.items.size());
    const int64_t ctas = (n_items + SA_WARPS_PER_CTA - 1) / SA_WARPS_PER_CTA;
    if (ctas == 0) return cudaSuccess;
    constexpr size_t smem = size_t(SA_WARPS_PER_CTA) * G::NS * G::STAGE * sizeof(float);
    auto kern = sddmm_spmm_kernel<K, L>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess)
        return cudaGetLastError();
    kern<<<(unsigned)ctas, 256, smem, stream>>>(wl.d_items, n_items, t->d_pos[1], t->d_crd[1], t->d_vals, ops[0].ptr,
                                               uint32_t(ops[0].ld), ops[1].ptr, uint32_t(ops[1].ld), ops[2].ptr,
                                               uint32_t(ops[2].ld), out, partial, sampled,
                                               sa_make_limits(t, t->dims[1], t->dims[0], wl.n_slots));
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
    for (int i = 0; i < 3; ++i)                       // the kernel addresses dense rows with 32-bit byte offsets
        if (ops[i].rows * ops[i].ld >= (int64_t(1) << 30)) return SA_E_UNSUPPORTED;
    if (materialize)
        sampled = reinterpret_cast<float *>(static_cast<char *>(ws) + sa_align256(size_t(t->wl_main.n_slots) * size_t(L) * sizeof(float)));
    cudaError_t e = cudaErrorInvalidValue;
#define SA_CASE(a, b) if (K == a && L == b) e = launch<a, b>(t, ops, out, partial, sampled, stream);
    SA_CASE(32, 32) SA_CASE(32, 64) SA_CASE(32, 128) SA_CASE(64, 32) SA_CASE(64, 64) SA_CASE(64, 128)
    SA_CASE(128, 32) SA_CASE(128, 64) SA_CASE(128, 128)
#undef SA_CASE
    if (e != cudaSuccess) return SA_E_CUDA;
    *launches = t->wl_main.items.empty() ? 0 : 1;
    if (!t->wl_main.fix.empty()) {
        if (sa_launch_fixup(t->wl_main, partial, out, int(L), stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}

// ---- kernel 2 <SDDMM,SpMM,GEMM>:  A(i,m) = sum_{j,k,l} B(i,j) C(i,k) D(j,k) E(j,l) F(l,m), the two-level
// schedule  i < T(l) ; j' < t ; k: ... , l: T(l) += t E(j,l) > , m,l: A(i,m) += T(l) F(l,m) >  of the paper's
// Table of kernels: the row temporary T is what the fused kernel above produces per row; here it goes
// through the workspace (I x L floats) to a tensor-core product with F instead of staying in registers.
// workspace: [T: I x L][partial rows of long-row pieces]
size_t sa_ws_sddmm_spmm_gemm(const sa_tensor *t, const sa_dense *ops)
{
    return sa_align256(size_t(t->dims[0]) * size_t(ops[2].cols) * sizeof(float)) + sa_ws_sddmm_spmm(t, ops, false);
}

sa_status sa_launch_sddmm_spmm_gemm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                                    cudaStream_t stream, int *launches)
{
    const int64_t I = t->dims[0], L = ops[2].cols, M = ops[3].cols;
    const size_t t_bytes = sa_align256(size_t(I) * size_t(L) * sizeof(float));
    float *T = static_cast<float *>(ws);
    int n1 = 0;
    const sa_status s = sa_launch_sddmm_spmm(t, ops, T, static_cast<char *>(ws) + t_bytes, ws_bytes - t_bytes, false, stream, &n1);
    if (s != SA_OK) return s;
    const sa_status g = sa_launch_dense_gemm(I, T, L, ops[3].ptr, ops[3].ld, L, M, out, t->d_status, stream);
    if (g != SA_OK) return g;
    *launches = n1 + 1;
    return SA_OK;
}
