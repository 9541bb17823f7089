// Kernel 6 <SpTTM,TTM>:  A(i,l,m) = sum_{j,k} B(i,j,k) C(j,l) D(k,m), scheduled as the branched
// nest  i, j' < t ; k': t += B(i,j,k) D(k,m) , l: A(i,l,m) += t C(j,l) >  of the paper's Table of
// kernels (Section 6).
//
// Producer (SpTTM, fp32 ALU).  A warp is four independent lane groups ("streams") of eight lanes.  Every
// stream walks its own contiguous part of the unit's nonzeros, sixteen per round (the per-round bookkeeping
// costs more instructions than the sixteen steps themselves); a lane holds M/8 consecutive entries of the
// fiber temporary t(:), so the eight lanes of a stream fetch one row D(k,:) with a single vector load and the
// row is consumed from registers eight steps after it was requested (eight rows in flight per lane).  The
// index, value and end-of-fiber-bit arrays reach the streams through a per-warp cp.async ring in shared
// memory that runs three rounds ahead and continues across the units of a task, so a warp that evaluates
// many small slices never drains its pipelines.
// Consumer (TTM, tensor cores).  A stream that meets an end-of-fiber bit parks t(:) and the fiber's C row
// offset in a ring of rows in shared memory; eight parked rows at a time update the slice tile as
// A(i,:,:) += Cg^T (L x 8) . T (8 x M) with m16n8k8 TF32 MMAs, each operand split into a high and a low
// TF32 part (three products), which keeps fp32-level accuracy.  The order-3 intermediate T(i,j,m) is
// never stored.
#include <algorithm>
#include <type_traits>

#include "sa_device.cuh"

namespace {

// Limits for the checks of the self-checking build (SA_CHK, sa_device.cuh).
struct dbg_limits {
    int32_t *status;
    uint32_t c_rows, d_rows, n_fibers, n_slices_dim;
    int64_t nnz;
};


template <int L, int M>
struct cfg {
    // Thread blocks per SM the register budget is set for: 4 (16 warps, 128 registers).  The 16 x 16 kernel also
    // compiles without spills for 6 blocks (24 warps, 80 registers); that variant is slower on long units but
    // faster when the units are short (many unit switches, whose latencies more warps hide): the launcher picks.
    static constexpr int MINCTAS = 4;
    static constexpr int MINCTAS_SHORT = (L == 16 && M == 16) ? 6 : 4;
    static constexpr int MT = L / 16;            // m16 tiles over l
    static constexpr int NT = M / 8;             // n8 tiles over m
    static constexpr int NS = SA_STREAMS;        // streams per warp
    static constexpr int VEC = M / 8;            // floats of a factor row per lane (eight lanes per row)
    static constexpr int RS = M + 8;             // row stride of the ring of parked temporaries and of a warp's
                                                 // tile in the CTA reduction; word M of a ring row = C row offset
    static constexpr int STEPS = SA_ROUND;       // nonzeros per stream and round
    static constexpr int RING = 8 + 4 * STEPS;   // rows parked fibers wait in: at most 7 rows are left over from the
                                                 // round before and a round parks at most 4 * STEPS more
    static constexpr int DEPTH = 4;              // rounds of index / value data in flight (cp.async ring)
    static constexpr int SLOT = 8 * STEPS + 16;  // bytes per (round, stream): 16 indices | 16 values | end bits | pad
    static_assert(STEPS == 16, "the step loop, the slot layout and the end-bit extraction are written for 16");
    static constexpr int OFF_KV = 0;
    static constexpr int OFF_RING = OFF_KV + DEPTH * NS * SLOT;
    static constexpr int WARP_BYTES = OFF_RING + RING * RS * 4;
    static_assert(L * RS * 4 <= WARP_BYTES, "the CTA reduction reuses a warp's region for its tile");
};

__device__ __forceinline__ void cp_async4_raw(uint32_t dst_smem, const void *src)
{
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst_smem), "l"(src) : "memory");
}
__device__ __forceinline__ uint32_t lds32(uint32_t a)
{
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t a)
{
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(a) : "memory");
    return v;
}
__device__ __forceinline__ void sts32(uint32_t a, uint32_t v) { asm volatile("st.shared.u32 [%0], %1;" ::"r"(a), "r"(v) : "memory"); }
__device__ __forceinline__ void prefetch_l1(const void *p) { asm volatile("prefetch.global.L1 [%0];" ::"l"(p)); }

// A lane's piece of a factor row: VEC = 4 or 2 consecutive floats.  Plain read-only loads: with the
// L1::no_allocate qualifier the rows also lost their place in L2 (hit rate 57 % instead of 87 %).
template <int VEC>
struct rowvec;
template <>
struct rowvec<4> {
    float x[4];
    __device__ __forceinline__ void load(const char *p)
    {
        asm volatile("ld.global.nc.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(x[0]), "=f"(x[1]), "=f"(x[2]), "=f"(x[3]) : "l"(p));
    }
    __device__ __forceinline__ void store_shared(uint32_t a) const
    {
        asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(a), "f"(x[0]), "f"(x[1]), "f"(x[2]), "f"(x[3]) : "memory");
    }
};
template <>
struct rowvec<2> {
    float x[2];
    __device__ __forceinline__ void load(const char *p)
    {
        asm volatile("ld.global.nc.v2.f32 {%0,%1}, [%2];" : "=f"(x[0]), "=f"(x[1]) : "l"(p));
    }
    __device__ __forceinline__ void store_shared(uint32_t a) const
    {
        asm volatile("st.shared.v2.f32 [%0], {%1,%2};" ::"r"(a), "f"(x[0]), "f"(x[1]) : "memory");
    }
};

// acc += Cg^T . T for the parked rows row0 + x, x = 0 .. 7, of which the first n are in use.
template <int L, int M>
__device__ __forceinline__ void ttm3_flush(float (&acc)[cfg<L, M>::MT][cfg<L, M>::NT][4], const float *__restrict__ ring,
                                           int row0, int n, const float *__restrict__ C, int lane, const dbg_limits &lim, uint32_t ldc)
{
    using K = cfg<L, M>;
    const int g = lane >> 2, t = lane & 3;
    const float *ra = ring + (row0 + t) * K::RS;
    const float *rb = ring + (row0 + t + 4) * K::RS;
    // the values of C this flush needs: rows of the fibers x = t and x = t + 4, columns 16 mt + g (+ 8)
    float cf[K::MT][4];
    {
        const bool va = t < n, vb = t + 4 < n;
        uint32_t oa = va ? __float_as_uint(ra[M]) : 0u, ob = vb ? __float_as_uint(rb[M]) : 0u;
        if (!SA_CHK(lim.status, oa < lim.c_rows * ldc, 1, oa)) oa = 0u;
        if (!SA_CHK(lim.status, ob < lim.c_rows * ldc, 2, ob)) ob = 0u;
        const float *ca = C + oa + g;
        const float *cb = C + ob + g;
#pragma unroll
        for (int mt = 0; mt < K::MT; ++mt) {
            cf[mt][0] = va ? __ldg(ca + 16 * mt) : 0.f;
            cf[mt][1] = va ? __ldg(ca + 16 * mt + 8) : 0.f;
            cf[mt][2] = vb ? __ldg(cb + 16 * mt) : 0.f;
            cf[mt][3] = vb ? __ldg(cb + 16 * mt + 8) : 0.f;
        }
    }
    uint32_t bh[K::NT][2], bl[K::NT][2];
#pragma unroll
    for (int nt = 0; nt < K::NT; ++nt) {
        split_tf32(ra[8 * nt + g], bh[nt][0], bl[nt][0]);
        split_tf32(rb[8 * nt + g], bh[nt][1], bl[nt][1]);
    }
#pragma unroll
    for (int mt = 0; mt < K::MT; ++mt) {
        uint32_t ah[4], al[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) split_tf32(cf[mt][x], ah[x], al[x]);
#pragma unroll
        for (int nt = 0; nt < K::NT; ++nt) {
            mma_m16n8k8_tf32(acc[mt][nt], al, bh[nt]);
            mma_m16n8k8_tf32(acc[mt][nt], ah, bl[nt]);
            mma_m16n8k8_tf32(acc[mt][nt], ah, bh[nt]);
        }
    }
}

// MTTKRP consumer (kernel 8): hacc(m) += sum over the parked rows row0 .. row0 + n - 1 of T(row, m) * C(j_row, m).
// M = 32: lane = m.  M = 16: lane & 15 = m, the two half-warps take alternate rows (summed at the unit end).
template <int M>
__device__ __forceinline__ void had_flush(float &hacc, const float *__restrict__ ring, int row0, int n,
                                          const float *__restrict__ C, int lane)
{
    constexpr int RS = M + 8;
    const int m = lane & (M - 1);
#pragma unroll
    for (int x = 0; x < 8; ++x) {
        const bool mine = x < n && (M == 32 || (x & 1) == (lane >> 4));
        const float *r = ring + (row0 + x) * RS;
        if (mine) hacc = fmaf(r[m], __ldg(C + __float_as_uint(r[M]) + m), hacc);
    }
}

// Store a slice tile held as MMA accumulator fragments (streaming stores: the output is written once).  The
// fragments go through the warp's ring of parked rows (empty at the end of a unit), so that every store instruction
// writes 512 contiguous bytes of the tile instead of eight 32-byte pieces of eight rows.
template <int L, int M>
__device__ __forceinline__ void store_tile(const float (&acc)[cfg<L, M>::MT][cfg<L, M>::NT][4], float *__restrict__ dst, int lane,
                                           float *__restrict__ ring)
{
    using K = cfg<L, M>;
    static_assert(L * K::RS <= K::RING * K::RS, "the tile fits the ring");
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int mt = 0; mt < K::MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < K::NT; ++nt) {
            const int l = 16 * mt + g, mm = 8 * nt + 2 * t;
            *reinterpret_cast<float2 *>(ring + l * K::RS + mm) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
            *reinterpret_cast<float2 *>(ring + (l + 8) * K::RS + mm) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
        }
    __syncwarp();
#pragma unroll
    for (int x = 4 * lane; x < L * M; x += 128)
        sa_st_cs4(dst + x, *reinterpret_cast<const float4 *>(ring + (x / M) * K::RS + (x % M)));
    __syncwarp();
}

template <int L, int M>
__device__ __forceinline__ void zero_tile(float (&acc)[cfg<L, M>::MT][cfg<L, M>::NT][4])
{
#pragma unroll
    for (int mt = 0; mt < cfg<L, M>::MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < cfg<L, M>::NT; ++nt)
#pragma unroll
            for (int x = 0; x < 4; ++x) acc[mt][nt][x] = 0.f;
}

// Where stream q of a unit runs: rounds, aligned start, and the clipped range [lo, hi) (see sa_unit3_streams).
struct stream_range {
    int rounds, base, lo, hi;
    int full;       // rounds 1 .. full - 2 lie inside every stream's part: nothing to mask, no cut fiber to close
};
__device__ __forceinline__ stream_range stream_of(int p0, int p1, int q)
{
    const int base = p0 & ~(SA_ROUND - 1), span = p1 - base;
    const int slen = ((span + SA_STREAMS - 1) / SA_STREAMS + SA_ROUND - 1) & ~(SA_ROUND - 1);
    stream_range r;
    r.rounds = slen / SA_ROUND;
    r.base = base + q * slen;
    r.lo = max(p0, r.base);
    r.hi = min(p1, r.base + slen);
    r.full = (span - (SA_STREAMS - 1) * slen) / SA_ROUND;
    return r;
}

// One warp evaluates the units [u0, u0 + nu) of its task.  `keep`: the (single) unit is a piece of a slice
// whose tile the caller reduces over the CTA, so it is left in acc; otherwise every unit is a whole slice
// and its tile is stored to `out` when the unit ends.
// What kernel 5 adds at the end of a unit (TTMC = true): the slice temporary T(i; m,n) in `acc` is not stored but
// contracted with C(i,:) into the block's accumulator of the whole output, accs[l][m][n] += C(i,l) T(i; m,n).
struct ttmc_sink {
    const float *C3;        // C of kernel 5 (rows by i)
    uint32_t ldc3;
    int L3;                 // its columns
    float *accs;            // shared memory, L3 x L x M floats
};

// Several warps of a block add to the same accumulator at unrelated times: shared-memory atomic adds.
template <int L, int M>
__device__ __forceinline__ void ttmc_accumulate(const float (&acc)[cfg<L, M>::MT][cfg<L, M>::NT][4], const ttmc_sink &sk, int row, int lane)
{
    using K = cfg<L, M>;
    const int g = lane >> 2, t = lane & 3;
    const float *crow = sk.C3 + uint32_t(row) * sk.ldc3;
    for (int l = 0; l < sk.L3; ++l) {
        const float c = __ldg(crow + l);
        float *base = sk.accs + l * (L * M) + g * M + 2 * t;
#pragma unroll
        for (int mt = 0; mt < K::MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < K::NT; ++nt) {
                float *p = base + (16 * mt) * M + 8 * nt;
                atomicAdd(p, c * acc[mt][nt][0]);
                atomicAdd(p + 1, c * acc[mt][nt][1]);
                atomicAdd(p + 8 * M, c * acc[mt][nt][2]);
                atomicAdd(p + 8 * M + 1, c * acc[mt][nt][3]);
            }
    }
}

template <int L, int M, bool HAD, bool TTMC = false>
__device__ __forceinline__ void ttm3_warp_task(const sa_unit3 *__restrict__ units, int u0, int nu,
                                               const int32_t *__restrict__ crd_j, const int32_t *__restrict__ crd_k,
                                               const float *__restrict__ vals, const uint32_t *__restrict__ endbits,
                                               const float *__restrict__ C, uint32_t ldc, const float *__restrict__ D,
                                               uint32_t ldd, unsigned char *__restrict__ wsm,
                                               float (&acc)[cfg<L, M>::MT][cfg<L, M>::NT][4], float &hacc, const bool keep,
                                               float *__restrict__ out, const dbg_limits &lim, const ttmc_sink *sink = nullptr)
{
    using K = cfg<L, M>;
    constexpr int VEC = K::VEC, DEPTH = K::DEPTH;
    const int lane = threadIdx.x & 31;
    const int q = lane >> 3, c = lane & 7;
    const uint32_t s_base = smem_u32(wsm), s_kv = s_base + K::OFF_KV + q * K::SLOT, s_ring = s_base + K::OFF_RING;
    float *ring = reinterpret_cast<float *>(wsm + K::OFF_RING);
    // the index / value ring starts as zeros: a stream that has nothing to fetch in some round still
    // turns the indices it finds there into (unused) row loads, which must stay inside D
    for (int x = lane; x < DEPTH * K::NS * K::SLOT / 16; x += 32)
        *reinterpret_cast<uint4 *>(wsm + K::OFF_KV + 16 * x) = make_uint4(0u, 0u, 0u, 0u);
    __syncwarp();
    // unit records are read straight from global memory, one unit ahead of their use
    struct unit_head { int row, p0, p1; };
    auto load_head = [&](int u) {
        const int4 w = __ldg(reinterpret_cast<const int4 *>(units + u0 + u));   // out_row, dest, p0, p1
        unit_head h;
        h.row = w.x; h.p0 = w.z; h.p1 = w.w;
        return h;
    };
    auto load_sf = [&](int u) { return __ldg(&units[u0 + u].sf[q]); };

    // ---- fetcher: copies the data of one round (of this or a later unit) into ring slot `slot`
    int fu = 0, fr = 0;
    const unit_head h0 = load_head(0);
    unit_head fnext = load_head(nu > 1 ? 1 : 0);             // the unit the fetcher turns to next
    stream_range fs = stream_of(h0.p0, h0.p1, q);
    auto fetch_round = [&](int slot) {
        if (fu < nu) {
            const int pg = fs.base + K::STEPS * fr;
            if (pg < fs.hi && pg + K::STEPS > fs.lo && SA_CHK(lim.status, pg >= 0 && pg <= lim.nnz, 3, pg)) {
                const uint32_t dst = s_kv + slot * (K::NS * K::SLOT);
                // lanes 0 .. 3 of the stream copy the sixteen indices, lanes 4 .. 7 the sixteen values
                cp_async16_raw(dst + 16 * c, (c < 4 ? reinterpret_cast<const char *>(crd_k) : reinterpret_cast<const char *>(vals)) + 4 * int64_t(pg) + 16 * (c & 3));
                if (c == 0) cp_async4_raw(dst + 8 * K::STEPS, endbits + (pg >> 5));
            }
            if (++fr == fs.rounds) {
                fr = 0;
                if (++fu < nu) {
                    fs = stream_of(fnext.p0, fnext.p1, q);
                    if (fu + 1 < nu) fnext = load_head(fu + 1);
                }
            }
        }
        cp_async_commit();
    };
#pragma unroll
    for (int r = 0; r < DEPTH - 1; ++r) fetch_round(r);

    // ---- consumer state
    int cu = 0, cr = 0;
    stream_range cs = stream_of(h0.p0, h0.p1, q);
    int crow = h0.row;                                  // output row of the unit being consumed
    unit_head cnext = load_head(nu > 1 ? 1 : 0);        // the unit the consumer turns to next
    int fnext_q = load_sf(nu > 1 ? 1 : 0);              // and the fiber its stream q starts in
    int fq = load_sf(0);                                // next fiber this stream parks
    if (!SA_CHK(lim.status, uint32_t(fq) <= lim.n_fibers, 4, fq)) fq = 0;
    int jreg = __ldg(crd_j + fq + c);                   // C rows of the next eight fibers of the stream, one per lane
    const char *dlane = reinterpret_cast<const char *>(D + c * VEC);
    const uint32_t row_bytes = ldd * 4u;
    cp_async_wait<DEPTH - 2>();
    __syncwarp();
    rowvec<VEC> buf[8];                                  // rows of the round about to be consumed
    {
        const uint4 ka = lds128(s_kv), kb = lds128(s_kv + 16);
        const uint32_t k8[8] = {ka.x, ka.y, ka.z, ka.w, kb.x, kb.y, kb.z, kb.w};
#pragma unroll
        for (int s = 0; s < 8; ++s) buf[s].load(dlane + uint64_t(SA_CHK(lim.status, k8[s] < lim.d_rows, 5, k8[s]) ? k8[s] : 0u) * row_bytes);
    }
    float T[VEC];
#pragma unroll
    for (int x = 0; x < VEC; ++x) T[x] = 0.f;
    int rbase = 0, npend = 0, sc = 0;               // parked rows waiting for the tensor cores: rbase .. rbase + npend - 1
#ifdef SA_DEBUG_BOUNDS
    int dbg_rounds = 0;
#endif
    while (cu < nu) {
      const int rounds = cs.rounds;
#pragma unroll 1
      for (cr = 0; cr < rounds; ++cr) {
#ifdef SA_DEBUG_BOUNDS
        if (!SA_CHK(lim.status, ++dbg_rounds <= (1 << 16), 9, cs.rounds)) return;    // a task has at most ~300 rounds
#endif
        fetch_round(sc == 0 ? DEPTH - 1 : sc - 1);
        cp_async_wait<DEPTH - 2>();
        __syncwarp();
        const int sn = sc == DEPTH - 1 ? 0 : sc + 1;
        const uint32_t slot_c = s_kv + sc * (K::NS * K::SLOT), slot_n = s_kv + sn * (K::NS * K::SLOT);
        const uint32_t fw = lds32(slot_c + 8 * K::STEPS);
        // which of the sixteen positions pg .. pg + 15 belong to the stream, and which of them end a fiber
        const int pg = cs.base + K::STEPS * cr;
        const bool interior = cr >= 1 && cr < cs.full - 1;      // warp-uniform
        uint32_t vm = 0xffffu, e8 = (fw >> (pg & 16)) & 0xffffu;
        if (!interior) {
            const int a = min(max(cs.lo - pg, 0), K::STEPS), b = min(max(cs.hi - pg, 0), K::STEPS);
            vm = ((1u << b) - 1u) & ~((1u << a) - 1u);
            e8 &= vm;
            if (cs.hi > cs.lo && uint32_t(cs.hi - pg - 1) < uint32_t(K::STEPS)) e8 |= 1u << (cs.hi - pg - 1);   // the part's last nonzero closes its (possibly cut) fiber
        }
        // ring rows for the fibers this round parks: stream-major
        const int cnt = __popc(e8);
        int incl = cnt;
        {
            int o = __shfl_up_sync(SA_FULL_MASK, incl, 8);
            if (lane >= 8) incl += o;
            o = __shfl_up_sync(SA_FULL_MASK, incl, 16);
            if (lane >= 16) incl += o;
        }
        const int total = __shfl_sync(SA_FULL_MASK, incl, 31);
        if (rbase + npend + total > K::RING) {
            // move the (at most seven) rows left over to the front so that this round's rows fit behind them
            constexpr int CH = K::RS / 4;                          // 16-byte pieces per row
            for (int x = lane; x < npend * CH; x += 32) {
                const int r = x / CH, ch = x - r * CH;
                const uint4 w = lds128(s_ring + ((rbase + r) * K::RS) * 4 + 16 * ch);
                asm volatile("st.shared.v4.u32 [%0], {%1,%2,%3,%4};" ::"r"(s_ring + (r * K::RS) * 4 + 16 * ch), "r"(w.x), "r"(w.y), "r"(w.z), "r"(w.w) : "memory");
            }
            rbase = 0;
            __syncwarp();
        }
        const int slot = rbase + npend + incl - cnt;          // first row of this stream's fibers in this round
        npend += total;
        uint32_t waddr = s_ring + (slot * K::RS + c * VEC) * 4;
        if (c < cnt) {
            const uint32_t off = uint32_t(jreg) * ldc;
            sts32(s_ring + ((slot + c) * K::RS + M) * 4, off);
            prefetch_l1(C + off);
            if (c + 8 < cnt)                                  // more than eight fibers of one stream end in this round
                sts32(s_ring + ((slot + c + 8) * K::RS + M) * 4, uint32_t(__ldg(crd_j + fq + c + 8)) * ldc);
        }
        fq += cnt;
        const bool last = cr + 1 == rounds;
        if (last && cu + 1 < nu) fq = fnext_q;
        if (!SA_CHK(lim.status, uint32_t(fq) <= lim.n_fibers, 6, fq)) fq = 0;
        const int jnext = __ldg(crd_j + fq + c);
        // Sixteen steps: consume the row requested eight steps ago, then request the row eight steps ahead (of
        // this round, or of the first half of the next one) into the same registers.  MASKED: some stream of
        // the warp is at a ragged end of its part; positions outside the part contribute nothing (their rows
        // are not even read as numbers).
        auto steps = [&](auto masked) {
            constexpr bool MASKED = decltype(masked)::value;
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const uint4 vv = lds128(slot_c + 4 * K::STEPS + 16 * h);
                const uint4 kk = h < 2 ? lds128(slot_c + 32 + 16 * h) : lds128(slot_n + 16 * (h - 2));
                const float v4[4] = {__uint_as_float(vv.x), __uint_as_float(vv.y), __uint_as_float(vv.z), __uint_as_float(vv.w)};
                const uint32_t k4[4] = {kk.x, kk.y, kk.z, kk.w};
#pragma unroll
                for (int s4 = 0; s4 < 4; ++s4) {
                    const int s = 4 * h + s4, b = s & 7;
                    if (!MASKED || ((vm >> s) & 1u)) {
#pragma unroll
                        for (int x = 0; x < VEC; ++x) T[x] = fmaf(v4[s4], buf[b].x[x], T[x]);
                    }
                    buf[b].load(dlane + uint64_t(SA_CHK(lim.status, k4[s4] < lim.d_rows, 7, k4[s4]) ? k4[s4] : 0u) * row_bytes);
                    if (e8 & (1u << s)) {
                        rowvec<VEC> tv;
#pragma unroll
                        for (int x = 0; x < VEC; ++x) { tv.x[x] = T[x]; T[x] = 0.f; }
                        tv.store_shared(waddr);
                        waddr += K::RS * 4;
                    }
                }
            }
        };
        if (!interior && __any_sync(SA_FULL_MASK, vm != 0xffffu)) steps(std::true_type{});
        else steps(std::false_type{});
        __syncwarp();
        while (npend >= 8) {
            if (HAD) had_flush<M>(hacc, ring, rbase, 8, C, lane);
            else ttm3_flush<L, M>(acc, ring, rbase, 8, C, lane, lim, ldc);
            rbase += 8;
            npend -= 8;
        }
        __syncwarp();
        jreg = jnext;
        sc = sn;
      }
      // the unit ends: the open group of parked rows, the tile, the next unit
      {
        const int n = npend;
        if (n > 0) {
            if (HAD) {
                had_flush<M>(hacc, ring, rbase, n, C, lane);
            } else {
                for (int x = n; x < 8; ++x) ring[(rbase + x) * K::RS + lane % M] = 0.f;
                __syncwarp();
                ttm3_flush<L, M>(acc, ring, rbase, n, C, lane, lim, ldc);
            }
            __syncwarp();
        }
        rbase = npend = 0;
        if (!keep) {
            if (HAD) {
                if (M == 16) hacc += __shfl_xor_sync(SA_FULL_MASK, hacc, 16);
                if (lane < M && SA_CHK(lim.status, uint32_t(crow) < lim.n_slices_dim, 8, crow)) sa_st_cs(out + int64_t(crow) * M + lane, hacc);
                hacc = 0.f;
            } else if (TTMC) {
                if (SA_CHK(lim.status, uint32_t(crow) < lim.n_slices_dim, 8, crow)) ttmc_accumulate<L, M>(acc, *sink, crow, lane);
                zero_tile<L, M>(acc);
            } else {
                if (SA_CHK(lim.status, uint32_t(crow) < lim.n_slices_dim, 8, crow)) store_tile<L, M>(acc, out + int64_t(crow) * (L * M), lane, ring);
                zero_tile<L, M>(acc);
            }
        }
        ++cu;
        if (cu < nu) {
            cs = stream_of(cnext.p0, cnext.p1, q);
            crow = cnext.row;
            SA_CHK(lim.status, cs.rounds >= 1, 10, cu);
            if (cu + 1 < nu) {
                cnext = load_head(cu + 1);
                fnext_q = load_sf(cu + 1);
            }
        }
      }
    }
    cp_async_wait<0>();
    __syncwarp();
}

template <int L, int M, int NCTA, bool HAD>
__global__ void __launch_bounds__(32 * SA_TTM3_WARPS, NCTA)
ttm3_kernel(const sa_unit3 *__restrict__ units, const int32_t *__restrict__ task_start, int64_t n_tasks, int n_group_ctas,
            const int32_t *__restrict__ crd_j, const int32_t *__restrict__ crd_k, const float *__restrict__ vals,
            const uint32_t *__restrict__ endbits, const float *__restrict__ C, uint32_t ldc,
            const float *__restrict__ D, uint32_t ldd, float *__restrict__ out, float *__restrict__ partial,
            const dbg_limits lim)
{
    using K = cfg<L, M>;
    constexpr int TILE = HAD ? M : L * M;
    extern __shared__ __align__(16) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    unsigned char *wsm = smem + warp * K::WARP_BYTES;
    const int64_t task = int64_t(blockIdx.x) * SA_TTM3_WARPS + warp;
    const bool group = int(blockIdx.x) < n_group_ctas;
    float acc[K::MT][K::NT][4];
    float hacc = 0.f;
    zero_tile<L, M>(acc);
    int u0 = 0, u1 = 0;
    if (task < n_tasks) { u0 = task_start[task]; u1 = task_start[task + 1]; }
    if (u1 > u0)
        ttm3_warp_task<L, M, HAD>(units, u0, u1 - u0, crd_j, crd_k, vals, endbits, C, ldc, D, ldd, wsm, acc, hacc, group, out, lim);
    if (!group) return;                 // whole small slices: every tile was stored when its unit ended
    if (HAD) {
        // the warps hold partial rows of the same slice: sum them in a fixed order
        float *rows = reinterpret_cast<float *>(smem);
        if (M == 16) hacc += __shfl_xor_sync(SA_FULL_MASK, hacc, 16);
        __syncthreads();                // every warp is done with its shared memory
        if (lane < M) rows[warp * M + lane] = hacc;
        __syncthreads();
        const sa_unit3 lead = units[task_start[int64_t(blockIdx.x) * SA_TTM3_WARPS]];
        if (threadIdx.x < M) {
            float sum = rows[threadIdx.x];
#pragma unroll
            for (int w = 1; w < SA_TTM3_WARPS; ++w) sum += rows[w * M + threadIdx.x];
            float *dst = lead.dest >= 0 ? partial + int64_t(lead.dest) * TILE : out + int64_t(lead.out_row) * TILE;
            dst[threadIdx.x] = sum;
        }
        return;
    }
    // the CTA's warps hold partial tiles of the same slice: sum them in a fixed order
    float *wt = reinterpret_cast<float *>(wsm);
#pragma unroll
    for (int mt = 0; mt < K::MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < K::NT; ++nt) {
            const int l = 16 * mt + g, mm = 8 * nt + 2 * t;
            *reinterpret_cast<float2 *>(wt + l * K::RS + mm) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
            *reinterpret_cast<float2 *>(wt + (l + 8) * K::RS + mm) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
        }
    __syncthreads();
    const sa_unit3 lead = units[task_start[int64_t(blockIdx.x) * SA_TTM3_WARPS]];   // warp 0 always has a unit
    float *dst = lead.dest >= 0 ? partial + int64_t(lead.dest) * TILE : out + int64_t(lead.out_row) * TILE;
    const float *all = reinterpret_cast<const float *>(smem);
    for (int x = threadIdx.x * 4; x < TILE; x += 32 * SA_TTM3_WARPS * 4) {
        const int off = (x / M) * K::RS + (x % M);
        float4 s = *reinterpret_cast<const float4 *>(all + off);
#pragma unroll
        for (int w = 1; w < SA_TTM3_WARPS; ++w) {
            const float4 v = *reinterpret_cast<const float4 *>(all + w * (K::WARP_BYTES / 4) + off);
            s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
        }
        if (lead.dest >= 0) *reinterpret_cast<float4 *>(dst + x) = s;
        else sa_st_cs4(dst + x, s);
    }
}

// Kernel 5 with the loop over i kept fused (second schedule of the 3-D TTMC row of the Table of kernels, the slice
// temporary never leaving the chip): the slice stage of kernel 6 with (D, E) as factors, whose finished temporaries
// T(i; m,n) are contracted with C(i,:) into an L3 x L x M accumulator in the block's shared memory.  Blocks are
// persistent (block b takes the block-tasks b, b + grid, ...: chunks of large slices first, then tasks of small
// slices) and write their accumulators to `partials` (grid x L3 x L x M), which a second kernel adds in block order.
// Nothing is needed for split slices: the contraction is linear, every chunk adds its share.
template <int L, int M, int NCTA>
__global__ void __launch_bounds__(32 * SA_TTM3_WARPS, NCTA)
ttmc3_fused_kernel(const sa_unit3 *__restrict__ units, const int32_t *__restrict__ task_start, int64_t n_tasks, int n_group_ctas,
                   const int32_t *__restrict__ crd_j, const int32_t *__restrict__ crd_k, const float *__restrict__ vals,
                   const uint32_t *__restrict__ endbits, const float *__restrict__ C, uint32_t ldc,
                   const float *__restrict__ D, uint32_t ldd, const float *__restrict__ C3, uint32_t ldc3, int L3,
                   float *__restrict__ partials, const dbg_limits lim)
{
    using K = cfg<L, M>;
    constexpr int TILE = L * M;
    extern __shared__ __align__(16) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    unsigned char *wsm = smem + warp * K::WARP_BYTES;
    float *accs = reinterpret_cast<float *>(smem + SA_TTM3_WARPS * K::WARP_BYTES);
    const int n_acc = L3 * TILE;
    for (int x = threadIdx.x; x < n_acc; x += 32 * SA_TTM3_WARPS) accs[x] = 0.f;
    __syncthreads();
    ttmc_sink sink;
    sink.C3 = C3; sink.ldc3 = ldc3; sink.L3 = L3; sink.accs = accs;
    const int64_t n_block_tasks = (n_tasks + SA_TTM3_WARPS - 1) / SA_TTM3_WARPS;
    for (int64_t bt = blockIdx.x; bt < n_block_tasks; bt += gridDim.x) {
        const int64_t task = bt * SA_TTM3_WARPS + warp;
        const bool group = bt < n_group_ctas;          // the same for all warps of the block
        float acc[K::MT][K::NT][4];
        float hacc = 0.f;
        zero_tile<L, M>(acc);
        int u0 = 0, u1 = 0;
        if (task < n_tasks) { u0 = task_start[task]; u1 = task_start[task + 1]; }
        if (u1 > u0)
            ttm3_warp_task<L, M, false, true>(units, u0, u1 - u0, crd_j, crd_k, vals, endbits, C, ldc, D, ldd, wsm, acc, hacc, group,
                                              nullptr, lim, &sink);
        if (!group) continue;              // whole small slices: added to the accumulator when their units ended
        // the block's warps hold partial temporaries of the same slice: sum them, then one rank-1 update
        __syncthreads();                   // every warp is done with its shared-memory region
        float *wt = reinterpret_cast<float *>(wsm);
#pragma unroll
        for (int mt = 0; mt < K::MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < K::NT; ++nt) {
                const int l = 16 * mt + g, mm = 8 * nt + 2 * t;
                *reinterpret_cast<float2 *>(wt + l * K::RS + mm) = make_float2(acc[mt][nt][0], acc[mt][nt][1]);
                *reinterpret_cast<float2 *>(wt + (l + 8) * K::RS + mm) = make_float2(acc[mt][nt][2], acc[mt][nt][3]);
            }
        __syncthreads();
        const int row = units[task_start[bt * SA_TTM3_WARPS]].out_row;       // warp 0 always has a unit
        const float *all = reinterpret_cast<const float *>(smem);
        if (SA_CHK(lim.status, uint32_t(row) < lim.n_slices_dim, 8, row)) {
            const float *crow = C3 + uint32_t(row) * ldc3;
            for (int x = threadIdx.x * 4; x < TILE; x += 32 * SA_TTM3_WARPS * 4) {
                const int off = (x / M) * K::RS + (x % M);
                float4 s = *reinterpret_cast<const float4 *>(all + off);
#pragma unroll
                for (int w = 1; w < SA_TTM3_WARPS; ++w) {
                    const float4 v = *reinterpret_cast<const float4 *>(all + w * (K::WARP_BYTES / 4) + off);
                    s.x += v.x; s.y += v.y; s.z += v.z; s.w += v.w;
                }
                for (int l = 0; l < L3; ++l) {          // no other warp touches the accumulator during a chunk
                    const float c = __ldg(crow + l);
                    float4 *a = reinterpret_cast<float4 *>(accs + l * TILE + x);
                    float4 o = *a;
                    o.x = fmaf(c, s.x, o.x); o.y = fmaf(c, s.y, o.y); o.z = fmaf(c, s.z, o.z); o.w = fmaf(c, s.w, o.w);
                    *a = o;
                }
            }
        }
        __syncthreads();                   // the next block-task reuses the warps' regions
    }
    __syncthreads();
    float *dst = partials + int64_t(blockIdx.x) * n_acc;
    for (int x = threadIdx.x; x < n_acc; x += 32 * SA_TTM3_WARPS) dst[x] = accs[x];
}

template <int L, int M, bool HAD>
cudaError_t launch(const sa_ttm3_view &v, const sa_dense &first, const sa_dense &second, float *out, float *partial,
                   cudaStream_t stream)
{
    const sa_worklist &wl = *v.wl;
    const int64_t n_tasks = int64_t(wl.task_start.size()) - 1;
    const int64_t ctas = (n_tasks + SA_TTM3_WARPS - 1) / SA_TTM3_WARPS;
    if (ctas <= 0) return cudaSuccess;
    constexpr size_t smem = size_t(SA_TTM3_WARPS) * cfg<L, M>::WARP_BYTES;
    const bool short_units = v.nnz < int64_t(512) * int64_t(wl.items.size());          // mean unit below 512 nonzeros
    auto kern = short_units ? ttm3_kernel<L, M, cfg<L, M>::MINCTAS_SHORT, HAD> : ttm3_kernel<L, M, cfg<L, M>::MINCTAS, HAD>;
    static bool attr_long[SA_MAX_DEVICE_FLAGS], attr_short[SA_MAX_DEVICE_FLAGS];     // per instantiation of this launcher
    if (!sa_set_smem_once(kern, int(smem), short_units ? attr_short : attr_long)) return cudaGetLastError();
    dbg_limits lim;
    lim.status = v.status;
    lim.c_rows = uint32_t(first.rows); lim.d_rows = uint32_t(second.rows);
    lim.n_fibers = uint32_t(v.n_fibers); lim.n_slices_dim = uint32_t(v.n_out_rows);
    lim.nnz = v.nnz_total;
    kern<<<(unsigned)ctas, 32 * SA_TTM3_WARPS, smem, stream>>>(wl.d_units3, wl.d_task_start, n_tasks, int(wl.n_group_ctas), v.crd_fiber,
                                                              v.crd_nz, v.vals, v.endbits, first.ptr, uint32_t(first.ld), second.ptr,
                                                              uint32_t(second.ld), out, partial, lim);
    return cudaGetLastError();
}

}  // namespace

bool sa_ranks_ok_ttm3(int64_t L, int64_t M) { return (L == 16 || L == 32) && (M == 16 || M == 32); }

size_t sa_ws_ttm3(const sa_tensor *t, const sa_dense *ops)
{
    return sa_align256(size_t(t->wl_main.n_slots) * size_t(ops[0].cols * ops[1].cols) * sizeof(float));
}

sa_status sa_launch_ttm3_view(const sa_ttm3_view &v, const sa_dense &first, const sa_dense &second, float *out,
                              float *partial, cudaStream_t stream, int *launches)
{
    const int64_t L = first.cols, M = second.cols;
    // the kernel addresses factor rows with 32-bit offsets
    if (first.rows * first.ld >= (int64_t(1) << 30) || second.rows * second.ld >= (int64_t(1) << 30)) return SA_E_UNSUPPORTED;
    if (!v.endbits) return SA_E_UNSUPPORTED;
    cudaError_t e;
    if (L == 16 && M == 16) e = launch<16, 16, false>(v, first, second, out, partial, stream);
    else if (L == 32 && M == 16) e = launch<32, 16, false>(v, first, second, out, partial, stream);
    else if (L == 16 && M == 32) e = launch<16, 32, false>(v, first, second, out, partial, stream);
    else if (L == 32 && M == 32) e = launch<32, 32, false>(v, first, second, out, partial, stream);
    else return SA_E_UNSUPPORTED;
    if (e != cudaSuccess) return SA_E_CUDA;
    *launches = v.wl->items.empty() ? 0 : 1;
    if (!v.wl->fix.empty()) {
        if (sa_launch_fixup(*v.wl, partial, out, int(L * M), stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}

sa_status sa_launch_ttm3(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t ws_bytes,
                         cudaStream_t stream, int *launches)
{
    (void)ws_bytes;
    sa_ttm3_view v;
    v.wl = &t->wl_main;
    v.crd_fiber = t->d_crd[1];
    v.crd_nz = t->d_crd[2];
    v.vals = t->d_vals;
    v.endbits = t->d_endbits;
    v.n_fibers = t->count[1];
    v.n_out_rows = t->dims[0];
    v.nnz = t->nnz;
    v.nnz_total = t->nnz;
    v.status = t->d_status;
    return sa_launch_ttm3_view(v, ops[0], ops[1], out, static_cast<float *>(ws), stream, launches);
}

// Kernel 5, fused over i: grid size and shared memory of ttmc3_fused_kernel for temporaries of M x N and L3 columns of C.
template <int L, int M>
static bool ttmc3_fused_shape(int L3, int *grid, size_t *smem_bytes)
{
    const size_t smem = size_t(SA_TTM3_WARPS) * cfg<L, M>::WARP_BYTES + size_t(L3) * L * M * sizeof(float);
    auto kern = ttmc3_fused_kernel<L, M, 4>;
    int dev = 0, sms = 148, per_sm = 0;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) != cudaSuccess ||
        cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 32 * SA_TTM3_WARPS, smem) != cudaSuccess || per_sm < 1) {
        cudaGetLastError();
        return false;
    }
    *grid = sms * per_sm;
    *smem_bytes = smem;
    return true;
}

// Accumulator elements the fused schedule of kernel 5 keeps per block; beyond this only the fissioned schedule runs.
constexpr int64_t SA_TTMC3_FUSED_MAX = 8192;
// Upper bound on the blocks of the fused schedule (sizes the workspace without asking the device).
constexpr int SA_TTMC3_MAX_BLOCKS = 148 * 6 * 2;

bool sa_ttmc3_fused_ok(int64_t L3, int64_t M, int64_t N) { return L3 * M * N <= SA_TTMC3_FUSED_MAX; }
size_t sa_ws_ttmc3_fused(int64_t L3, int64_t M, int64_t N) { return sa_align256(size_t(SA_TTMC3_MAX_BLOCKS) * size_t(L3 * M * N) * sizeof(float)); }

// Launches ttmc3_fused_kernel; *n_blocks receives the number of partial accumulators written to `partials`.
sa_status sa_launch_ttmc3_fused_stage(const sa_tensor *t, const sa_dense &C3, const sa_dense &D, const sa_dense &E, float *partials,
                                      cudaStream_t stream, int *n_blocks)
{
    const int64_t M = D.cols, N = E.cols;
    if (D.rows * D.ld >= (int64_t(1) << 30) || E.rows * E.ld >= (int64_t(1) << 30) || C3.rows * C3.ld >= (int64_t(1) << 30)) return SA_E_UNSUPPORTED;
    if (!t->d_endbits || !sa_ttmc3_fused_ok(C3.cols, M, N)) return SA_E_UNSUPPORTED;
    const sa_worklist &wl = t->wl_main;
    const int64_t n_tasks = int64_t(wl.task_start.size()) - 1;
    const int64_t n_block_tasks = (n_tasks + SA_TTM3_WARPS - 1) / SA_TTM3_WARPS;
    *n_blocks = 0;
    if (n_block_tasks <= 0) return SA_OK;
    dbg_limits lim;
    lim.status = t->d_status;
    lim.c_rows = uint32_t(D.rows); lim.d_rows = uint32_t(E.rows);
    lim.n_fibers = uint32_t(t->count[1]); lim.n_slices_dim = uint32_t(t->dims[0]);
    lim.nnz = t->nnz;
    int grid = 0;
    size_t smem = 0;
#define SA_TTMC_CASE(m, n)                                                                                                        \
    if (M == m && N == n) {                                                                                                       \
        if (!ttmc3_fused_shape<m, n>(int(C3.cols), &grid, &smem)) return SA_E_CUDA;                                               \
        grid = int(std::min<int64_t>(std::min<int64_t>(grid, SA_TTMC3_MAX_BLOCKS), n_block_tasks));                               \
        ttmc3_fused_kernel<m, n, 4><<<unsigned(grid), 32 * SA_TTM3_WARPS, smem, stream>>>(                                        \
            wl.d_units3, wl.d_task_start, n_tasks, int(wl.n_group_ctas), t->d_crd[1], t->d_crd[2], t->d_vals, t->d_endbits, D.ptr, \
            uint32_t(D.ld), E.ptr, uint32_t(E.ld), C3.ptr, uint32_t(C3.ld), int(C3.cols), partials, lim);                         \
        if (cudaGetLastError() != cudaSuccess) return SA_E_CUDA;                                                                  \
        *n_blocks = grid;                                                                                                         \
        return SA_OK;                                                                                                             \
    }
    SA_TTMC_CASE(16, 16) SA_TTMC_CASE(16, 32) SA_TTMC_CASE(32, 16)
#undef SA_TTMC_CASE
    return SA_E_UNSUPPORTED;
}

// Kernel 8, first stage (MTTKRP): T(i,r) = sum_{j,k} B(i,j,k) C(j,r) D(k,r), R = 32 or 16 columns, one row of R
// floats per slice written to `out` (empty slices zero), partial rows of split slices to `partial`.
sa_status sa_launch_mttkrp_rows(const sa_tensor *t, const sa_dense &C, const sa_dense &D, float *out, float *partial,
                                cudaStream_t stream, int *launches)
{
    const int64_t R = C.cols;
    if (D.cols != R || (R != 32 && R != 16)) return SA_E_UNSUPPORTED;
    if (C.rows * C.ld >= (int64_t(1) << 30) || D.rows * D.ld >= (int64_t(1) << 30) || !t->d_endbits) return SA_E_UNSUPPORTED;
    sa_ttm3_view v;
    v.wl = &t->wl_main;
    v.crd_fiber = t->d_crd[1];
    v.crd_nz = t->d_crd[2];
    v.vals = t->d_vals;
    v.endbits = t->d_endbits;
    v.n_fibers = t->count[1];
    v.n_out_rows = t->dims[0];
    v.nnz = t->nnz;
    v.nnz_total = t->nnz;
    v.status = t->d_status;
    const cudaError_t e = R == 32 ? launch<16, 32, true>(v, C, D, out, partial, stream) : launch<16, 16, true>(v, C, D, out, partial, stream);
    if (e != cudaSuccess) return SA_E_CUDA;
    *launches = v.wl->items.empty() ? 0 : 1;
    if (!v.wl->fix.empty()) {
        if (sa_launch_fixup(*v.wl, partial, out, int(R), stream) != cudaSuccess) return SA_E_CUDA;
        *launches += 1;
    }
    return SA_OK;
}

// ------------------------------------------------------------------ entry point without allocation

// Scratch for sa_run_ttm3_static_scratch: part of the library image, so every device that loads the
// library carries these 4 MiB until the process exits.
constexpr size_t SA_STATIC_SCRATCH_BYTES = size_t(4) << 20;
static __device__ __align__(256) float sa_static_scratch[SA_STATIC_SCRATCH_BYTES / sizeof(float)];

namespace {

constexpr int SA_MAX_DEVICES = 64;
float *g_static_scratch_addr[SA_MAX_DEVICES];   // device address of sa_static_scratch, per device; set once

// In host code `sa_static_scratch` only names the symbol; the address a kernel can use has to be
// asked for, with the owning device current.
sa_status static_scratch_address(int device, float **addr)
{
    if (device < 0 || device >= SA_MAX_DEVICES) return SA_E_ARG;
    if (!g_static_scratch_addr[device]) {
        float *p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void **>(&p), sa_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return SA_E_CUDA;
        }
        g_static_scratch_addr[device] = p;
    }
    *addr = g_static_scratch_addr[device];
    return SA_OK;
}

}  // namespace

extern "C" sa_status sa_run_ttm3_static_scratch(const sa_tensor *t, const sa_dense *ops, int n_ops, float *out,
                                                void *cuda_stream)
{
    if (!t || !ops || !out || n_ops != 2 || t->device < 0) return SA_E_ARG;
    if (reinterpret_cast<uintptr_t>(out) % 16) return SA_E_ARG;
    if (t->fmt != SA_FMT_CSF || t->order != 3) return SA_E_FORMAT;
    for (int i = 0; i < 2; ++i) {
        if (!ops[i].ptr) return SA_E_ARG;
        if (ops[i].rows != t->dims[i + 1] || ops[i].cols <= 0 || ops[i].ld < ops[i].cols || ops[i].ld % 4 ||
            reinterpret_cast<uintptr_t>(ops[i].ptr) % 16)
            return SA_E_SHAPE;
    }
    if (!sa_ranks_ok_ttm3(ops[0].cols, ops[1].cols)) return SA_E_UNSUPPORTED;
    const size_t need = sa_ws_ttm3(t, ops);
    if (need > SA_STATIC_SCRATCH_BYTES) return SA_E_WORKSPACE;   // the partial tiles do not fit the built-in scratch
    int prev = -1;
    if (cudaGetDevice(&prev) != cudaSuccess) { cudaGetLastError(); return SA_E_CUDA; }
    if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) { cudaGetLastError(); return SA_E_CUDA; }
    float *scratch = nullptr;
    sa_status s = static_scratch_address(t->device, &scratch);
    int launches = 0;
    if (s == SA_OK)
        s = sa_launch_ttm3(t, ops, out, scratch, SA_STATIC_SCRATCH_BYTES, static_cast<cudaStream_t>(cuda_stream), &launches);
    if (s == SA_E_CUDA) cudaGetLastError();
    if (s == SA_OK) t->last_launches = launches;
    if (prev != t->device) cudaSetDevice(prev);
    return s;
}
