// RMSNorm forward device kernels (paper Table 3 "rmsnorm": warp-shuffle reduction + fast
// rsqrt, weight multiply fused into the epilogue per Section 7.3 Tier 3).
//
//   y[r, j] = rne( x[r, j] * rsqrt(mean_k x[r, k]^2 + eps) * w[j] )
//
// One DRAM read and one DRAM write per element, fp32 accumulation, fixed-order reductions.
// Every kernel takes the element type DT (bf16, fp16 or fp32) as a template parameter; sizes
// are counted in 16-byte vectors (8 or 4 elements).  The phase-staged and the multi-pass
// kernels address 2-byte elements and serve the 16-bit types; fp32 rows that are not 16-byte
// aligned go to rmsnorm_generic32_kernel.
#pragma once

#include "ak_common.cuh"

namespace ak {

// Vector helpers, one 16-byte vector at a time, per element type.
//
// 16-bit types use the mixed-precision forms (sm_100): the multiply-add reads its bf16 / fp16
// operands straight from the two halves of a packed word and accumulates in fp32, so no
// widening instruction is spent.  x*x + s and x*w are exact products (8-bit x 8-bit or
// 11-bit x 11-bit significands) with one rounding.  (The packed f32x2 formulation measured 2 %
// slower sustained with 14 more registers.)
__device__ __forceinline__ void halves(uint32_t u, uint16_t& lo, uint16_t& hi) {
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(u));
}
template <int DT>
__device__ __forceinline__ float sumsq_v(const uint4& v) {
    if constexpr (DT == AK_DTYPE_F32) {
        const float a = __uint_as_float(v.x), b = __uint_as_float(v.y), c = __uint_as_float(v.z), d = __uint_as_float(v.w);
        return fmaf(c, c, a * a) + fmaf(d, d, b * b);
    } else {
        using E = Elem<DT>;
        uint16_t a0, a1, a2, a3, a4, a5, a6, a7;
        halves(v.x, a0, a1); halves(v.y, a2, a3); halves(v.z, a4, a5); halves(v.w, a6, a7);
        float s0 = E::fma_h(a0, a0, 0.0f), s1 = E::fma_h(a1, a1, 0.0f);
        s0 = E::fma_h(a2, a2, s0); s1 = E::fma_h(a3, a3, s1);
        s0 = E::fma_h(a4, a4, s0); s1 = E::fma_h(a5, a5, s1);
        s0 = E::fma_h(a6, a6, s0); s1 = E::fma_h(a7, a7, s1);
        return s0 + s1;
    }
}
template <int DT>
__device__ __forceinline__ uint32_t scale2(uint32_t x, uint32_t w, f32x2 rstd2) {
    using E = Elem<DT>;
    uint16_t x0, x1, w0, w1;
    halves(x, x0, x1); halves(w, w0, w1);
    const f32x2 p = mul2(pack2(E::fma_h(x0, w0, 0.0f), E::fma_h(x1, w1, 0.0f)), rstd2);
    float lo, hi;
    unpack2(p, lo, hi);
    return E::pack(lo, hi);
}
// (x * w) * rstd per element, one rounding to the output type (fp32: (x * rstd) * w)
template <int DT>
__device__ __forceinline__ uint4 scale_v(const uint4& x, const uint4& w, float rstd) {
    if constexpr (DT == AK_DTYPE_F32) {
        return make_uint4(__float_as_uint(__uint_as_float(x.x) * rstd * __uint_as_float(w.x)),
                          __float_as_uint(__uint_as_float(x.y) * rstd * __uint_as_float(w.y)),
                          __float_as_uint(__uint_as_float(x.z) * rstd * __uint_as_float(w.z)),
                          __float_as_uint(__uint_as_float(x.w) * rstd * __uint_as_float(w.w)));
    } else {
        const f32x2 r2 = pack2(rstd, rstd);
        return make_uint4(scale2<DT>(x.x, w.x, r2), scale2<DT>(x.y, w.y, r2), scale2<DT>(x.z, w.z, r2),
                          scale2<DT>(x.w, w.w, r2));
    }
}

// ------------------------------------------------------------------ row in registers
// A CTA of THREADS threads is cut into THREADS / GROUP groups; one group owns one row and
// each of its threads holds VPT 16-byte vectors of it as packed bf16 (vector i of the row
// lives in thread i % GROUP, slot i / GROUP, so every load instruction is a contiguous
// GROUP * 16-byte segment).  GROUP == 32 is the warp-per-row layout (no barrier at all),
// GROUP == THREADS the CTA-per-row layout.  All of a thread's loads are issued before the
// first use.  The weight vectors are fetched through L1 (they are shared by every row)
// either before the reduction (W_EARLY: latency hidden behind the row loads, 4 * VPT more
// live registers) or after it.  MINB is the launch-bounds occupancy hint that caps the
// register count.  The grid may be smaller than the number of row slots: groups then walk
// the rows with a grid stride.  FULL: nvec == VPT * GROUP, the rows fill the CTAs' groups exactly
// and the grid has one CTA per group of rows, so nothing tests a bound and the body runs once.
template <int THREADS, int GROUP, int VPT, int MINB, bool W_EARLY, int DT = AK_DTYPE_BF16, bool FULL = false>
__global__ void __launch_bounds__(THREADS, MINB)
rmsnorm_reg_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w, uint4* __restrict__ y,
                   int64_t rows, int nvec, float inv_D, float eps, int first_wave) {
    constexpr int GROUPS = THREADS / GROUP;
    constexpr int WARPS_PER_GROUP = GROUP / kWarp;
    static_assert(GROUP % kWarp == 0 && THREADS % GROUP == 0, "groups are whole warps");
    __shared__ float slots[2][THREADS / kWarp];
    {
        const int64_t r0 = (int64_t)blockIdx.x * GROUPS;
        const int64_t nr = rows - r0 < GROUPS ? rows - r0 : GROUPS;
        pdl_prologue(x + r0 * nvec, nr * nvec * 16, first_wave);
    }
    const int g = threadIdx.x / GROUP;
    const int t = threadIdx.x % GROUP;
    const int lane = threadIdx.x & 31;
    const int warp_in_group = t >> 5;

    uint4 wv[VPT];
    if constexpr (W_EARLY) {
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = t + k * GROUP;
            wv[k] = (FULL || i < nvec) ? __ldg(w + i) : make_uint4(0, 0, 0, 0);
        }
    }
    int phase = 0;
    // Whole CTAs iterate together (rows beyond the end are masked, not skipped) so the
    // barrier below is reached by every thread.
    for (int64_t row0 = (int64_t)blockIdx.x * GROUPS; FULL || row0 < rows; row0 += (int64_t)gridDim.x * GROUPS) {
        const int64_t row = row0 + g;
        const bool live = FULL || row < rows;
        const uint4* xr = x + row * nvec;
        uint4 xv[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = t + k * GROUP;
            xv[k] = (FULL || (live && i < nvec)) ? ld_stream(xr + i) : make_uint4(0, 0, 0, 0);
        }
        float ss = 0.0f;
#pragma unroll
        for (int k = 0; k < VPT; ++k) ss += sumsq_v<DT>(xv[k]);
        ss = warp_sum(ss);
        if constexpr (WARPS_PER_GROUP > 1) {
            float* s = slots[phase] + g * WARPS_PER_GROUP;
            if (lane == 0) s[warp_in_group] = ss;
            __syncthreads();
            float v = (lane < WARPS_PER_GROUP) ? s[lane] : 0.0f;
            ss = warp_sum(v);
            phase ^= 1;
        }
        const float rstd = rsqrtf(fmaf(ss, inv_D, eps));
        uint4* yr = y + row * nvec;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = t + k * GROUP;
            if (FULL || (live && i < nvec)) {
                const uint4 wq = W_EARLY ? wv[k] : __ldg(w + i);
                st_stream(yr + i, scale_v<DT>(xv[k], wq, rstd));
            }
        }
        if constexpr (FULL) break;   // the grid has one CTA per group of rows
    }
}

// ------------------------------------------------------------------ long rows staged in shared memory
// One CTA per row.  One thread asks the copy engine for the whole row (bulk copies of at
// most kBulkChunk bytes, all counted in by one mbarrier), so the bytes in flight per SM
// are bounded by shared memory (resident CTAs x row bytes), not by registers.  The row is
// then read twice from shared memory: sum of squares, then scale and store.  Needs
// 16-byte aligned rows (D % 8 == 0).  Dynamic shared memory = nvec * 16 bytes.
constexpr uint32_t kBulkChunk = 32768;

template <int THREADS, int MINB, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(THREADS, MINB)
rmsnorm_smem_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w, uint4* __restrict__ y,
                    int nvec, float inv_D, float eps) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint4* row = reinterpret_cast<uint4*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[2 * kWarp];
    const int64_t r = blockIdx.x;
    if (threadIdx.x == 0) mbar_init(&bar, 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t bytes = (uint32_t)nvec * 16u;
        mbar_expect_tx(&bar, bytes);
        const unsigned char* src = reinterpret_cast<const unsigned char*>(x + r * nvec);
        for (uint32_t off = 0; off < bytes; off += kBulkChunk)
            bulk_load(smem_raw + off, src + off, min(kBulkChunk, bytes - off), &bar);
    }
    if (!mbar_wait(&bar, 0)) return;  // gave up (flag set, see ak_wait_timeouts): a thread that exits no longer counts at later barriers
    float ss = 0.0f;
#pragma unroll 4
    for (int i = threadIdx.x; i < nvec; i += THREADS) ss += sumsq_v<DT>(row[i]);
    ss = cta_sum<THREADS>(ss, slots, 0);
    const float rstd = rsqrtf(fmaf(ss, inv_D, eps));
    uint4* yr = y + r * nvec;
#pragma unroll 4
    for (int i = threadIdx.x; i < nvec; i += THREADS) st_stream(yr + i, scale_v<DT>(row[i], __ldg(w + i), rstd));
}

// ------------------------------------------------------------------ rows split over a cluster
// C CTAs of a thread-block cluster share one row: few rows then still fill the GPU, and rows of
// up to C x 224 KiB are normalised in one pass over DRAM.  CTA c stages vectors
// [nvec * c / C, nvec * (c + 1) / C) in its shared memory by bulk copies, sums its squares, and
// the C partial sums meet through distributed shared memory (a mailbox exchange; added in rank
// order in every CTA, so all hold the same bits).  grid = rows * C, cluster = C.  Dynamic shared memory = the
// largest slice, ceil(nvec / C) * 16 bytes.
template <int THREADS, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(THREADS)
rmsnorm_cluster_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w, uint4* __restrict__ y,
                       int nvec, int C, float inv_D, float eps) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint4* row = reinterpret_cast<const uint4*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[2 * kWarp];
    __shared__ float box[kMaxCluster];
    __shared__ uint64_t xbar;
    const uint32_t c = cluster_rank();
    const int64_t r = blockIdx.x / C;
    const int v0 = (int)((int64_t)nvec * c / C);
    const int n = (int)((int64_t)nvec * (c + 1) / C) - v0;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mailbox_arm(&xbar, C);
    }
    __syncthreads();
    if (threadIdx.x == 0) bulk_load_span(smem_raw, x + r * nvec + v0, (uint32_t)n * 16u, &bar);
    cluster_arrive_relaxed();
    // a wait that gave up (never expected) contributes nothing and writes nothing, but still posts
    int nn = mbar_wait(&bar, 0) ? n : 0;
    float ss = 0.0f;
#pragma unroll 4
    for (int i = threadIdx.x; i < nn; i += THREADS) ss += sumsq_v<DT>(row[i]);
    ss = cta_sum<THREADS>(ss, slots, 0);
    cluster_wait();   // every CTA of the cluster runs, its mailboxes armed, before anything is posted to it
    if (!mailbox_exchange(ss, box, &xbar, C, c)) nn = 0;
    float tot = 0.0f;
    for (int i = 0; i < C; ++i) tot += box[i];
    const float rstd = rsqrtf(fmaf(tot, inv_D, eps));
    uint4* yr = y + r * nvec + v0;
    const uint4* wr = w + v0;
#pragma unroll 4
    for (int i = threadIdx.x; i < nn; i += THREADS) st_stream(yr + i, scale_v<DT>(row[i], __ldg(wr + i), rstd));
}

// ------------------------------------------------------------------ rows of any length streamed by a cluster
// Rows too long for the shared memory of eight CTAs: the C CTAs of a cluster each stream their
// slice of the row from global memory twice, once for the sum of squares (partial sums through the
// mailbox) and once more to scale and store; the second read finds what the caches kept (nothing
// is staged).  Needs 16-byte aligned rows.  grid = rows * C, cluster = C.
template <int T, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(T, 1)
rmsnorm_cluster_stream_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w, uint4* __restrict__ y,
                              int64_t nvec, int C, float inv_D, float eps) {
    __shared__ float slots[2 * kWarp];
    __shared__ float box[kMaxCluster];
    __shared__ uint64_t xbar;
    const uint32_t c = cluster_rank();
    const int64_t r = blockIdx.x / C;
    const int64_t v0 = nvec / C * c + min((int64_t)c, nvec % C);
    const int64_t v1 = v0 + nvec / C + ((int64_t)c < nvec % C ? 1 : 0);
    if (threadIdx.x == 0) mailbox_arm(&xbar, C);
    __syncthreads();
    cluster_arrive_relaxed();
    const uint4* xr = x + r * nvec;
    float ss = 0.0f;
#pragma unroll 8
    for (int64_t i = v0 + threadIdx.x; i < v1; i += T) ss += sumsq_v<DT>(xr[i]);
    ss = cta_sum<T>(ss, slots, 0);
    cluster_wait();   // every CTA of the cluster runs, its mailbox armed, before anything is posted to it
    const bool ok = mailbox_exchange(ss, box, &xbar, C, c);
    float tot = 0.0f;
    for (int i = 0; i < C; ++i) tot += box[i];
    const float rstd = rsqrtf(fmaf(tot, inv_D, eps));
    if (!ok) return;   // a wait that gave up (never expected): nothing is written
    uint4* yr = y + r * nvec;
#pragma unroll 4
    for (int64_t i = v0 + threadIdx.x; i < v1; i += T) st_stream(yr + i, scale_v<DT>(ld_stream(xr + i), __ldg(w + i), rstd));
}

// ------------------------------------------------------------------ unaligned rows staged in shared memory
// D % 8 != 0 (or a misaligned base) makes the 16-byte phase of a row change from row to row.
// One CTA per row copies the row into shared memory in the phase it has in global memory:
// vector k of the staging buffer holds row elements [8k - phase, 8k - phase + 8), so the run of
// fully-inside vectors is 16-byte aligned on both sides and arrives by bulk (TMA) copies, and,
// because x and y rows share the phase here, every one of them leaves by an aligned 16-byte store.  The (at most two) edge vectors are filled element
// by element, zeros standing in for the neighbours' bytes, and written back element by
// element, so nothing outside the row is ever read or written.  Weights for an inside vector
// start at the odd or even element 8k - phase: four 4-byte loads (phase even) or five plus
// funnel shifts (phase odd), all L1 hits.  Needs w 4-byte aligned and the row to fit.
// (T threads per CTA: 128 up to D = 8192, where many small CTAs per SM matter most, more above)

__device__ __forceinline__ uint4 load_w_shifted(const uint16_t* __restrict__ w, int64_t j0) {
    // j0 >= 0: first weight index of the vector; w is 4-byte aligned
    const uint32_t* ww = reinterpret_cast<const uint32_t*>(w) + (j0 >> 1);
    if ((j0 & 1) == 0) return make_uint4(__ldg(ww), __ldg(ww + 1), __ldg(ww + 2), __ldg(ww + 3));
    // the fifth word would reach one element past j0 + 7 (possibly past the end of w): only
    // its low half is needed, so fetch that half alone
    const uint32_t a = __ldg(ww), b = __ldg(ww + 1), c = __ldg(ww + 2), d = __ldg(ww + 3);
    const uint32_t e = (uint32_t)__ldg(w + j0 + 7);
    return make_uint4(__funnelshift_r(a, b, 16), __funnelshift_r(b, c, 16), __funnelshift_r(c, d, 16),
                      __funnelshift_r(d, e, 16));
}

template <int T, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(T)
rmsnorm_stage_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w, uint16_t* __restrict__ y,
                     int64_t D, float inv_D, float eps, int first_wave) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint4* row = reinterpret_cast<uint4*>(smem_raw);
    uint16_t* row16 = reinterpret_cast<uint16_t*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[2 * kWarp];
    const int64_t r = blockIdx.x;
    pdl_prologue(x + r * D, D * 2, first_wave);
    const uint16_t* xr = x + r * D;
    uint16_t* yr = y + r * D;
    const int phase = (int)((reinterpret_cast<uintptr_t>(xr) >> 1) & 7);
    const int nv = (int)((phase + D + 7) >> 3);
    const int k_lo = phase ? 1 : 0;                      // first fully-inside vector
    const int k_hi = ((phase + D) & 7) ? nv - 1 : nv;    // one past the last fully-inside vector
    const uint4* xa = reinterpret_cast<const uint4*>(xr - phase);
    uint4* ya = reinterpret_cast<uint4*>(yr - phase);

    // the fully-inside vectors are 16-byte aligned on both sides: the copy engine brings them in
    // while sixteen threads fill the edge vectors
    stage_interior_bulk(smem_raw, xa, k_lo, k_hi, &bar);
    if (threadIdx.x < 16) {  // edge vectors: 8 lanes for the first, 8 for the last
        const int k = (threadIdx.x < 8) ? 0 : nv - 1;
        const bool edge = (threadIdx.x < 8) ? (k_lo == 1) : (k_hi == nv - 1 && !(nv == 1 && k_lo == 1));
        if (edge) {
            const int e = threadIdx.x & 7;
            const int64_t j = (int64_t)k * 8 - phase + e;
            row16[k * 8 + e] = (j >= 0 && j < D) ? ld_stream_u16(xr + j) : (uint16_t)0;
        }
    }
    __syncthreads();
    if (!mbar_wait(&bar, 0)) return;  // gave up (flag set, see ak_wait_timeouts): a thread that exits no longer counts at later barriers
    float ss = 0.0f;
    for (int k = threadIdx.x; k < nv; k += T) ss += sumsq_v<DT>(row[k]);
    ss = cta_sum<T>(ss, slots, 0);
    const float rstd = rsqrtf(fmaf(ss, inv_D, eps));
    for (int k = k_lo + threadIdx.x; k < k_hi; k += T)
        st_stream(ya + k, scale_v<DT>(row[k], load_w_shifted(w, (int64_t)k * 8 - phase), rstd));
    if (threadIdx.x < 16) {
        const int k = (threadIdx.x < 8) ? 0 : nv - 1;
        const bool edge = (threadIdx.x < 8) ? (k_lo == 1) : (k_hi == nv - 1 && !(nv == 1 && k_lo == 1));
        const int e = threadIdx.x & 7;
        const int64_t j = (int64_t)k * 8 - phase + e;
        if (edge && j >= 0 && j < D)
            yr[j] = Elem<DT>::from_float(Elem<DT>::to_float(row16[k * 8 + e]) * Elem<DT>::to_float(__ldg(w + j)) * rstd);
    }
}

// ------------------------------------------------------------------ unaligned rows split over a cluster
// The phase layout of rmsnorm_stage_kernel with the covering vectors of a row split over the C
// CTAs of a thread-block cluster: CTA c stages covering vectors [nv * c / C, nv * (c + 1) / C),
// the fully-inside ones by bulk copies; the first CTA fills the head edge vector and the last one
// the tail edge vector element by element (zeros in the padding).  The partial sums of squares
// meet through the mailbox of rmsnorm_cluster_kernel.  For unaligned rows longer than one CTA's
// shared memory (up to eight) and for a few long unaligned rows.  Needs x and y rows in the same
// phase, w 4-byte aligned and nv >= C.  grid = rows * C, cluster = C.  Dynamic shared memory =
// ceil(max nv / C) * 16 bytes.
template <int T, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(T)
rmsnorm_cluster_stage_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w, uint16_t* __restrict__ y,
                             int64_t D, int C, float inv_D, float eps) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint4* row = reinterpret_cast<uint4*>(smem_raw);
    uint16_t* row16 = reinterpret_cast<uint16_t*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[2 * kWarp];
    __shared__ float box[kMaxCluster];
    __shared__ uint64_t xbar;
    const uint32_t c = cluster_rank();
    const int64_t r = blockIdx.x / C;
    const uint16_t* xr = x + r * D;
    uint16_t* yr = y + r * D;
    const int phase = (int)((reinterpret_cast<uintptr_t>(xr) >> 1) & 7);
    const int nv = (int)((phase + D + 7) >> 3);
    const int k_lo = phase ? 1 : 0;
    const int k_hi = ((phase + D) & 7) ? nv - 1 : nv;
    const uint4* xa = reinterpret_cast<const uint4*>(xr - phase);
    uint4* ya = reinterpret_cast<uint4*>(yr - phase);
    const int v0 = (int)((int64_t)nv * c / C), v1 = (int)((int64_t)nv * (c + 1) / C);
    const int n = v1 - v0;                                   // covering vectors of this CTA
    const int i0 = max(v0, k_lo), i1 = min(v1, k_hi);        // the fully-inside ones
    // edge element of this thread: threads 0..7 the head vector (CTA 0), 8..15 the tail vector (last CTA)
    const int ek = (threadIdx.x < 8) ? 0 : nv - 1;
    const bool evec = (threadIdx.x < 8) ? (k_lo == 1 && v0 == 0) : (k_hi == nv - 1 && v1 == nv && !(nv == 1 && k_lo == 1));
    const int64_t ej = (int64_t)ek * 8 - phase + (threadIdx.x & 7);
    const bool my_edge = threadIdx.x < 16 && evec;
    const bool my_elem = my_edge && ej >= 0 && ej < D;

    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mailbox_arm(&xbar, C);
    }
    __syncthreads();
    if (threadIdx.x == 0)
        bulk_load_span(smem_raw + (size_t)(i0 - v0) * 16, xa + i0, i1 > i0 ? (uint32_t)(i1 - i0) * 16u : 0u, &bar);
    cluster_arrive_relaxed();
    if (my_edge) row16[(ek - v0) * 8 + (threadIdx.x & 7)] = my_elem ? ld_stream_u16(xr + ej) : (uint16_t)0;
    __syncthreads();
    // a wait that gave up (never expected) contributes nothing and writes nothing, but still posts
    bool ok = mbar_wait(&bar, 0);
    const int nn = ok ? n : 0;
    float ss = 0.0f;
    for (int k = threadIdx.x; k < nn; k += T) ss += sumsq_v<DT>(row[k]);
    ss = cta_sum<T>(ss, slots, 0);
    cluster_wait();   // every CTA of the cluster runs, its mailbox armed, before anything is posted to it
    if (!mailbox_exchange(ss, box, &xbar, C, c)) ok = false;
    float tot = 0.0f;
    for (int i = 0; i < C; ++i) tot += box[i];
    const float rstd = rsqrtf(fmaf(tot, inv_D, eps));
    if (!ok) return;
    for (int k = i0 + threadIdx.x; k < i1; k += T)
        st_stream(ya + k, scale_v<DT>(row[k - v0], load_w_shifted(w, (int64_t)k * 8 - phase), rstd));
    if (my_elem)
        yr[ej] = Elem<DT>::from_float(Elem<DT>::to_float(row16[(ek - v0) * 8 + (threadIdx.x & 7)]) *
                                      Elem<DT>::to_float(__ldg(w + ej)) * rstd);
}

// ------------------------------------------------------------------ unaligned rows in registers
// The phase layout of rmsnorm_stage_kernel without the trip through shared memory, for rows
// short enough to sit in registers: every interior vector is loaded before the first use and
// the edge elements are single values in sixteen threads, outside the unrolled slots.  Needs x
// and y rows in the same phase, w 4-byte aligned and at most THREADS * VPT covering vectors.
template <int THREADS, int VPT, int DT>
__global__ void __launch_bounds__(THREADS)
rmsnorm_regp_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w, uint16_t* __restrict__ y,
                    int64_t D, float inv_D, float eps, int first_wave) {
    __shared__ float slots[2 * kWarp];
    const int64_t r = blockIdx.x;
    pdl_prologue(x + r * D, D * 2, first_wave);
    const uint16_t* xr = x + r * D;
    uint16_t* yr = y + r * D;
    // interior vectors k_lo .. k_hi - 1 live in registers (slot i of thread t holds vector
    // k_lo + t + i * THREADS); the up to 14 edge elements belong to threads 0..15, one each
    const int phase = (int)((reinterpret_cast<uintptr_t>(xr) >> 1) & 7);
    const int nv = (int)((phase + D + 7) >> 3);
    const int k_lo = phase ? 1 : 0;
    const int k_hi = ((phase + D) & 7) ? nv - 1 : nv;
    const uint4* xa = reinterpret_cast<const uint4*>(xr - phase);
    uint4* ya = reinterpret_cast<uint4*>(yr - phase);
    const int ek = (threadIdx.x < 8) ? 0 : nv - 1;
    const bool evec = (threadIdx.x < 8) ? (k_lo == 1) : (k_hi == nv - 1 && !(nv == 1 && k_lo == 1));
    const int64_t ej = (int64_t)ek * 8 - phase + (threadIdx.x & 7);
    const bool edge = threadIdx.x < 16 && evec && ej >= 0 && ej < D;
    uint4 xv[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int k = k_lo + threadIdx.x + i * THREADS;
        xv[i] = (k < k_hi) ? ld_stream(xa + k) : make_uint4(0, 0, 0, 0);
    }
    const float xe = edge ? Elem<DT>::to_float(ld_stream_u16(xr + ej)) : 0.0f;
    float ss = xe * xe;
#pragma unroll
    for (int i = 0; i < VPT; ++i) ss += sumsq_v<DT>(xv[i]);
    ss = cta_sum<THREADS>(ss, slots, 0);
    const float rstd = rsqrtf(fmaf(ss, inv_D, eps));
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int k = k_lo + threadIdx.x + i * THREADS;
        if (k < k_hi) st_stream(ya + k, scale_v<DT>(xv[i], load_w_shifted(w, (int64_t)k * 8 - phase), rstd));
    }
    if (edge) yr[ej] = Elem<DT>::from_float(xe * Elem<DT>::to_float(__ldg(w + ej)) * rstd);
}

// ------------------------------------------------------------------ generic
// Any D and any 2-byte alignment.  Row r starts at element r*D, so its 16-byte phase
// changes from row to row: up to 7 head elements and 7 tail elements are handled with
// 2-byte accesses, the body with 16-byte vectors (when x and y share the phase).  The
// second pass re-reads the row, which this CTA has just pulled through L1/L2.
constexpr int kRmsGenericThreads = 256;

template <int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(kRmsGenericThreads)
rmsnorm_generic_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w,
                       uint16_t* __restrict__ y, int64_t rows, int64_t D, float inv_D, float eps) {
    constexpr int T = kRmsGenericThreads;
    __shared__ float slots[2 * kWarp];
    int phase = 0;
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint16_t* xr = x + row * D;
        uint16_t* yr = y + row * D;
        const int xph = (int)((reinterpret_cast<uintptr_t>(xr) >> 1) & 7);
        const int yph = (int)((reinterpret_cast<uintptr_t>(yr) >> 1) & 7);
        const bool vec_ok = (xph == yph);
        int64_t head = vec_ok ? ((8 - xph) & 7) : D;
        if (head > D) head = D;
        const int64_t nbody = (D - head) >> 3;
        const int64_t tail0 = head + (nbody << 3);
        const uint4* xb = reinterpret_cast<const uint4*>(xr + head);

        float ss = 0.0f;
        for (int64_t i = threadIdx.x; i < nbody; i += T) ss += sumsq_v<DT>(xb[i]);
        for (int64_t j = threadIdx.x; j < head; j += T) {
            const float v = Elem<DT>::to_float(xr[j]);
            ss = fmaf(v, v, ss);
        }
        for (int64_t j = tail0 + threadIdx.x; j < D; j += T) {
            const float v = Elem<DT>::to_float(xr[j]);
            ss = fmaf(v, v, ss);
        }
        ss = cta_sum<T>(ss, slots, phase);
        phase ^= 1;
        const float rstd = rsqrtf(fmaf(ss, inv_D, eps));

        uint4* yb = reinterpret_cast<uint4*>(yr + head);
        for (int64_t i = threadIdx.x; i < nbody; i += T) {
            const uint4 v = xb[i];
            const uint16_t* wj = w + head + (i << 3);
            uint4 wq;
            wq.x = (uint32_t)__ldg(wj + 0) | ((uint32_t)__ldg(wj + 1) << 16);
            wq.y = (uint32_t)__ldg(wj + 2) | ((uint32_t)__ldg(wj + 3) << 16);
            wq.z = (uint32_t)__ldg(wj + 4) | ((uint32_t)__ldg(wj + 5) << 16);
            wq.w = (uint32_t)__ldg(wj + 6) | ((uint32_t)__ldg(wj + 7) << 16);
            st_stream(yb + i, scale_v<DT>(v, wq, rstd));
        }
        for (int64_t j = threadIdx.x; j < head; j += T)
            yr[j] = Elem<DT>::from_float(Elem<DT>::to_float(xr[j]) * rstd * Elem<DT>::to_float(__ldg(w + j)));
        for (int64_t j = tail0 + threadIdx.x; j < D; j += T)
            yr[j] = Elem<DT>::from_float(Elem<DT>::to_float(xr[j]) * rstd * Elem<DT>::to_float(__ldg(w + j)));
    }
}

// fp32 rows with no 16-byte alignment (D % 4 != 0 or a misaligned base): element-wise, two
// passes, the second from L1/L2.
__global__ void __launch_bounds__(kRmsGenericThreads)
rmsnorm_generic32_kernel(const float* __restrict__ x, const float* __restrict__ w, float* __restrict__ y,
                         int64_t rows, int64_t D, float inv_D, float eps) {
    constexpr int T = kRmsGenericThreads;
    __shared__ float slots[2 * kWarp];
    int phase = 0;
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const float* xr = x + row * D;
        float* yr = y + row * D;
        float s0 = 0.0f, s1 = 0.0f;
        int64_t j = threadIdx.x;
        for (; j + T < D; j += 2 * T) {
            const float a = xr[j], b = xr[j + T];
            s0 = fmaf(a, a, s0);
            s1 = fmaf(b, b, s1);
        }
        if (j < D) s0 = fmaf(xr[j], xr[j], s0);
        const float ss = cta_sum<T>(s0 + s1, slots, phase);
        phase ^= 1;
        const float rstd = rsqrtf(fmaf(ss, inv_D, eps));
        for (int64_t k = threadIdx.x; k < D; k += T) yr[k] = xr[k] * rstd * __ldg(w + k);
    }
}

}  // namespace ak
