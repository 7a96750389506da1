// LayerNorm forward device kernels (paper Table 3 "layernorm"; Table 4 rows "layernorm").
//
//   mu = mean_k x[r, k];  var = mean_k (x[r, k] - mu)^2  (biased);
//   y[r, j] = rne( (x[r, j] - mu) * rsqrt(var + eps) * gamma[j] + beta[j] )
//
// The paper's kernel is a single-pass Welford.  Here the row already sits in registers (or
// shared memory) after its one trip from HBM, so the moments are taken in two exact-order
// passes over that copy, which is both simpler and more accurate: first the mean, computed
// as K + mean(x - K) with K the row's first element (for a constant row every difference is
// exactly zero and mu == K exactly; in general the partial sums stay small, so fp32 does not
// lose the low bits of large activations), then the sum of squared deviations from mu.
// One DRAM read and one DRAM write per element.  Differences x - K and x - mu come straight
// from the packed 16-bit halves with the mixed-precision subtract (no widening instruction).
// Kernels take the element type DT (bf16, fp16, fp32) as a template parameter; the phase-staged
// and multi-pass kernels serve the 16-bit types, unaligned fp32 rows go to
// layernorm_generic32_kernel.
#pragma once

#include "ak_common.cuh"

namespace ak {

// Vector helpers per element type DT (16-byte vectors: 8 bf16 / fp16 or 4 fp32 elements).
__device__ __forceinline__ void ln_halves(uint32_t u, uint16_t& lo, uint16_t& hi) {
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(u));
}
// x - c with x a 16-bit element: exact operand, one rounding
template <int DT>
__device__ __forceinline__ float sub_h(uint16_t x, float c) {
    float d;
    if constexpr (DT == AK_DTYPE_F16) asm("sub.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(x), "f"(c));
    else asm("sub.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(x), "f"(c));
    return d;
}
template <int DT>
__device__ __forceinline__ f32x2 dev2(uint32_t u, float c) {
    uint16_t lo, hi;
    ln_halves(u, lo, hi);
    return pack2(sub_h<DT>(lo, c), sub_h<DT>(hi, c));
}
// s += (x - c), q += (x - c)^2 over the elements of a vector, lane-wise in packed pairs
template <int DT>
__device__ __forceinline__ void moments_v(const uint4& v, float c, f32x2& s, f32x2& q) {
    if constexpr (DT == AK_DTYPE_F32) {
        const f32x2 c2 = pack2(c, c);
        const f32x2 a = sub2(pack2(__uint_as_float(v.x), __uint_as_float(v.y)), c2);
        const f32x2 b = sub2(pack2(__uint_as_float(v.z), __uint_as_float(v.w)), c2);
        s = add2(s, add2(a, b));
        q = fma2(b, b, fma2(a, a, q));
    } else {
        // word by word: two live temporaries instead of eight
        f32x2 d = dev2<DT>(v.x, c);
        s = add2(s, d);
        q = fma2(d, d, q);
        d = dev2<DT>(v.y, c);
        s = add2(s, d);
        q = fma2(d, d, q);
        d = dev2<DT>(v.z, c);
        s = add2(s, d);
        q = fma2(d, d, q);
        d = dev2<DT>(v.w, c);
        s = add2(s, d);
        q = fma2(d, d, q);
    }
}
// The shift of the one-sweep moments: the mean of the row's first 16 bytes.  Exactly c for a
// constant row (every term is c scaled by a power of two and the partial sums are multiples of
// it); scaled before summing so that eight large values cannot overflow.
template <int DT>
__device__ __forceinline__ float head_mean(const uint4 v) {
    if constexpr (DT == AK_DTYPE_F32) {
        return (__uint_as_float(v.x) * 0.25f + __uint_as_float(v.y) * 0.25f) +
               (__uint_as_float(v.z) * 0.25f + __uint_as_float(v.w) * 0.25f);
    } else {
        const float a = Elem<DT>::lo(v.x) * 0.125f + Elem<DT>::hi(v.x) * 0.125f;
        const float b = Elem<DT>::lo(v.y) * 0.125f + Elem<DT>::hi(v.y) * 0.125f;
        const float c = Elem<DT>::lo(v.z) * 0.125f + Elem<DT>::hi(v.z) * 0.125f;
        const float d = Elem<DT>::lo(v.w) * 0.125f + Elem<DT>::hi(v.w) * 0.125f;
        return (a + b) + (c + d);
    }
}
// Mean and variance from the one-sweep sums s = sum(x - K), q = sum((x - K)^2).  False when the
// shift is so far from the mean (or something is not a number) that the subtraction
// q/D - (s/D)^2 would lose accuracy: the caller then sweeps again with the shift mu (refine_stats).
template <int DT>
__device__ __forceinline__ bool sweep_stats(float s, float q, float inv_D, float K, float& mu, float& mc,
                                            float& var) {
    const float m = s * inv_D;   // mean - K
    if constexpr (DT == AK_DTYPE_F32) {
        mu = K;
        mc = m;
    } else {
        mu = K + m;
        mc = 0.0f;
    }
    var = fmaf(q, inv_D, -(m * m));
    return m * m <= var;
}
// The second sweep of such a row is shifted by the first estimate of the mean (one float): s and
// q are now sums of x - mu and (x - mu)^2, what is left of the mean is tiny against the spread,
// and the subtraction is harmless.  16-bit element types add the residual to mu.  fp32 keeps the
// mean in two parts, mu + mc with mc of the order of the spread at most, and its output subtracts
// them one after the other: a mean far above the spread does not fit one float to the accuracy
// of an fp32 result (1024 +- 8 would lose 1e-5 of it), while the rounding of a 16-bit output is
// coarser than that.
template <int DT>
__device__ __forceinline__ float second_shift(float& mu, float mc) {   // the shift of the second sweep
    if constexpr (DT == AK_DTYPE_F32) mu += mc;
    return mu;
}
template <int DT>
__device__ __forceinline__ void refine_stats(float s, float q, float inv_D, float& mu, float& mc, float& var) {
    const float m = s * inv_D;
    if constexpr (DT == AK_DTYPE_F32) mc = m;
    else mu += m;
    var = fmaxf(fmaf(q, inv_D, -(m * m)), 0.0f);
}
// the lane sums of packed accumulators, added over the CTA with one barrier (two sets of slots)
template <int THREADS>
__device__ __forceinline__ void cta_sum2(f32x2 sp, f32x2 qp, float* slots, float& s, float& q) {
    constexpr int NW = THREADS / kWarp;
    float lo, hi;
    unpack2(sp, lo, hi);
    s = warp_sum(lo + hi);
    unpack2(qp, lo, hi);
    q = warp_sum(lo + hi);
    if constexpr (NW > 1) {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        if (lane == 0) {
            slots[warp] = s;
            slots[kWarp + warp] = q;
        }
        __syncthreads();
        s = warp_sum((lane < NW) ? slots[lane] : 0.0f);
        q = warp_sum((lane < NW) ? slots[kWarp + lane] : 0.0f);
    }
}
// sum over the elements of (x - c)
template <int DT>
__device__ __forceinline__ float sumdev_v(const uint4& v, float c) {
    float lo, hi;
    if constexpr (DT == AK_DTYPE_F32) {
        const f32x2 c2 = pack2(c, c);
        unpack2(add2(sub2(pack2(__uint_as_float(v.x), __uint_as_float(v.y)), c2),
                     sub2(pack2(__uint_as_float(v.z), __uint_as_float(v.w)), c2)), lo, hi);
    } else {
        unpack2(add2(add2(dev2<DT>(v.x, c), dev2<DT>(v.y, c)), add2(dev2<DT>(v.z, c), dev2<DT>(v.w, c))), lo, hi);
    }
    return lo + hi;
}
// sum over the elements of (x - c)^2
template <int DT>
__device__ __forceinline__ float sqdev_v(const uint4& v, float c) {
    float lo, hi;
    if constexpr (DT == AK_DTYPE_F32) {
        const f32x2 c2 = pack2(c, c);
        const f32x2 a = sub2(pack2(__uint_as_float(v.x), __uint_as_float(v.y)), c2);
        const f32x2 b = sub2(pack2(__uint_as_float(v.z), __uint_as_float(v.w)), c2);
        unpack2(fma2(b, b, mul2(a, a)), lo, hi);
    } else {
        const f32x2 a = dev2<DT>(v.x, c), b = dev2<DT>(v.y, c), d = dev2<DT>(v.z, c), e = dev2<DT>(v.w, c);
        f32x2 s = mul2(a, a);
        s = fma2(b, b, s);
        s = fma2(d, d, s);
        s = fma2(e, e, s);
        unpack2(s, lo, hi);
    }
    return lo + hi;
}
// ((x - mean) * rstd) * gamma + beta per element, rounded once to the output type; mean = mu + mc
template <int DT>
__device__ __forceinline__ uint32_t ln_out2(uint32_t x, uint32_t g, uint32_t b, float mu, f32x2 rstd2) {
    const f32x2 t = fma2(mul2(dev2<DT>(x, mu), rstd2), widen2_t<DT>(g), widen2_t<DT>(b));
    float lo, hi;
    unpack2(t, lo, hi);
    return Elem<DT>::pack(lo, hi);
}
template <int DT>
__device__ __forceinline__ uint4 ln_out_v(const uint4& x, const uint4& g, const uint4& b, float mu, float mc, float rstd) {
    const f32x2 r2 = pack2(rstd, rstd);
    if constexpr (DT == AK_DTYPE_F32) {
        const f32x2 m2 = pack2(mu, mu), c2 = pack2(mc, mc);
        float o0, o1, o2, o3;
        unpack2(fma2(mul2(sub2(sub2(pack2(__uint_as_float(x.x), __uint_as_float(x.y)), m2), c2), r2),
                     pack2(__uint_as_float(g.x), __uint_as_float(g.y)), pack2(__uint_as_float(b.x), __uint_as_float(b.y))), o0, o1);
        unpack2(fma2(mul2(sub2(sub2(pack2(__uint_as_float(x.z), __uint_as_float(x.w)), m2), c2), r2),
                     pack2(__uint_as_float(g.z), __uint_as_float(g.w)), pack2(__uint_as_float(b.z), __uint_as_float(b.w))), o2, o3);
        return make_uint4(__float_as_uint(o0), __float_as_uint(o1), __float_as_uint(o2), __float_as_uint(o3));
    } else {
        // 16-bit types: mu is the whole mean (see refine_stats)
        return make_uint4(ln_out2<DT>(x.x, g.x, b.x, mu, r2), ln_out2<DT>(x.y, g.y, b.y, mu, r2),
                          ln_out2<DT>(x.z, g.z, b.z, mu, r2), ln_out2<DT>(x.w, g.w, b.w, mu, r2));
    }
}
template <int DT>
__device__ __forceinline__ float ln_out1(uint16_t x, uint16_t g, uint16_t b, float mu, float mc, float rstd) {
    (void)mc;   // 16-bit types only: mu is the whole mean
    return fmaf(sub_h<DT>(x, mu) * rstd, Elem<DT>::to_float(g), Elem<DT>::to_float(b));
}
// first element of a row (any element type), the shift K of the mean
template <int DT>
__device__ __forceinline__ float first_elem(const void* row) {
    if constexpr (DT == AK_DTYPE_F32) return __ldg(static_cast<const float*>(row));
    else return Elem<DT>::to_float(__ldg(static_cast<const uint16_t*>(row)));
}

// ------------------------------------------------------------------ row in registers
// Same thread layout as the RMSNorm register kernel (a group of GROUP threads owns a row,
// thread t holds vectors t, t + GROUP, ...).
//
// Groups of one or two warps (short rows) make two centred reductions: the mean from
// sum(x - K) with K the row's first element, then sum((x - mean)^2).
//
// Groups of 128 threads and more (a CTA per row) make ONE sweep over the registers and one
// barrier: s = sum(x - K) and q = sum((x - K)^2) with K the mean of the row's first 16 bytes,
// mean = K + s/D, variance = q/D - (s/D)^2.  The subtraction loses accuracy only when the shift
// is far from the mean, so the result is kept when (s/D)^2 <= variance (the relative error of
// the variance is then at most three times that of q); otherwise the registers are swept once
// more with the shift K := mean estimate, which corrects the mean as well (a whole row at a
// time, so the branch does not diverge).  A constant row gives s = q = 0 exactly, hence the
// output beta bit for bit.
//
// P_EARLY: gamma and beta are requested together with the row instead of after the reductions
// (8 * VPT more live registers; for launches too small to fill the GPU, where latency counts).
// FULL: every thread holds exactly VPT vectors of a live row (nvec == VPT * GROUP, the rows fill
// the CTAs' groups, one CTA per group of rows), so the loads and the sweep test no bounds; with AHEAD neither does the output phase,
// which lets the compiler fetch gamma and beta several vectors ahead (at the cost of registers).
template <int THREADS, int GROUP, int VPT, int MINB, int DT = AK_DTYPE_BF16, bool P_EARLY = false, bool FULL = false,
          bool AHEAD = false>
__global__ void __launch_bounds__(THREADS, MINB)
layernorm_reg_kernel(const uint4* __restrict__ x, const uint4* __restrict__ gamma, const uint4* __restrict__ beta,
                     uint4* __restrict__ y, int64_t rows, int nvec, float inv_D, float eps, int first_wave) {
    constexpr int GROUPS = THREADS / GROUP;
    constexpr int WARPS_PER_GROUP = GROUP / kWarp;
    constexpr bool SWEEP1 = GROUP >= 128;
    static_assert(GROUP % kWarp == 0 && THREADS % GROUP == 0, "groups are whole warps");
    // SWEEP1 alternates between two sets of slots by row, so that one barrier per row is enough:
    // a warp can be at most one barrier ahead of the slowest reader
    __shared__ float slots2[2][4][THREADS / kWarp];
    int par = 0;
    {
        const int64_t r0 = (int64_t)blockIdx.x * GROUPS;
        const int64_t nr = rows - r0 < GROUPS ? rows - r0 : GROUPS;
        pdl_prologue(x + r0 * nvec, nr * nvec * 16, first_wave);
    }
    const int g = threadIdx.x / GROUP;
    const int t = threadIdx.x % GROUP;
    const int lane = threadIdx.x & 31;
    const int warp_in_group = t >> 5;

    uint4 gv[P_EARLY ? VPT : 1], bv[P_EARLY ? VPT : 1];
    if constexpr (P_EARLY) {
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = t + k * GROUP;
            if (FULL || i < nvec) {
                gv[k] = __ldg(gamma + i);
                bv[k] = __ldg(beta + i);
            }
        }
    }
    // FULL: the grid has one CTA per row, so the loop body runs once
    for (int64_t row0 = (int64_t)blockIdx.x * GROUPS; FULL || row0 < rows; row0 += (int64_t)gridDim.x * GROUPS) {
        const int64_t row = row0 + g;
        const bool live = FULL || row < rows;
        const uint4* xr = x + row * nvec;
        float (*slots)[THREADS / kWarp] = slots2[par];
        // sum over the group of a per-thread partial (slot set `which`, one barrier)
        auto group_sum = [&](float v, int which) {
            v = warp_sum(v);
            if constexpr (WARPS_PER_GROUP > 1) {
                float* s = slots[which] + g * WARPS_PER_GROUP;
                if (lane == 0) s[warp_in_group] = v;
                __syncthreads();
                v = warp_sum((lane < WARPS_PER_GROUP) ? s[lane] : 0.0f);
            }
            return v;
        };
        const float K = !live ? 0.0f : (SWEEP1 ? head_mean<DT>(__ldg(xr)) : first_elem<DT>(xr));
        uint4 xv[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = t + k * GROUP;
            if (FULL || (live && i < nvec)) xv[k] = ld_stream(xr + i);
        }
        float mu, mc = 0.0f, var;
        if constexpr (SWEEP1) {
            f32x2 sp = pack2(0.0f, 0.0f), qp = sp;
#pragma unroll
            for (int k = 0; k < VPT; ++k)
                if (FULL || (live && t + k * GROUP < nvec)) moments_v<DT>(xv[k], K, sp, qp);
            float s1, q1, lo, hi;
            unpack2(sp, lo, hi);
            s1 = warp_sum(lo + hi);
            unpack2(qp, lo, hi);
            q1 = warp_sum(lo + hi);
            {
                float* s = slots[0] + g * WARPS_PER_GROUP;
                float* q = slots[1] + g * WARPS_PER_GROUP;
                if (lane == 0) {
                    s[warp_in_group] = s1;
                    q[warp_in_group] = q1;
                }
                __syncthreads();
                s1 = warp_sum((lane < WARPS_PER_GROUP) ? s[lane] : 0.0f);
                q1 = warp_sum((lane < WARPS_PER_GROUP) ? q[lane] : 0.0f);
            }
            if (!sweep_stats<DT>(s1, q1, inv_D, K, mu, mc, var)) {
                second_shift<DT>(mu, mc);   // the second sweep is shifted by the first estimate of the mean
                sp = pack2(0.0f, 0.0f);
                qp = sp;
#pragma unroll
                for (int k = 0; k < VPT; ++k)
                    if (FULL || (live && t + k * GROUP < nvec)) moments_v<DT>(xv[k], mu, sp, qp);
                unpack2(sp, lo, hi);
                s1 = warp_sum(lo + hi);
                unpack2(qp, lo, hi);
                q1 = warp_sum(lo + hi);
                float* s = slots[2] + g * WARPS_PER_GROUP;
                float* q = slots[3] + g * WARPS_PER_GROUP;
                if (lane == 0) {
                    s[warp_in_group] = s1;
                    q[warp_in_group] = q1;
                }
                __syncthreads();
                s1 = warp_sum((lane < WARPS_PER_GROUP) ? s[lane] : 0.0f);
                q1 = warp_sum((lane < WARPS_PER_GROUP) ? q[lane] : 0.0f);
                refine_stats<DT>(s1, q1, inv_D, mu, mc, var);
            }
            par ^= 1;
        } else {
            float s1 = 0.0f;
#pragma unroll
            for (int k = 0; k < VPT; ++k)
                if (live && t + k * GROUP < nvec) s1 += sumdev_v<DT>(xv[k], K);
            mu = fmaf(group_sum(s1, 0), inv_D, K);
            // the second pass also sums x - mu: what the first element as shift cost the mean
            // (it may be an outlier) is corrected, see refine_stats
            f32x2 sp = pack2(0.0f, 0.0f), qp = sp;
#pragma unroll
            for (int k = 0; k < VPT; ++k)
                if (live && t + k * GROUP < nvec) moments_v<DT>(xv[k], mu, sp, qp);
            float lo, hi;
            unpack2(sp, lo, hi);
            float s2 = warp_sum(lo + hi);
            unpack2(qp, lo, hi);
            float q2 = warp_sum(lo + hi);
            if constexpr (WARPS_PER_GROUP > 1) {
                float* s = slots[1] + g * WARPS_PER_GROUP;
                float* q = slots[2] + g * WARPS_PER_GROUP;
                if (lane == 0) {
                    s[warp_in_group] = s2;
                    q[warp_in_group] = q2;
                }
                __syncthreads();
                s2 = warp_sum((lane < WARPS_PER_GROUP) ? s[lane] : 0.0f);
                q2 = warp_sum((lane < WARPS_PER_GROUP) ? q[lane] : 0.0f);
            }
            refine_stats<DT>(s2, q2, inv_D, mu, mc, var);
        }
        const float rstd = rsqrtf(var + eps);
        // FULL: the row index is read again rather than kept in registers across the reductions
        uint4* yr = y + (FULL ? (int64_t)cta_id_x() * GROUPS + g : row) * nvec;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = t + k * GROUP;
            if ((FULL && (P_EARLY || AHEAD)) || (live && i < nvec)) {
                if constexpr (P_EARLY) st_stream(yr + i, ln_out_v<DT>(xv[k], gv[k], bv[k], mu, mc, rstd));
                else st_stream(yr + i, ln_out_v<DT>(xv[k], __ldg(gamma + i), __ldg(beta + i), mu, mc, rstd));
            }
        }
        if constexpr (FULL) break;
    }
}

// ------------------------------------------------------------------ long rows staged in shared memory
// One CTA per row; the row is brought into shared memory by bulk (TMA) copies counted in by
// one mbarrier, then read three times from there.  Needs 16-byte aligned rows (D % 8 == 0).
// Dynamic shared memory = nvec * 16 bytes.
constexpr uint32_t kLnBulkChunk = 32768;

template <int THREADS, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(THREADS, 1)
layernorm_smem_kernel(const uint4* __restrict__ x, const uint4* __restrict__ gamma, const uint4* __restrict__ beta,
                      uint4* __restrict__ y, int nvec, float inv_D, float eps) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint4* row = reinterpret_cast<const uint4*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[4 * kWarp];
    const int64_t r = blockIdx.x;
    if (threadIdx.x == 0) mbar_init(&bar, 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t bytes = (uint32_t)nvec * 16u;
        mbar_expect_tx(&bar, bytes);
        const unsigned char* src = reinterpret_cast<const unsigned char*>(x + r * nvec);
        for (uint32_t off = 0; off < bytes; off += kLnBulkChunk)
            bulk_load(smem_raw + off, src + off, min(kLnBulkChunk, bytes - off), &bar);
    }
    if (!mbar_wait(&bar, 0)) return;  // gave up (flag set, see ak_wait_timeouts): a thread that exits no longer counts at later barriers
    const float K = head_mean<DT>(row[0]);
    f32x2 sp = pack2(0.0f, 0.0f), qp = sp;
#pragma unroll 4
    for (int i = threadIdx.x; i < nvec; i += THREADS) moments_v<DT>(row[i], K, sp, qp);
    float s1, q1, mu, mc = 0.0f, var;
    cta_sum2<THREADS>(sp, qp, slots, s1, q1);
    if (!sweep_stats<DT>(s1, q1, inv_D, K, mu, mc, var)) {
        second_shift<DT>(mu, mc);   // the second sweep is shifted by the first estimate of the mean
        sp = pack2(0.0f, 0.0f);
        qp = sp;
#pragma unroll 4
        for (int i = threadIdx.x; i < nvec; i += THREADS) moments_v<DT>(row[i], mu, sp, qp);
        cta_sum2<THREADS>(sp, qp, slots + 2 * kWarp, s1, q1);
        refine_stats<DT>(s1, q1, inv_D, mu, mc, var);
    }
    const float rstd = rsqrtf(var + eps);
    uint4* yr = y + r * nvec;
#pragma unroll 2
    for (int i = threadIdx.x; i < nvec; i += THREADS)
        st_stream(yr + i, ln_out_v<DT>(row[i], __ldg(gamma + i), __ldg(beta + i), mu, mc, rstd));
}

// ------------------------------------------------------------------ rows split over a cluster
// C CTAs of a thread-block cluster share one row (few rows still fill the GPU; rows of up to
// C x 224 KiB are done in one pass over DRAM).  CTA c stages vectors
// [nvec * c / C, nvec * (c + 1) / C) in its shared memory by bulk copies; the slice sums of
// x - K (K = the row's first element, read by every CTA) and then of (x - mu)^2 meet through
// distributed shared memory and are added in rank order in every CTA.  grid = rows * C,
// cluster = C.  Dynamic shared memory = ceil(nvec / C) * 16 bytes.
// Register cap: six CTAs of 256 threads per SM (40 registers; 32 KiB slices let shared memory hold
// seven).  Occupancy is what this kernel lives on: five CTAs (48 registers, the compiler's choice
// when asked for two) measured 1.5-3 % slower, seven (32 registers, spills) 9 % slower.
template <int THREADS, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(THREADS, THREADS <= 256 ? 6 : 2)
layernorm_cluster_kernel(const uint4* __restrict__ x, const uint4* __restrict__ gamma, const uint4* __restrict__ beta,
                         uint4* __restrict__ y, int nvec, int C, float inv_D, float eps) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint4* row = reinterpret_cast<const uint4*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[4 * kWarp];
    __shared__ __align__(8) float2 box1[kMaxCluster], box2[kMaxCluster];
    __shared__ uint64_t xbar1, xbar2;
    const uint32_t c = cluster_rank();
    const int64_t r = blockIdx.x / C;
    const int v0 = (int)((int64_t)nvec * c / C);
    const int n = (int)((int64_t)nvec * (c + 1) / C) - v0;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mailbox_arm2(&xbar1, C);
        mailbox_arm2(&xbar2, C);
    }
    __syncthreads();
    if (threadIdx.x == 0) bulk_load_span(smem_raw, x + r * nvec + v0, (uint32_t)n * 16u, &bar);
    const float K = head_mean<DT>(__ldg(x + r * nvec));
    cluster_arrive_relaxed();
    // a wait that gave up (never expected) contributes nothing and writes nothing, but still posts
    int nn = mbar_wait(&bar, 0) ? n : 0;
    f32x2 sp = pack2(0.0f, 0.0f), qp = sp;
#pragma unroll 4
    for (int i = threadIdx.x; i < nn; i += THREADS) moments_v<DT>(row[i], K, sp, qp);
    float s1, q1;
    cta_sum2<THREADS>(sp, qp, slots, s1, q1);
    cluster_wait();   // every CTA of the cluster runs, its mailboxes armed, before anything is posted to it
    if (!mailbox_exchange2(s1, q1, box1, &xbar1, C, c)) nn = 0;
    float t1 = 0.0f, tq = 0.0f;
    for (int i = 0; i < C; ++i) {
        t1 += box1[i].x;
        tq += box1[i].y;
    }
    float mu, mc = 0.0f, var;
    // every CTA adds the same values in the same order, so the whole cluster takes the same branch
    if (!sweep_stats<DT>(t1, tq, inv_D, K, mu, mc, var)) {
        second_shift<DT>(mu, mc);   // the second sweep is shifted by the first estimate of the mean
        sp = pack2(0.0f, 0.0f);
        qp = sp;
#pragma unroll 4
        for (int i = threadIdx.x; i < nn; i += THREADS) moments_v<DT>(row[i], mu, sp, qp);
        cta_sum2<THREADS>(sp, qp, slots + 2 * kWarp, s1, q1);
        if (!mailbox_exchange2(s1, q1, box2, &xbar2, C, c)) nn = 0;
        t1 = 0.0f;
        tq = 0.0f;
        for (int i = 0; i < C; ++i) {
            t1 += box2[i].x;
            tq += box2[i].y;
        }
        refine_stats<DT>(t1, tq, inv_D, mu, mc, var);
    }
    const float rstd = rsqrtf(var + eps);
    uint4* yr = y + r * nvec + v0;
    const uint4* gr = gamma + v0;
    const uint4* br = beta + v0;
#pragma unroll 2
    for (int i = threadIdx.x; i < nn; i += THREADS)
        st_stream(yr + i, ln_out_v<DT>(row[i], __ldg(gr + i), __ldg(br + i), mu, mc, rstd));
}

// ------------------------------------------------------------------ rows of any length streamed by a cluster
// Rows too long for the shared memory of eight CTAs: the C CTAs of a cluster each stream their
// slice of the row from global memory three times (sum of x - K, sum of (x - mu)^2, normalise and
// store; partial sums through the mailboxes); the later reads find what the caches kept.  Needs
// 16-byte aligned rows.  grid = rows * C, cluster = C.
template <int T, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(T)
layernorm_cluster_stream_kernel(const uint4* __restrict__ x, const uint4* __restrict__ gamma,
                                const uint4* __restrict__ beta, uint4* __restrict__ y, int64_t nvec, int C,
                                float inv_D, float eps) {
    __shared__ float slots[4 * kWarp];
    __shared__ __align__(8) float2 box1[kMaxCluster], box2[kMaxCluster];
    __shared__ uint64_t xbar1, xbar2;
    const uint32_t c = cluster_rank();
    const int64_t r = blockIdx.x / C;
    const int64_t v0 = nvec / C * c + min((int64_t)c, nvec % C);
    const int64_t v1 = v0 + nvec / C + ((int64_t)c < nvec % C ? 1 : 0);
    if (threadIdx.x == 0) {
        mailbox_arm2(&xbar1, C);
        mailbox_arm2(&xbar2, C);
    }
    __syncthreads();
    cluster_arrive_relaxed();
    const uint4* xr = x + r * nvec;
    const float K = head_mean<DT>(__ldg(xr));
    f32x2 sp = pack2(0.0f, 0.0f), qp = sp;
#pragma unroll 8
    for (int64_t i = v0 + threadIdx.x; i < v1; i += T) moments_v<DT>(xr[i], K, sp, qp);
    float s1, q1;
    cta_sum2<T>(sp, qp, slots, s1, q1);
    cluster_wait();   // every CTA of the cluster runs, its mailboxes armed, before anything is posted to it
    bool ok = mailbox_exchange2(s1, q1, box1, &xbar1, C, c);
    float t1 = 0.0f, tq = 0.0f;
    for (int i = 0; i < C; ++i) {
        t1 += box1[i].x;
        tq += box1[i].y;
    }
    float mu, mc = 0.0f, var;
    // every CTA adds the same values in the same order, so the whole cluster takes the same branch
    if (!sweep_stats<DT>(t1, tq, inv_D, K, mu, mc, var)) {
        second_shift<DT>(mu, mc);   // the second sweep is shifted by the first estimate of the mean
        sp = pack2(0.0f, 0.0f);
        qp = sp;
#pragma unroll 8
        for (int64_t i = v0 + threadIdx.x; i < v1; i += T) moments_v<DT>(xr[i], mu, sp, qp);
        cta_sum2<T>(sp, qp, slots + 2 * kWarp, s1, q1);
        if (!mailbox_exchange2(s1, q1, box2, &xbar2, C, c)) ok = false;
        t1 = 0.0f;
        tq = 0.0f;
        for (int i = 0; i < C; ++i) {
            t1 += box2[i].x;
            tq += box2[i].y;
        }
        refine_stats<DT>(t1, tq, inv_D, mu, mc, var);
    }
    const float rstd = rsqrtf(var + eps);
    if (!ok) return;   // a wait that gave up (never expected): nothing is written
    uint4* yr = y + r * nvec;
#pragma unroll 2
    for (int64_t i = v0 + threadIdx.x; i < v1; i += T)
        st_stream(yr + i, ln_out_v<DT>(ld_stream(xr + i), __ldg(gamma + i), __ldg(beta + i), mu, mc, rstd));
}

// ------------------------------------------------------------------ unaligned rows staged in shared memory
// D % 8 != 0 (or a misaligned base): one CTA per row copies the row into shared memory in the
// 16-byte phase it has in global memory, so interior vectors are aligned 16-byte loads and
// (x and y rows sharing the phase) aligned 16-byte stores; the at most two edge vectors are
// handled element by element by 16 threads, so nothing outside the row is read or written and
// the padding never enters a sum.  gamma and beta for an interior vector start at element
// 8k - phase: 4-byte loads plus funnel shifts.  Needs gamma and beta 4-byte aligned.
__device__ __forceinline__ uint4 ln_load_shifted(const uint16_t* __restrict__ p, int64_t j0) {
    const uint32_t* pw = reinterpret_cast<const uint32_t*>(p) + (j0 >> 1);
    if ((j0 & 1) == 0) return make_uint4(__ldg(pw), __ldg(pw + 1), __ldg(pw + 2), __ldg(pw + 3));
    // odd start: the fifth word would reach past element j0 + 7; fetch only its low half
    const uint32_t a = __ldg(pw), b = __ldg(pw + 1), c = __ldg(pw + 2), d = __ldg(pw + 3);
    const uint32_t e = (uint32_t)__ldg(p + j0 + 7);
    return make_uint4(__funnelshift_r(a, b, 16), __funnelshift_r(b, c, 16), __funnelshift_r(c, d, 16),
                      __funnelshift_r(d, e, 16));
}

// TAB: gamma and beta of the inside vectors come pre-shifted from the table of shift_params_kernel,
// whose programmatic dependent this kernel then is (only the output phase waits for the table).
template <int T, int DT = AK_DTYPE_BF16, bool TAB = false>
__global__ void __launch_bounds__(T)
layernorm_stage_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ gamma,
                       const uint16_t* __restrict__ beta, uint16_t* __restrict__ y, int64_t D, float inv_D,
                       float eps, const uint4* tab, int nvp) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint4* row = reinterpret_cast<uint4*>(smem_raw);
    uint16_t* row16 = reinterpret_cast<uint16_t*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[4 * kWarp];
    const int64_t r = blockIdx.x;
    const uint16_t* xr = x + r * D;
    uint16_t* yr = y + r * D;
    const int phase = (int)((reinterpret_cast<uintptr_t>(xr) >> 1) & 7);
    const int nv = (int)((phase + D + 7) >> 3);
    const int k_lo = phase ? 1 : 0;                      // first fully-inside vector
    const int k_hi = ((phase + D) & 7) ? nv - 1 : nv;    // one past the last fully-inside vector
    const uint4* xa = reinterpret_cast<const uint4*>(xr - phase);
    uint4* ya = reinterpret_cast<uint4*>(yr - phase);

    // edge element owned by this thread (threads 0..7: first vector, 8..15: last vector)
    const int ek = (threadIdx.x < 8) ? 0 : nv - 1;
    const bool is_edge_vec = (threadIdx.x < 8) ? (k_lo == 1) : (k_hi == nv - 1 && !(nv == 1 && k_lo == 1));
    const int64_t ej = (int64_t)ek * 8 - phase + (threadIdx.x & 7);
    const bool edge = threadIdx.x < 16 && is_edge_vec && ej >= 0 && ej < D;

    stage_interior_bulk(smem_raw, xa, k_lo, k_hi, &bar);   // the copy engine brings the inside vectors
    if (edge) row16[ek * 8 + (threadIdx.x & 7)] = ld_stream_u16(xr + ej);
    __syncthreads();
    if (!mbar_wait(&bar, 0)) return;  // gave up (flag set, see ak_wait_timeouts): a thread that exits no longer counts at later barriers
    // the shift of the one-sweep moments: the mean of the first inside vector, or the row's first
    // element when there is none
    const float K = (k_lo < k_hi) ? head_mean<DT>(row[k_lo]) : Elem<DT>::to_float(row16[phase]);
    const float d0 = edge ? sub_h<DT>(row16[ek * 8 + (threadIdx.x & 7)], K) : 0.0f;
    f32x2 sp = pack2(d0, 0.0f), qp = pack2(d0 * d0, 0.0f);
#pragma unroll 4
    for (int k = k_lo + threadIdx.x; k < k_hi; k += T) moments_v<DT>(row[k], K, sp, qp);
    float s1, q1, mu, mc = 0.0f, var;
    cta_sum2<T>(sp, qp, slots, s1, q1);
    if (!sweep_stats<DT>(s1, q1, inv_D, K, mu, mc, var)) {
        second_shift<DT>(mu, mc);   // the second sweep is shifted by the first estimate of the mean
        const float d1 = edge ? sub_h<DT>(row16[ek * 8 + (threadIdx.x & 7)], mu) : 0.0f;
        sp = pack2(d1, 0.0f);
        qp = pack2(d1 * d1, 0.0f);
#pragma unroll 4
        for (int k = k_lo + threadIdx.x; k < k_hi; k += T) moments_v<DT>(row[k], mu, sp, qp);
        cta_sum2<T>(sp, qp, slots + 2 * kWarp, s1, q1);
        refine_stats<DT>(s1, q1, inv_D, mu, mc, var);
    }
    const float rstd = rsqrtf(var + eps);
    if constexpr (TAB) {
        pdl_wait();   // the table is complete and visible; plain loads (cached in L1), not the read-only path
        const uint4* gt = tab + (size_t)phase * nvp;
        const uint4* bt = tab + (size_t)(8 + phase) * nvp;
#pragma unroll 2
        for (int k = k_lo + threadIdx.x; k < k_hi; k += T)
            st_stream(ya + k, ln_out_v<DT>(row[k], gt[k], bt[k], mu, mc, rstd));
    } else {
        for (int k = k_lo + threadIdx.x; k < k_hi; k += T) {
            const int64_t j0 = (int64_t)k * 8 - phase;
            st_stream(ya + k, ln_out_v<DT>(row[k], ln_load_shifted(gamma, j0), ln_load_shifted(beta, j0), mu, mc, rstd));
        }
    }
    if (edge)
        yr[ej] = Elem<DT>::from_float(ln_out1<DT>(row16[ek * 8 + (threadIdx.x & 7)], __ldg(gamma + ej), __ldg(beta + ej), mu, mc, rstd));
}

// ------------------------------------------------------------------ unaligned rows split over a cluster
// The phase layout of layernorm_stage_kernel with the covering vectors of a row split over the C
// CTAs of a thread-block cluster: CTA c stages covering vectors [nv * c / C, nv * (c + 1) / C),
// the fully-inside ones by bulk copies; the edge elements (head: first CTA, tail: last CTA) are
// single values in sixteen threads.  The partial sums meet through the mailboxes of
// layernorm_cluster_kernel.  For unaligned rows longer than one CTA's shared memory (up to eight)
// and for a few long unaligned rows.  Needs x and y rows in the same phase, gamma and beta 4-byte
// aligned and nv >= C.  TAB as in layernorm_stage_kernel.  grid = rows * C, cluster = C.  Dynamic
// shared memory = ceil(max nv / C) * 16 bytes.
template <int T, int DT = AK_DTYPE_BF16, bool TAB = false>
__global__ void __launch_bounds__(T, 2)
layernorm_cluster_stage_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ gamma,
                               const uint16_t* __restrict__ beta, uint16_t* __restrict__ y, int64_t D, int C,
                               float inv_D, float eps, const uint4* tab, int nvp) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint4* row = reinterpret_cast<uint4*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[4 * kWarp];
    __shared__ __align__(8) float2 box1[kMaxCluster], box2[kMaxCluster];
    __shared__ uint64_t xbar1, xbar2;
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
    const int i0 = max(v0, k_lo), i1 = min(v1, k_hi);        // the fully-inside vectors of this CTA
    // edge element of this thread: threads 0..7 the head vector (CTA 0), 8..15 the tail vector (last CTA)
    const int ek = (threadIdx.x < 8) ? 0 : nv - 1;
    const bool evec = (threadIdx.x < 8) ? (k_lo == 1 && v0 == 0) : (k_hi == nv - 1 && v1 == nv && !(nv == 1 && k_lo == 1));
    const int64_t ej = (int64_t)ek * 8 - phase + (threadIdx.x & 7);
    const bool edge = threadIdx.x < 16 && evec && ej >= 0 && ej < D;

    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mailbox_arm2(&xbar1, C);
        mailbox_arm2(&xbar2, C);
    }
    __syncthreads();
    if (threadIdx.x == 0)
        bulk_load_span(smem_raw + (size_t)(i0 - v0) * 16, xa + i0, i1 > i0 ? (uint32_t)(i1 - i0) * 16u : 0u, &bar);
    cluster_arrive_relaxed();
    // the shift of the one-sweep moments, the same in every CTA of the cluster: the mean of the
    // row's first inside vector, or its first element when there is none
    const float K = (k_lo < k_hi) ? head_mean<DT>(__ldg(xa + k_lo)) : first_elem<DT>(xr);
    const uint16_t xe = edge ? ld_stream_u16(xr + ej) : (uint16_t)0;
    // a wait that gave up (never expected) contributes nothing and writes nothing, but still posts
    bool ok = mbar_wait(&bar, 0);
    const int j0 = i0 - v0, j1 = ok ? i1 - v0 : j0;          // local indices of the fully-inside vectors
    const float d0 = edge ? sub_h<DT>(xe, K) : 0.0f;
    f32x2 sp = pack2(d0, 0.0f), qp = pack2(d0 * d0, 0.0f);
#pragma unroll 4
    for (int k = j0 + threadIdx.x; k < j1; k += T) moments_v<DT>(row[k], K, sp, qp);
    float s1, q1;
    cta_sum2<T>(sp, qp, slots, s1, q1);
    cluster_wait();   // every CTA of the cluster runs, its mailboxes armed, before anything is posted to it
    if (!mailbox_exchange2(s1, q1, box1, &xbar1, C, c)) ok = false;
    float t1 = 0.0f, tq = 0.0f;
    for (int i = 0; i < C; ++i) {
        t1 += box1[i].x;
        tq += box1[i].y;
    }
    float mu, mc = 0.0f, var;
    // every CTA adds the same values in the same order, so the whole cluster takes the same branch
    if (!sweep_stats<DT>(t1, tq, inv_D, K, mu, mc, var)) {
        second_shift<DT>(mu, mc);   // the second sweep is shifted by the first estimate of the mean
        const float d1 = edge ? sub_h<DT>(xe, mu) : 0.0f;
        sp = pack2(d1, 0.0f);
        qp = pack2(d1 * d1, 0.0f);
#pragma unroll 4
        for (int k = j0 + threadIdx.x; k < j1; k += T) moments_v<DT>(row[k], mu, sp, qp);
        cta_sum2<T>(sp, qp, slots + 2 * kWarp, s1, q1);
        if (!mailbox_exchange2(s1, q1, box2, &xbar2, C, c)) ok = false;
        t1 = 0.0f;
        tq = 0.0f;
        for (int i = 0; i < C; ++i) {
            t1 += box2[i].x;
            tq += box2[i].y;
        }
        refine_stats<DT>(t1, tq, inv_D, mu, mc, var);
    }
    const float rstd = rsqrtf(var + eps);
    if (!ok) return;
    if constexpr (TAB) {
        pdl_wait();   // the table is complete and visible; plain loads (cached in L1), not the read-only path
        const uint4* gt = tab + (size_t)phase * nvp;
        const uint4* bt = tab + (size_t)(8 + phase) * nvp;
#pragma unroll 2
        for (int k = i0 + threadIdx.x; k < i1; k += T)
            st_stream(ya + k, ln_out_v<DT>(row[k - v0], gt[k], bt[k], mu, mc, rstd));
    } else {
        for (int k = i0 + threadIdx.x; k < i1; k += T) {
            const int64_t e0 = (int64_t)k * 8 - phase;
            st_stream(ya + k, ln_out_v<DT>(row[k - v0], ln_load_shifted(gamma, e0), ln_load_shifted(beta, e0), mu, mc, rstd));
        }
    }
    if (edge) yr[ej] = Elem<DT>::from_float(ln_out1<DT>(xe, __ldg(gamma + ej), __ldg(beta + ej), mu, mc, rstd));
}

// ------------------------------------------------------------------ unaligned rows in registers
// The phase layout of layernorm_stage_kernel without the trip through shared memory, for rows
// short enough to sit in registers: interior vectors are loaded before the first use, the edge
// elements are single values in sixteen threads.  Needs x and y rows in the same phase, gamma
// and beta 4-byte aligned and at most THREADS * VPT covering vectors.  TAB: gamma and beta of the
// interior vectors come pre-shifted from the table of shift_params_kernel (this kernel then runs
// as its programmatic dependent: the statistics need no parameters, so only the output phase
// waits for the table).
template <int THREADS, int VPT, int MINB, int DT = AK_DTYPE_BF16, bool TAB = false>
__global__ void __launch_bounds__(THREADS, MINB)
layernorm_regp_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ gamma,
                      const uint16_t* __restrict__ beta, uint16_t* __restrict__ y, int64_t D, float inv_D, float eps,
                      const uint4* tab, int nvp) {
    __shared__ float slots[3 * kWarp];
    const int64_t r = blockIdx.x;
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
    const float K = Elem<DT>::to_float(__ldg(xr));
    uint4 xv[VPT];
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int k = k_lo + threadIdx.x + i * THREADS;
        if (k < k_hi) xv[i] = ld_stream(xa + k);
    }
    const uint16_t xe = edge ? ld_stream_u16(xr + ej) : (uint16_t)0;
    float s1 = edge ? sub_h<DT>(xe, K) : 0.0f;
#pragma unroll
    for (int i = 0; i < VPT; ++i)
        if (k_lo + (int)threadIdx.x + i * THREADS < k_hi) s1 += sumdev_v<DT>(xv[i], K);
    s1 = cta_sum<THREADS>(s1, slots, 0);
    float mu = fmaf(s1, inv_D, K), mc = 0.0f, var;
    // the second pass also sums x - mu: what the first element as shift cost the mean (it may
    // be an outlier) is corrected, see refine_stats
    const float de = edge ? sub_h<DT>(xe, mu) : 0.0f;
    f32x2 sp = pack2(de, 0.0f), qp = pack2(de * de, 0.0f);
#pragma unroll
    for (int i = 0; i < VPT; ++i)
        if (k_lo + (int)threadIdx.x + i * THREADS < k_hi) moments_v<DT>(xv[i], mu, sp, qp);
    float s2, q2;
    cta_sum2<THREADS>(sp, qp, slots + kWarp, s2, q2);
    refine_stats<DT>(s2, q2, inv_D, mu, mc, var);
    const float rstd = rsqrtf(var + eps);
    if constexpr (TAB) {
        pdl_wait();   // the table is complete and visible; plain loads (cached in L1), not the read-only path
        const uint4* gt = tab + (size_t)phase * nvp;
        const uint4* bt = tab + (size_t)(8 + phase) * nvp;
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int k = k_lo + threadIdx.x + i * THREADS;
            if (k < k_hi) st_stream(ya + k, ln_out_v<DT>(xv[i], gt[k], bt[k], mu, mc, rstd));
        }
    } else {
#pragma unroll
        for (int i = 0; i < VPT; ++i) {
            const int k = k_lo + threadIdx.x + i * THREADS;
            if (k < k_hi) {
                const int64_t j0 = (int64_t)k * 8 - phase;
                st_stream(ya + k, ln_out_v<DT>(xv[i], ln_load_shifted(gamma, j0), ln_load_shifted(beta, j0), mu, mc, rstd));
            }
        }
    }
    if (edge) yr[ej] = Elem<DT>::from_float(ln_out1<DT>(xe, __ldg(gamma + ej), __ldg(beta + ej), mu, mc, rstd));
}

// ------------------------------------------------------------------ generic
// Any D and any 2-byte alignment: element-wise 2-byte accesses, three passes over the row
// (the second and third are served by L1/L2).  The slow, always-correct fallback; aligned
// shapes never reach it.
constexpr int kLnGenericThreads = 256;

template <int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(kLnGenericThreads)
layernorm_generic_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ gamma,
                         const uint16_t* __restrict__ beta, uint16_t* __restrict__ y, int64_t rows, int64_t D,
                         float inv_D, float eps) {
    constexpr int T = kLnGenericThreads;
    __shared__ float slots[3 * kWarp];
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint16_t* xr = x + row * D;
        uint16_t* yr = y + row * D;
        const float K = Elem<DT>::to_float(xr[0]);
        float s1 = 0.0f;
        for (int64_t j = threadIdx.x; j < D; j += T) s1 += sub_h<DT>(xr[j], K);
        s1 = cta_sum<T>(s1, slots, 0);
        float mu = fmaf(s1, inv_D, K), mc = 0.0f, var;
        float r2 = 0.0f, s2 = 0.0f;   // the second pass also sums x - mu, see refine_stats
        for (int64_t j = threadIdx.x; j < D; j += T) {
            const float d = sub_h<DT>(xr[j], mu);
            r2 += d;
            s2 = fmaf(d, d, s2);
        }
        r2 = cta_sum<T>(r2, slots, 1);
        s2 = cta_sum<T>(s2, slots, 2);
        refine_stats<DT>(r2, s2, inv_D, mu, mc, var);
        const float rstd = rsqrtf(var + eps);
        for (int64_t j = threadIdx.x; j < D; j += T)
            yr[j] = Elem<DT>::from_float(ln_out1<DT>(xr[j], __ldg(gamma + j), __ldg(beta + j), mu, mc, rstd));
    }
}

// fp32 rows with no 16-byte alignment: element-wise, three passes (the last two from L1/L2).
__global__ void __launch_bounds__(kLnGenericThreads)
layernorm_generic32_kernel(const float* __restrict__ x, const float* __restrict__ gamma, const float* __restrict__ beta,
                           float* __restrict__ y, int64_t rows, int64_t D, float inv_D, float eps) {
    constexpr int T = kLnGenericThreads;
    __shared__ float slots[3 * kWarp];
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const float* xr = x + row * D;
        float* yr = y + row * D;
        const float K = xr[0];
        float s1 = 0.0f;
        for (int64_t j = threadIdx.x; j < D; j += T) s1 += xr[j] - K;
        s1 = cta_sum<T>(s1, slots, 0);
        float mu = fmaf(s1, inv_D, K), mc = 0.0f, var;
        float r2 = 0.0f, s2 = 0.0f;   // the second pass also sums x - mu, see refine_stats
        for (int64_t j = threadIdx.x; j < D; j += T) {
            const float d = xr[j] - mu;
            r2 += d;
            s2 = fmaf(d, d, s2);
        }
        r2 = cta_sum<T>(r2, slots, 1);
        s2 = cta_sum<T>(s2, slots, 2);
        refine_stats<AK_DTYPE_F32>(r2, s2, inv_D, mu, mc, var);
        const float rstd = rsqrtf(var + eps);
        for (int64_t j = threadIdx.x; j < D; j += T) yr[j] = fmaf(((xr[j] - mu) - mc) * rstd, __ldg(gamma + j), __ldg(beta + j));
    }
}

}  // namespace ak
