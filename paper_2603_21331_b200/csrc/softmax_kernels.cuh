// Last-dim softmax forward device kernels (paper Table 3 "softmax": warp-shuffle
// reductions, packed 16-bit loads).
//
//   m = max_k x[r, k];  y[r, j] = rne( exp(x[r, j] - m) / sum_k exp(x[r, k] - m) )
//
// Every kernel takes the element type DT (bf16, fp16 or fp32) as a template parameter; sizes
// are counted in 16-byte vectors.  The phase-staged and multi-pass kernels address 2-byte
// elements (16-bit types); unaligned fp32 rows go to softmax_generic32_kernel.
//
// exp is evaluated as 2^(x*log2e - rn(m*log2e)) with one FMA feeding the SFU.  Rounding
// m*log2e once scales every term of the row by the same factor, which cancels in the
// ratio.  -inf entries give 2^(-inf) = 0 exactly; an all -inf row, +inf or NaN gives NaN
// through inf - inf, as IEEE arithmetic on the definition would.
#pragma once

#include "ak_common.cuh"

namespace ak {

// Vector helpers per element type DT (16-byte vectors: 8 bf16 / fp16 or 4 fp32 elements).
// The running maximum travels as one 32-bit word: a packed pair for the 16-bit types (the
// packed max instruction is exact), the float's bits for fp32.
template <int DT>
__device__ __forceinline__ constexpr uint32_t neg_inf_word() {
    if constexpr (DT == AK_DTYPE_F32) return 0xFF800000u; else return Elem<DT>::kNegInf2;
}
template <int DT>
__device__ __forceinline__ uint32_t max_w(uint32_t a, uint32_t b) {   // drops a NaN operand
    if constexpr (DT == AK_DTYPE_F32) return __float_as_uint(fmaxf(__uint_as_float(a), __uint_as_float(b)));
    else return Elem<DT>::max2(a, b);
}
template <int DT>
__device__ __forceinline__ uint32_t max_v(const uint4& v) {
    return max_w<DT>(max_w<DT>(v.x, v.y), max_w<DT>(v.z, v.w));
}
template <int DT>
__device__ __forceinline__ float hmax_of(uint32_t m) {
    if constexpr (DT == AK_DTYPE_F32) return __uint_as_float(m);
    else return fmaxf(Elem<DT>::lo(m), Elem<DT>::hi(m));
}
template <int DT>
__device__ __forceinline__ uint4 neg_inf_vec() {
    return make_uint4(neg_inf_word<DT>(), neg_inf_word<DT>(), neg_inf_word<DT>(), neg_inf_word<DT>());
}

// e[..] = the values 2^(x*log2e - m2) of one vector as packed pairs (four pairs for the 16-bit
// types, two for fp32); returns their sum (fixed association: even elements in the low lane,
// odd in the high lane).  Multiply-adds, sums and the final scaling run as packed f32x2
// instructions.
__device__ __forceinline__ f32x2 exp_of_pair(f32x2 x2, f32x2 l2, f32x2 nm2) {
    float t0, t1;
    unpack2(fma2(x2, l2, nm2), t0, t1);
    return pack2(fast_exp2(t0), fast_exp2(t1));
}
// The same on the FMA pipe: t = x*log2e - m2 <= 0 is clamped at -160, rounded to the nearest
// integer n (the 1.5 * 2^23 trick), 2^(t - n) comes from a degree-4 minimax polynomial on
// [-0.5, 0.5] (relative error 2.7e-6, far below the rounding of a 16-bit output), and n goes into
// the exponent field.  Below the normal range the result is zero (the signed maximum with zero
// catches the exponent field running negative: every t < -127.5) or, in the one binade under
// 2^-126, a subnormal within 2^-126 of the true value; `ex2.approx.ftz` gives zero there.
__device__ __forceinline__ f32x2 exp_of_pair_poly(f32x2 x2, f32x2 l2, f32x2 nm2) {
    float t0, t1;
    unpack2(fma2(x2, l2, nm2), t0, t1);
    const f32x2 tc = pack2(fmaxf(t0, -160.0f), fmaxf(t1, -160.0f));
    const f32x2 magic = pack2(12582912.0f, 12582912.0f);
    const f32x2 z = add2(tc, magic);
    const f32x2 n = sub2(z, magic);
    const f32x2 f = sub2(tc, n);
    f32x2 p = pack2(0.009570079855620861f, 0.009570079855620861f);
    p = fma2(p, f, pack2(0.05591783672571182f, 0.05591783672571182f));
    p = fma2(p, f, pack2(0.240247443318367f, 0.240247443318367f));
    p = fma2(p, f, pack2(0.6931217908859253f, 0.6931217908859253f));
    p = fma2(p, f, pack2(0.9999992847442627f, 0.9999992847442627f));
    float p0, p1, z0, z1;
    unpack2(p, p0, p1);
    unpack2(z, z0, z1);
    p0 = __int_as_float(max(__float_as_int(p0) + (__float_as_int(z0) << 23), 0));
    p1 = __int_as_float(max(__float_as_int(p1) + (__float_as_int(z1) << 23), 0));
    return pack2(p0, p1);
}
// pairs per recomputed vector that the aligned cluster kernel evaluates on the FMA pipe (the unaligned
// one, which is not bound by the transcendental pipe, gained nothing from it)
template <int DT> constexpr int kClusterPolyPairs = DT == AK_DTYPE_F32 ? 0 : 1;
// exp_v with the first NP of the four pairs of a 16-bit vector on the FMA pipe (NP = 0: exp_v)
template <int DT, int NP>
__device__ __forceinline__ float exp_v_mix(const uint4& v, float m2, f32x2* e) {
    static_assert(DT != AK_DTYPE_F32 || NP == 0, "the polynomial is for 16-bit outputs");
    const f32x2 l2 = pack2(kLog2e, kLog2e), nm2 = pack2(-m2, -m2);
    float lo, hi;
    if constexpr (DT == AK_DTYPE_F32) {
        e[0] = exp_of_pair(pack2(__uint_as_float(v.x), __uint_as_float(v.y)), l2, nm2);
        e[1] = exp_of_pair(pack2(__uint_as_float(v.z), __uint_as_float(v.w)), l2, nm2);
        unpack2(add2(e[0], e[1]), lo, hi);
    } else {
        e[0] = NP > 0 ? exp_of_pair_poly(widen2_t<DT>(v.x), l2, nm2) : exp_of_pair(widen2_t<DT>(v.x), l2, nm2);
        e[1] = NP > 1 ? exp_of_pair_poly(widen2_t<DT>(v.y), l2, nm2) : exp_of_pair(widen2_t<DT>(v.y), l2, nm2);
        e[2] = NP > 2 ? exp_of_pair_poly(widen2_t<DT>(v.z), l2, nm2) : exp_of_pair(widen2_t<DT>(v.z), l2, nm2);
        e[3] = NP > 3 ? exp_of_pair_poly(widen2_t<DT>(v.w), l2, nm2) : exp_of_pair(widen2_t<DT>(v.w), l2, nm2);
        unpack2(add2(add2(e[0], e[1]), add2(e[2], e[3])), lo, hi);
    }
    return lo + hi;
}
template <int DT>
__device__ __forceinline__ float exp_v(const uint4& v, float m2, f32x2* e) {
    const f32x2 l2 = pack2(kLog2e, kLog2e), nm2 = pack2(-m2, -m2);
    float lo, hi;
    if constexpr (DT == AK_DTYPE_F32) {
        e[0] = exp_of_pair(pack2(__uint_as_float(v.x), __uint_as_float(v.y)), l2, nm2);
        e[1] = exp_of_pair(pack2(__uint_as_float(v.z), __uint_as_float(v.w)), l2, nm2);
        unpack2(add2(e[0], e[1]), lo, hi);
    } else {
        e[0] = exp_of_pair(widen2_t<DT>(v.x), l2, nm2);
        e[1] = exp_of_pair(widen2_t<DT>(v.y), l2, nm2);
        e[2] = exp_of_pair(widen2_t<DT>(v.z), l2, nm2);
        e[3] = exp_of_pair(widen2_t<DT>(v.w), l2, nm2);
        unpack2(add2(add2(e[0], e[1]), add2(e[2], e[3])), lo, hi);
    }
    return lo + hi;
}
template <int DT>
__device__ __forceinline__ uint4 norm_v(const f32x2* e, float inv) {
    const f32x2 inv2 = pack2(inv, inv);
    if constexpr (DT == AK_DTYPE_F32) {
        float a, b, c, d;
        unpack2(mul2(e[0], inv2), a, b);
        unpack2(mul2(e[1], inv2), c, d);
        return make_uint4(__float_as_uint(a), __float_as_uint(b), __float_as_uint(c), __float_as_uint(d));
    } else {
        uint32_t o[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            float lo, hi;
            unpack2(mul2(e[i], inv2), lo, hi);
            o[i] = Elem<DT>::pack(lo, hi);
        }
        return make_uint4(o[0], o[1], o[2], o[3]);
    }
}
// exponentials kept per vector: four pairs (16-bit types) or two (fp32)
template <int DT> constexpr int kExpPairs = (DT == AK_DTYPE_F32) ? 2 : 4;

// ------------------------------------------------------------------ row in registers
// Same thread layout as the RMSNorm register kernel: a group of GROUP threads owns a row,
// thread t holds vectors t, t + GROUP, ...  Two reductions per row (max, then sum).
// RECOMPUTE == false keeps the eight exponentials of every vector in fp32 registers so
// each is evaluated once; RECOMPUTE == true keeps only the packed inputs and evaluates the
// exponentials a second time in the epilogue (half the registers, twice the SFU work) for
// rows too long to hold in fp32.
template <int THREADS, int GROUP, int VPT, int MINB, bool RECOMPUTE, int DT = AK_DTYPE_BF16, bool FULL = false>
__global__ void __launch_bounds__(THREADS, MINB)
softmax_reg_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int64_t rows, int nvec, int first_wave) {
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

    // FULL: nvec == VPT * GROUP, the rows fill the groups exactly and the grid has one CTA per group of
    // rows: nothing tests a bound and the body runs once
    for (int64_t row0 = (int64_t)blockIdx.x * GROUPS; FULL || row0 < rows; row0 += (int64_t)gridDim.x * GROUPS) {
        const int64_t row = row0 + g;
        const bool live = FULL || row < rows;
        const uint4* xr = x + row * nvec;
        uint4 xv[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = t + k * GROUP;
            xv[k] = (FULL || (live && i < nvec)) ? ld_stream(xr + i) : neg_inf_vec<DT>();
        }
        uint32_t mx = neg_inf_word<DT>();
#pragma unroll
        for (int k = 0; k < VPT; ++k) mx = max_w<DT>(mx, max_v<DT>(xv[k]));
        float m = warp_max(hmax_of<DT>(mx));
        if constexpr (WARPS_PER_GROUP > 1) {
            float* s = slots[0] + g * WARPS_PER_GROUP;
            if (lane == 0) s[warp_in_group] = m;
            __syncthreads();
            m = warp_max((lane < WARPS_PER_GROUP) ? s[lane] : -INFINITY);
        }
        const float m2 = m * kLog2e;
        f32x2 e[RECOMPUTE ? 1 : VPT][kExpPairs<DT>];
        float sum = 0.0f;
#pragma unroll
        for (int k = 0; k < VPT; ++k) sum += exp_v<DT>(xv[k], m2, e[RECOMPUTE ? 0 : k]);
        sum = warp_sum(sum);
        if constexpr (WARPS_PER_GROUP > 1) {
            float* s = slots[1] + g * WARPS_PER_GROUP;
            if (lane == 0) s[warp_in_group] = sum;
            __syncthreads();
            sum = warp_sum((lane < WARPS_PER_GROUP) ? s[lane] : 0.0f);
        }
        const float inv = 1.0f / sum;
        uint4* yr = y + row * nvec;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = t + k * GROUP;
            if constexpr (RECOMPUTE) exp_v<DT>(xv[k], m2, e[0]);
            if (FULL || (live && i < nvec)) st_stream(yr + i, norm_v<DT>(e[RECOMPUTE ? 0 : k], inv));
        }
        if constexpr (FULL) break;
    }
}

// ------------------------------------------------------------------ long rows staged in shared memory
// One CTA per row; the row is brought into shared memory by bulk copies counted in by one
// mbarrier (bytes in flight bounded by shared memory, not registers), then read three
// times from there: maximum, sum of exponentials, normalise + store.  The first KEEP
// vectors of every thread keep their exponentials in fp32 registers between the second and
// third pass; the rest are evaluated twice.  Needs 16-byte aligned rows (D % 8 == 0).
// Dynamic shared memory = nvec * 16 bytes.
constexpr uint32_t kSmBulkChunk = 32768;

template <int THREADS, int MINB, int KEEP, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(THREADS, MINB)
softmax_smem_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int nvec, int first_wave) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint4* row = reinterpret_cast<const uint4*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[2 * kWarp];
    const int64_t r = blockIdx.x;
    pdl_prologue(x + r * nvec, (int64_t)nvec * 16, first_wave);
    if (threadIdx.x == 0) mbar_init(&bar, 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t bytes = (uint32_t)nvec * 16u;
        mbar_expect_tx(&bar, bytes);
        const unsigned char* src = reinterpret_cast<const unsigned char*>(x + r * nvec);
        for (uint32_t off = 0; off < bytes; off += kSmBulkChunk)
            bulk_load(smem_raw + off, src + off, min(kSmBulkChunk, bytes - off), &bar);
    }
    if (!mbar_wait(&bar, 0)) return;  // gave up (flag set, see ak_wait_timeouts): a thread that exits no longer counts at later barriers

    uint32_t mx = neg_inf_word<DT>();
#pragma unroll 4
    for (int i = threadIdx.x; i < nvec; i += THREADS) mx = max_w<DT>(mx, max_v<DT>(row[i]));
    const float m = cta_max<THREADS>(hmax_of<DT>(mx), slots, 0);
    const float m2 = m * kLog2e;

    f32x2 kept[KEEP > 0 ? KEEP : 1][kExpPairs<DT>];
    float sum = 0.0f;
    f32x2 e[kExpPairs<DT>];
#pragma unroll
    for (int k = 0; k < KEEP; ++k) {
        const int i = threadIdx.x + k * THREADS;
        if (i < nvec) sum += exp_v<DT>(row[i], m2, kept[k]);
    }
#pragma unroll 2
    for (int i = threadIdx.x + KEEP * THREADS; i < nvec; i += THREADS) sum += exp_v<DT>(row[i], m2, e);
    sum = cta_sum<THREADS>(sum, slots, 1);
    const float inv = 1.0f / sum;

    uint4* yr = y + r * nvec;
#pragma unroll
    for (int k = 0; k < KEEP; ++k) {
        const int i = threadIdx.x + k * THREADS;
        if (i < nvec) st_stream(yr + i, norm_v<DT>(kept[k], inv));
    }
#pragma unroll 2
    for (int i = threadIdx.x + KEEP * THREADS; i < nvec; i += THREADS) {
        exp_v<DT>(row[i], m2, e);
        st_stream(yr + i, norm_v<DT>(e, inv));
    }
}

// ------------------------------------------------------------------ rows split over a cluster
// C CTAs of a thread-block cluster share one row (few rows still fill the GPU; rows of up to
// C x 224 KiB, a 128K vocabulary among them, are done in one pass over DRAM).  CTA c stages
// vectors [nvec * c / C, nvec * (c + 1) / C) in its shared memory by bulk copies; the slice
// maxima and then the slice sums meet through distributed shared memory and are combined in
// rank order in every CTA.  The first KEEP vectors of a thread keep their exponentials in
// registers.  grid = rows * C, cluster = C.  Dynamic shared memory = ceil(nvec / C) * 16 bytes.
template <int THREADS, int KEEP, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(THREADS, THREADS <= 128 ? 7 : (THREADS <= 256 ? 3 : 1))
softmax_cluster_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int nvec, int C) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    const uint4* row = reinterpret_cast<const uint4*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[2 * kWarp];
    __shared__ float box_m[kMaxCluster], box_s[kMaxCluster];
    __shared__ uint64_t xbar_m, xbar_s;
    const uint32_t c = cluster_rank();
    const int64_t r = blockIdx.x / C;
    const int v0 = (int)((int64_t)nvec * c / C);
    const int n = (int)((int64_t)nvec * (c + 1) / C) - v0;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mailbox_arm(&xbar_m, C);
        mailbox_arm(&xbar_s, C);
    }
    __syncthreads();
    if (threadIdx.x == 0) bulk_load_span(smem_raw, x + r * nvec + v0, (uint32_t)n * 16u, &bar);
    cluster_arrive_relaxed();
    // a wait that gave up (never expected) contributes nothing and writes nothing, but still posts
    int nn = mbar_wait(&bar, 0) ? n : 0;

    uint32_t mx = neg_inf_word<DT>();
#pragma unroll 4
    for (int i = threadIdx.x; i < nn; i += THREADS) mx = max_w<DT>(mx, max_v<DT>(row[i]));
    const float m_cta = cta_max<THREADS>(hmax_of<DT>(mx), slots, 0);
    cluster_wait();   // every CTA of the cluster runs, its mailboxes armed, before anything is posted to it
    if (!mailbox_exchange(m_cta, box_m, &xbar_m, C, c)) nn = 0;
    float m = box_m[0];
    for (int i = 1; i < C; ++i) m = fmaxf(m, box_m[i]);
    const float m2 = m * kLog2e;

    f32x2 kept[KEEP > 0 ? KEEP : 1][kExpPairs<DT>];
    float sum = 0.0f;
    f32x2 e[kExpPairs<DT>];
#pragma unroll
    for (int k = 0; k < KEEP; ++k) {
        const int i = threadIdx.x + k * THREADS;
        if (i < nn) sum += exp_v<DT>(row[i], m2, kept[k]);
    }
    // The vectors that are not kept are evaluated twice, which makes the transcendental pipe the
    // busiest unit of this kernel (63 % of its peak over the whole kernel); one of their four pairs
    // goes to the FMA pipe instead (4096 x 65536: 168.6 -> 165.5 us; two pairs: 171.0 us).
    constexpr int NP = kClusterPolyPairs<DT>;
#pragma unroll 2
    for (int i = threadIdx.x + KEEP * THREADS; i < nn; i += THREADS) sum += exp_v_mix<DT, NP>(row[i], m2, e);
    sum = cta_sum<THREADS>(sum, slots, 1);
    if (!mailbox_exchange(sum, box_s, &xbar_s, C, c)) nn = 0;
    float tot = 0.0f;
    for (int i = 0; i < C; ++i) tot += box_s[i];
    const float inv = 1.0f / tot;

    uint4* yr = y + r * nvec + v0;
#pragma unroll
    for (int k = 0; k < KEEP; ++k) {
        const int i = threadIdx.x + k * THREADS;
        if (i < nn) st_stream(yr + i, norm_v<DT>(kept[k], inv));
    }
#pragma unroll 2
    for (int i = threadIdx.x + KEEP * THREADS; i < nn; i += THREADS) {
        exp_v_mix<DT, NP>(row[i], m2, e);
        st_stream(yr + i, norm_v<DT>(e, inv));
    }
}

// ------------------------------------------------------------------ rows of any length streamed by a cluster
// Rows too long for the shared memory of eight CTAs: the C CTAs of a cluster each stream their
// slice of the row from global memory three times (maximum, sum of exponentials, normalise and
// store; maxima and sums through the mailboxes); the later reads find what the caches kept.
// Needs 16-byte aligned rows.  grid = rows * C, cluster = C.
template <int T, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(T)
softmax_cluster_stream_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int64_t nvec, int C) {
    __shared__ float slots[2 * kWarp];
    __shared__ float box_m[kMaxCluster], box_s[kMaxCluster];
    __shared__ uint64_t xbar_m, xbar_s;
    const uint32_t c = cluster_rank();
    const int64_t r = blockIdx.x / C;
    const int64_t v0 = nvec / C * c + min((int64_t)c, nvec % C);
    const int64_t v1 = v0 + nvec / C + ((int64_t)c < nvec % C ? 1 : 0);
    if (threadIdx.x == 0) {
        mailbox_arm(&xbar_m, C);
        mailbox_arm(&xbar_s, C);
    }
    __syncthreads();
    cluster_arrive_relaxed();
    const uint4* xr = x + r * nvec;
    uint32_t mx = neg_inf_word<DT>();
#pragma unroll 8
    for (int64_t i = v0 + threadIdx.x; i < v1; i += T) mx = max_w<DT>(mx, max_v<DT>(xr[i]));
    const float m_cta = cta_max<T>(hmax_of<DT>(mx), slots, 0);
    cluster_wait();   // every CTA of the cluster runs, its mailboxes armed, before anything is posted to it
    bool ok = mailbox_exchange(m_cta, box_m, &xbar_m, C, c);
    float m = box_m[0];
    for (int i = 1; i < C; ++i) m = fmaxf(m, box_m[i]);
    const float m2 = m * kLog2e;
    float sum = 0.0f;
    f32x2 e[kExpPairs<DT>];
#pragma unroll 4
    for (int64_t i = v0 + threadIdx.x; i < v1; i += T) sum += exp_v<DT>(xr[i], m2, e);
    sum = cta_sum<T>(sum, slots, 1);
    if (!mailbox_exchange(sum, box_s, &xbar_s, C, c)) ok = false;
    float tot = 0.0f;
    for (int i = 0; i < C; ++i) tot += box_s[i];
    const float inv = 1.0f / tot;
    if (!ok) return;   // a wait that gave up (never expected): nothing is written
    uint4* yr = y + r * nvec;
#pragma unroll 4
    for (int64_t i = v0 + threadIdx.x; i < v1; i += T) {
        exp_v<DT>(ld_stream(xr + i), m2, e);
        st_stream(yr + i, norm_v<DT>(e, inv));
    }
}

// ------------------------------------------------------------------ unaligned rows staged in shared memory
// Same staging as the RMSNorm kernel of that name: the row sits in shared memory in the
// 16-byte phase it has in global memory (x and y rows share it), fully-inside vectors move
// with aligned 16-byte loads and stores, the edge vectors element by element with -inf
// standing in for the neighbours' bytes.  Three passes over shared memory.
template <int T, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(T)
softmax_stage_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ y, int64_t D, int first_wave) {
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
    const int k_lo = phase ? 1 : 0;
    const int k_hi = ((phase + D) & 7) ? nv - 1 : nv;
    const uint4* xa = reinterpret_cast<const uint4*>(xr - phase);
    uint4* ya = reinterpret_cast<uint4*>(yr - phase);
    const int my_edge_k = (threadIdx.x < 8) ? 0 : nv - 1;
    const bool my_edge = (threadIdx.x < 16) &&
                         ((threadIdx.x < 8) ? (k_lo == 1) : (k_hi == nv - 1 && !(nv == 1 && k_lo == 1)));
    const int64_t my_j = (int64_t)my_edge_k * 8 - phase + (threadIdx.x & 7);

    stage_interior_bulk(smem_raw, xa, k_lo, k_hi, &bar);   // the copy engine brings the inside vectors
    if (my_edge) row16[my_edge_k * 8 + (threadIdx.x & 7)] = (my_j >= 0 && my_j < D) ? ld_stream_u16(xr + my_j) : Elem<DT>::kNegInf;
    __syncthreads();
    if (!mbar_wait(&bar, 0)) return;  // gave up (flag set, see ak_wait_timeouts): a thread that exits no longer counts at later barriers

    uint32_t mx = neg_inf_word<DT>();
    for (int k = threadIdx.x; k < nv; k += T) mx = max_w<DT>(mx, max_v<DT>(row[k]));
    const float m = cta_max<T>(hmax_of<DT>(mx), slots, 0);
    const float m2 = m * kLog2e;
    float sum = 0.0f;
    f32x2 e[kExpPairs<DT>];
    for (int k = threadIdx.x; k < nv; k += T) sum += exp_v<DT>(row[k], m2, e);
    sum = cta_sum<T>(sum, slots, 1);
    const float inv = 1.0f / sum;
    for (int k = k_lo + threadIdx.x; k < k_hi; k += T) {
        exp_v<DT>(row[k], m2, e);
        st_stream(ya + k, norm_v<DT>(e, inv));
    }
    if (my_edge && my_j >= 0 && my_j < D)
        yr[my_j] = Elem<DT>::from_float(fast_exp2(fmaf(Elem<DT>::to_float(row16[my_edge_k * 8 + (threadIdx.x & 7)]), kLog2e, -m2)) * inv);
}

// ------------------------------------------------------------------ unaligned rows split over a cluster
// The phase layout of softmax_stage_kernel with the covering vectors of a row (vector k = row
// elements 8k - phase .. 8k - phase + 7) split over the C CTAs of a thread-block cluster: CTA c
// stages covering vectors [nv * c / C, nv * (c + 1) / C), the fully-inside ones by bulk copies;
// the first CTA fills the head edge vector and the last one the tail edge vector element by
// element (-inf in the padding).  Maxima and sums meet through the mailboxes of
// softmax_cluster_kernel.  For unaligned rows longer than one CTA's shared memory (up to eight) and
// for a few long unaligned rows.  Needs x and y rows in the same phase and nv >= C.
// grid = rows * C, cluster = C.  Dynamic shared memory = ceil(max nv / C) * 16 bytes.
template <int T, int DT = AK_DTYPE_BF16, int KEEP = 0>
__global__ void __launch_bounds__(T)
softmax_cluster_stage_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ y, int64_t D, int C) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint4* row = reinterpret_cast<uint4*>(smem_raw);
    uint16_t* row16 = reinterpret_cast<uint16_t*>(smem_raw);
    __shared__ uint64_t bar;
    __shared__ float slots[2 * kWarp];
    __shared__ float box_m[kMaxCluster], box_s[kMaxCluster];
    __shared__ uint64_t xbar_m, xbar_s;
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
        mailbox_arm(&xbar_m, C);
        mailbox_arm(&xbar_s, C);
    }
    __syncthreads();
    if (threadIdx.x == 0)
        bulk_load_span(smem_raw + (size_t)(i0 - v0) * 16, xa + i0, i1 > i0 ? (uint32_t)(i1 - i0) * 16u : 0u, &bar);
    cluster_arrive_relaxed();
    if (my_edge) row16[(ek - v0) * 8 + (threadIdx.x & 7)] = my_elem ? ld_stream_u16(xr + ej) : Elem<DT>::kNegInf;
    __syncthreads();
    // a wait that gave up (never expected) contributes nothing and writes nothing, but still posts
    bool ok = mbar_wait(&bar, 0);
    const int nn = ok ? n : 0;

    uint32_t mx = neg_inf_word<DT>();
    for (int k = threadIdx.x; k < nn; k += T) mx = max_w<DT>(mx, max_v<DT>(row[k]));
    const float m_cta = cta_max<T>(hmax_of<DT>(mx), slots, 0);
    cluster_wait();   // every CTA of the cluster runs, its mailboxes armed, before anything is posted to it
    if (!mailbox_exchange(m_cta, box_m, &xbar_m, C, c)) ok = false;
    float m = box_m[0];
    for (int i = 1; i < C; ++i) m = fmaxf(m, box_m[i]);
    const float m2 = m * kLog2e;
    float sum = 0.0f;
    f32x2 kept[KEEP > 0 ? KEEP : 1][kExpPairs<DT>];
    f32x2 e[kExpPairs<DT>];
#pragma unroll
    for (int j = 0; j < KEEP; ++j) {
        const int k = threadIdx.x + j * T;
        if (k < nn) sum += exp_v<DT>(row[k], m2, kept[j]);
    }
    for (int k = threadIdx.x + KEEP * T; k < nn; k += T) sum += exp_v<DT>(row[k], m2, e);
    sum = cta_sum<T>(sum, slots, 1);
    if (!mailbox_exchange(sum, box_s, &xbar_s, C, c)) ok = false;
    float tot = 0.0f;
    for (int i = 0; i < C; ++i) tot += box_s[i];
    const float inv = 1.0f / tot;
    if (!ok) return;
    // local vector k is covering vector v0 + k of the row; only the fully-inside ones are stored whole
#pragma unroll
    for (int j = 0; j < KEEP; ++j) {
        const int k = v0 + threadIdx.x + j * T;
        if (k >= i0 && k < i1) st_stream(ya + k, norm_v<DT>(kept[j], inv));
    }
    for (int k = v0 + threadIdx.x + KEEP * T; k < i1; k += T) {
        if (k < i0) continue;
        exp_v<DT>(row[k - v0], m2, e);
        st_stream(ya + k, norm_v<DT>(e, inv));
    }
    if (my_elem)
        yr[ej] = Elem<DT>::from_float(fast_exp2(fmaf(Elem<DT>::to_float(row16[(ek - v0) * 8 + (threadIdx.x & 7)]), kLog2e, -m2)) * inv);
}

// ------------------------------------------------------------------ unaligned rows in registers
// The phase layout of softmax_stage_kernel without the trip through shared memory, for rows
// short enough to sit in registers (exponentials kept in fp32): interior vectors are loaded
// before the first use, the edge elements are single values in sixteen threads.  Needs x and y
// rows in the same phase and at most THREADS * VPT covering vectors.
template <int THREADS, int VPT, int MINB, int DT>
__global__ void __launch_bounds__(THREADS, MINB)
softmax_regp_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ y, int64_t D, int first_wave) {
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
        xv[i] = (k < k_hi) ? ld_stream(xa + k) : neg_inf_vec<DT>();
    }
    const float xe = edge ? Elem<DT>::to_float(ld_stream_u16(xr + ej)) : -INFINITY;
    uint32_t mx = neg_inf_word<DT>();
#pragma unroll
    for (int i = 0; i < VPT; ++i) mx = max_w<DT>(mx, max_v<DT>(xv[i]));
    const float m = cta_max<THREADS>(fmaxf(hmax_of<DT>(mx), xe), slots, 0);
    const float m2 = m * kLog2e;
    f32x2 e[VPT][4];
    const float ee = fast_exp2(fmaf(xe, kLog2e, -m2));   // 0 for the threads without an edge element
    float sum = ee;
#pragma unroll
    for (int i = 0; i < VPT; ++i) sum += exp_v<DT>(xv[i], m2, e[i]);
    sum = cta_sum<THREADS>(sum, slots, 1);
    const float inv = 1.0f / sum;
#pragma unroll
    for (int i = 0; i < VPT; ++i) {
        const int k = k_lo + threadIdx.x + i * THREADS;
        if (k < k_hi) st_stream(ya + k, norm_v<DT>(e[i], inv));
    }
    if (edge) yr[ej] = Elem<DT>::from_float(ee * inv);
}

// ------------------------------------------------------------------ generic
// Any D / alignment: three passes over the row (max, sum, write); only the first comes
// from DRAM, the other two are served by L1/L2.
constexpr int kSmGenericThreads = 256;

template <int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(kSmGenericThreads)
softmax_generic_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ y, int64_t rows, int64_t D) {
    constexpr int T = kSmGenericThreads;
    __shared__ float slots[2 * kWarp];
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

        uint32_t mx = neg_inf_word<DT>();
        for (int64_t i = threadIdx.x; i < nbody; i += T) mx = max_w<DT>(mx, max_v<DT>(xb[i]));
        float m = hmax_of<DT>(mx);
        for (int64_t j = threadIdx.x; j < head; j += T) m = fmaxf(m, Elem<DT>::to_float(xr[j]));
        for (int64_t j = tail0 + threadIdx.x; j < D; j += T) m = fmaxf(m, Elem<DT>::to_float(xr[j]));
        m = cta_max<T>(m, slots, 0);
        const float m2 = m * kLog2e;

        float s = 0.0f;
        f32x2 e[kExpPairs<DT>];
        for (int64_t i = threadIdx.x; i < nbody; i += T) s += exp_v<DT>(xb[i], m2, e);
        for (int64_t j = threadIdx.x; j < head; j += T) s += fast_exp2(fmaf(Elem<DT>::to_float(xr[j]), kLog2e, -m2));
        for (int64_t j = tail0 + threadIdx.x; j < D; j += T) s += fast_exp2(fmaf(Elem<DT>::to_float(xr[j]), kLog2e, -m2));
        s = cta_sum<T>(s, slots, 1);
        const float inv = 1.0f / s;

        uint4* yb = reinterpret_cast<uint4*>(yr + head);
        for (int64_t i = threadIdx.x; i < nbody; i += T) {
            exp_v<DT>(xb[i], m2, e);
            st_stream(yb + i, norm_v<DT>(e, inv));
        }
        for (int64_t j = threadIdx.x; j < head; j += T)
            yr[j] = Elem<DT>::from_float(fast_exp2(fmaf(Elem<DT>::to_float(xr[j]), kLog2e, -m2)) * inv);
        for (int64_t j = tail0 + threadIdx.x; j < D; j += T)
            yr[j] = Elem<DT>::from_float(fast_exp2(fmaf(Elem<DT>::to_float(xr[j]), kLog2e, -m2)) * inv);
    }
}

// fp32 rows with no 16-byte alignment: element-wise, three passes (the last two from L1/L2).
__global__ void __launch_bounds__(kSmGenericThreads)
softmax_generic32_kernel(const float* __restrict__ x, float* __restrict__ y, int64_t rows, int64_t D) {
    constexpr int T = kSmGenericThreads;
    __shared__ float slots[2 * kWarp];
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const float* xr = x + row * D;
        float* yr = y + row * D;
        float m = -INFINITY;
        for (int64_t j = threadIdx.x; j < D; j += T) m = fmaxf(m, xr[j]);
        m = cta_max<T>(m, slots, 0);
        const float m2 = m * kLog2e;
        float s = 0.0f;
        for (int64_t j = threadIdx.x; j < D; j += T) s += fast_exp2(fmaf(xr[j], kLog2e, -m2));
        s = cta_sum<T>(s, slots, 1);
        const float inv = 1.0f / s;
        for (int64_t j = threadIdx.x; j < D; j += T) yr[j] = fast_exp2(fmaf(xr[j], kLog2e, -m2)) * inv;
    }
}

}  // namespace ak
