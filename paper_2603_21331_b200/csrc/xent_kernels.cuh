// Fused cross-entropy forward device kernels (paper Table 3 "cross_ent": online log-sum-exp
// fused with the NLL gather; a single pass over the logits).
//
//   loss[r] = (m - x[r, t]) + log( sum_k exp(x[r, k] - m) ),  m = max_k x[r, k]
//
// Kernels take the element type DT of the logits (bf16, fp16 or fp32) as a template parameter.
//
// Each thread streams 16-byte vectors of its row (or of its slice of the row) and keeps an
// online pair: the running maximum m (always a value of the element type) and s = sum 2^(x*log2e - mf)
// with mf = rn(m*log2e).  Rescaling by 2^(mf_old - mf_new) happens once per batch of
// vectors, only when the maximum moved.  Working in the rounded log2 domain is exact up to
// one per-row constant: x*log2e - m*log2e = (x*log2e - mf) - err with
// err = fma(m, log2e, -mf) (the rounding error of a product is representable), so
//   log sum exp(x - m) = ln2 * (log2(s) - err).
// The loss is assembled as (m - x_t) + that term: both parts are >= 0, and no large
// magnitude is ever added to a small one.
//
// The kernel is co-bound by HBM and by the SFU: one exponential per two bytes keeps the
// transcendental pipe ~78 % busy at 5.8 TB/s.  POLY of every 8 exponentials are therefore
// evaluated on the FMA pipe instead (round-to-nearest range reduction + degree-4 minimax
// polynomial, relative error 2.7e-6, the split is fixed per element so results stay
// deterministic), and the multiply-adds and the summation use the packed f32x2 forms to
// halve the instruction count.
#pragma once

#include "ak_common.cuh"

namespace ak {

constexpr float kFloor2 = -1.0e30f;  // finite stand-in for "no maximum yet" in the log2 domain
constexpr int kXentThreads = 256;

// Per element type DT: the storage type of one element, the -inf padding word, and the
// NaN-propagating maximum of a 16-byte vector (a NaN logit must surface as a NaN loss).  The
// running maximum of a batch travels as one 32-bit word (a packed pair for the 16-bit types,
// the float's bits for fp32).
template <int DT> struct XElem { using type = uint16_t; };
template <> struct XElem<AK_DTYPE_F32> { using type = float; };
template <int DT>
__device__ __forceinline__ constexpr uint32_t xneg_inf_word() {
    if constexpr (DT == AK_DTYPE_F32) return 0xFF800000u; else return Elem<DT>::kNegInf2;
}
template <int DT>
__device__ __forceinline__ uint4 xneg_inf_vec() {
    return make_uint4(xneg_inf_word<DT>(), xneg_inf_word<DT>(), xneg_inf_word<DT>(), xneg_inf_word<DT>());
}
template <int DT>
__device__ __forceinline__ uint32_t xmax_w(uint32_t a, uint32_t b) {
    if constexpr (DT == AK_DTYPE_F32) {
        uint32_t r;
        asm("max.NaN.f32 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    } else {
        return Elem<DT>::max2_nan(a, b);
    }
}
template <int DT>
__device__ __forceinline__ uint32_t xmax_v(const uint4& v) {
    return xmax_w<DT>(xmax_w<DT>(v.x, v.y), xmax_w<DT>(v.z, v.w));
}
template <int DT>
__device__ __forceinline__ float xhmax_of(uint32_t m2) {
    if constexpr (DT == AK_DTYPE_F32) {
        return __uint_as_float(m2);
    } else {
        const float a = Elem<DT>::lo(m2), b = Elem<DT>::hi(m2);
        return (a != a || b != b) ? __int_as_float(0x7fc00000) : fmaxf(a, b);
    }
}
template <int DT>
__device__ __forceinline__ float xload(const typename XElem<DT>::type* p) {   // one element, streaming
    if constexpr (DT == AK_DTYPE_F32) return __ldcs(p); else return Elem<DT>::to_float(ld_stream_u16(p));
}
template <int DT>
__device__ __forceinline__ float xread(const typename XElem<DT>::type* p) {   // one element, cached
    if constexpr (DT == AK_DTYPE_F32) return *p; else return Elem<DT>::to_float(*p);
}

// 2^t for a pair, t <= ~0, on the FMA pipe.  t is clamped at -125 (2^-125 stands in for
// anything smaller, including 2^-inf: negligible against a sum that is >= 1), rounded to
// the nearest integer n with the 1.5 * 2^23 trick, and 2^(t - n) comes from a degree-4
// minimax polynomial on [-0.5, 0.5]; n is added to the exponent field.
__device__ __forceinline__ f32x2 poly_exp2_pair(f32x2 t2) {
    float t0, t1;
    unpack2(t2, t0, t1);
    const f32x2 tc = pack2(fmaxf(t0, -125.0f), fmaxf(t1, -125.0f));
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
    p0 = __int_as_float(__float_as_int(p0) + (__float_as_int(z0) << 23));
    p1 = __int_as_float(__float_as_int(p1) + (__float_as_int(z1) << 23));
    return pack2(p0, p1);
}
__device__ __forceinline__ f32x2 sfu_exp2_pair(f32x2 t2) {
    float t0, t1;
    unpack2(t2, t0, t1);
    return pack2(fast_exp2(t0), fast_exp2(t1));
}

// sum over the elements of one vector of 2^(x*log2e - mf), as a packed pair of partial sums.
// 16-bit types: four pairs, the first POLY / 2 of them take the polynomial, the rest the SFU.
// fp32: two pairs and half as many exponentials per byte, so the SFU keeps up: pair k takes
// the polynomial only if POLY >= 4 * (k + 1).
template <int POLY, int DT>
__device__ __forceinline__ f32x2 sumexp_v(const uint4& v, f32x2 l2, f32x2 nmf2) {
    static_assert(POLY % 2 == 0 && POLY >= 0 && POLY <= 8, "pairs");
    if constexpr (DT == AK_DTYPE_F32) {
        const f32x2 t0 = fma2(pack2(__uint_as_float(v.x), __uint_as_float(v.y)), l2, nmf2);
        const f32x2 t1 = fma2(pack2(__uint_as_float(v.z), __uint_as_float(v.w)), l2, nmf2);
        const f32x2 e0 = (POLY >= 4) ? poly_exp2_pair(t0) : sfu_exp2_pair(t0);
        const f32x2 e1 = (POLY >= 8) ? poly_exp2_pair(t1) : sfu_exp2_pair(t1);
        return add2(e0, e1);
    } else {
        const f32x2 t0 = fma2(widen2_t<DT>(v.x), l2, nmf2);
        const f32x2 t1 = fma2(widen2_t<DT>(v.y), l2, nmf2);
        const f32x2 t2 = fma2(widen2_t<DT>(v.z), l2, nmf2);
        const f32x2 t3 = fma2(widen2_t<DT>(v.w), l2, nmf2);
        const f32x2 e0 = (POLY >= 2) ? poly_exp2_pair(t0) : sfu_exp2_pair(t0);
        const f32x2 e1 = (POLY >= 4) ? poly_exp2_pair(t1) : sfu_exp2_pair(t1);
        const f32x2 e2 = (POLY >= 6) ? poly_exp2_pair(t2) : sfu_exp2_pair(t2);
        const f32x2 e3 = (POLY >= 8) ? poly_exp2_pair(t3) : sfu_exp2_pair(t3);
        return add2(add2(e0, e1), add2(e2, e3));
    }
}

struct Online {
    float m;    // running maximum (bf16-valued; -inf when nothing finite seen; NaN sticks)
    float mf;   // max(rn(m * log2e), kFloor2)
    f32x2 s2;   // two partial sums of 2^(x*log2e - mf)
};

__device__ __forceinline__ void raise_max(Online& o, float vm) {
    const float vmf = fmaxf(vm * kLog2e, kFloor2);
    if (vmf > o.mf) {
        const float r = fast_exp2(o.mf - vmf);
        o.s2 = fma2(o.s2, pack2(r, r), pack2(0.0f, 0.0f));
        o.mf = vmf;
    }
    o.m = (vm != vm) ? vm : fmaxf(o.m, vm);  // NaN sticks (fmaxf alone would drop it)
}
__device__ __forceinline__ void absorb_scalar(Online& o, float v) {
    raise_max(o, v);
    o.s2 = add2(o.s2, pack2(fast_exp2(fmaf(v, kLog2e, -o.mf)), 0.0f));
}

// ---- plain form: the masked last batch is a whole batch (used unless the row's last batch is
// mostly padding; see the trimmed form below, which gives the same bits).
// A slice = elements [begin, end) of one row, cut into up to kPerVec - 1 head elements (single
// loads until the address is 16-byte aligned), nbody aligned 16-byte vectors, and up to
// kPerVec - 1 tail elements.  One batch = UNROLL vectors per thread, all loaded before the
// first use.  Full batches run without any per-vector bounds test (constant offsets from one
// moving pointer); a single masked batch finishes the slice.
template <int DT>
struct SliceF {
    const typename XElem<DT>::type* p;
    int64_t n, head, nbody, tail0, nfull;
    const uint4* body;
    int rest;  // vectors in the masked last batch, < T * UNROLL
};
template <int UNROLL, int T, int DT>
__device__ __forceinline__ SliceF<DT> make_slice_full(const typename XElem<DT>::type* __restrict__ xr, int64_t begin, int64_t end) {
    constexpr int PV = Elem<DT>::kPerVec;
    constexpr int LOG_PV = (PV == 8) ? 3 : 2, LOG_BYTES = (Elem<DT>::kBytes == 2) ? 1 : 2;
    SliceF<DT> s;
    s.p = xr + begin;
    s.n = end - begin;
    s.head = (PV - (int)((reinterpret_cast<uintptr_t>(s.p) >> LOG_BYTES) & (PV - 1))) & (PV - 1);
    if (s.head > s.n) s.head = s.n;
    s.nbody = (s.n - s.head) >> LOG_PV;
    s.tail0 = s.head + (s.nbody << LOG_PV);
    s.body = reinterpret_cast<const uint4*>(s.p + s.head);
    s.nfull = s.nbody / ((int64_t)T * UNROLL);
    s.rest = (int)(s.nbody - s.nfull * T * UNROLL);
    return s;
}
// The slice's first batch (full if there is a full batch, otherwise the masked one).
template <int UNROLL, int T, int DT>
__device__ __forceinline__ void load_first_batch_full(const SliceF<DT>& s, uint4 (&q)[UNROLL]) {
    const uint4* src = s.body + threadIdx.x;
    if (s.nfull > 0) {
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) q[k] = ld_stream(src + k * T);
    } else {
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) {
            const int i = (int)threadIdx.x + k * T;
            q[k] = (i < s.rest) ? ld_stream(src + k * T) : xneg_inf_vec<DT>();
        }
    }
}

// One thread's online (m, s) over its share of a slice whose first batch `q` is already in flight:
// every batch, the masked last one included, absorbs all UNROLL slots (padding adds exact zeros).
template <int UNROLL, int POLY, int T, int DT>
__device__ __forceinline__ Online slice_stream_full(const SliceF<DT>& sl, uint4 (&q)[UNROLL]) {
    Online o{-INFINITY, kFloor2, pack2(0.0f, 0.0f)};
    const f32x2 l2 = pack2(kLog2e, kLog2e);
    auto absorb_batch = [&](const uint4 (&v)[UNROLL]) {
        uint32_t mx = xmax_v<DT>(v[0]);
#pragma unroll
        for (int k = 1; k < UNROLL; ++k) mx = xmax_w<DT>(mx, xmax_v<DT>(v[k]));
        raise_max(o, xhmax_of<DT>(mx));
        const f32x2 nmf2 = pack2(-o.mf, -o.mf);
        f32x2 acc = sumexp_v<POLY, DT>(v[0], l2, nmf2);
#pragma unroll
        for (int k = 1; k < UNROLL; ++k) acc = add2(acc, sumexp_v<POLY, DT>(v[k], l2, nmf2));
        o.s2 = add2(o.s2, acc);
    };
    // (taken before the loop as two small ints and a pointer: with the 64-bit fields kept alive
    // across the loop the compiler needs a spill slot)
    const int ihead = (int)sl.head, ntail = (int)(sl.n - sl.tail0);
    const typename XElem<DT>::type* ptail = sl.p + sl.tail0;
    absorb_batch(q);  // batch 0 (all padding when the slice has no body)
    const uint4* src = sl.body + threadIdx.x + T * UNROLL;
    for (int64_t b = 1; b < sl.nfull; ++b, src += T * UNROLL) {
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) q[k] = ld_stream(src + k * T);
        absorb_batch(q);
    }
    if (sl.nfull > 0 && sl.rest > 0) {
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) {
            const int i = (int)threadIdx.x + k * T;
            q[k] = (i < sl.rest) ? ld_stream(src + k * T) : xneg_inf_vec<DT>();
        }
        absorb_batch(q);
    }
    if ((int)threadIdx.x < ihead) absorb_scalar(o, xload<DT>(sl.p + threadIdx.x));
    if ((int)threadIdx.x < ntail) absorb_scalar(o, xload<DT>(ptail + threadIdx.x));
    return o;
}

// ---- trimmed form
// A slice = elements [begin, end) of one row, cut into up to kPerVec - 1 head elements (single
// loads until the address is 16-byte aligned), nbody aligned 16-byte vectors, and up to
// kPerVec - 1 tail elements.  One batch = UNROLL vectors per thread, all loaded before the
// first use.  Full batches run without any per-vector bounds test (constant offsets from one
// moving pointer); a single masked batch finishes the slice.
template <int DT>
struct Slice {
    const typename XElem<DT>::type* p;   // first element
    int64_t n;                           // elements
    int head, ntail;                     // single elements before / after the aligned body (< kPerVec each)
    int rest;                            // vectors in the masked last batch, < T * UNROLL
    const uint4* body;                   // first aligned vector
    const uint4* full_end;               // end of the full batches (== body when there is none)
};
template <int UNROLL, int T, int DT>
__device__ __forceinline__ Slice<DT> make_slice(const typename XElem<DT>::type* __restrict__ xr, int64_t begin, int64_t end) {
    constexpr int PV = Elem<DT>::kPerVec;
    constexpr int LOG_PV = (PV == 8) ? 3 : 2, LOG_BYTES = (Elem<DT>::kBytes == 2) ? 1 : 2;
    Slice<DT> s;
    s.p = xr + begin;
    s.n = end - begin;
    int64_t head = (PV - (int)((reinterpret_cast<uintptr_t>(s.p) >> LOG_BYTES) & (PV - 1))) & (PV - 1);
    if (head > s.n) head = s.n;
    const int64_t nbody = (s.n - head) >> LOG_PV;
    s.head = (int)head;
    s.ntail = (int)(s.n - head - (nbody << LOG_PV));
    s.body = reinterpret_cast<const uint4*>(s.p + head);
    const int64_t nfull = nbody / ((int64_t)T * UNROLL);
    s.rest = (int)(nbody - nfull * T * UNROLL);
    s.full_end = s.body + nfull * T * UNROLL;
    return s;
}
// The masked batch holds `rest` vectors: thread i owns vectors i, i + T, ... below `rest`, so only
// the first ceil(rest / T) of a thread's UNROLL slots can hold data, the same number for every
// thread of the CTA.  Loading and absorbing stop there (a row of 50304 bf16 is 6.14 batches of
// 16 KiB: its seventh batch fills 2 of 8 slots); the skipped slots would have added exact zeros.
template <int T>
__device__ __forceinline__ int masked_slots(int rest) { return (rest + T - 1) / T; }
template <int UNROLL, int T, int DT>
__device__ __forceinline__ void load_masked_batch(const uint4* src, int rest, int nk, uint4 (&q)[UNROLL]) {
#pragma unroll
    for (int k = 0; k < UNROLL; ++k) {
        if (k < nk) {
            const int i = (int)threadIdx.x + k * T;
            q[k] = (i < rest) ? ld_stream(src + k * T) : xneg_inf_vec<DT>();
        }
    }
}
// The slice's first batch (full if there is a full batch, otherwise the masked one; slot 0 is
// always defined, all padding when the slice has no body).
template <int UNROLL, int T, int DT>
__device__ __forceinline__ void load_first_batch(const Slice<DT>& s, uint4 (&q)[UNROLL]) {
    const uint4* src = s.body + threadIdx.x;
    if (s.full_end != s.body) {
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) q[k] = ld_stream(src + k * T);
    } else {
        q[0] = xneg_inf_vec<DT>();
        load_masked_batch<UNROLL, T, DT>(src, s.rest, masked_slots<T>(s.rest), q);
    }
}

// One thread's online (m, s) over its share of a slice whose first batch `q` is already in
// flight.  After it returns q is free again (the caller may put the next row's first batch there).
template <int UNROLL, int POLY, int T, int DT>
__device__ __forceinline__ Online slice_stream(const Slice<DT>& sl, uint4 (&q)[UNROLL]) {
    Online o{-INFINITY, kFloor2, pack2(0.0f, 0.0f)};
    const f32x2 l2 = pack2(kLog2e, kLog2e);
    auto absorb_batch = [&](const uint4 (&v)[UNROLL]) {
        uint32_t mx = xmax_v<DT>(v[0]);
#pragma unroll
        for (int k = 1; k < UNROLL; ++k) mx = xmax_w<DT>(mx, xmax_v<DT>(v[k]));
        raise_max(o, xhmax_of<DT>(mx));
        const f32x2 nmf2 = pack2(-o.mf, -o.mf);
        f32x2 acc = sumexp_v<POLY, DT>(v[0], l2, nmf2);
#pragma unroll
        for (int k = 1; k < UNROLL; ++k) acc = add2(acc, sumexp_v<POLY, DT>(v[k], l2, nmf2));
        o.s2 = add2(o.s2, acc);
    };
    // slots 0 .. nk - 1 only (nk >= 1, uniform over the CTA)
    auto absorb_masked = [&](const uint4 (&v)[UNROLL], int nk) {
        uint32_t mx = xmax_v<DT>(v[0]);
#pragma unroll
        for (int k = 1; k < UNROLL; ++k)
            if (k < nk) mx = xmax_w<DT>(mx, xmax_v<DT>(v[k]));
        raise_max(o, xhmax_of<DT>(mx));
        const f32x2 nmf2 = pack2(-o.mf, -o.mf);
        f32x2 acc = sumexp_v<POLY, DT>(v[0], l2, nmf2);
#pragma unroll
        for (int k = 1; k < UNROLL; ++k)
            if (k < nk) acc = add2(acc, sumexp_v<POLY, DT>(v[k], l2, nmf2));
        o.s2 = add2(o.s2, acc);
    };
    const int nk = masked_slots<T>(sl.rest);
    if (sl.full_end != sl.body) {
        absorb_batch(q);
        // this thread's vector k of batch b sits at body + b * T * UNROLL + k * T + threadIdx.x
        const uint4* src = sl.body + threadIdx.x + T * UNROLL;
        for (; src < sl.full_end; src += T * UNROLL) {
#pragma unroll
            for (int k = 0; k < UNROLL; ++k) q[k] = ld_stream(src + k * T);
            absorb_batch(q);
        }
        if (nk > 0) {
            load_masked_batch<UNROLL, T, DT>(sl.full_end + threadIdx.x, sl.rest, nk, q);
            absorb_masked(q, nk);
        }
    } else {
        absorb_masked(q, nk > 0 ? nk : 1);   // the first batch was the masked one
    }
    if ((int)threadIdx.x < sl.head) absorb_scalar(o, xload<DT>(sl.p + threadIdx.x));
    if ((int)threadIdx.x < sl.ntail) absorb_scalar(o, xload<DT>(sl.p + (sl.n - sl.ntail) + threadIdx.x));
    return o;
}

// The threads' pairs combined over the CTA: returns, in every thread, the maximum M and the sum S
// relative to MF = max(rn(M*log2e), kFloor2).  Every warp first combines its own lanes (the
// maximum, then the sums rescaled to the warp's maximum); the warps' pairs meet in shared memory
// behind a single barrier and every thread combines them in warp order, so all threads hold the
// same bits.  (A CTA-wide maximum followed by a CTA-wide sum costs a second barrier: 0.1-0.4 us
// per launch slower.)  `slots` = 2 * 32 floats of shared memory; a CTA calls this once, or with
// a barrier of its own between calls.
template <int T>
__device__ __forceinline__ void slice_combine(const Online& o, float* slots, float& M, float& S) {
    constexpr int NW = T / kWarp;
    // NaN must win the max: fmaxf would drop it, so it travels as +inf plus a flag
    const bool has_nan = (o.m != o.m) || (o.m == INFINITY);  // +inf makes inf - inf: NaN row as well
    float s0, s1;
    unpack2(o.s2, s0, s1);
    const float mw = warp_max(has_nan ? INFINITY : o.m);
    const float mfw = fmaxf(mw * kLog2e, kFloor2);
    float s = (s0 + s1) * fast_exp2(o.mf - mfw);
    if (has_nan) s = __int_as_float(0x7fc00000);
    s = warp_sum(s);
    if constexpr (NW == 1) {
        M = mw;
        S = s;
    } else {
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        if (lane == 0) { slots[warp] = mw; slots[kWarp + warp] = s; }
        __syncthreads();
        float m = slots[0];
#pragma unroll
        for (int w = 1; w < NW; ++w) m = fmaxf(m, slots[w]);
        const float MF = fmaxf(m * kLog2e, kFloor2);
        float sum = 0.0f;
#pragma unroll
        for (int w = 0; w < NW; ++w) sum += slots[kWarp + w] * fast_exp2(fmaxf(slots[w] * kLog2e, kFloor2) - MF);
        M = m;
        S = sum;
    }
}

// CTA-wide online (m, s) over elements [begin, end) of the row at xr: the first batch is requested,
// `early` runs (loads that should sit under the row's own traffic, not after the reduction), the
// slice is streamed and the threads' pairs are combined.  TRIM picks the form of the masked last
// batch (same bits either way).
template <int UNROLL, int POLY, int T, int DT, bool TRIM, typename Early>
__device__ __forceinline__ void row_lse(const typename XElem<DT>::type* xr, int64_t begin, int64_t end, float* slots,
                                        float& M, float& S, Early early) {
    uint4 q[UNROLL];
    Online o;
    if constexpr (TRIM) {
        const Slice<DT> sl = make_slice<UNROLL, T, DT>(xr, begin, end);
        load_first_batch<UNROLL, T, DT>(sl, q);
        early();
        o = slice_stream<UNROLL, POLY, T, DT>(sl, q);
    } else {
        const SliceF<DT> sl = make_slice_full<UNROLL, T, DT>(xr, begin, end);
        load_first_batch_full<UNROLL, T, DT>(sl, q);
        early();
        o = slice_stream_full<UNROLL, POLY, T, DT>(sl, q);
    }
    slice_combine<T>(o, slots, M, S);
}

// loss from the row's (M, S) and the target logit.
__device__ __forceinline__ float finish_loss(float M, float S, float xt) {
    const float MF = fmaxf(M * kLog2e, kFloor2);
    const float err = fmaf(M, kLog2e, -MF);
    // The exact value is >= 0 (the maximum contributes 1 to the sum); approximation error
    // can leave it a few 1e-7 below.  Clamp without swallowing a NaN.
    float lse = kLn2 * (log2f(S) - err);
    if (lse < 0.0f) lse = 0.0f;
    return (M - xt) + lse;
}

// ------------------------------------------------------------------ one CTA per row
// Launched as a programmatic dependent of whatever precedes it in the stream: nothing is read
// or written before griddepcontrol.wait, and its own dependents (the finish kernel) are let in
// only after the wait, so that they may read this kernel's inputs before their own wait.
template <int UNROLL, int POLY, int MINB = 1, int T = kXentThreads, int DT = AK_DTYPE_BF16, bool TRIM = false>
__global__ void __launch_bounds__(T, MINB)
xent_row_kernel(const typename XElem<DT>::type* __restrict__ logits, const int64_t* __restrict__ targets,
                int64_t ignore_index, float* __restrict__ loss_rows, int64_t V, int first_wave) {
    __shared__ float slots[2 * kWarp];
    if (blockIdx.x < first_wave) {
        // The CTAs of the first wave (as many as the device holds at once) become resident while
        // the grids before this one drain, and would idle at the wait.  Meanwhile they ask for the
        // first 128 bytes per thread of their row (one batch is eight times that) and for the
        // target to be brought into L2: a prefetch reads nothing architecturally, so it may precede
        // the wait.  Later CTAs start on a busy machine and skip it; prefetching more than this,
        // or in every CTA, measured slower.
        const int64_t row0 = blockIdx.x;
        const char* head = reinterpret_cast<const char*>(logits + row0 * V);
        const int64_t left = ((int64_t)gridDim.x - row0) * V * (int64_t)sizeof(typename XElem<DT>::type);
        const int64_t off = (int64_t)threadIdx.x * 128;
        if (off < left) prefetch_l2(head + off);
        if (threadIdx.x == 0) prefetch_l2(targets + row0);
    }
    pdl_wait();
    pdl_launch_dependents();
    const int64_t row = cta_id_x();   // read again, so that nothing computed above stays in registers
    const typename XElem<DT>::type* xr = logits + row * V;
    const int64_t t = targets[row];
    // (The compiler keeps this kernel inside its 64 registers without spilling only in this
    // if / else form; an early return for the rows that are not read costs a spill slot.)
    if (t != ignore_index && t >= 0 && t < V) {  // uniform across the CTA
        // (Requesting the first batch before the target is known was measured: no gain, and
        // ignored rows would be touched.)
        float xt = 0.0f, M, S;
        // the target logit is fetched under the row's own traffic, not after the reduction
        row_lse<UNROLL, POLY, T, DT, TRIM>(xr, 0, V, slots, M, S, [&] { if (threadIdx.x == 0) xt = xread<DT>(xr + t); });
        if (threadIdx.x == 0) loss_rows[row] = finish_loss(M, S, xt);
    } else if (threadIdx.x == 0) {   // nothing of the row is read
        loss_rows[row] = (t == ignore_index) ? 0.0f : __int_as_float(0x7fc00000);
    }
}

// ------------------------------------------------------------------ split row, phase 1
// grid = (nsplit, rows).  Slice boundaries are multiples of 8 elements so an aligned row
// keeps aligned slices.  partial[row * nsplit + split] = (M, S) of the slice.
template <int UNROLL, int POLY, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(kXentThreads)
xent_split_kernel(const typename XElem<DT>::type* __restrict__ logits, const int64_t* __restrict__ targets,
                  int64_t ignore_index, float2* __restrict__ partial, int64_t V, int nsplit) {
    __shared__ float slots[2 * kWarp];
    pdl_wait();
    pdl_launch_dependents();
    const int64_t row = blockIdx.y;
    const int sp = blockIdx.x;
    const int64_t t = targets[row];
    if (t == ignore_index || t < 0 || t >= V) return;
    const int64_t groups = (V + 7) >> 3;
    int64_t begin = ((groups * sp) / nsplit) << 3;
    int64_t end = ((groups * (sp + 1)) / nsplit) << 3;
    if (end > V) end = V;
    float M, S;
    row_lse<UNROLL, POLY, kXentThreads, DT, false>(logits + row * V, begin, end, slots, M, S, [] {});
    if (threadIdx.x == 0) partial[row * nsplit + sp] = make_float2(M, S);
}

// ------------------------------------------------------------------ finish: merge + mean
// One CTA, launched as a programmatic dependent of the streaming kernel.  For the split layout
// thread i first merges the partials of rows i, i + T, ... in split order and writes the losses.
// Then (if out_mean / out_pair is given) the counted losses are added in fp64 in ONE fixed order,
// whatever the CTA's size T: "virtual" thread v of kFinishVirtual = 1024 adds rows v, v + 1024, ...
// in that order; a butterfly adds the 32 lanes of each virtual warp; a second butterfly adds the
// 32 warp sums.  Physical thread i plays virtual threads i, i + T, ...: its lane is their lane,
// so the butterflies are the same and every T gives the same bits.  A small CTA (T = 256) finds a
// free slot on an SM, and lets the next kernel of the stream in, while the streaming kernel's
// last CTAs are still running; a 1024-thread CTA with its registers needs a whole empty SM.
// out_mean = sum / count (0/0 = NaN); out_pair = {sum, count}.
constexpr int kFinishVirtual = 1024;
constexpr int kFinishThreads = 256;        // fewer than kFinishSmallRows rows
constexpr int kFinishThreadsMany = 1024;
constexpr int64_t kFinishSmallRows = 1024;

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <int DT, int T>
__global__ void __launch_bounds__(T)
xent_finish_kernel(const typename XElem<DT>::type* __restrict__ logits, const int64_t* __restrict__ targets,
                   int64_t ignore_index, const float2* __restrict__ partial, int nsplit,
                   float* __restrict__ loss_rows, int64_t rows, int64_t V,
                   float* __restrict__ out_mean, double* __restrict__ out_pair) {
    constexpr int J = kFinishVirtual / T;   // virtual threads per thread
    constexpr int KB = 16 / J;              // 16 rows per thread and batch: independent loads in flight
    __shared__ double ssum[kFinishVirtual / kWarp];
    __shared__ int scnt[T / kWarp];
    pdl_launch_dependents();   // the next kernel may take free slots now (it reads nothing before its own wait)
    const bool want_sum = out_mean != nullptr || out_pair != nullptr;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // The targets are inputs of the streaming kernel, final before it let this kernel in: which
    // rows count is worked out before the wait, while that kernel is still running.  The first
    // batch's flags are kept; later batches (more than 1024 * KB rows) read their targets again.
    uint32_t counted0 = 0;
    int n_counted = 0;
    if (want_sum) {
        for (int64_t base = 0; base < rows; base += (int64_t)kFinishVirtual * KB) {
            int64_t tt[KB][J];   // all of a batch's targets are requested before the first is looked at
#pragma unroll
            for (int k = 0; k < KB; ++k)
#pragma unroll
                for (int j = 0; j < J; ++j) {
                    const int64_t r = base + (int64_t)k * kFinishVirtual + j * T + threadIdx.x;
                    tt[k][j] = (r < rows) ? targets[r] : ignore_index;
                }
#pragma unroll
            for (int k = 0; k < KB; ++k)
#pragma unroll
                for (int j = 0; j < J; ++j)
                    if (tt[k][j] != ignore_index) {
                        ++n_counted;
                        if (base == 0) counted0 |= 1u << (k * J + j);
                    }
        }
        n_counted = __reduce_add_sync(0xffffffffu, n_counted);
        if (lane == 0) scnt[warp] = n_counted;
    }
    pdl_wait();  // everything the streaming kernel wrote is visible from here on
    if (nsplit > 0) {
        for (int64_t r = threadIdx.x; r < rows; r += T) {
            const int64_t t = targets[r];
            float loss;
            if (t == ignore_index) {
                loss = 0.0f;
            } else if (t < 0 || t >= V) {
                loss = __int_as_float(0x7fc00000);
            } else {
                const float2* pr = partial + r * nsplit;
                float M = -INFINITY;
                for (int i = 0; i < nsplit; ++i) M = fmaxf(M, __ldcg(pr + i).x);
                const float MF = fmaxf(M * kLog2e, kFloor2);
                float S = 0.0f;
                for (int i = 0; i < nsplit; ++i) {
                    const float2 ps = __ldcg(pr + i);
                    S += ps.y * fast_exp2(fmaxf(ps.x * kLog2e, kFloor2) - MF);
                }
                loss = finish_loss(M, S, xread<DT>(logits + r * V + t));
            }
            loss_rows[r] = loss;
        }
        // virtual thread v = i + j * T reads rows written by thread (v mod T) = i: its own
    }
    if (!want_sum) return;
    double acc[J];
#pragma unroll
    for (int j = 0; j < J; ++j) acc[j] = 0.0;
    {   // the first batch: the counted rows are known already
        float ll[KB][J];
#pragma unroll
        for (int k = 0; k < KB; ++k)
#pragma unroll
            for (int j = 0; j < J; ++j) {
                const int64_t r = (int64_t)k * kFinishVirtual + j * T + threadIdx.x;
                ll[k][j] = (r < rows) ? __ldcg(loss_rows + r) : 0.0f;  // L2: written by the grid we depend on
            }
#pragma unroll
        for (int k = 0; k < KB; ++k)
#pragma unroll
            for (int j = 0; j < J; ++j)
                if (counted0 & (1u << (k * J + j))) acc[j] += (double)ll[k][j];
    }
    for (int64_t base = (int64_t)kFinishVirtual * KB; base < rows; base += (int64_t)kFinishVirtual * KB) {
        int64_t tt[KB][J];
        float ll[KB][J];
#pragma unroll
        for (int k = 0; k < KB; ++k)
#pragma unroll
            for (int j = 0; j < J; ++j) {
                const int64_t r = base + (int64_t)k * kFinishVirtual + j * T + threadIdx.x;
                tt[k][j] = (r < rows) ? targets[r] : ignore_index;
                ll[k][j] = (r < rows) ? __ldcg(loss_rows + r) : 0.0f;
            }
#pragma unroll
        for (int k = 0; k < KB; ++k)
#pragma unroll
            for (int j = 0; j < J; ++j)
                if (tt[k][j] != ignore_index) acc[j] += (double)ll[k][j];
    }
#pragma unroll
    for (int j = 0; j < J; ++j) {
        const double v = warp_sum_f64(acc[j]);
        if (lane == 0) ssum[warp + j * (T / kWarp)] = v;
    }
    __syncthreads();
    if (warp == 0) {
        const double total = warp_sum_f64(ssum[lane]);
        int c = (lane < T / kWarp) ? scnt[lane] : 0;
        c = __reduce_add_sync(0xffffffffu, c);
        if (lane == 0) {
            const double cnt = (double)c;
            if (out_mean) out_mean[0] = (cnt > 0.0) ? (float)(total / cnt) : __int_as_float(0x7fc00000);
            if (out_pair) { out_pair[0] = total; out_pair[1] = cnt; }
        }
    }
}

// Mean over row shards: pairs[i] = {sum_i, count_i}; added in index order by one thread.
static __global__ void xent_mean_merge_kernel(const double* __restrict__ pairs, int64_t n, float* __restrict__ out_mean) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double total = 0.0, count = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        total += pairs[2 * i];
        count += pairs[2 * i + 1];
    }
    out_mean[0] = (count > 0.0) ? (float)(total / count) : __int_as_float(0x7fc00000);
}

}  // namespace ak
