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

// A slice = elements [begin, end) of one row, cut into up to kPerVec - 1 head elements (single
// loads until the address is 16-byte aligned), nbody aligned 16-byte vectors, and up to
// kPerVec - 1 tail elements.  One batch = UNROLL vectors per thread, all loaded before the
// first use.  Full batches run without any per-vector bounds test (constant offsets from one
// moving pointer); a single masked batch finishes the slice.
template <int DT>
struct Slice {
    const typename XElem<DT>::type* p;
    int64_t n, head, nbody, tail0, nfull;
    const uint4* body;
    int rest;  // vectors in the masked last batch, < T * UNROLL
};
template <int UNROLL, int T, int DT>
__device__ __forceinline__ Slice<DT> make_slice(const typename XElem<DT>::type* __restrict__ xr, int64_t begin, int64_t end) {
    constexpr int PV = Elem<DT>::kPerVec;
    constexpr int LOG_PV = (PV == 8) ? 3 : 2, LOG_BYTES = (Elem<DT>::kBytes == 2) ? 1 : 2;
    Slice<DT> s;
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
__device__ __forceinline__ void load_first_batch(const Slice<DT>& s, uint4 (&q)[UNROLL]) {
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

// CTA-wide online (m, s) over a slice whose first batch `q` is already in flight.  Returns,
// in every thread, the maximum M and the sum S relative to MF = max(rn(M*log2e), kFloor2).
// Uses both slot sets (max then sum).
template <int UNROLL, int POLY, int T, int DT>
__device__ __forceinline__ void slice_lse(const Slice<DT>& sl, uint4 (&q)[UNROLL], float* slots, float& M, float& S) {
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
    if ((int64_t)threadIdx.x < sl.head) absorb_scalar(o, xload<DT>(sl.p + threadIdx.x));
    if (sl.tail0 + threadIdx.x < sl.n) absorb_scalar(o, xload<DT>(sl.p + sl.tail0 + threadIdx.x));

    // NaN must win the max: fmaxf in cta_max would drop it, so it travels as +inf plus a flag
    const bool has_nan = (o.m != o.m) || (o.m == INFINITY);  // +inf makes inf - inf: NaN row as well
    M = cta_max<T>(has_nan ? INFINITY : o.m, slots, 0);
    const float MF = fmaxf(M * kLog2e, kFloor2);
    float s0, s1;
    unpack2(o.s2, s0, s1);
    float s = (s0 + s1) * fast_exp2(o.mf - MF);
    if (has_nan) s = __int_as_float(0x7fc00000);
    S = cta_sum<T>(s, slots, 1);
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
template <int UNROLL, int POLY, int MINB = 1, int T = kXentThreads, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(T, MINB)
xent_row_kernel(const typename XElem<DT>::type* __restrict__ logits, const int64_t* __restrict__ targets,
                int64_t ignore_index, float* __restrict__ loss_rows, int64_t V) {
    __shared__ float slots[2 * kWarp];
    pdl_launch_dependents();
    const int64_t row = blockIdx.x;
    const typename XElem<DT>::type* xr = logits + row * V;
    const int64_t t = targets[row];
    if (t == ignore_index || t < 0 || t >= V) {  // uniform across the CTA: nothing is read
        if (threadIdx.x == 0) loss_rows[row] = (t == ignore_index) ? 0.0f : __int_as_float(0x7fc00000);
        return;
    }
    // (Requesting the first batch before the target is known was measured: no gain, and
    // ignored rows would be touched.)
    const Slice<DT> sl = make_slice<UNROLL, T, DT>(xr, 0, V);
    uint4 q[UNROLL];
    load_first_batch<UNROLL, T, DT>(sl, q);
    // the target logit is fetched now, under the row's own traffic, not after the reduction
    const float xt = (threadIdx.x == 0) ? xread<DT>(xr + t) : 0.0f;
    float M, S;
    slice_lse<UNROLL, POLY, T, DT>(sl, q, slots, M, S);
    if (threadIdx.x == 0) loss_rows[row] = finish_loss(M, S, xt);
}

// ------------------------------------------------------------------ split row, phase 1
// grid = (nsplit, rows).  Slice boundaries are multiples of 8 elements so an aligned row
// keeps aligned slices.  partial[row * nsplit + split] = (M, S) of the slice.
template <int UNROLL, int POLY, int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(kXentThreads)
xent_split_kernel(const typename XElem<DT>::type* __restrict__ logits, const int64_t* __restrict__ targets,
                  int64_t ignore_index, float2* __restrict__ partial, int64_t V, int nsplit) {
    __shared__ float slots[2 * kWarp];
    pdl_launch_dependents();
    const int64_t row = blockIdx.y;
    const int sp = blockIdx.x;
    const int64_t t = targets[row];
    if (t == ignore_index || t < 0 || t >= V) return;
    const int64_t groups = (V + 7) >> 3;
    int64_t begin = ((groups * sp) / nsplit) << 3;
    int64_t end = ((groups * (sp + 1)) / nsplit) << 3;
    if (end > V) end = V;
    const Slice<DT> sl = make_slice<UNROLL, kXentThreads, DT>(logits + row * V, begin, end);
    uint4 q[UNROLL];
    load_first_batch<UNROLL, kXentThreads, DT>(sl, q);
    float M, S;
    slice_lse<UNROLL, POLY, kXentThreads, DT>(sl, q, slots, M, S);
    if (threadIdx.x == 0) partial[row * nsplit + sp] = make_float2(M, S);
}

// ------------------------------------------------------------------ finish: merge + mean
// One CTA, launched as a programmatic dependent of the streaming kernel.  Thread i owns
// rows i, i + T, i + 2T, ...: for the split layout it first merges the row's partials in
// split order and writes the loss; then (if out_mean / out_pair is given) it adds its
// rows' counted losses in fp64 in that order, and a fixed shuffle + shared-memory tree
// adds the threads.  out_mean = sum / count (0/0 = NaN); out_pair = {sum, count}.
constexpr int kFinishThreads = 1024;

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <int DT = AK_DTYPE_BF16>
__global__ void __launch_bounds__(kFinishThreads)
xent_finish_kernel(const typename XElem<DT>::type* __restrict__ logits, const int64_t* __restrict__ targets,
                   int64_t ignore_index, const float2* __restrict__ partial, int nsplit,
                   float* __restrict__ loss_rows, int64_t rows, int64_t V,
                   float* __restrict__ out_mean, double* __restrict__ out_pair) {
    constexpr int T = kFinishThreads;
    __shared__ double ssum[T / kWarp];
    __shared__ double scnt[T / kWarp];
    // The targets are inputs, not results of the streaming kernel: which of this thread's first
    // sixteen rows count is worked out before the wait, while that kernel is still running.
    constexpr int B = 16;
    uint32_t counted0 = 0;
    if (out_mean != nullptr || out_pair != nullptr) {
#pragma unroll
        for (int k = 0; k < B; ++k) {
            const int64_t r = threadIdx.x + (int64_t)k * T;
            if (r < rows && targets[r] != ignore_index) counted0 |= 1u << k;
        }
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
    }
    if (out_mean == nullptr && out_pair == nullptr) return;
    // Mean: batches of independent loads (a lone CTA is latency-bound, so sixteen rows are in
    // flight per thread), added in row order per thread.  A thread re-reads only rows it
    // wrote itself above, so program order makes them visible.
    double acc = 0.0, cnt = 0.0;
    {   // the first batch: the counted rows are known already
        float ll[B];
#pragma unroll
        for (int k = 0; k < B; ++k) {
            const int64_t r = threadIdx.x + (int64_t)k * T;
            ll[k] = (r < rows) ? __ldcg(loss_rows + r) : 0.0f;  // L2 read: written by the grid we depend on
        }
#pragma unroll
        for (int k = 0; k < B; ++k) {
            if (counted0 & (1u << k)) {
                acc += (double)ll[k];
                cnt += 1.0;
            }
        }
    }
    for (int64_t base = threadIdx.x + (int64_t)T * B; base < rows; base += (int64_t)T * B) {
        int64_t tt[B];
        float ll[B];
#pragma unroll
        for (int k = 0; k < B; ++k) {
            const int64_t r = base + (int64_t)k * T;
            tt[k] = (r < rows) ? targets[r] : ignore_index;
            ll[k] = (r < rows) ? __ldcg(loss_rows + r) : 0.0f;
        }
#pragma unroll
        for (int k = 0; k < B; ++k) {
            if (tt[k] != ignore_index) {
                acc += (double)ll[k];
                cnt += 1.0;
            }
        }
    }
    acc = warp_sum_f64(acc);
    cnt = warp_sum_f64(cnt);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) { ssum[warp] = acc; scnt[warp] = cnt; }
    __syncthreads();
    if (warp == 0) {
        acc = warp_sum_f64(ssum[lane]);
        cnt = warp_sum_f64(scnt[lane]);
        if (lane == 0) {
            if (out_mean) out_mean[0] = (cnt > 0.0) ? (float)(acc / cnt) : __int_as_float(0x7fc00000);
            if (out_pair) { out_pair[0] = acc; out_pair[1] = cnt; }
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
