// Rotary position embedding forward (paper Table 3 "rotary_emb": interleaved rotation,
// sincosf; Table 4 rows "rotary", batch x heads x sequence x head_dim).
//
//   x: [n_seq, S, Dh];  pair i = elements (2i, 2i + 1) of the head vector at position
//   p = pos_offset + s is rotated by theta = p * base^(-2i / Dh).
//
// One read and one write of every element.  The angle of a pair depends on (s, i) only, not
// on the sequence (batch x head) index, so a thread owns one 16-byte vector slot (s, four or
// two pairs) and evaluates its sines and cosines ONCE, then walks the sequences that share
// them: the transcendental work is amortised over n_seq / chunks rows and the inner loop is
// a handful of packed multiply-adds per 16 bytes.  Since the trigonometry is off the hot loop
// it can afford to be exact: the frequencies base^(-2i/Dh) are computed on the host in double
// and travel as kernel parameters; the angle is the double product fl(p * f) - the angle an
// fp64 evaluation of the definition uses - reduced to [-pi, pi] in double with a two-term 2 pi,
// and only the reduced argument goes to single-precision sincosf (its accurate small-argument
// branch).  The cosine and sine OF THAT ANGLE are right to fp32 rounding at any position up to
// 2^52.  Against the real-number product the angle itself carries the rounding of the double
// multiplication, at most p * f * 2^-53 rad: below fp32's own rounding while p * f < 2^28, 6e-5
// rad at p * f = 2^40.  (Carrying the product's low part would remove that, and would then
// disagree with every fp64 evaluation of p * f by the same amount: not done.)
#include <cmath>

#include "ak_common.cuh"

namespace ak {
namespace {

constexpr int kRopeMaxPairs = 256;   // Dh <= 512: the frequency table stays within 2 KiB of parameters
constexpr int kRopeThreads = 128;

struct RopeFreq {
    double inv_freq[kRopeMaxPairs];
};

__device__ __forceinline__ void angle_sincos(double pos, double inv_freq, float& c, float& s) {
    const double a = pos * inv_freq;
    const double k = rint(a * 0.15915494309189535);           // a / (2 pi)
    double r = fma(-k, 6.283185307179586, a);                  // 2 pi, high part
    r = fma(-k, 2.4492935982947064e-16, r);                    // 2 pi, low part
    sincosf((float)r, &s, &c);
}

// (x0, x1) -> (x0 c - x1 s, x0 s + x1 c) on a packed pair
__device__ __forceinline__ f32x2 rotate(f32x2 x, f32x2 cc, f32x2 ns_s) {
    float x0, x1;
    unpack2(x, x0, x1);
    return fma2(pack2(x1, x0), ns_s, mul2(x, cc));
}

template <int DT>
__device__ __forceinline__ uint4 rotate_vec(const uint4& v, const f32x2* cc, const f32x2* ns) {
    if constexpr (DT == AK_DTYPE_F32) {
        float a, b, c, d;
        unpack2(rotate(pack2(__uint_as_float(v.x), __uint_as_float(v.y)), cc[0], ns[0]), a, b);
        unpack2(rotate(pack2(__uint_as_float(v.z), __uint_as_float(v.w)), cc[1], ns[1]), c, d);
        return make_uint4(__float_as_uint(a), __float_as_uint(b), __float_as_uint(c), __float_as_uint(d));
    } else {
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint32_t o[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float lo, hi;
            unpack2(rotate(widen2_t<DT>(w[k]), cc[k], ns[k]), lo, hi);
            o[k] = Elem<DT>::pack(lo, hi);
        }
        return make_uint4(o[0], o[1], o[2], o[3]);
    }
}

// grid = (ceil(S * vpr / T), chunks of sequences).  vpr = 16-byte vectors per head vector.
template <int DT, int UNROLL>
__global__ void __launch_bounds__(kRopeThreads)
rope_vec_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int64_t n_seq, int64_t nvs, int vpr,
                int64_t pos_offset, int seq_per_cta, const __grid_constant__ RopeFreq freq) {
    constexpr int PPV = Elem<DT>::kPerVec / 2;   // pairs per vector
    const int64_t v = (int64_t)blockIdx.x * kRopeThreads + threadIdx.x;
    int64_t n = (int64_t)blockIdx.y * seq_per_cta;
    int64_t n_end = n + seq_per_cta;
    if (n_end > n_seq) n_end = n_seq;
    const uint4* xp = x + n * nvs + v;
    uint4* yp = y + n * nvs + v;
    // Launched as a programmatic dependent; nothing is read or written before the wait.  (The
    // prefetch of the first wave that the row kernels do before their wait is left out here: for
    // these strided 2 KiB segments it measured 0.8-1.4 us slower per launch.)
    pdl_wait();
    pdl_launch_dependents();
    if (v >= nvs) return;
    const int64_t s = v / vpr;
    const int j = (int)(v - s * vpr);
    // the first batch of loads is in flight while the sines and cosines are evaluated
    uint4 q[UNROLL];
    const bool full_first = n + UNROLL <= n_end;
    if (full_first) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) q[u] = ld_stream(xp + u * nvs);
    }
    const double pos = (double)(pos_offset + s);
    f32x2 cc[PPV], ns[PPV];
#pragma unroll
    for (int k = 0; k < PPV; ++k) {
        float c, sn;
        angle_sincos(pos, freq.inv_freq[j * PPV + k], c, sn);
        cc[k] = pack2(c, c);
        ns[k] = pack2(-sn, sn);
    }
    if (full_first) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) st_stream(yp + u * nvs, rotate_vec<DT>(q[u], cc, ns));
        n += UNROLL, xp += UNROLL * nvs, yp += UNROLL * nvs;
    }
    for (; n + UNROLL <= n_end; n += UNROLL, xp += UNROLL * nvs, yp += UNROLL * nvs) {
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) q[u] = ld_stream(xp + u * nvs);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) st_stream(yp + u * nvs, rotate_vec<DT>(q[u], cc, ns));
    }
    for (; n < n_end; ++n, xp += nvs, yp += nvs) st_stream(yp, rotate_vec<DT>(ld_stream(xp), cc, ns));
}

// Any alignment of the element type and any even Dh: one thread per pair slot (s, i), single
// element accesses.  The slow, always-correct fallback.
template <int DT>
__global__ void __launch_bounds__(kRopeThreads)
rope_pair_kernel(const void* __restrict__ xv, void* __restrict__ yv, int64_t n_seq, int64_t nps, int half,
                 int64_t pos_offset, int seq_per_cta, const __grid_constant__ RopeFreq freq) {
    const int64_t p = (int64_t)blockIdx.x * kRopeThreads + threadIdx.x;
    if (p >= nps) return;
    const int64_t s = p / half;
    const int i = (int)(p - s * half);
    float c, sn;
    angle_sincos((double)(pos_offset + s), freq.inv_freq[i], c, sn);
    int64_t n = (int64_t)blockIdx.y * seq_per_cta;
    int64_t n_end = n + seq_per_cta;
    if (n_end > n_seq) n_end = n_seq;
    for (; n < n_end; ++n) {
        const int64_t e = (n * nps + p) * 2;
        if constexpr (DT == AK_DTYPE_F32) {
            const float* xs = static_cast<const float*>(xv);
            float* ys = static_cast<float*>(yv);
            const float a = xs[e], b = xs[e + 1];
            ys[e] = fmaf(-b, sn, a * c);
            ys[e + 1] = fmaf(a, sn, b * c);
        } else {
            const uint16_t* xs = static_cast<const uint16_t*>(xv);
            uint16_t* ys = static_cast<uint16_t*>(yv);
            const float a = Elem<DT>::to_float(xs[e]), b = Elem<DT>::to_float(xs[e + 1]);
            ys[e] = Elem<DT>::from_float(fmaf(-b, sn, a * c));
            ys[e + 1] = Elem<DT>::from_float(fmaf(a, sn, b * c));
        }
    }
}

// Sequences are cut into chunks (grid.y) so that the grid fills the GPU (about 32 CTAs of 128
// threads per SM in total), but a chunk keeps at least eight sequences where it can (one full
// batch of loads, in flight while the trigonometry runs), so the trigonometry stays amortised.
// (Timed on B200 for 296 .. 4736 CTAs and 4 / 8 / 16 sequences: within 10 % of each other; this
// choice was best or tied on every shape.)
void chunking(int64_t gx, int64_t n_seq, int* seq_per_cta, unsigned* gy) {
    const int64_t target = (int64_t)sm_count() * 32;
    constexpr int64_t minseq = 8;
    int64_t want = (target + gx - 1) / gx;
    int64_t most = n_seq / minseq > 1 ? n_seq / minseq : 1;
    if (want > most) want = most;
    if (want > 65535) want = 65535;
    if (want < 1) want = 1;
    int64_t per = (n_seq + want - 1) / want;
    if (per > 2147483647LL) per = 2147483647LL;
    *seq_per_cta = (int)per;
    *gy = (unsigned)((n_seq + per - 1) / per);
}

template <int DT>
int rope_t(const void* x, void* y, int64_t n_seq, int64_t S, int64_t Dh, int64_t pos_offset, const RopeFreq& freq,
           cudaStream_t st) {
    constexpr int PV = Elem<DT>::kPerVec;
    int seq_per_cta;
    unsigned gy;
    if (Dh % PV == 0 && is_aligned(x, 16) && is_aligned(y, 16)) {
        const int vpr = (int)(Dh / PV);
        const int64_t nvs = S * vpr;
        const int64_t gx = (nvs + kRopeThreads - 1) / kRopeThreads;
        if (gx > 2147483647LL) return AK_ERR_SHAPE;
        chunking(gx, n_seq, &seq_per_cta, &gy);
        if ((n_seq + seq_per_cta - 1) / seq_per_cta > 65535) return AK_ERR_SHAPE;
        auto kernel = rope_vec_kernel<DT, 8>;
        const cudaError_t e = launch_dependent(kernel, dim3((unsigned)gx, gy), dim3(kRopeThreads), 0, st,
                                               static_cast<const uint4*>(x), static_cast<uint4*>(y), n_seq, nvs, vpr,
                                               pos_offset, seq_per_cta, freq);
        count_launch();
        return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
    } else {
        const int half = (int)(Dh / 2);
        const int64_t nps = S * half;
        const int64_t gx = (nps + kRopeThreads - 1) / kRopeThreads;
        if (gx > 2147483647LL) return AK_ERR_SHAPE;
        chunking(gx, n_seq, &seq_per_cta, &gy);
        if ((n_seq + seq_per_cta - 1) / seq_per_cta > 65535) return AK_ERR_SHAPE;
        rope_pair_kernel<DT><<<dim3((unsigned)gx, gy), kRopeThreads, 0, st>>>(x, y, n_seq, nps, half, pos_offset,
                                                                             seq_per_cta, freq);
    }
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

}  // namespace

int rope_dispatch(const void* x, void* y, int64_t n_seq, int64_t S, int64_t Dh, float base, int64_t pos_offset,
                  int dtype, cudaStream_t st) {
    if (Dh / 2 > kRopeMaxPairs) return AK_ERR_SHAPE;
    RopeFreq freq;
    for (int i = 0; i < kRopeMaxPairs; ++i)
        freq.inv_freq[i] = (2 * i < Dh) ? std::pow((double)base, -2.0 * (double)i / (double)Dh) : 0.0;
    switch (dtype) {
        case AK_DTYPE_BF16: return rope_t<AK_DTYPE_BF16>(x, y, n_seq, S, Dh, pos_offset, freq, st);
        case AK_DTYPE_F16: return rope_t<AK_DTYPE_F16>(x, y, n_seq, S, Dh, pos_offset, freq, st);
        case AK_DTYPE_F32: return rope_t<AK_DTYPE_F32>(x, y, n_seq, S, Dh, pos_offset, freq, st);
        default: return AK_ERR_ARG;
    }
}

}  // namespace ak
