// Last-dim softmax forward kernels (paper Table 3 "softmax": warp-shuffle reductions,
// packed 16-bit loads).
//
//   m = max_k x[r, k];  y[r, j] = bf16_rne( exp(x[r, j] - m) / sum_k exp(x[r, k] - m) )
//
// exp is evaluated as 2^(x*log2e - rn(m*log2e)) with one FMA feeding the SFU.  Rounding
// m*log2e once scales every term of the row by the same factor, which cancels in the
// ratio.  -inf entries give 2^(-inf) = 0 exactly; an all -inf row, +inf or NaN gives NaN
// through inf - inf, as IEEE arithmetic on the definition would.
//
// Paths mirror RMSNorm: warp per row, CTA per row (row in registers: the exponentials
// are kept in fp32 so each is computed once), and a generic three-pass path for any
// D / alignment whose re-reads are served by L1/L2.
#include "ak_common.cuh"

namespace ak {
namespace {

constexpr uint32_t kNegInf2 = 0xFF80FF80u;  // two bf16 -inf

__device__ __forceinline__ uint32_t max8(const uint4& v) {
    return bf16x2_max(bf16x2_max(v.x, v.y), bf16x2_max(v.z, v.w));
}
__device__ __forceinline__ float hmax_of(uint32_t m2) { return fmaxf(bf16lo(m2), bf16hi(m2)); }

// e[0..7] = 2^(x*log2e - m2); returns their sum (fixed association).
__device__ __forceinline__ float exp8(const uint4& v, float m2, float* e) {
    e[0] = fast_exp2(fmaf(bf16lo(v.x), kLog2e, -m2));
    e[1] = fast_exp2(fmaf(bf16hi(v.x), kLog2e, -m2));
    e[2] = fast_exp2(fmaf(bf16lo(v.y), kLog2e, -m2));
    e[3] = fast_exp2(fmaf(bf16hi(v.y), kLog2e, -m2));
    e[4] = fast_exp2(fmaf(bf16lo(v.z), kLog2e, -m2));
    e[5] = fast_exp2(fmaf(bf16hi(v.z), kLog2e, -m2));
    e[6] = fast_exp2(fmaf(bf16lo(v.w), kLog2e, -m2));
    e[7] = fast_exp2(fmaf(bf16hi(v.w), kLog2e, -m2));
    return ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
}
__device__ __forceinline__ uint4 norm8(const float* e, float inv) {
    return make_uint4(pack_bf16x2(e[0] * inv, e[1] * inv), pack_bf16x2(e[2] * inv, e[3] * inv),
                      pack_bf16x2(e[4] * inv, e[5] * inv), pack_bf16x2(e[6] * inv, e[7] * inv));
}

// ------------------------------------------------------------------ CTA per row
template <int THREADS, int VPT>
__global__ void __launch_bounds__(THREADS)
softmax_cta_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int64_t rows, int nvec) {
    __shared__ float slots[2 * kWarp];
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint4* xr = x + row * nvec;
        uint4 xv[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = threadIdx.x + k * THREADS;
            xv[k] = (i < nvec) ? ld_stream(xr + i) : make_uint4(kNegInf2, kNegInf2, kNegInf2, kNegInf2);
        }
        uint32_t mx = kNegInf2;
#pragma unroll
        for (int k = 0; k < VPT; ++k) mx = bf16x2_max(mx, max8(xv[k]));
        const float m = cta_max<THREADS>(hmax_of(mx), slots, 0);
        const float m2 = m * kLog2e;
        float e[VPT][8];
        float s = 0.0f;
#pragma unroll
        for (int k = 0; k < VPT; ++k) s += exp8(xv[k], m2, e[k]);
        s = cta_sum<THREADS>(s, slots, 1);
        const float inv = 1.0f / s;
        uint4* yr = y + row * nvec;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = threadIdx.x + k * THREADS;
            if (i < nvec) st_stream(yr + i, norm8(e[k], inv));
        }
    }
}

// ------------------------------------------------------------------ warp per row
template <int WARPS, int VPT>
__global__ void __launch_bounds__(WARPS * kWarp)
softmax_warp_kernel(const uint4* __restrict__ x, uint4* __restrict__ y, int64_t rows, int nvec) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * WARPS + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * WARPS;
    for (int64_t row = warp0; row < rows; row += nwarps) {
        const uint4* xr = x + row * nvec;
        uint4 xv[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = lane + k * kWarp;
            xv[k] = (i < nvec) ? ld_stream(xr + i) : make_uint4(kNegInf2, kNegInf2, kNegInf2, kNegInf2);
        }
        uint32_t mx = kNegInf2;
#pragma unroll
        for (int k = 0; k < VPT; ++k) mx = bf16x2_max(mx, max8(xv[k]));
        const float m = warp_max(hmax_of(mx));
        const float m2 = m * kLog2e;
        float e[VPT][8];
        float s = 0.0f;
#pragma unroll
        for (int k = 0; k < VPT; ++k) s += exp8(xv[k], m2, e[k]);
        s = warp_sum(s);
        const float inv = 1.0f / s;
        uint4* yr = y + row * nvec;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = lane + k * kWarp;
            if (i < nvec) st_stream(yr + i, norm8(e[k], inv));
        }
    }
}

// ------------------------------------------------------------------ generic
constexpr int kGenericThreads = 256;

__global__ void __launch_bounds__(kGenericThreads)
softmax_generic_kernel(const uint16_t* __restrict__ x, uint16_t* __restrict__ y, int64_t rows, int64_t D) {
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

        // pass 1: row maximum (DRAM read; leaves the row in L1/L2)
        uint32_t mx = kNegInf2;
        for (int64_t i = threadIdx.x; i < nbody; i += kGenericThreads) mx = bf16x2_max(mx, max8(xb[i]));
        float m = hmax_of(mx);
        for (int64_t j = threadIdx.x; j < head; j += kGenericThreads) m = fmaxf(m, bf16_to_float(xr[j]));
        for (int64_t j = tail0 + threadIdx.x; j < D; j += kGenericThreads) m = fmaxf(m, bf16_to_float(xr[j]));
        m = cta_max<kGenericThreads>(m, slots, 0);
        const float m2 = m * kLog2e;

        // pass 2: sum of exponentials
        float s = 0.0f, e[8];
        for (int64_t i = threadIdx.x; i < nbody; i += kGenericThreads) s += exp8(xb[i], m2, e);
        for (int64_t j = threadIdx.x; j < head; j += kGenericThreads)
            s += fast_exp2(fmaf(bf16_to_float(xr[j]), kLog2e, -m2));
        for (int64_t j = tail0 + threadIdx.x; j < D; j += kGenericThreads)
            s += fast_exp2(fmaf(bf16_to_float(xr[j]), kLog2e, -m2));
        s = cta_sum<kGenericThreads>(s, slots, 1);
        const float inv = 1.0f / s;

        // pass 3: normalise and store
        uint4* yb = reinterpret_cast<uint4*>(yr + head);
        for (int64_t i = threadIdx.x; i < nbody; i += kGenericThreads) {
            exp8(xb[i], m2, e);
            st_stream(yb + i, norm8(e, inv));
        }
        for (int64_t j = threadIdx.x; j < head; j += kGenericThreads)
            yr[j] = float_to_bf16(fast_exp2(fmaf(bf16_to_float(xr[j]), kLog2e, -m2)) * inv);
        for (int64_t j = tail0 + threadIdx.x; j < D; j += kGenericThreads)
            yr[j] = float_to_bf16(fast_exp2(fmaf(bf16_to_float(xr[j]), kLog2e, -m2)) * inv);
        // the barrier inside the next row's cta_max (slot set 0) is preceded by this row's
        // cta_sum barrier (slot set 1), so both slot sets are free again here
    }
}

// ------------------------------------------------------------------ launch helpers
template <typename K>
int resident_ctas(K kernel, int threads) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, 0) != cudaSuccess ||
        per_sm < 1)
        per_sm = 1;
    return per_sm * sm_count();
}

template <int THREADS, int VPT>
int launch_cta(const void* x, void* y, int64_t rows, int nvec, cudaStream_t st) {
    static const int resident = resident_ctas(softmax_cta_kernel<THREADS, VPT>, THREADS);
    const int grid = (int)(rows < resident || !persistent_grid() ? rows : resident);
    softmax_cta_kernel<THREADS, VPT><<<grid, THREADS, 0, st>>>(
        static_cast<const uint4*>(x), static_cast<uint4*>(y), rows, nvec);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

template <int THREADS>
int launch_cta_vpt(int vpt, const void* x, void* y, int64_t rows, int nvec, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_cta<THREADS, 1>(x, y, rows, nvec, st);
        case 2: return launch_cta<THREADS, 2>(x, y, rows, nvec, st);
        case 3: return launch_cta<THREADS, 3>(x, y, rows, nvec, st);
        case 4: return launch_cta<THREADS, 4>(x, y, rows, nvec, st);
        default: break;
    }
    if constexpr (THREADS == 512) {
        switch (vpt) {
            case 5: return launch_cta<512, 5>(x, y, rows, nvec, st);
            case 6: return launch_cta<512, 6>(x, y, rows, nvec, st);
            case 7: return launch_cta<512, 7>(x, y, rows, nvec, st);
            case 8: return launch_cta<512, 8>(x, y, rows, nvec, st);
            default: break;
        }
    }
    return AK_ERR_SHAPE;
}

constexpr int kWarpsPerCta = 4;

template <int VPT>
int launch_warp(const void* x, void* y, int64_t rows, int nvec, cudaStream_t st) {
    static const int resident =
        resident_ctas(softmax_warp_kernel<kWarpsPerCta, VPT>, kWarpsPerCta * kWarp);
    const int64_t need = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
    const int grid = (int)(need < resident || !persistent_grid() ? need : resident);
    softmax_warp_kernel<kWarpsPerCta, VPT><<<grid, kWarpsPerCta * kWarp, 0, st>>>(
        static_cast<const uint4*>(x), static_cast<uint4*>(y), rows, nvec);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

}  // namespace

int softmax_choose(int64_t rows, int64_t D, bool aligned16) {
    (void)rows;
    if (!aligned16 || (D & 7) != 0 || D > 32768) return AK_PATH_GENERIC;
    return D <= 1024 ? AK_PATH_WARP : AK_PATH_CTA;
}

int softmax_dispatch(const void* x, void* y, int64_t rows, int64_t D, cudaStream_t st, int path) {
    const bool aligned16 = is_aligned(x, 16) && is_aligned(y, 16);
    if (path == AK_PATH_AUTO) path = softmax_choose(rows, D, aligned16);
    if (path == AK_PATH_WARP || path == AK_PATH_CTA) {
        if ((D & 7) != 0) return AK_ERR_SHAPE;
        if (!aligned16) return AK_ERR_ALIGN;
    }
    switch (path) {
        case AK_PATH_WARP: {
            if (D > 2048) return AK_ERR_SHAPE;
            const int nvec = (int)(D >> 3);
            switch ((nvec + 31) / 32) {
                case 1: return launch_warp<1>(x, y, rows, nvec, st);
                case 2: return launch_warp<2>(x, y, rows, nvec, st);
                case 3: return launch_warp<3>(x, y, rows, nvec, st);
                case 4: return launch_warp<4>(x, y, rows, nvec, st);
                case 5: return launch_warp<5>(x, y, rows, nvec, st);
                case 6: return launch_warp<6>(x, y, rows, nvec, st);
                case 7: return launch_warp<7>(x, y, rows, nvec, st);
                default: return launch_warp<8>(x, y, rows, nvec, st);
            }
        }
        case AK_PATH_CTA: {
            if (D > 32768) return AK_ERR_SHAPE;
            const int nvec = (int)(D >> 3);
            int threads, vpt;
            cta_shape(nvec, &threads, &vpt);
            if (threads == 128) return launch_cta_vpt<128>(vpt, x, y, rows, nvec, st);
            if (threads == 256) return launch_cta_vpt<256>(vpt, x, y, rows, nvec, st);
            return launch_cta_vpt<512>(vpt, x, y, rows, nvec, st);
        }
        case AK_PATH_GENERIC: {
            static const int resident = resident_ctas(softmax_generic_kernel, kGenericThreads);
            const int grid = (int)(rows < resident ? rows : resident);
            softmax_generic_kernel<<<grid, kGenericThreads, 0, st>>>(
                static_cast<const uint16_t*>(x), static_cast<uint16_t*>(y), rows, D);
            count_launch();
            return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
        }
        default:
            return AK_ERR_ARG;
    }
}

}  // namespace ak
