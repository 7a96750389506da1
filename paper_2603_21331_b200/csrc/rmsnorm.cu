// RMSNorm forward kernels (paper Table 3 "rmsnorm": warp-shuffle reduction + fast rsqrt,
// weight multiply fused into the epilogue per Section 7.3 Tier 3).
//
//   y[r, j] = bf16_rne( x[r, j] * rsqrt(mean_k x[r, k]^2 + eps) * w[j] )
//
// Three paths, all one DRAM read + one DRAM write per element, fp32 accumulation,
// fixed-order reductions:
//   warp    one warp owns a row (D <= 2048): no barriers; weights live in registers
//   cta     one CTA owns a row (D <= 32768): row in registers as packed bf16, weights too
//   generic any D / alignment: scalar head and tail, 16-byte body, second pass from L1/L2
// Register paths are persistent: a CTA (warp) walks rows with a grid stride so the
// per-column weights are fetched once per CTA instead of once per row.
#include "ak_common.cuh"

namespace ak {
namespace {

__device__ __forceinline__ float sumsq8(const uint4& v) {
    float a0 = bf16lo(v.x), a1 = bf16hi(v.x), a2 = bf16lo(v.y), a3 = bf16hi(v.y);
    float a4 = bf16lo(v.z), a5 = bf16hi(v.z), a6 = bf16lo(v.w), a7 = bf16hi(v.w);
    float s0 = a0 * a0, s1 = a1 * a1;
    s0 = fmaf(a2, a2, s0); s1 = fmaf(a3, a3, s1);
    s0 = fmaf(a4, a4, s0); s1 = fmaf(a5, a5, s1);
    s0 = fmaf(a6, a6, s0); s1 = fmaf(a7, a7, s1);
    return s0 + s1;
}

__device__ __forceinline__ uint32_t scale2(uint32_t x, uint32_t w, float rstd) {
    return pack_bf16x2(bf16lo(x) * rstd * bf16lo(w), bf16hi(x) * rstd * bf16hi(w));
}
__device__ __forceinline__ uint4 scale8(const uint4& x, const uint4& w, float rstd) {
    return make_uint4(scale2(x.x, w.x, rstd), scale2(x.y, w.y, rstd),
                      scale2(x.z, w.z, rstd), scale2(x.w, w.w, rstd));
}

// ------------------------------------------------------------------ CTA per row
template <int THREADS, int VPT>
__global__ void __launch_bounds__(THREADS)
rmsnorm_cta_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w, uint4* __restrict__ y,
                   int64_t rows, int nvec, float inv_D, float eps) {
    __shared__ float slots[2 * kWarp];
    uint4 wv[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int i = threadIdx.x + k * THREADS;
        wv[k] = (i < nvec) ? __ldg(w + i) : make_uint4(0, 0, 0, 0);
    }
    int phase = 0;
    for (int64_t row = blockIdx.x; row < rows; row += gridDim.x) {
        const uint4* xr = x + row * nvec;
        uint4 xv[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = threadIdx.x + k * THREADS;
            xv[k] = (i < nvec) ? ld_stream(xr + i) : make_uint4(0, 0, 0, 0);
        }
        float ss = 0.0f;
#pragma unroll
        for (int k = 0; k < VPT; ++k) ss += sumsq8(xv[k]);
        ss = cta_sum<THREADS>(ss, slots, phase);
        phase ^= 1;
        const float rstd = rsqrtf(fmaf(ss, inv_D, eps));
        uint4* yr = y + row * nvec;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = threadIdx.x + k * THREADS;
            if (i < nvec) st_stream(yr + i, scale8(xv[k], wv[k], rstd));
        }
    }
}

// ------------------------------------------------------------------ warp per row
template <int WARPS, int VPT>
__global__ void __launch_bounds__(WARPS * kWarp)
rmsnorm_warp_kernel(const uint4* __restrict__ x, const uint4* __restrict__ w, uint4* __restrict__ y,
                    int64_t rows, int nvec, float inv_D, float eps) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = (int64_t)blockIdx.x * WARPS + (threadIdx.x >> 5);
    const int64_t nwarps = (int64_t)gridDim.x * WARPS;
    uint4 wv[VPT];
#pragma unroll
    for (int k = 0; k < VPT; ++k) {
        const int i = lane + k * kWarp;
        wv[k] = (i < nvec) ? __ldg(w + i) : make_uint4(0, 0, 0, 0);
    }
    for (int64_t row = warp0; row < rows; row += nwarps) {
        const uint4* xr = x + row * nvec;
        uint4 xv[VPT];
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = lane + k * kWarp;
            xv[k] = (i < nvec) ? ld_stream(xr + i) : make_uint4(0, 0, 0, 0);
        }
        float ss = 0.0f;
#pragma unroll
        for (int k = 0; k < VPT; ++k) ss += sumsq8(xv[k]);
        ss = warp_sum(ss);
        const float rstd = rsqrtf(fmaf(ss, inv_D, eps));
        uint4* yr = y + row * nvec;
#pragma unroll
        for (int k = 0; k < VPT; ++k) {
            const int i = lane + k * kWarp;
            if (i < nvec) st_stream(yr + i, scale8(xv[k], wv[k], rstd));
        }
    }
}

// ------------------------------------------------------------------ generic
// Any D and any 2-byte alignment.  Row r starts at element r*D, so its 16-byte phase
// changes from row to row: up to 7 head elements and 7 tail elements are handled with
// 2-byte accesses, the body with 16-byte vectors (when x and y share the phase).  The
// second pass re-reads the row, which one CTA has just pulled through L1/L2.
constexpr int kGenericThreads = 256;

__global__ void __launch_bounds__(kGenericThreads)
rmsnorm_generic_kernel(const uint16_t* __restrict__ x, const uint16_t* __restrict__ w,
                       uint16_t* __restrict__ y, int64_t rows, int64_t D, float inv_D, float eps) {
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
        for (int64_t i = threadIdx.x; i < nbody; i += kGenericThreads) ss += sumsq8(xb[i]);
        for (int64_t j = threadIdx.x; j < head; j += kGenericThreads) {
            const float v = bf16_to_float(xr[j]);
            ss = fmaf(v, v, ss);
        }
        for (int64_t j = tail0 + threadIdx.x; j < D; j += kGenericThreads) {
            const float v = bf16_to_float(xr[j]);
            ss = fmaf(v, v, ss);
        }
        ss = cta_sum<kGenericThreads>(ss, slots, phase);
        phase ^= 1;
        const float rstd = rsqrtf(fmaf(ss, inv_D, eps));

        uint4* yb = reinterpret_cast<uint4*>(yr + head);
        for (int64_t i = threadIdx.x; i < nbody; i += kGenericThreads) {
            const uint4 v = xb[i];
            const uint16_t* wj = w + head + (i << 3);
            uint4 wq;
            wq.x = (uint32_t)__ldg(wj + 0) | ((uint32_t)__ldg(wj + 1) << 16);
            wq.y = (uint32_t)__ldg(wj + 2) | ((uint32_t)__ldg(wj + 3) << 16);
            wq.z = (uint32_t)__ldg(wj + 4) | ((uint32_t)__ldg(wj + 5) << 16);
            wq.w = (uint32_t)__ldg(wj + 6) | ((uint32_t)__ldg(wj + 7) << 16);
            st_stream(yb + i, scale8(v, wq, rstd));
        }
        for (int64_t j = threadIdx.x; j < head; j += kGenericThreads)
            yr[j] = float_to_bf16(bf16_to_float(xr[j]) * rstd * bf16_to_float(__ldg(w + j)));
        for (int64_t j = tail0 + threadIdx.x; j < D; j += kGenericThreads)
            yr[j] = float_to_bf16(bf16_to_float(xr[j]) * rstd * bf16_to_float(__ldg(w + j)));
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
int launch_cta(const void* x, const void* w, void* y, int64_t rows, int nvec, float inv_D, float eps,
               cudaStream_t st) {
    static const int resident = resident_ctas(rmsnorm_cta_kernel<THREADS, VPT>, THREADS);
    const int grid = (int)(rows < resident || !persistent_grid() ? rows : resident);
    rmsnorm_cta_kernel<THREADS, VPT><<<grid, THREADS, 0, st>>>(
        static_cast<const uint4*>(x), static_cast<const uint4*>(w), static_cast<uint4*>(y),
        rows, nvec, inv_D, eps);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

template <int THREADS>
int launch_cta_vpt(int vpt, const void* x, const void* w, void* y, int64_t rows, int nvec, float inv_D,
                   float eps, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_cta<THREADS, 1>(x, w, y, rows, nvec, inv_D, eps, st);
        case 2: return launch_cta<THREADS, 2>(x, w, y, rows, nvec, inv_D, eps, st);
        case 3: return launch_cta<THREADS, 3>(x, w, y, rows, nvec, inv_D, eps, st);
        case 4: return launch_cta<THREADS, 4>(x, w, y, rows, nvec, inv_D, eps, st);
        default: break;
    }
    if constexpr (THREADS == 512) {
        switch (vpt) {
            case 5: return launch_cta<512, 5>(x, w, y, rows, nvec, inv_D, eps, st);
            case 6: return launch_cta<512, 6>(x, w, y, rows, nvec, inv_D, eps, st);
            case 7: return launch_cta<512, 7>(x, w, y, rows, nvec, inv_D, eps, st);
            case 8: return launch_cta<512, 8>(x, w, y, rows, nvec, inv_D, eps, st);
            default: break;
        }
    }
    return AK_ERR_SHAPE;
}

constexpr int kWarpsPerCta = 4;

template <int VPT>
int launch_warp(const void* x, const void* w, void* y, int64_t rows, int nvec, float inv_D, float eps,
                cudaStream_t st) {
    static const int resident =
        resident_ctas(rmsnorm_warp_kernel<kWarpsPerCta, VPT>, kWarpsPerCta * kWarp);
    const int64_t need = (rows + kWarpsPerCta - 1) / kWarpsPerCta;
    const int grid = (int)(need < resident || !persistent_grid() ? need : resident);
    rmsnorm_warp_kernel<kWarpsPerCta, VPT><<<grid, kWarpsPerCta * kWarp, 0, st>>>(
        static_cast<const uint4*>(x), static_cast<const uint4*>(w), static_cast<uint4*>(y),
        rows, nvec, inv_D, eps);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

}  // namespace

// CTA shape for the register path: threads chosen from the vector count, then the number
// of 16-byte vectors each thread holds.
void cta_shape(int nvec, int* threads, int* vpt) {
    int t = nvec <= 512 ? 128 : nvec <= 1024 ? 256 : 512;
    *threads = t;
    *vpt = (nvec + t - 1) / t;
}

int rmsnorm_choose(int64_t rows, int64_t D, bool aligned16) {
    (void)rows;
    if (!aligned16 || (D & 7) != 0 || D > 32768) return AK_PATH_GENERIC;
    return D <= 1024 ? AK_PATH_WARP : AK_PATH_CTA;
}

int rmsnorm_dispatch(const void* x, const void* w, void* y, int64_t rows, int64_t D, float eps,
                     cudaStream_t st, int path) {
    const bool aligned16 = is_aligned(x, 16) && is_aligned(y, 16) && is_aligned(w, 16);
    if (path == AK_PATH_AUTO) path = rmsnorm_choose(rows, D, aligned16);
    const float inv_D = 1.0f / (float)D;
    if (path == AK_PATH_WARP || path == AK_PATH_CTA) {
        if ((D & 7) != 0) return AK_ERR_SHAPE;
        if (!aligned16) return AK_ERR_ALIGN;
    }
    switch (path) {
        case AK_PATH_WARP: {
            if (D > 2048) return AK_ERR_SHAPE;
            const int nvec = (int)(D >> 3);
            switch ((nvec + 31) / 32) {
                case 1: return launch_warp<1>(x, w, y, rows, nvec, inv_D, eps, st);
                case 2: return launch_warp<2>(x, w, y, rows, nvec, inv_D, eps, st);
                case 3: return launch_warp<3>(x, w, y, rows, nvec, inv_D, eps, st);
                case 4: return launch_warp<4>(x, w, y, rows, nvec, inv_D, eps, st);
                case 5: return launch_warp<5>(x, w, y, rows, nvec, inv_D, eps, st);
                case 6: return launch_warp<6>(x, w, y, rows, nvec, inv_D, eps, st);
                case 7: return launch_warp<7>(x, w, y, rows, nvec, inv_D, eps, st);
                default: return launch_warp<8>(x, w, y, rows, nvec, inv_D, eps, st);
            }
        }
        case AK_PATH_CTA: {
            if (D > 32768) return AK_ERR_SHAPE;
            const int nvec = (int)(D >> 3);
            int threads, vpt;
            cta_shape(nvec, &threads, &vpt);
            if (threads == 128) return launch_cta_vpt<128>(vpt, x, w, y, rows, nvec, inv_D, eps, st);
            if (threads == 256) return launch_cta_vpt<256>(vpt, x, w, y, rows, nvec, inv_D, eps, st);
            return launch_cta_vpt<512>(vpt, x, w, y, rows, nvec, inv_D, eps, st);
        }
        case AK_PATH_GENERIC: {
            static const int resident = resident_ctas(rmsnorm_generic_kernel, kGenericThreads);
            const int grid = (int)(rows < resident ? rows : resident);
            rmsnorm_generic_kernel<<<grid, kGenericThreads, 0, st>>>(
                static_cast<const uint16_t*>(x), static_cast<const uint16_t*>(w),
                static_cast<uint16_t*>(y), rows, D, inv_D, eps);
            count_launch();
            return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
        }
        default:
            return AK_ERR_ARG;
    }
}

}  // namespace ak
