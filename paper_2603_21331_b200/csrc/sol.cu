// Speed-of-light measurement aids: a plain streaming copy and a plain streaming read, with
// the same 16-byte streaming accesses and small one-shot CTAs as the row kernels.  They do
// no arithmetic of the ops; the benchmark times them in the same process to show the HBM
// ceiling this GPU offers for 1:1 read/write traffic and for read-only traffic.
#include "ak_common.cuh"

namespace ak {
namespace {

constexpr int kSolThreads = 256;

// every thread moves UNROLL 16-byte vectors; a CTA covers one contiguous 8 KiB (copy) span
template <int UNROLL>
__global__ void __launch_bounds__(kSolThreads)
sol_copy_kernel(const uint4* __restrict__ in, uint4* __restrict__ out, size_t nvec) {
    const size_t base = (size_t)blockIdx.x * kSolThreads * UNROLL + threadIdx.x;
    uint4 v[UNROLL];
#pragma unroll
    for (int k = 0; k < UNROLL; ++k) {
        const size_t i = base + (size_t)k * kSolThreads;
        if (i < nvec) v[k] = ld_stream(in + i);
    }
#pragma unroll
    for (int k = 0; k < UNROLL; ++k) {
        const size_t i = base + (size_t)k * kSolThreads;
        if (i < nvec) st_stream(out + i, v[k]);
    }
}

// every CTA reads one contiguous span of `per_cta` vectors and folds it into one word
template <int UNROLL>
__global__ void __launch_bounds__(kSolThreads)
sol_read_kernel(const uint4* __restrict__ in, uint32_t* __restrict__ sink, size_t nvec, size_t per_cta) {
    const size_t b0 = (size_t)blockIdx.x * per_cta;
    const size_t b1 = (b0 + per_cta < nvec) ? b0 + per_cta : nvec;
    uint32_t acc = 0;
    for (size_t base = b0 + threadIdx.x; base < b1; base += (size_t)kSolThreads * UNROLL) {
        uint4 v[UNROLL];
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) {
            const size_t i = base + (size_t)k * kSolThreads;
            v[k] = (i < b1) ? ld_stream(in + i) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int k = 0; k < UNROLL; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
    }
    // keeps the loads alive; the comparison is never true for the benchmark's data
    if (acc == 0x9E3779B9u) sink[0] = acc;
}

}  // namespace
}  // namespace ak

using namespace ak;

extern "C" int ak_sol_copy(const void* src, void* dst, size_t bytes, void* cuda_stream) {
    if (!src || !dst) return AK_ERR_NULL;
    if (!is_aligned(src, 16) || !is_aligned(dst, 16) || (bytes & 15) != 0) return AK_ERR_ALIGN;
    if (bytes == 0) return AK_OK;
    const size_t nvec = bytes / 16;
    const size_t grid = (nvec + kSolThreads * 2 - 1) / (kSolThreads * 2);
    if (grid > 2147483647u) return AK_ERR_SHAPE;
    sol_copy_kernel<2><<<(unsigned)grid, kSolThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const uint4*>(src), static_cast<uint4*>(dst), nvec);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

extern "C" int ak_sol_read(const void* src, size_t bytes, void* sink4, void* cuda_stream) {
    if (!src || !sink4) return AK_ERR_NULL;
    if (!is_aligned(src, 16) || !is_aligned(sink4, 4) || (bytes & 15) != 0) return AK_ERR_ALIGN;
    if (bytes == 0) return AK_OK;
    const size_t nvec = bytes / 16;
    const size_t per_cta = 16384;  // 256 KiB per CTA, the size of a 128K-vocabulary row
    const size_t grid = (nvec + per_cta - 1) / per_cta;
    if (grid > 2147483647u) return AK_ERR_SHAPE;
    sol_read_kernel<4><<<(unsigned)grid, kSolThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const uint4*>(src), static_cast<uint32_t*>(sink4), nvec, per_cta);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}
