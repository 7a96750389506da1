// LayerNorm forward: host dispatch.  Kernels live in layernorm_kernels.cuh.
//
// Same dispatch structure as RMSNorm (the op moves the same bytes: one read of x, one write
// of y, gamma and beta from L1/L2): a warp per row for short rows, a CTA per row with the
// row in registers up to 32 KiB, the row staged in shared memory by bulk copies beyond, and
// the phase-staged kernel for rows that are not 16-byte aligned.
#include "layernorm_kernels.cuh"

namespace ak {
namespace {

template <int THREADS, int GROUP, int VPT, int MINB>
int launch_reg(const void* x, const void* g, const void* b, void* y, int64_t rows, int nvec, float inv_D,
               float eps, cudaStream_t st) {
    constexpr int GROUPS = THREADS / GROUP;
    const int64_t grid = (rows + GROUPS - 1) / GROUPS;
    layernorm_reg_kernel<THREADS, GROUP, VPT, MINB><<<(unsigned)grid, THREADS, 0, st>>>(
        static_cast<const uint4*>(x), static_cast<const uint4*>(g), static_cast<const uint4*>(b),
        static_cast<uint4*>(y), rows, nvec, inv_D, eps);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// vectors per thread 1..8 for a fixed (THREADS, GROUP); the minimum-CTAs-per-SM hint (a register
// cap) is given per vector count: M14 for 1..4 vectors, M56 for 5..6, M7 and M8 for 7 and 8
template <int THREADS, int GROUP, int M14, int M56, int M7, int M8>
int launch_reg_vpt(int vpt, const void* x, const void* g, const void* b, void* y, int64_t rows, int nvec,
                   float inv_D, float eps, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_reg<THREADS, GROUP, 1, M14>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 2: return launch_reg<THREADS, GROUP, 2, M14>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 3: return launch_reg<THREADS, GROUP, 3, M14>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 4: return launch_reg<THREADS, GROUP, 4, M14>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 5: return launch_reg<THREADS, GROUP, 5, M56>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 6: return launch_reg<THREADS, GROUP, 6, M56>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 7: return launch_reg<THREADS, GROUP, 7, M7>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 8: return launch_reg<THREADS, GROUP, 8, M8>(x, g, b, y, rows, nvec, inv_D, eps, st);
        default: return AK_ERR_SHAPE;
    }
}

template <int THREADS>
int launch_smem(const void* x, const void* g, const void* b, void* y, int64_t rows, int nvec, float inv_D,
                float eps, cudaStream_t st) {
    const size_t smem = (size_t)nvec * 16;
    static const bool configured = [] {
        return cudaFuncSetAttribute(layernorm_smem_kernel<THREADS>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    kMaxRowSmemBytes) == cudaSuccess;
    }();
    if (!configured) return AK_ERR_CUDA;
    layernorm_smem_kernel<THREADS><<<(unsigned)rows, THREADS, smem, st>>>(
        static_cast<const uint4*>(x), static_cast<const uint4*>(g), static_cast<const uint4*>(b),
        static_cast<uint4*>(y), nvec, inv_D, eps);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

template <int T>
int launch_stage(const uint16_t* x, const uint16_t* g, const uint16_t* b, uint16_t* y, int64_t rows, int64_t D,
                 size_t stage_bytes, float inv_D, float eps, cudaStream_t st) {
    static const bool configured = [] {
        return cudaFuncSetAttribute(layernorm_stage_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    kMaxRowSmemBytes) == cudaSuccess;
    }();
    if (!configured) return AK_ERR_CUDA;
    layernorm_stage_kernel<T><<<(unsigned)rows, T, stage_bytes, st>>>(x, g, b, y, D, inv_D, eps);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

template <int THREADS, int VPT, int MINB>
int launch_regp(const uint16_t* x, const uint16_t* g, const uint16_t* b, uint16_t* y, int64_t rows, int64_t D,
                float inv_D, float eps, cudaStream_t st) {
    layernorm_regp_kernel<THREADS, VPT, MINB><<<(unsigned)rows, THREADS, 0, st>>>(x, g, b, y, D, inv_D, eps);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}
// unaligned rows held in registers: vectors per thread 1..8 for a CTA of THREADS threads
// (register caps: M14 for 1..5 vectors, M58 for 6..8)
template <int THREADS, int M14, int M58>
int launch_regp_vpt(int vpt, const uint16_t* x, const uint16_t* g, const uint16_t* b, uint16_t* y, int64_t rows,
                    int64_t D, float inv_D, float eps, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_regp<THREADS, 1, M14>(x, g, b, y, rows, D, inv_D, eps, st);
        case 2: return launch_regp<THREADS, 2, M14>(x, g, b, y, rows, D, inv_D, eps, st);
        case 3: return launch_regp<THREADS, 3, M14>(x, g, b, y, rows, D, inv_D, eps, st);
        case 4: return launch_regp<THREADS, 4, M14>(x, g, b, y, rows, D, inv_D, eps, st);
        case 5: return launch_regp<THREADS, 5, M14>(x, g, b, y, rows, D, inv_D, eps, st);
        case 6: return launch_regp<THREADS, 6, M58>(x, g, b, y, rows, D, inv_D, eps, st);
        case 7: return launch_regp<THREADS, 7, M58>(x, g, b, y, rows, D, inv_D, eps, st);
        case 8: return launch_regp<THREADS, 8, M58>(x, g, b, y, rows, D, inv_D, eps, st);
        default: return AK_ERR_SHAPE;
    }
}

}  // namespace

int layernorm_choose(int64_t rows, int64_t D, bool aligned16) {
    (void)rows;
    if (!aligned16 || (D & 7) != 0 || D * 2 > kMaxRowSmemBytes) return AK_PATH_GENERIC;
    if (D <= 2048) return AK_PATH_WARP;
    if (D <= 16384) return AK_PATH_CTA;
    return AK_PATH_SMEM;
}

int layernorm_dispatch(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t D,
                       float eps, cudaStream_t st, int path) {
    const bool aligned16 = is_aligned(x, 16) && is_aligned(y, 16) && is_aligned(gamma, 16) && is_aligned(beta, 16);
    if (path == AK_PATH_AUTO) path = layernorm_choose(rows, D, aligned16);
    const float inv_D = 1.0f / (float)D;
    if (path != AK_PATH_GENERIC) {
        if ((D & 7) != 0) return AK_ERR_SHAPE;
        if (!aligned16) return AK_ERR_ALIGN;
    }
    if (rows > 2147483647LL) return AK_ERR_SHAPE;  // grid.x limit of the one-row-per-CTA layouts
    const int nvec = (int)(D >> 3);
    switch (path) {
        // Launch shapes and register caps below were picked by timing each candidate in the
        // sustained (power-capped) regime of a long run.
        case AK_PATH_WARP:
            if (D > 2048) return AK_ERR_SHAPE;
            if (nvec <= 128)   // a warp per row, 8 rows per CTA, 46 registers
                return launch_reg_vpt<256, 32, 5, 1, 1, 1>((nvec + 31) / 32, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            // two warps per row, 4 rows per CTA
            return launch_reg_vpt<256, 64, 5, 1, 1, 1>((nvec + 63) / 64, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
        case AK_PATH_CTA:
            if (D > 32768) return AK_ERR_SHAPE;
            if (nvec <= 1024)  // 128 threads x up to 8 vectors: many small CTAs per SM
                return launch_reg_vpt<128, 128, 10, 8, 6, 8>((nvec + 127) / 128, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            if (nvec <= 2048)
                return launch_reg_vpt<256, 256, 5, 4, 4, 4>((nvec + 255) / 256, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            return launch_reg_vpt<512, 512, 1, 2, 2, 2>((nvec + 511) / 512, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
        case AK_PATH_SMEM:
            if (D * 2 > kMaxRowSmemBytes) return AK_ERR_SHAPE;
            if (nvec <= 4096) return launch_smem<256>(x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            return launch_smem<512>(x, gamma, beta, y, rows, nvec, inv_D, eps, st);
        case AK_PATH_GENERIC: {
            const size_t stage_bytes = (size_t)((D + 14) >> 3) * 16;
            const bool same_phase = ((reinterpret_cast<uintptr_t>(x) ^ reinterpret_cast<uintptr_t>(y)) & 15) == 0;
            const uint16_t* xs = static_cast<const uint16_t*>(x);
            const uint16_t* gs = static_cast<const uint16_t*>(gamma);
            const uint16_t* bs = static_cast<const uint16_t*>(beta);
            uint16_t* ys = static_cast<uint16_t*>(y);
            // rows of up to 1024 covering vectors stay in the registers of a 128-thread CTA
            const int64_t max_nv = (D + 14) >> 3;   // vectors covering the row at the worst phase
            if (same_phase && is_aligned(gamma, 4) && is_aligned(beta, 4) && max_nv <= 1024)
                return launch_regp_vpt<128, 10, 6>((int)((max_nv + 127) / 128), xs, gs, bs, ys, rows, D, inv_D, eps, st);
            if (same_phase && is_aligned(gamma, 4) && is_aligned(beta, 4) && stage_bytes <= (size_t)kMaxRowSmemBytes) {
                if (D <= 8192) return launch_stage<128>(xs, gs, bs, ys, rows, D, stage_bytes, inv_D, eps, st);
                if (D <= 32768) return launch_stage<256>(xs, gs, bs, ys, rows, D, stage_bytes, inv_D, eps, st);
                return launch_stage<512>(xs, gs, bs, ys, rows, D, stage_bytes, inv_D, eps, st);
            }
            static const int resident = [] {
                int per_sm = 0;
                if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, layernorm_generic_kernel,
                                                                  kLnGenericThreads, 0) != cudaSuccess || per_sm < 1)
                    per_sm = 1;
                return per_sm * sm_count();
            }();
            const int grid = (int)(rows < resident ? rows : resident);
            layernorm_generic_kernel<<<grid, kLnGenericThreads, 0, st>>>(xs, gs, bs, ys, rows, D, inv_D, eps);
            count_launch();
            return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
        }
        default:
            return AK_ERR_ARG;
    }
}

}  // namespace ak
