// LayerNorm forward: host dispatch.  Kernels live in layernorm_kernels.cuh.
//
// Same dispatch structure as RMSNorm (the op moves the same bytes: one read of x, one write
// of y, gamma and beta from L1/L2): a warp (or two) per row for short rows, a CTA per row with
// the row in registers up to 64 KiB, longer rows (and a few long rows) split over a thread-block
// cluster whose CTAs stage their slices in shared memory by bulk copies, and the phase kernels
// for rows that are not 16-byte aligned.  Thresholds are in row bytes,
// so they hold for every element type.
#include "layernorm_kernels.cuh"

namespace ak {
namespace {

// A launch of at most this many rows and bytes does not fill the GPU and is latency-bound: gamma
// and beta are then requested together with the row instead of after the reductions, without a
// register cap (1 x 1024 .. 512 x 4096: 5-32 % faster, e.g. 8 x 8192 4.3 -> 3.0 us; beyond 4 MiB
// the uncapped registers cost occupancy: 1024 x 8192 8.1 -> 13.3 us, so those keep the late fetch).
constexpr int64_t kEarlyParamRows = 1024, kEarlyParamBytes = 4 << 20;

template <int DT, int THREADS, int GROUP, int VPT, int MINB, bool PE = false>
int launch_reg(const void* x, const void* g, const void* b, void* y, int64_t rows, int nvec, float inv_D,
               float eps, cudaStream_t st) {
    constexpr int GROUPS = THREADS / GROUP;
    const int64_t grid = (rows + GROUPS - 1) / GROUPS;
    auto kernel = layernorm_reg_kernel<THREADS, GROUP, VPT, MINB, DT, PE>;
    // Every thread holds exactly VPT vectors: the form without bounds tests.  Its output phase may
    // fetch gamma and beta several vectors ahead, which at 4 and 8 vectors per thread (fp32: 6 and 7 too)
    // needs a few registers more than MINB CTAs per SM leave: one CTA fewer there (measured faster: 8192 x 8192
    // 45.5 -> 41.9 us), and bounds-tested output for the 512-thread shape, which has no CTA to give.
    if constexpr (GROUPS == 1) {
        constexpr bool tight = (VPT == 8 || VPT == 4 || ((VPT == 6 || VPT == 7) && DT == AK_DTYPE_F32)) && !PE;
        constexpr bool ahead = !(tight && THREADS == 512);
        constexpr int minb = (tight && THREADS < 512) ? MINB - 1 : MINB;
        if (nvec == VPT * GROUP) kernel = layernorm_reg_kernel<THREADS, GROUP, VPT, minb, DT, PE, true, ahead>;
    } else {
        // warp groups (several rows per CTA): the same form when the rows fill the groups exactly
        // (16384 x 256 5.8 -> 4.8 us, 8192 x 1024 7.9 -> 7.6 us); at four vectors per thread the output
        // loop keeps its bounds test, which keeps the kernel inside its register cap
        constexpr bool ahead = VPT != 4 || PE;
        if (nvec == VPT * GROUP && rows % GROUPS == 0) kernel = layernorm_reg_kernel<THREADS, GROUP, VPT, MINB, DT, PE, true, ahead>;
    }
    const cudaError_t e = launch_dependent(kernel, dim3((unsigned)grid), dim3(THREADS), 0, st,
                                           static_cast<const uint4*>(x), static_cast<const uint4*>(g),
                                           static_cast<const uint4*>(b), static_cast<uint4*>(y), rows, nvec, inv_D, eps,
                                           first_wave_ctas(kernel, THREADS, 0));
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// vectors per thread 1..8 for a fixed (THREADS, GROUP); the minimum-CTAs-per-SM hint (a register
// cap) is given per vector count: M14 for 1..4 vectors, M56 for 5..6, M7 and M8 for 7 and 8
template <int DT, int THREADS, int GROUP, int M14, int M56, int M7, int M8, bool PE = false>
int launch_reg_vpt(int vpt, const void* x, const void* g, const void* b, void* y, int64_t rows, int nvec,
                   float inv_D, float eps, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_reg<DT, THREADS, GROUP, 1, M14, PE>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 2: return launch_reg<DT, THREADS, GROUP, 2, M14, PE>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 3: return launch_reg<DT, THREADS, GROUP, 3, M14, PE>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 4: return launch_reg<DT, THREADS, GROUP, 4, M14, PE>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 5: return launch_reg<DT, THREADS, GROUP, 5, M56, PE>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 6: return launch_reg<DT, THREADS, GROUP, 6, M56, PE>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 7: return launch_reg<DT, THREADS, GROUP, 7, M7, PE>(x, g, b, y, rows, nvec, inv_D, eps, st);
        case 8: return launch_reg<DT, THREADS, GROUP, 8, M8, PE>(x, g, b, y, rows, nvec, inv_D, eps, st);
        default: return AK_ERR_SHAPE;
    }
}

template <int DT, int THREADS>
int launch_smem(const void* x, const void* g, const void* b, void* y, int64_t rows, int nvec, float inv_D,
                float eps, cudaStream_t st) {
    const size_t smem = (size_t)nvec * 16;
    if (!allow_big_smem(layernorm_smem_kernel<THREADS, DT>)) return AK_ERR_CUDA;
    layernorm_smem_kernel<THREADS, DT><<<(unsigned)rows, THREADS, smem, st>>>(
        static_cast<const uint4*>(x), static_cast<const uint4*>(g), static_cast<const uint4*>(b),
        static_cast<uint4*>(y), nvec, inv_D, eps);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// a cluster of C CTAs per row (C from cluster_ctas, at least 2)
template <int DT, int THREADS>
int launch_cluster_rows(const void* x, const void* g, const void* b, void* y, int64_t rows, int nvec, int C, float inv_D,
                        float eps, cudaStream_t st) {
    if (!allow_big_smem(layernorm_cluster_kernel<THREADS, DT>)) return AK_ERR_CUDA;
    const size_t smem = (size_t)((nvec + C - 1) / C) * 16;
    const cudaError_t e = launch_cluster(layernorm_cluster_kernel<THREADS, DT>, (unsigned)(rows * C), THREADS, smem, C, st,
                                         static_cast<const uint4*>(x), static_cast<const uint4*>(g),
                                         static_cast<const uint4*>(b), static_cast<uint4*>(y), nvec, C, inv_D, eps);
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// Rows that are not 16-byte aligned need gamma and beta shifted to the row's phase.  From
// `min_rows` rows on they are shifted once per launch, for all eight phases, into a table in
// stream-ordered scratch (16 x the row's vectors) instead of once per output vector; the row
// kernel then runs as the programmatic dependent of the kernel that writes the table.  Returns
// null (and launches nothing) for fewer rows or when the scratch cannot be had.
const uint4* shift_table(const uint16_t* g, const uint16_t* b, int64_t rows, int64_t D, int64_t min_rows,
                         cudaStream_t st, int* nvp_out) {
    const int nvp = (int)((D + 14) >> 3);
    *nvp_out = nvp;
    if (rows < min_rows) return nullptr;
    void* tab = nullptr;
    if (scratch_alloc(&tab, (size_t)16 * nvp * sizeof(uint4), st) != cudaSuccess) {
        (void)cudaGetLastError();
        return nullptr;
    }
    shift_params_kernel<<<(16 * nvp + kShiftThreads - 1) / kShiftThreads, kShiftThreads, 0, st>>>(
        g, b, D, nvp, static_cast<uint4*>(tab));
    count_launch();
    if (cudaGetLastError() != cudaSuccess) {
        cudaFreeAsync(tab, st);
        return nullptr;
    }
    return static_cast<const uint4*>(tab);
}
constexpr int64_t kShiftMinRowsRegs = 1024;    // rows of up to 64 KiB in registers
constexpr int64_t kShiftMinRowsStaged = 256;   // longer rows staged in shared memory

template <int DT, int T>
int launch_stage(const uint16_t* x, const uint16_t* g, const uint16_t* b, uint16_t* y, int64_t rows, int64_t D,
                 size_t stage_bytes, float inv_D, float eps, cudaStream_t st) {
    if (!allow_big_smem(layernorm_stage_kernel<T, DT, false>) || !allow_big_smem(layernorm_stage_kernel<T, DT, true>)) return AK_ERR_CUDA;
    int nvp = 0;
    if (const uint4* tab = shift_table(g, b, rows, D, kShiftMinRowsStaged, st, &nvp)) {
        const cudaError_t e = launch_dependent(layernorm_stage_kernel<T, DT, true>, dim3((unsigned)rows), dim3(T),
                                               stage_bytes, st, x, g, b, y, D, inv_D, eps, tab, nvp);
        count_launch();
        cudaFreeAsync(const_cast<uint4*>(tab), st);
        return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
    }
    layernorm_stage_kernel<T, DT, false><<<(unsigned)rows, T, stage_bytes, st>>>(x, g, b, y, D, inv_D, eps, nullptr, 0);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// unaligned rows split over a cluster of C CTAs (covering vectors of the worst phase: max_nv);
// gamma and beta from the shift table from kShiftMinRowsStaged rows on
template <int DT, int T>
int launch_cluster_stage(const uint16_t* x, const uint16_t* g, const uint16_t* b, uint16_t* y, int64_t rows, int64_t D,
                         int64_t max_nv, int C, float inv_D, float eps, cudaStream_t st) {
    if (!allow_big_smem(layernorm_cluster_stage_kernel<T, DT, false>) || !allow_big_smem(layernorm_cluster_stage_kernel<T, DT, true>)) return AK_ERR_CUDA;
    const size_t smem = (size_t)((max_nv + C - 1) / C) * 16;
    int nvp = 0;
    if (const uint4* tab = shift_table(g, b, rows, D, kShiftMinRowsStaged, st, &nvp)) {
        const cudaError_t e = launch_cluster_dependent(layernorm_cluster_stage_kernel<T, DT, true>, (unsigned)(rows * C), T,
                                                       smem, C, st, x, g, b, y, D, C, inv_D, eps, tab, nvp);
        count_launch();
        cudaFreeAsync(const_cast<uint4*>(tab), st);
        return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
    }
    const cudaError_t e = launch_cluster(layernorm_cluster_stage_kernel<T, DT, false>, (unsigned)(rows * C), T, smem, C, st,
                                         x, g, b, y, D, C, inv_D, eps, static_cast<const uint4*>(nullptr), 0);
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

template <int DT, int THREADS, int VPT, int MINB>
int launch_regp(const uint16_t* x, const uint16_t* g, const uint16_t* b, uint16_t* y, int64_t rows, int64_t D,
                float inv_D, float eps, cudaStream_t st) {
    int nvp = 0;
    if (const uint4* tab = shift_table(g, b, rows, D, kShiftMinRowsRegs, st, &nvp)) {
        const cudaError_t e = launch_dependent(layernorm_regp_kernel<THREADS, VPT, MINB, DT, true>, dim3((unsigned)rows),
                                               dim3(THREADS), 0, st, x, g, b, y, D, inv_D, eps, tab, nvp);
        count_launch();
        cudaFreeAsync(const_cast<uint4*>(tab), st);
        return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
    }
    layernorm_regp_kernel<THREADS, VPT, MINB, DT, false><<<(unsigned)rows, THREADS, 0, st>>>(x, g, b, y, D, inv_D, eps,
                                                                                            nullptr, 0);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}
// unaligned rows held in registers: one to four vectors per thread of a CTA of THREADS threads
// (MINB: the minimum-CTAs-per-SM hint, a register cap)
template <int DT, int THREADS, int MINB>
int launch_regp_vpt(int vpt, const uint16_t* x, const uint16_t* g, const uint16_t* b, uint16_t* y, int64_t rows,
                    int64_t D, float inv_D, float eps, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_regp<DT, THREADS, 1, MINB>(x, g, b, y, rows, D, inv_D, eps, st);
        case 2: return launch_regp<DT, THREADS, 2, MINB>(x, g, b, y, rows, D, inv_D, eps, st);
        case 3: return launch_regp<DT, THREADS, 3, MINB>(x, g, b, y, rows, D, inv_D, eps, st);
        case 4: return launch_regp<DT, THREADS, 4, MINB>(x, g, b, y, rows, D, inv_D, eps, st);
        default: return AK_ERR_SHAPE;
    }
}

template <int DT>
int dispatch_t(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t D, float eps,
               cudaStream_t st, int path) {
    const int64_t row_bytes = D * Elem<DT>::kBytes;
    const bool aligned16 = is_aligned(x, 16) && is_aligned(y, 16) && is_aligned(gamma, 16) && is_aligned(beta, 16);
    if (path == AK_PATH_AUTO) {
        path = layernorm_choose(rows, D, aligned16, DT);
        if (path == AK_PATH_CLUSTER) {
            const int s = dispatch_t<DT>(x, gamma, beta, y, rows, D, eps, st, AK_PATH_CLUSTER);
            if (s != AK_ERR_CUDA) return s;
            // a device (or a partition of one) that cannot co-schedule the cluster: one CTA per row
            // or, for rows beyond its shared memory, the multi-pass kernel
            (void)cudaGetLastError();
            path = row_bytes <= 65536 ? AK_PATH_CTA : (row_bytes <= kMaxRowSmemBytes ? AK_PATH_SMEM : AK_PATH_GENERIC);
        }
    }
    const float inv_D = 1.0f / (float)D;
    if (path != AK_PATH_GENERIC) {
        if ((row_bytes & 15) != 0) return AK_ERR_SHAPE;
        if (!aligned16) return AK_ERR_ALIGN;
    }
    if (rows > 2147483647LL) return AK_ERR_SHAPE;  // grid.x limit of the one-row-per-CTA layouts
    const int nvec = (int)(row_bytes >> 4);
    switch (path) {
        // Launch shapes and register caps below were picked by timing each candidate in the
        // sustained (power-capped) regime of a long run.
        case AK_PATH_WARP:
            if (row_bytes > 4096) return AK_ERR_SHAPE;
            if (rows <= kEarlyParamRows && rows * row_bytes <= kEarlyParamBytes) {
                if (nvec <= 128) return launch_reg_vpt<DT, 256, 32, 1, 1, 1, 1, true>((nvec + 31) / 32, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
                return launch_reg_vpt<DT, 256, 64, 1, 1, 1, 1, true>((nvec + 63) / 64, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            }
            if (nvec <= 128)   // a warp per row, 8 rows per CTA, 46 registers
                return launch_reg_vpt<DT, 256, 32, 5, 1, 1, 1>((nvec + 31) / 32, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            // two warps per row, 4 rows per CTA
            return launch_reg_vpt<DT, 256, 64, 5, 1, 1, 1>((nvec + 63) / 64, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
        case AK_PATH_CTA:
            if (row_bytes > 65536) return AK_ERR_SHAPE;
            if (rows <= kEarlyParamRows && rows * row_bytes <= kEarlyParamBytes) {
                if (nvec <= 1024) return launch_reg_vpt<DT, 128, 128, 1, 1, 1, 1, true>((nvec + 127) / 128, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
                if (nvec <= 2048) return launch_reg_vpt<DT, 256, 256, 1, 1, 1, 1, true>((nvec + 255) / 256, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            }
            if (nvec <= 1024)  // 128 threads x up to 8 vectors: many small CTAs per SM
                return launch_reg_vpt<DT, 128, 128, 10, 8, 6, 8>((nvec + 127) / 128, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            if (nvec <= 2048)
                return launch_reg_vpt<DT, 256, 256, 5, 4, 4, 4>((nvec + 255) / 256, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            return launch_reg_vpt<DT, 512, 512, 2, 2, 2, 2>((nvec + 511) / 512, x, gamma, beta, y, rows, nvec, inv_D, eps, st);
        case AK_PATH_SMEM:
            if (row_bytes > kMaxRowSmemBytes) return AK_ERR_SHAPE;
            if (nvec <= 4096) return launch_smem<DT, 256>(x, gamma, beta, y, rows, nvec, inv_D, eps, st);
            return launch_smem<DT, 512>(x, gamma, beta, y, rows, nvec, inv_D, eps, st);
        case AK_PATH_CLUSTER: {
            int C = cluster_ctas(rows, row_bytes, kClusterFrom);
            if (C < 2) C = 2;   // forced by the caller
            if ((row_bytes >> 4) < C || rows * C > 2147483647LL) return AK_ERR_SHAPE;
            if (row_bytes > (int64_t)C * kMaxRowSmemBytes) {   // too long to stage: streamed
                const cudaError_t e = launch_cluster(layernorm_cluster_stream_kernel<512, DT>, (unsigned)(rows * C), 512, 0, C, st,
                                                     static_cast<const uint4*>(x), static_cast<const uint4*>(gamma),
                                                     static_cast<const uint4*>(beta), static_cast<uint4*>(y),
                                                     (int64_t)(row_bytes >> 4), C, inv_D, eps);
                count_launch();
                return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
            }
            if ((nvec + C - 1) / C <= 4096)
                return launch_cluster_rows<DT, 256>(x, gamma, beta, y, rows, nvec, C, inv_D, eps, st);
            return launch_cluster_rows<DT, 512>(x, gamma, beta, y, rows, nvec, C, inv_D, eps, st);
        }
        case AK_PATH_GENERIC: {
            if constexpr (DT == AK_DTYPE_F32) {
                const int resident = resident_ctas(layernorm_generic32_kernel, kLnGenericThreads, 0);
                const int grid = (int)(rows < resident ? rows : resident);
                layernorm_generic32_kernel<<<grid, kLnGenericThreads, 0, st>>>(
                    static_cast<const float*>(x), static_cast<const float*>(gamma), static_cast<const float*>(beta),
                    static_cast<float*>(y), rows, D, inv_D, eps);
                count_launch();
                return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
            } else {
                const size_t stage_bytes = (size_t)((D + 14) >> 3) * 16;
                const bool same_phase = ((reinterpret_cast<uintptr_t>(x) ^ reinterpret_cast<uintptr_t>(y)) & 15) == 0;
                const bool params4 = is_aligned(gamma, 4) && is_aligned(beta, 4);
                const uint16_t* xs = static_cast<const uint16_t*>(x);
                const uint16_t* gs = static_cast<const uint16_t*>(gamma);
                const uint16_t* bs = static_cast<const uint16_t*>(beta);
                uint16_t* ys = static_cast<uint16_t*>(y);
                const int64_t max_nv = (D + 14) >> 3;   // vectors covering the row at the worst phase
                // long rows (up to eight CTAs' shared memory), and a few rows (at most 64) of 32 KiB or
                // more: the covering vectors split over a thread-block cluster;
                // unaligned rows are split over a cluster from 160 KiB on (4096 x 100001: 376 -> 348 us; at 128 KiB
                // and below one CTA per row is as fast or faster)
                const int Cu = cluster_ctas(rows, (int64_t)stage_bytes, 163840 + 16);
                if (same_phase && params4 && Cu > 1 && stage_bytes <= (size_t)kMaxCluster * kMaxRowSmemBytes && rows * Cu <= 2147483647LL) {
                    if (launch_cluster_stage<DT, 256>(xs, gs, bs, ys, rows, D, max_nv, Cu, inv_D, eps, st) == AK_OK) return AK_OK;
                    (void)cudaGetLastError();   // the cluster cannot be co-scheduled here: the kernels below
                }
                // Rows of up to 512 covering vectors (D <= about 4090) stay in the registers of a 128-thread
                // CTA; longer ones are staged in shared memory: with both moments taken in one pass over the
                // staged row that kernel is the faster one from there on (8192 x 4099 28.3 -> 27.2 us, 8192 x 7001
                // 48.3 -> 45.0 us, 4096 x 28001 96.7 -> 87.2 us against rows held by 128 or 512 threads).
                if (same_phase && params4 && max_nv <= 512)
                    return launch_regp_vpt<DT, 128, 10>((int)((max_nv + 127) / 128), xs, gs, bs, ys, rows, D, inv_D, eps, st);
                if (same_phase && params4 && stage_bytes <= (size_t)kMaxRowSmemBytes) {
                    if (D <= 8192) return launch_stage<DT, 128>(xs, gs, bs, ys, rows, D, stage_bytes, inv_D, eps, st);
                    if (D <= 32768) return launch_stage<DT, 256>(xs, gs, bs, ys, rows, D, stage_bytes, inv_D, eps, st);
                    return launch_stage<DT, 512>(xs, gs, bs, ys, rows, D, stage_bytes, inv_D, eps, st);
                }
                const int resident = resident_ctas(layernorm_generic_kernel<DT>, kLnGenericThreads, 0);
                const int grid = (int)(rows < resident ? rows : resident);
                layernorm_generic_kernel<DT><<<grid, kLnGenericThreads, 0, st>>>(xs, gs, bs, ys, rows, D, inv_D, eps);
                count_launch();
                return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
            }
        }
        default:
            return AK_ERR_ARG;
    }
}

}  // namespace

int layernorm_choose(int64_t rows, int64_t D, bool aligned16, int dtype) {
    const int64_t bytes = D * dtype_bytes(dtype);
    if (!aligned16 || (bytes & 15) != 0) return AK_PATH_GENERIC;
    if (cluster_ctas(rows, bytes, kClusterFrom) > 1) return AK_PATH_CLUSTER;
    if (bytes > kMaxRowSmemBytes) return AK_PATH_GENERIC;   // only with clusters switched off
    if (bytes <= 4096) return AK_PATH_WARP;
    if (bytes <= 65536) return AK_PATH_CTA;   // up to 64 KiB the register layout beats the staged one
    return AK_PATH_SMEM;
}

int layernorm_dispatch(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t D,
                       float eps, cudaStream_t st, int path, int dtype) {
    switch (dtype) {
        case AK_DTYPE_BF16: return dispatch_t<AK_DTYPE_BF16>(x, gamma, beta, y, rows, D, eps, st, path);
        case AK_DTYPE_F16: return dispatch_t<AK_DTYPE_F16>(x, gamma, beta, y, rows, D, eps, st, path);
        case AK_DTYPE_F32: return dispatch_t<AK_DTYPE_F32>(x, gamma, beta, y, rows, D, eps, st, path);
        default: return AK_ERR_ARG;
    }
}

AK_DEFINE_WAIT_TIMEOUT_READER(layernorm_wait_timeouts)

}  // namespace ak
