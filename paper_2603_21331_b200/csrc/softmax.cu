// Last-dim softmax forward: host dispatch.  Kernels live in softmax_kernels.cuh.
//
// Launch shapes come from CUDA-graph timed sweeps on B200 (see rmsnorm.cu for the
// reasoning): one row per warp up to 4 KiB rows, one row per CTA in registers up to
// 16 KiB rows (exponentials kept in fp32, register cap chosen for five CTAs per SM), rows
// up to 64 KiB staged in shared memory by the copy engine, longer rows (and a few long rows)
// split over a thread-block cluster.  The thresholds are in row bytes, so they hold for every
// element type.
#include "softmax_kernels.cuh"

namespace ak {
namespace {

template <int DT, int THREADS, int GROUP, int VPT, int MINB>
int launch_reg(const void* x, void* y, int64_t rows, int nvec, cudaStream_t st) {
    constexpr int GROUPS = THREADS / GROUP;
    const int64_t grid = (rows + GROUPS - 1) / GROUPS;
    auto kernel = softmax_reg_kernel<THREADS, GROUP, VPT, MINB, false, DT>;
    // every thread holds exactly VPT vectors of a live row: the form without bounds tests (16384 x 512
    // 6.4 -> 5.9 us, 16384 x 4096 40.9 -> 40.4 us, 262144 x 4096 640 -> 618 us; at eight vectors per thread
    // it measured 0.5 us slower at 16384 x 8192 and is not taken)
    if constexpr (VPT < 8)
        if (nvec == VPT * GROUP && rows % GROUPS == 0) kernel = softmax_reg_kernel<THREADS, GROUP, VPT, MINB, false, DT, true>;
    const cudaError_t e = launch_dependent(kernel, dim3((unsigned)grid), dim3(THREADS), 0, st,
                                           static_cast<const uint4*>(x), static_cast<uint4*>(y), rows, nvec,
                                           first_wave_ctas(kernel, THREADS, 0));
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

template <int DT, int THREADS, int GROUP, int MINB_LO, int MINB_HI>
int launch_reg_vpt(int vpt, const void* x, void* y, int64_t rows, int nvec, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_reg<DT, THREADS, GROUP, 1, MINB_LO>(x, y, rows, nvec, st);
        case 2: return launch_reg<DT, THREADS, GROUP, 2, MINB_LO>(x, y, rows, nvec, st);
        case 3: return launch_reg<DT, THREADS, GROUP, 3, MINB_LO>(x, y, rows, nvec, st);
        case 4: return launch_reg<DT, THREADS, GROUP, 4, MINB_LO>(x, y, rows, nvec, st);
        case 5: return launch_reg<DT, THREADS, GROUP, 5, MINB_HI>(x, y, rows, nvec, st);
        case 6: return launch_reg<DT, THREADS, GROUP, 6, MINB_HI>(x, y, rows, nvec, st);
        case 7: return launch_reg<DT, THREADS, GROUP, 7, MINB_HI>(x, y, rows, nvec, st);
        case 8: return launch_reg<DT, THREADS, GROUP, 8, MINB_HI>(x, y, rows, nvec, st);
        default: return AK_ERR_SHAPE;
    }
}

template <int DT, int THREADS, int KEEP>
int launch_smem(const void* x, void* y, int64_t rows, int nvec, cudaStream_t st) {
    const size_t smem = (size_t)nvec * 16;
    if (!allow_big_smem(softmax_smem_kernel<THREADS, 1, KEEP, DT>)) return AK_ERR_CUDA;
    auto kernel = softmax_smem_kernel<THREADS, 1, KEEP, DT>;
    const cudaError_t e = launch_dependent(kernel, dim3((unsigned)rows), dim3(THREADS), smem, st,
                                           static_cast<const uint4*>(x), static_cast<uint4*>(y), nvec,
                                           first_wave_ctas(kernel, THREADS, smem));
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

template <int DT, int T>
int launch_stage(const uint16_t* x, uint16_t* y, int64_t rows, int64_t D, size_t stage_bytes, cudaStream_t st) {
    if (!allow_big_smem(softmax_stage_kernel<T, DT>)) return AK_ERR_CUDA;
    auto kernel = softmax_stage_kernel<T, DT>;
    const cudaError_t e = launch_dependent(kernel, dim3((unsigned)rows), dim3(T), stage_bytes, st, x, y, D,
                                           first_wave_ctas(kernel, T, stage_bytes));
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// unaligned rows split over a cluster of C CTAs (covering vectors of the worst phase: max_nv)
template <int DT, int T, int KEEP>
int launch_cluster_stage(const uint16_t* x, uint16_t* y, int64_t rows, int64_t D, int64_t max_nv, int C, cudaStream_t st) {
    if (!allow_big_smem(softmax_cluster_stage_kernel<T, DT, KEEP>)) return AK_ERR_CUDA;
    const size_t smem = (size_t)((max_nv + C - 1) / C) * 16;
    const cudaError_t e = launch_cluster(softmax_cluster_stage_kernel<T, DT, KEEP>, (unsigned)(rows * C), T, smem, C, st, x, y, D, C);
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

template <int DT, int THREADS, int VPT, int MINB>
int launch_regp(const uint16_t* x, uint16_t* y, int64_t rows, int64_t D, cudaStream_t st) {
    auto kernel = softmax_regp_kernel<THREADS, VPT, MINB, DT>;
    const cudaError_t e = launch_dependent(kernel, dim3((unsigned)rows), dim3(THREADS), 0, st, x, y, D,
                                           first_wave_ctas(kernel, THREADS, 0));
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}
// a cluster of C CTAs per row (C from cluster_ctas, at least 2)
template <int DT, int THREADS, int KEEP>
int launch_cluster_rows(const void* x, void* y, int64_t rows, int nvec, int C, cudaStream_t st) {
    if (!allow_big_smem(softmax_cluster_kernel<THREADS, KEEP, DT>)) return AK_ERR_CUDA;
    const size_t smem = (size_t)((nvec + C - 1) / C) * 16;
    const cudaError_t e = launch_cluster(softmax_cluster_kernel<THREADS, KEEP, DT>, (unsigned)(rows * C), THREADS, smem, C, st,
                                         static_cast<const uint4*>(x), static_cast<uint4*>(y), nvec, C);
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// unaligned rows held in registers: vectors per thread 1..8 for a CTA of THREADS threads
template <int DT, int THREADS, int MINB>
int launch_regp_vpt(int vpt, const uint16_t* x, uint16_t* y, int64_t rows, int64_t D, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_regp<DT, THREADS, 1, 1>(x, y, rows, D, st);
        case 2: return launch_regp<DT, THREADS, 2, 1>(x, y, rows, D, st);
        case 3: return launch_regp<DT, THREADS, 3, 1>(x, y, rows, D, st);
        case 4: return launch_regp<DT, THREADS, 4, 1>(x, y, rows, D, st);
        case 5: return launch_regp<DT, THREADS, 5, MINB>(x, y, rows, D, st);
        case 6: return launch_regp<DT, THREADS, 6, MINB>(x, y, rows, D, st);
        case 7: return launch_regp<DT, THREADS, 7, MINB>(x, y, rows, D, st);
        case 8: return launch_regp<DT, THREADS, 8, MINB>(x, y, rows, D, st);
        default: return AK_ERR_SHAPE;
    }
}

template <int DT>
int dispatch_t(const void* x, void* y, int64_t rows, int64_t D, cudaStream_t st, int path) {
    const int64_t row_bytes = D * Elem<DT>::kBytes;
    const bool aligned16 = is_aligned(x, 16) && is_aligned(y, 16);
    if (path == AK_PATH_AUTO) {
        path = softmax_choose(rows, D, aligned16, DT);
        if (path == AK_PATH_CLUSTER) {
            const int s = dispatch_t<DT>(x, y, rows, D, st, AK_PATH_CLUSTER);
            if (s != AK_ERR_CUDA) return s;
            // a device (or a partition of one) that cannot co-schedule the cluster: one CTA per row
            // or, for rows beyond its shared memory, the multi-pass kernel
            (void)cudaGetLastError();
            path = row_bytes <= 16384 ? AK_PATH_CTA : (row_bytes <= kMaxRowSmemBytes ? AK_PATH_SMEM : AK_PATH_GENERIC);
        }
    }
    if (path != AK_PATH_GENERIC) {
        if ((row_bytes & 15) != 0) return AK_ERR_SHAPE;
        if (!aligned16) return AK_ERR_ALIGN;
    }
    if (rows > 2147483647LL) return AK_ERR_SHAPE;  // grid.x limit of the one-row-per-CTA layouts
    const int nvec = (int)(row_bytes >> 4);
    switch (path) {
        case AK_PATH_WARP:
            if (row_bytes > 4096) return AK_ERR_SHAPE;
            return launch_reg_vpt<DT, 128, 32, 1, 1>((nvec + 31) / 32, x, y, rows, nvec, st);
        case AK_PATH_CTA:
            if (row_bytes > 65536) return AK_ERR_SHAPE;
            // 128 threads with up to 8 vectors each (exponentials of the whole share in fp32
            // registers, capped at 102 registers for five CTAs per SM): the best sustained shape
            // up to 16 KiB rows
            if (nvec <= 1024) return launch_reg_vpt<DT, 128, 128, 1, 5>((nvec + 127) / 128, x, y, rows, nvec, st);
            if (nvec <= 2048) return launch_reg_vpt<DT, 256, 256, 1, 1>((nvec + 255) / 256, x, y, rows, nvec, st);
            return launch_reg_vpt<DT, 512, 512, 1, 1>((nvec + 511) / 512, x, y, rows, nvec, st);
        case AK_PATH_SMEM:
            if (row_bytes > kMaxRowSmemBytes) return AK_ERR_SHAPE;
            // 256 threads keeping the first four vectors' exponentials in registers: best both in
            // short bursts and under the power cap of a long run up to 64 KiB rows
            if (nvec <= 4096) return launch_smem<DT, 256, 4>(x, y, rows, nvec, st);
            return launch_smem<DT, 512, 0>(x, y, rows, nvec, st);
        case AK_PATH_CLUSTER: {
            int C = cluster_ctas(rows, row_bytes, kClusterFrom);
            if (C < 2) C = 2;   // forced by the caller
            if ((row_bytes >> 4) < C || rows * C > 2147483647LL) return AK_ERR_SHAPE;
            if (row_bytes > (int64_t)C * kMaxRowSmemBytes) {   // too long to stage: streamed
                const cudaError_t e = launch_cluster(softmax_cluster_stream_kernel<512, DT>, (unsigned)(rows * C), 512, 0, C, st,
                                                     static_cast<const uint4*>(x), static_cast<uint4*>(y),
                                                     (int64_t)(row_bytes >> 4), C);
                count_launch();
                return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
            }
            // many rows in slices of up to 32 KiB: 128-thread CTAs measured 2-12 % faster than 256
            // (and 64 slower); a few rows are better off with 256
            // kept exponentials per thread picked by timing (4096 x 65536: 4 kept 177 us, 6 kept 166 us,
            // 8 kept 179 us: 72 registers still leave the seven CTAs per SM that shared memory allows)
            if ((nvec + C - 1) / C <= 2048 && rows > 64) return launch_cluster_rows<DT, 128, 6>(x, y, rows, nvec, C, st);
            if ((nvec + C - 1) / C <= 4096) return launch_cluster_rows<DT, 256, 7>(x, y, rows, nvec, C, st);
            return launch_cluster_rows<DT, 512, 0>(x, y, rows, nvec, C, st);
        }
        case AK_PATH_GENERIC: {
            if constexpr (DT == AK_DTYPE_F32) {
                const int resident = resident_ctas(softmax_generic32_kernel, kSmGenericThreads, 0);
                const int grid = (int)(rows < resident ? rows : resident);
                softmax_generic32_kernel<<<grid, kSmGenericThreads, 0, st>>>(
                    static_cast<const float*>(x), static_cast<float*>(y), rows, D);
                count_launch();
                return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
            } else {
                // rows staged in shared memory when x and y rows share their 16-byte phase and a
                // row (plus up to 14 bytes of phase padding) fits
                const size_t stage_bytes = (size_t)((D + 14) >> 3) * 16;
                const bool same_phase = ((reinterpret_cast<uintptr_t>(x) ^ reinterpret_cast<uintptr_t>(y)) & 15) == 0;
                const uint16_t* xs = static_cast<const uint16_t*>(x);
                uint16_t* ys = static_cast<uint16_t*>(y);
                // rows of up to 512 covering vectors stay in the registers of a 128-thread CTA (from
                // there on the staged kernel, whose row arrives by bulk copies, measured 3-6 % faster)
                const int64_t max_nv = (D + 14) >> 3;   // vectors covering the row at the worst phase
                if (same_phase && max_nv <= 512)
                    return launch_regp_vpt<DT, 128, 5>((int)((max_nv + 127) / 128), xs, ys, rows, D, st);
                // rows of more than 96 KiB (up to eight CTAs' shared memory), and a few long rows: the
                // covering vectors split over a thread-block cluster (4096 x 65539: 257 us staged by one
                // CTA, 207 us in clusters; 4096 x 40001: 115 us against 126 us)
                const int Cu = cluster_ctas(rows, (int64_t)stage_bytes, 98304 + 16);
                if (same_phase && Cu > 1 && stage_bytes <= (size_t)kMaxCluster * kMaxRowSmemBytes && rows * Cu <= 2147483647LL) {
                    // exponentials kept per thread as in the aligned cluster kernel; a few rows (latency-
                    // bound) are better off with fewer registers (64 x 128257: 4 kept 11.7 us, 7 kept 14.3 us)
                    const int s = rows <= 64 ? launch_cluster_stage<DT, 256, 4>(xs, ys, rows, D, max_nv, Cu, st)
                                  : (max_nv + Cu - 1) / Cu <= 2048
                                      ? launch_cluster_stage<DT, 128, 6>(xs, ys, rows, D, max_nv, Cu, st)
                                      : launch_cluster_stage<DT, 256, 7>(xs, ys, rows, D, max_nv, Cu, st);
                    if (s == AK_OK) return AK_OK;
                    (void)cudaGetLastError();   // the cluster cannot be co-scheduled here: the kernels below
                }
                if (same_phase && stage_bytes <= (size_t)kMaxRowSmemBytes) {
                    if (D <= 8192) return launch_stage<DT, 128>(xs, ys, rows, D, stage_bytes, st);
                    if (D <= 32768) return launch_stage<DT, 256>(xs, ys, rows, D, stage_bytes, st);
                    return launch_stage<DT, 512>(xs, ys, rows, D, stage_bytes, st);
                }
                const int resident = resident_ctas(softmax_generic_kernel<DT>, kSmGenericThreads, 0);
                const int grid = (int)(rows < resident ? rows : resident);
                softmax_generic_kernel<DT><<<grid, kSmGenericThreads, 0, st>>>(xs, ys, rows, D);
                count_launch();
                return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
            }
        }
        default:
            return AK_ERR_ARG;
    }
}

}  // namespace

int softmax_choose(int64_t rows, int64_t D, bool aligned16, int dtype) {
    const int64_t bytes = D * dtype_bytes(dtype);
    if (!aligned16 || (bytes & 15) != 0) return AK_PATH_GENERIC;
    if (cluster_ctas(rows, bytes, kClusterFrom) > 1) return AK_PATH_CLUSTER;
    if (bytes > kMaxRowSmemBytes) return AK_PATH_GENERIC;   // only with clusters switched off
    if (bytes <= 4096) return AK_PATH_WARP;
    if (bytes <= 16384) return AK_PATH_CTA;
    return AK_PATH_SMEM;
}

int softmax_dispatch(const void* x, void* y, int64_t rows, int64_t D, cudaStream_t st, int path, int dtype) {
    switch (dtype) {
        case AK_DTYPE_BF16: return dispatch_t<AK_DTYPE_BF16>(x, y, rows, D, st, path);
        case AK_DTYPE_F16: return dispatch_t<AK_DTYPE_F16>(x, y, rows, D, st, path);
        case AK_DTYPE_F32: return dispatch_t<AK_DTYPE_F32>(x, y, rows, D, st, path);
        default: return AK_ERR_ARG;
    }
}

AK_DEFINE_WAIT_TIMEOUT_READER(softmax_wait_timeouts)

}  // namespace ak
