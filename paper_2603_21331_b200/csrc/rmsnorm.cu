// RMSNorm forward: host dispatch.  Kernels live in rmsnorm_kernels.cuh.
//
// The launch shapes below were chosen by measurement on B200 (CUDA-graph timed sweeps over
// threads per CTA, threads per row, vectors per thread and register caps): what decides
// the bandwidth is how many bytes each SM keeps in flight, i.e. resident CTAs x bytes per
// CTA, so weights are fetched late (fewer live registers, more CTAs), one row (or one row
// per warp) per CTA beats grid-stride persistence, and rows beyond 64 KiB are split over a
// thread-block cluster whose CTAs stage slices of at most 32 KiB in shared memory by the copy
// engine (as are a few long rows, which one CTA each would not spread over the GPU).
#include "rmsnorm_kernels.cuh"

namespace ak {
namespace {

// A launch of at most this many rows and bytes does not fill the GPU and is latency-bound: the
// weights are then requested together with the row instead of after the reduction (no register
// cap to keep: 1 x 1024 .. 1024 x 4096 run 5-47 % faster, e.g. 8 x 2048 3.2 -> 1.7 us; from 2048
// rows or 8 MiB on the late fetch with its tighter register budget is as fast or faster).
// unaligned rows split over a cluster of C CTAs (covering vectors of the worst phase: max_nv)
template <int DT, int T>
int launch_cluster_stage(const uint16_t* x, const uint16_t* w, uint16_t* y, int64_t rows, int64_t D, int64_t max_nv, int C,
                         float inv_D, float eps, cudaStream_t st) {
    if (!allow_big_smem(rmsnorm_cluster_stage_kernel<T, DT>)) return AK_ERR_CUDA;
    const size_t smem = (size_t)((max_nv + C - 1) / C) * 16;
    const cudaError_t e = launch_cluster(rmsnorm_cluster_stage_kernel<T, DT>, (unsigned)(rows * C), T, smem, C, st, x, w, y,
                                         D, C, inv_D, eps);
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

constexpr int64_t kEarlyWeightRows = 1024, kEarlyWeightBytes = 8 << 20;

template <int DT, int THREADS, int GROUP, int VPT, int MINB, bool WE = false>
int launch_reg(const void* x, const void* w, void* y, int64_t rows, int nvec, float inv_D, float eps,
               cudaStream_t st) {
    constexpr int GROUPS = THREADS / GROUP;
    const int64_t grid = (rows + GROUPS - 1) / GROUPS;
    auto kernel = rmsnorm_reg_kernel<THREADS, GROUP, VPT, MINB, WE, DT>;
    // every thread holds exactly VPT vectors of a live row: the form without bounds tests (the loads
    // of x and w are then issued without waiting for predicates: 8192 x 2048 13.3 -> 11.7 us,
    // 8192 x 8192 41.1 -> 40.6 us)
    if (nvec == VPT * GROUP && rows % GROUPS == 0) kernel = rmsnorm_reg_kernel<THREADS, GROUP, VPT, MINB, WE, DT, true>;
    const cudaError_t e = launch_dependent(kernel, dim3((unsigned)grid), dim3(THREADS), 0, st,
                                           static_cast<const uint4*>(x), static_cast<const uint4*>(w),
                                           static_cast<uint4*>(y), rows, nvec, inv_D, eps,
                                           first_wave_ctas(kernel, THREADS, 0));
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// vectors per thread 1..MAXV for a fixed (THREADS, GROUP)
template <int DT, int THREADS, int GROUP, int MINB_LO, int MINB_HI, bool WE = false>
int launch_reg_vpt(int vpt, const void* x, const void* w, void* y, int64_t rows, int nvec, float inv_D,
                   float eps, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_reg<DT, THREADS, GROUP, 1, MINB_LO, WE>(x, w, y, rows, nvec, inv_D, eps, st);
        case 2: return launch_reg<DT, THREADS, GROUP, 2, MINB_LO, WE>(x, w, y, rows, nvec, inv_D, eps, st);
        case 3: return launch_reg<DT, THREADS, GROUP, 3, MINB_LO, WE>(x, w, y, rows, nvec, inv_D, eps, st);
        case 4: return launch_reg<DT, THREADS, GROUP, 4, MINB_LO, WE>(x, w, y, rows, nvec, inv_D, eps, st);
        case 5: return launch_reg<DT, THREADS, GROUP, 5, MINB_HI, WE>(x, w, y, rows, nvec, inv_D, eps, st);
        case 6: return launch_reg<DT, THREADS, GROUP, 6, MINB_HI, WE>(x, w, y, rows, nvec, inv_D, eps, st);
        case 7: return launch_reg<DT, THREADS, GROUP, 7, MINB_HI, WE>(x, w, y, rows, nvec, inv_D, eps, st);
        case 8: return launch_reg<DT, THREADS, GROUP, 8, MINB_HI, WE>(x, w, y, rows, nvec, inv_D, eps, st);
        default: return AK_ERR_SHAPE;
    }
}

template <int DT, int THREADS>
int launch_smem(const void* x, const void* w, void* y, int64_t rows, int nvec, float inv_D, float eps,
                cudaStream_t st) {
    const size_t smem = (size_t)nvec * 16;
    if (!allow_big_smem(rmsnorm_smem_kernel<THREADS, 1, DT>)) return AK_ERR_CUDA;
    rmsnorm_smem_kernel<THREADS, 1, DT><<<(unsigned)rows, THREADS, smem, st>>>(
        static_cast<const uint4*>(x), static_cast<const uint4*>(w), static_cast<uint4*>(y), nvec, inv_D, eps);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// a cluster of C CTAs per row (C from cluster_ctas, at least 2)
template <int DT, int THREADS>
int launch_cluster_rows(const void* x, const void* w, void* y, int64_t rows, int nvec, int C, float inv_D, float eps,
                        cudaStream_t st) {
    if (!allow_big_smem(rmsnorm_cluster_kernel<THREADS, DT>)) return AK_ERR_CUDA;
    const size_t smem = (size_t)((nvec + C - 1) / C) * 16;
    const cudaError_t e = launch_cluster(rmsnorm_cluster_kernel<THREADS, DT>, (unsigned)(rows * C), THREADS, smem, C, st,
                                         static_cast<const uint4*>(x), static_cast<const uint4*>(w),
                                         static_cast<uint4*>(y), nvec, C, inv_D, eps);
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

// unaligned rows held in registers: vectors per thread 1..8 for a CTA of THREADS threads
template <int DT, int THREADS, int VPT>
int launch_regp(const uint16_t* x, const uint16_t* w, uint16_t* y, int64_t rows, int64_t D, float inv_D, float eps,
                cudaStream_t st) {
    auto kernel = rmsnorm_regp_kernel<THREADS, VPT, DT>;
    const cudaError_t e = launch_dependent(kernel, dim3((unsigned)rows), dim3(THREADS), 0, st, x, w, y, D, inv_D, eps,
                                           first_wave_ctas(kernel, THREADS, 0));
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}
template <int DT, int THREADS>
int launch_regp_vpt(int vpt, const uint16_t* x, const uint16_t* w, uint16_t* y, int64_t rows, int64_t D, float inv_D,
                    float eps, cudaStream_t st) {
    switch (vpt) {
        case 1: return launch_regp<DT, THREADS, 1>(x, w, y, rows, D, inv_D, eps, st);
        case 2: return launch_regp<DT, THREADS, 2>(x, w, y, rows, D, inv_D, eps, st);
        case 3: return launch_regp<DT, THREADS, 3>(x, w, y, rows, D, inv_D, eps, st);
        case 4: return launch_regp<DT, THREADS, 4>(x, w, y, rows, D, inv_D, eps, st);
        case 5: return launch_regp<DT, THREADS, 5>(x, w, y, rows, D, inv_D, eps, st);
        case 6: return launch_regp<DT, THREADS, 6>(x, w, y, rows, D, inv_D, eps, st);
        case 7: return launch_regp<DT, THREADS, 7>(x, w, y, rows, D, inv_D, eps, st);
        case 8: return launch_regp<DT, THREADS, 8>(x, w, y, rows, D, inv_D, eps, st);
        default: return AK_ERR_SHAPE;
    }
}

}  // namespace

int rmsnorm_choose(int64_t rows, int64_t D, bool aligned16, int dtype) {
    const int64_t bytes = D * dtype_bytes(dtype);   // row bytes decide the layout
    if (!aligned16 || (bytes & 15) != 0) return AK_PATH_GENERIC;
    if (cluster_ctas(rows, bytes, kClusterFrom) > 1) return AK_PATH_CLUSTER;
    if (bytes > kMaxRowSmemBytes) return AK_PATH_GENERIC;   // only with clusters switched off
    if (bytes <= 4096) return AK_PATH_WARP;
    if (bytes <= 65536) return AK_PATH_CTA;   // up to 64 KiB the register layout beats the staged one
    return AK_PATH_SMEM;
}

namespace {

template <int DT>
int dispatch_t(const void* x, const void* w, void* y, int64_t rows, int64_t D, float eps, cudaStream_t st, int path) {
    constexpr int kBytes = Elem<DT>::kBytes;
    const int64_t row_bytes = D * kBytes;
    const bool aligned16 = is_aligned(x, 16) && is_aligned(y, 16) && is_aligned(w, 16);
    if (path == AK_PATH_AUTO) {
        path = rmsnorm_choose(rows, D, aligned16, DT);
        if (path == AK_PATH_CLUSTER) {
            const int s = dispatch_t<DT>(x, w, y, rows, D, eps, st, AK_PATH_CLUSTER);
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
        case AK_PATH_WARP:
            if (row_bytes > 4096) return AK_ERR_SHAPE;
            if (rows <= kEarlyWeightRows && rows * row_bytes <= kEarlyWeightBytes) {
                if (nvec <= 128) return launch_reg_vpt<DT, 256, 32, 4, 1, true>((nvec + 31) / 32, x, w, y, rows, nvec, inv_D, eps, st);
                return launch_reg_vpt<DT, 128, 32, 1, 1, true>((nvec + 31) / 32, x, w, y, rows, nvec, inv_D, eps, st);
            }
            if (nvec <= 128) return launch_reg_vpt<DT, 256, 32, 4, 1>((nvec + 31) / 32, x, w, y, rows, nvec, inv_D, eps, st);
            return launch_reg_vpt<DT, 128, 32, 1, 1>((nvec + 31) / 32, x, w, y, rows, nvec, inv_D, eps, st);
        case AK_PATH_CTA:
            if (row_bytes > 65536) return AK_ERR_SHAPE;
            // Shapes chosen in the sustained (power-capped) regime of a long run: 128 threads x <= 4
            // vectors (46 registers); 256 threads x <= 4 vectors (46 registers, five CTAs per SM);
            // 256 threads x <= 8 vectors capped at 85 registers (62 used); 512 threads x <= 8 vectors
            // capped at 64 registers so that two CTAs share an SM (6.5 TB/s at 64 KiB rows against 6.2
            // for the shared-memory kernel).
            if (rows <= kEarlyWeightRows && rows * row_bytes <= kEarlyWeightBytes) {
                if (nvec <= 512) return launch_reg_vpt<DT, 128, 128, 1, 1, true>((nvec + 127) / 128, x, w, y, rows, nvec, inv_D, eps, st);
                if (nvec <= 2048) return launch_reg_vpt<DT, 256, 256, 1, 1, true>((nvec + 255) / 256, x, w, y, rows, nvec, inv_D, eps, st);
            }
            if (nvec <= 512) return launch_reg_vpt<DT, 128, 128, 1, 1>((nvec + 127) / 128, x, w, y, rows, nvec, inv_D, eps, st);
            if (nvec <= 2048) return launch_reg_vpt<DT, 256, 256, 1, 3>((nvec + 255) / 256, x, w, y, rows, nvec, inv_D, eps, st);
            return launch_reg_vpt<DT, 512, 512, 2, 2>((nvec + 511) / 512, x, w, y, rows, nvec, inv_D, eps, st);
        case AK_PATH_SMEM:
            if (row_bytes > kMaxRowSmemBytes) return AK_ERR_SHAPE;
            if (nvec <= 4096) return launch_smem<DT, 256>(x, w, y, rows, nvec, inv_D, eps, st);
            return launch_smem<DT, 512>(x, w, y, rows, nvec, inv_D, eps, st);
        case AK_PATH_CLUSTER: {
            int C = cluster_ctas(rows, row_bytes, kClusterFrom);
            if (C < 2) C = 2;   // forced by the caller
            if ((row_bytes >> 4) < C || rows * C > 2147483647LL) return AK_ERR_SHAPE;
            if (row_bytes > (int64_t)C * kMaxRowSmemBytes) {   // too long to stage: streamed
                const cudaError_t e = launch_cluster(rmsnorm_cluster_stream_kernel<512, DT>, (unsigned)(rows * C), 512, 0, C, st,
                                                     static_cast<const uint4*>(x), static_cast<const uint4*>(w),
                                                     static_cast<uint4*>(y), (int64_t)(row_bytes >> 4), C, inv_D, eps);
                count_launch();
                return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
            }
            if ((nvec + C - 1) / C <= 4096) return launch_cluster_rows<DT, 256>(x, w, y, rows, nvec, C, inv_D, eps, st);
            return launch_cluster_rows<DT, 512>(x, w, y, rows, nvec, C, inv_D, eps, st);
        }
        case AK_PATH_GENERIC: {
            if constexpr (DT == AK_DTYPE_F32) {
                const int resident32 = resident_ctas(rmsnorm_generic32_kernel, kRmsGenericThreads, 0);
                const int grid = (int)(rows < resident32 ? rows : resident32);
                rmsnorm_generic32_kernel<<<grid, kRmsGenericThreads, 0, st>>>(
                    static_cast<const float*>(x), static_cast<const float*>(w), static_cast<float*>(y), rows, D, inv_D, eps);
                count_launch();
                return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
            } else {
                // rows staged in shared memory when x and y rows share their 16-byte phase, w is
                // 4-byte aligned and a row (plus up to 14 bytes of phase padding) fits
                const size_t stage_bytes = (size_t)((D + 14) >> 3) * 16;
                const bool same_phase = ((reinterpret_cast<uintptr_t>(x) ^ reinterpret_cast<uintptr_t>(y)) & 15) == 0;
                const uint16_t* xs = static_cast<const uint16_t*>(x);
                const uint16_t* ws = static_cast<const uint16_t*>(w);
                uint16_t* ys = static_cast<uint16_t*>(y);
                const int64_t max_nv = (D + 14) >> 3;   // vectors covering the row at the worst phase
                // long rows (up to eight CTAs' shared memory), and a few rows (at most 64) of 32 KiB or
                // more: the covering vectors split over a thread-block cluster;
                // unaligned rows are split over a cluster from 128 KiB on (4096 x 65539: 235 -> 229 us, 4096 x 100001:
                // 337 -> 322 us; at 100 KiB one CTA per row is 4 % faster)
                const int Cu = cluster_ctas(rows, (int64_t)stage_bytes, 131072 + 16);
                if (same_phase && is_aligned(w, 4) && Cu > 1 && stage_bytes <= (size_t)kMaxCluster * kMaxRowSmemBytes && rows * Cu <= 2147483647LL) {
                    if (launch_cluster_stage<DT, 256>(xs, ws, ys, rows, D, max_nv, Cu, inv_D, eps, st) == AK_OK) return AK_OK;
                    (void)cudaGetLastError();   // the cluster cannot be co-scheduled here: the kernels below
                }
                // rows of up to 1024 covering vectors stay in the registers of a 128-thread CTA ...
                if (same_phase && is_aligned(w, 4) && max_nv <= 1024)
                    return launch_regp_vpt<DT, 128>((int)((max_nv + 127) / 128), xs, ws, ys, rows, D, inv_D, eps, st);
                if (same_phase && is_aligned(w, 4) && max_nv <= 2048)   // ... or of a 256-thread CTA up to 2048
                    return launch_regp_vpt<DT, 256>((int)((max_nv + 255) / 256), xs, ws, ys, rows, D, inv_D, eps, st);
                if (same_phase && is_aligned(w, 4) && max_nv <= 4096)   // ... 512 threads up to 4096
                    return launch_regp_vpt<DT, 512>((int)((max_nv + 511) / 512), xs, ws, ys, rows, D, inv_D, eps, st);
                if (same_phase && is_aligned(w, 4) && stage_bytes <= (size_t)kMaxRowSmemBytes) {
                    if (!allow_big_smem(rmsnorm_stage_kernel<128, DT>) || !allow_big_smem(rmsnorm_stage_kernel<256, DT>) || !allow_big_smem(rmsnorm_stage_kernel<512, DT>)) return AK_ERR_CUDA;
                    cudaError_t e;
                    if (D <= 8192)
                        e = launch_dependent(rmsnorm_stage_kernel<128, DT>, dim3((unsigned)rows), dim3(128), stage_bytes, st, xs, ws,
                                             ys, D, inv_D, eps, first_wave_ctas(rmsnorm_stage_kernel<128, DT>, 128, stage_bytes));
                    else if (D <= 32768)
                        e = launch_dependent(rmsnorm_stage_kernel<256, DT>, dim3((unsigned)rows), dim3(256), stage_bytes, st, xs, ws,
                                             ys, D, inv_D, eps, first_wave_ctas(rmsnorm_stage_kernel<256, DT>, 256, stage_bytes));
                    else
                        e = launch_dependent(rmsnorm_stage_kernel<512, DT>, dim3((unsigned)rows), dim3(512), stage_bytes, st, xs, ws,
                                             ys, D, inv_D, eps, first_wave_ctas(rmsnorm_stage_kernel<512, DT>, 512, stage_bytes));
                    count_launch();
                    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
                }
                const int resident = resident_ctas(rmsnorm_generic_kernel<DT>, kRmsGenericThreads, 0);
                const int grid = (int)(rows < resident ? rows : resident);
                rmsnorm_generic_kernel<DT><<<grid, kRmsGenericThreads, 0, st>>>(xs, ws, ys, rows, D, inv_D, eps);
                count_launch();
                return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
            }
        }
        default:
            return AK_ERR_ARG;
    }
}

}  // namespace

int rmsnorm_dispatch(const void* x, const void* w, void* y, int64_t rows, int64_t D, float eps,
                     cudaStream_t st, int path, int dtype) {
    switch (dtype) {
        case AK_DTYPE_BF16: return dispatch_t<AK_DTYPE_BF16>(x, w, y, rows, D, eps, st, path);
        case AK_DTYPE_F16: return dispatch_t<AK_DTYPE_F16>(x, w, y, rows, D, eps, st, path);
        case AK_DTYPE_F32: return dispatch_t<AK_DTYPE_F32>(x, w, y, rows, D, eps, st, path);
        default: return AK_ERR_ARG;
    }
}

AK_DEFINE_WAIT_TIMEOUT_READER(rmsnorm_wait_timeouts)

}  // namespace ak
