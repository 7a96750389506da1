// Fused cross-entropy forward: host dispatch.  Kernels live in xent_kernels.cuh.
//
// Two layouts:
//   row    one CTA per row streams the logits once and writes the loss itself
//   split  nsplit CTAs per row write partial (max, sum) pairs to scratch (few rows / very
//          long rows: keeps every SM busy)
// followed by one single-CTA "finish" kernel (split: merge the partials in split order;
// both: fixed-order fp64 mean), launched as a programmatic dependent so that its launch
// latency overlaps the streaming kernel.  Rows whose target is ignore_index are never read.
#include "xent_kernels.cuh"

namespace ak {
namespace {

// vectors in flight per thread, exponentials per 8 evaluated on the FMA pipe
constexpr int kUnroll = 4;
constexpr int kPoly = 2;
// Row layout: 128-thread CTAs with eight vectors in flight per thread; the occupancy hint of
// eight CTAs per SM caps the kernel at 64 registers.  (Without a hint the compiler spends
// registers on scheduling freedom and halves the CTAs in flight.)  Measured against 256
// threads x 4 vectors, 64 x 8, 512 x 4 and a persistent bulk-copy ring fed by one producer
// lane: this shape was the fastest or tied on every benchmark vocabulary; the ring lost
// 5-8 % because the arithmetic, not the loads, needs the resident warps.
constexpr int kRowThreads = 128;
constexpr int kRowUnroll = 8;
constexpr int kRowMinCtas = 8;

template <int DT>
int launch_finish(const typename XElem<DT>::type* logits, const int64_t* targets, int64_t ignore_index, const float2* partial,
                  int nsplit, float* loss_rows, int64_t rows, int64_t V, float* out_mean, double* out_pair,
                  cudaStream_t st, bool dependent) {
    const bool many = rows >= kFinishSmallRows;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(many ? kFinishThreadsMany : kFinishThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = dependent ? 1 : 0;
    cudaError_t e = many ? cudaLaunchKernelEx(&cfg, xent_finish_kernel<DT, kFinishThreadsMany>, logits, targets,
                                              ignore_index, partial, nsplit, loss_rows, rows, V, out_mean, out_pair)
                         : cudaLaunchKernelEx(&cfg, xent_finish_kernel<DT, kFinishThreads>, logits, targets,
                                              ignore_index, partial, nsplit, loss_rows, rows, V, out_mean, out_pair);
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

}  // namespace

// Split when one CTA per row cannot fill the machine (few rows) and the row is long
// enough for slices of about 16384 elements.  Pure function of (rows, V) and the device's SM count.  (Timed for 1 .. 512
// rows with 2 .. 64 slices: about four CTAs per SM in total and slices no shorter than that were
// best or tied: 64 x 128256 13.4 -> 9.6 us, 16 x 128256 8.7 -> 7.3 us against eight per SM / 8192.)
int xent_choose(int64_t rows, int64_t V, int* nsplit) {
    const int64_t kTargetCtas = (int64_t)sm_count() * 4;   // 592 on a full B200: a fixed number for a given device
    constexpr int64_t kMinSlice = 16384;      // elements
    int ns = 1;
    if (rows > 0 && rows < kTargetCtas) {
        int64_t want = (kTargetCtas + rows - 1) / rows;
        // slices of at most kMinSlice elements where the row is that long: two full batches of the
        // split kernel (a slice just over that would run a third, nearly empty one)
        int64_t cap = V >= 2 * kMinSlice ? (V + kMinSlice - 1) / kMinSlice : 1;
        if (want > cap) want = cap;
        if (want > 64) want = 64;
        if (want > 1) ns = (int)want;
    }
    if (nsplit) *nsplit = ns;
    return ns > 1 ? AK_XENT_SPLIT : AK_XENT_ROW;
}

namespace {

template <int DT>
int dispatch_t(const void* logits, const int64_t* targets, int64_t ignore_index,
               float* loss_rows, float* loss_mean, int64_t rows, int64_t V,
               void* workspace, size_t workspace_bytes, bool may_allocate,
               cudaStream_t st, int path, int nsplit) {
    using elem_t = typename XElem<DT>::type;
    int auto_ns = 1;
    const int auto_path = xent_choose(rows, V, &auto_ns);
    if (path == AK_XENT_AUTO) {
        path = auto_path;
        nsplit = auto_ns;
    } else if (path == AK_XENT_SPLIT) {
        if (nsplit == 0) nsplit = auto_ns > 1 ? auto_ns : 2;
        if (nsplit < 1 || nsplit > 64) return AK_ERR_ARG;
    } else if (path == AK_XENT_ROW) {
        nsplit = 1;
    } else {
        return AK_ERR_ARG;
    }
    if (rows > 2147483647LL) return AK_ERR_SHAPE;  // grid.x limit
    const elem_t* lg = static_cast<const elem_t*>(logits);

    if (rows == 0) {
        // nothing to stream; the mean of an empty batch is NaN
        if (loss_mean == nullptr) return AK_OK;
        return launch_finish<DT>(lg, targets, ignore_index, nullptr, 0, loss_rows, 0, V, loss_mean, nullptr, st, false);
    }
    if (path == AK_XENT_ROW) {
        // fp32 logits: seven CTAs per SM (72 registers); at eight the compiler spills
        constexpr int kMinCtas = (DT == AK_DTYPE_F32) ? kRowMinCtas - 1 : kRowMinCtas;
        // The last batch of a row is masked; when at most five of its eight slots per thread can
        // hold data (a 50304-column bf16 row: two) the kernel form that stops at the filled slots
        // is taken (1-2 us per launch there); otherwise the plain form, whose straight-line code is
        // 1-3 % faster when the last batch is full or nearly so.  Same bits either way.
        const int64_t nvec_row = V * (int64_t)sizeof(elem_t) / 16;
        const int64_t rest = nvec_row % ((int64_t)kRowThreads * kRowUnroll);
        const bool trim = nvec_row >= (int64_t)kRowThreads * kRowUnroll && rest > 0 && (rest + kRowThreads - 1) / kRowThreads <= 5;
        const int first_wave = first_wave_prefetch_enabled() ? kMinCtas * sm_count() : 0;
        const cudaError_t e =
            trim ? launch_dependent(xent_row_kernel<kRowUnroll, kPoly, kMinCtas, kRowThreads, DT, true>, dim3((unsigned)rows),
                                    dim3(kRowThreads), 0, st, lg, targets, ignore_index, loss_rows, V, first_wave)
                 : launch_dependent(xent_row_kernel<kRowUnroll, kPoly, kMinCtas, kRowThreads, DT, false>, dim3((unsigned)rows),
                                    dim3(kRowThreads), 0, st, lg, targets, ignore_index, loss_rows, V, first_wave);
        count_launch();
        if (e != cudaSuccess) return AK_ERR_CUDA;
        if (loss_mean == nullptr) return AK_OK;
        return launch_finish<DT>(lg, targets, ignore_index, nullptr, 0, loss_rows, rows, V, loss_mean, nullptr, st, true);
    }
    if (rows > 65535) return AK_ERR_SHAPE;  // grid.y limit; the dispatcher never splits that many rows
    const size_t need = (size_t)rows * (size_t)nsplit * sizeof(float2);
    float2* partial = static_cast<float2*>(workspace);
    bool own = false;
    if (partial == nullptr || workspace_bytes < need) {
        if (!may_allocate) return AK_ERR_NOMEM;
        void* p = nullptr;
        if (scratch_alloc(&p, need, st) != cudaSuccess) {
            (void)cudaGetLastError();
            return AK_ERR_NOMEM;
        }
        partial = static_cast<float2*>(p);
        own = true;
    }
    xent_split_kernel<kUnroll, kPoly, DT><<<dim3((unsigned)nsplit, (unsigned)rows), kXentThreads, 0, st>>>(
        lg, targets, ignore_index, partial, V, nsplit);
    count_launch();
    int status = cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
    if (status == AK_OK)
        status = launch_finish<DT>(lg, targets, ignore_index, partial, nsplit, loss_rows, rows, V, loss_mean, nullptr, st, true);
    if (own) cudaFreeAsync(partial, st);
    return status;
}

}  // namespace

int xent_dispatch(const void* logits, const int64_t* targets, int64_t ignore_index,
                  float* loss_rows, float* loss_mean, int64_t rows, int64_t V,
                  void* workspace, size_t workspace_bytes, bool may_allocate,
                  cudaStream_t st, int path, int nsplit, int dtype) {
    switch (dtype) {
        case AK_DTYPE_BF16:
            return dispatch_t<AK_DTYPE_BF16>(logits, targets, ignore_index, loss_rows, loss_mean, rows, V, workspace,
                                             workspace_bytes, may_allocate, st, path, nsplit);
        case AK_DTYPE_F16:
            return dispatch_t<AK_DTYPE_F16>(logits, targets, ignore_index, loss_rows, loss_mean, rows, V, workspace,
                                            workspace_bytes, may_allocate, st, path, nsplit);
        case AK_DTYPE_F32:
            return dispatch_t<AK_DTYPE_F32>(logits, targets, ignore_index, loss_rows, loss_mean, rows, V, workspace,
                                            workspace_bytes, may_allocate, st, path, nsplit);
        default:
            return AK_ERR_ARG;
    }
}

int xent_mean_launch(const float* loss_rows, const int64_t* targets, int64_t ignore_index, int64_t rows,
                     float* loss_mean, cudaStream_t st, bool dependent) {
    return launch_finish<AK_DTYPE_BF16>(nullptr, targets, ignore_index, nullptr, 0, const_cast<float*>(loss_rows), rows,
                                        0, loss_mean, nullptr, st, dependent);
}

int xent_sum_count_launch(const float* loss_rows, const int64_t* targets, int64_t ignore_index, int64_t rows,
                          double* sum_count, cudaStream_t st) {
    return launch_finish<AK_DTYPE_BF16>(nullptr, targets, ignore_index, nullptr, 0, const_cast<float*>(loss_rows), rows,
                                        0, nullptr, sum_count, st, false);
}

int xent_mean_merge_launch(const double* pairs, int64_t n, float* loss_mean, cudaStream_t st) {
    xent_mean_merge_kernel<<<1, 32, 0, st>>>(pairs, n, loss_mean);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

}  // namespace ak
