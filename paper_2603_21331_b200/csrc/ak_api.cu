// C ABI of libak: argument validation, dispatch, status strings, launch counter and the
// host-buffer variants (chunked copy-in / compute / copy-out pipeline).
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <map>
#include <mutex>
#include <set>
#include <tuple>

#include "ak_common.cuh"

namespace ak {

static std::atomic<int64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

// Stream-ordered scratch comes from a memory pool of the library's own, one per device, that
// keeps up to 256 MiB cached between calls.  (The device's default pool releases everything at
// the next synchronisation unless the application raised its threshold; each call after a
// synchronise would then pay for a fresh physical allocation, hundreds of microseconds.)
cudaError_t scratch_alloc(void** p, size_t bytes, cudaStream_t st) {
    static std::mutex mu;
    static cudaMemPool_t pools[64] = {};
    static bool tried[64] = {};
    int dev = 0;
    cudaMemPool_t pool = nullptr;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0 && dev < 64) {
        std::lock_guard<std::mutex> lock(mu);
        // the pool is not created while `st` is being captured (creating one is no stream
        // operation and could invalidate the capture); such a call uses the default pool
        cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
        if (!tried[dev] && cudaStreamIsCapturing(st, &cap) != cudaSuccess) {
            (void)cudaGetLastError();
            cap = cudaStreamCaptureStatusActive;
        }
        if (!tried[dev] && cap == cudaStreamCaptureStatusNone) {
            tried[dev] = true;
            cudaMemPoolProps props = {};
            props.allocType = cudaMemAllocationTypePinned;
            props.handleTypes = cudaMemHandleTypeNone;
            props.location.type = cudaMemLocationTypeDevice;
            props.location.id = dev;
            cudaMemPool_t created = nullptr;
            if (cudaMemPoolCreate(&created, &props) == cudaSuccess) {
                uint64_t keep = 256ull << 20;
                cudaMemPoolSetAttribute(created, cudaMemPoolAttrReleaseThreshold, &keep);
                pools[dev] = created;
            } else {
                (void)cudaGetLastError();
            }
        }
        pool = pools[dev];
    }
    if (pool != nullptr) return cudaMallocFromPoolAsync(p, bytes, pool, st);
    return cudaMallocAsync(p, bytes, st);
}

// How many CTAs of a cluster share a row.  Timed on B200 for 1 .. 4096 rows of 16 KiB .. 512 KiB
// with 1, 2, 4 and 8 CTAs per row:
//  (a) rows of `split_from` bytes or more (64 KiB: above what one CTA holds in registers) are always
//      split, into slices of at most 32 KiB where eight CTAs can do that: several CTAs then share an
//      SM and overlap their phases (4096 x 65536 softmax 235 -> 174 us, RMSNorm 186 -> 163 us;
//      rows beyond one CTA's shared memory, 4096 x 128256: softmax 677 -> 362 us);
//  (b) with at most 64 rows, rows of 32 KiB or more go to eight CTAs each (1.1x - 2.6x).
// 1 = one CTA per row.  Rows beyond eight CTAs' shared memory get eight CTAs too (the callers
// that cannot stage them stream them, or fall back, as they see fit).
int cluster_ctas(int64_t rows, int64_t row_bytes, int64_t split_from) {
    constexpr int64_t kSliceBytes = 32768, kFewRows = 64, kFewRowsMinBytes = 32768;
    // AK_DISABLE_CLUSTERS=1 in the environment (read once) keeps every row on one CTA: for devices
    // or partitions of one that cannot co-schedule clusters, and for comparing the layouts
    static const bool disabled = [] {
        const char* v = getenv("AK_DISABLE_CLUSTERS");
        return v != nullptr && v[0] != '\0' && v[0] != '0';
    }();
    if (rows < 1 || disabled) return 1;
    if (row_bytes > (int64_t)kMaxCluster * kMaxRowSmemBytes) return kMaxCluster;
    int C = 1;
    if (row_bytes >= split_from)
        while (C < kMaxCluster && row_bytes > (int64_t)C * kSliceBytes) C *= 2;
    if (rows <= kFewRows && row_bytes >= kFewRowsMinBytes) C = kMaxCluster;
    return C;
}

// false when AK_DISABLE_CLUSTERS switches the cluster layouts off
bool clusters_enabled() { return cluster_ctas(1, kClusterFrom, kClusterFrom) > 1; }

int sm_count() {
    static std::mutex mu;
    static int cached[64] = {0};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    std::lock_guard<std::mutex> lock(mu);
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

namespace {
constexpr int kMaxDev = 64;
int current_device() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) return -1;
    return dev;
}
}  // namespace

bool dyn_smem_configured(const void* kernel) {
    static std::mutex mu;
    static std::set<const void*> done[kMaxDev];
    const int dev = current_device();
    if (dev < 0) return false;
    std::lock_guard<std::mutex> lock(mu);
    if (done[dev].count(kernel)) return true;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxRowSmemBytes) != cudaSuccess) {
        (void)cudaGetLastError();
        return false;
    }
    done[dev].insert(kernel);
    return true;
}

// AK_DISABLE_PREFETCH=1 in the environment (read once) switches off the L2 prefetch the first
// wave of a kernel issues before its griddepcontrol.wait (for comparing, or where the kernel
// before in the stream should keep all of the memory system to itself until it ends).
bool first_wave_prefetch_enabled() {
    static const bool off = [] {
        const char* v = getenv("AK_DISABLE_PREFETCH");
        return v != nullptr && v[0] != '\0' && v[0] != '0';
    }();
    return !off;
}

int resident_ctas_of(const void* kernel, int threads, size_t dyn_smem) {
    static std::mutex mu;
    static std::map<std::tuple<const void*, int, size_t>, int> memo[kMaxDev];
    const int dev = current_device();
    const int sms = sm_count();
    if (dev < 0) return sms;
    std::lock_guard<std::mutex> lock(mu);
    const auto key = std::make_tuple(kernel, threads, dyn_smem);
    auto it = memo[dev].find(key);
    if (it != memo[dev].end()) return it->second;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, threads, dyn_smem) != cudaSuccess || per_sm < 1) {
        (void)cudaGetLastError();
        per_sm = 1;
    }
    memo[dev][key] = per_sm * sms;
    return per_sm * sms;
}

namespace {

int check_rows_cols(int64_t rows, int64_t D) {
    if (rows < 0 || D <= 0) return AK_ERR_SHAPE;
    // element offsets are 64-bit, but keep rows*D well inside int64 and vector counts inside int32
    if (rows > 0 && D > (int64_t)0x7fffffffffffLL / rows) return AK_ERR_SHAPE;
    return AK_OK;
}

bool known_dtype(int dtype) { return dtype == AK_DTYPE_BF16 || dtype == AK_DTYPE_F16 || dtype == AK_DTYPE_F32; }

int validate_rmsnorm(const void* x, const void* w, void* y, int64_t rows, int64_t D, float eps, size_t esize = 2) {
    if (rows != 0 && (!x || !w || !y)) return AK_ERR_NULL;  // an empty batch may carry NULL data pointers
    if (int s = check_rows_cols(rows, D)) return s;
    if (!is_aligned(x, esize) || !is_aligned(w, esize) || !is_aligned(y, esize)) return AK_ERR_ALIGN;
    if (!(eps >= 0.0f) || !std::isfinite(eps)) return AK_ERR_ARG;
    return AK_OK;
}
int validate_softmax(const void* x, void* y, int64_t rows, int64_t D, size_t esize = 2) {
    if (rows != 0 && (!x || !y)) return AK_ERR_NULL;
    if (int s = check_rows_cols(rows, D)) return s;
    if (!is_aligned(x, esize) || !is_aligned(y, esize)) return AK_ERR_ALIGN;
    return AK_OK;
}
}  // namespace

int validate_xent(const void* logits, const int64_t* targets, float* loss_rows, float* loss_mean,
                  int64_t rows, int64_t V, size_t esize) {
    if (rows != 0 && (!logits || !targets || !loss_rows)) return AK_ERR_NULL;
    if (int s = check_rows_cols(rows, V)) return s;
    if (!is_aligned(logits, esize) || !is_aligned(targets, 8) || !is_aligned(loss_rows, 4) ||
        (loss_mean && !is_aligned(loss_mean, 4)))
        return AK_ERR_ALIGN;
    return AK_OK;
}

}  // namespace ak

using namespace ak;

extern "C" {

int ak_rmsnorm_fwd_path(const void* x, const void* w, void* y, int64_t rows, int64_t D, float eps,
                        void* cuda_stream, int path) {
    if (int s = validate_rmsnorm(x, w, y, rows, D, eps)) return s;
    if (path < AK_PATH_AUTO || path > AK_PATH_CLUSTER) return AK_ERR_ARG;
    if (rows == 0) return AK_OK;
    return rmsnorm_dispatch(x, w, y, rows, D, eps, static_cast<cudaStream_t>(cuda_stream), path);
}
int ak_rmsnorm_fwd(const void* x, const void* w, void* y, int64_t rows, int64_t D, float eps,
                   void* cuda_stream) {
    return ak_rmsnorm_fwd_path(x, w, y, rows, D, eps, cuda_stream, AK_PATH_AUTO);
}

int ak_rmsnorm_fwd_dt(const void* x, const void* w, void* y, int64_t rows, int64_t D, float eps, int dtype,
                      void* cuda_stream, int path) {
    if (!known_dtype(dtype)) return AK_ERR_ARG;
    if (int s = validate_rmsnorm(x, w, y, rows, D, eps, (size_t)dtype_bytes(dtype))) return s;
    if (path < AK_PATH_AUTO || path > AK_PATH_CLUSTER) return AK_ERR_ARG;
    if (rows == 0) return AK_OK;
    return rmsnorm_dispatch(x, w, y, rows, D, eps, static_cast<cudaStream_t>(cuda_stream), path, dtype);
}
int ak_softmax_fwd_dt(const void* x, void* y, int64_t rows, int64_t D, int dtype, void* cuda_stream, int path) {
    if (!known_dtype(dtype)) return AK_ERR_ARG;
    if (int s = validate_softmax(x, y, rows, D, (size_t)dtype_bytes(dtype))) return s;
    if (path < AK_PATH_AUTO || path > AK_PATH_CLUSTER) return AK_ERR_ARG;
    if (rows == 0) return AK_OK;
    return softmax_dispatch(x, y, rows, D, static_cast<cudaStream_t>(cuda_stream), path, dtype);
}
int ak_xent_fwd_dt(const void* logits, const int64_t* targets, int64_t ignore_index, float* loss_rows,
                   float* loss_mean, int64_t rows, int64_t V, int dtype, void* cuda_stream, int path, int nsplit) {
    if (!known_dtype(dtype)) return AK_ERR_ARG;
    if (int s = validate_xent(logits, targets, loss_rows, loss_mean, rows, V, (size_t)dtype_bytes(dtype))) return s;
    if (path < AK_XENT_AUTO || path > AK_XENT_SPLIT || nsplit < 0 || nsplit > 64) return AK_ERR_ARG;
    return xent_dispatch(logits, targets, ignore_index, loss_rows, loss_mean, rows, V, nullptr, 0, true,
                         static_cast<cudaStream_t>(cuda_stream), path, nsplit, dtype);
}
int ak_layernorm_fwd_dt(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t D,
                        float eps, int dtype, void* cuda_stream, int path) {
    if (!known_dtype(dtype)) return AK_ERR_ARG;
    const size_t es = (size_t)dtype_bytes(dtype);
    if (int s = validate_rmsnorm(x, gamma, y, rows, D, eps, es)) return s;
    if (rows != 0 && !beta) return AK_ERR_NULL;
    if (!is_aligned(beta, es)) return AK_ERR_ALIGN;
    if (path < AK_PATH_AUTO || path > AK_PATH_CLUSTER) return AK_ERR_ARG;
    if (rows == 0) return AK_OK;
    return layernorm_dispatch(x, gamma, beta, y, rows, D, eps, static_cast<cudaStream_t>(cuda_stream), path, dtype);
}
int ak_rowsum_fwd_dt(const void* x, float* out, int64_t rows, int64_t D, int dtype, void* cuda_stream) {
    if (!known_dtype(dtype)) return AK_ERR_ARG;
    if (rows != 0 && (!x || !out)) return AK_ERR_NULL;
    if (int s = check_rows_cols(rows, D)) return s;
    if (!is_aligned(x, (size_t)dtype_bytes(dtype)) || !is_aligned(out, 4)) return AK_ERR_ALIGN;
    if (rows == 0) return AK_OK;
    return rowsum_dispatch(x, out, rows, D, static_cast<cudaStream_t>(cuda_stream), dtype);
}
int ak_rope_fwd(const void* x, void* y, int64_t n_seq, int64_t S, int64_t Dh, float base, int64_t pos_offset,
                int dtype, void* cuda_stream) {
    if (!known_dtype(dtype)) return AK_ERR_ARG;
    if (n_seq < 0 || S < 0 || Dh <= 0 || (Dh & 1) || Dh > 512) return AK_ERR_SHAPE;
    if (n_seq != 0 && S != 0 && (!x || !y)) return AK_ERR_NULL;
    if (n_seq > 0 && S > 0 && (S > (int64_t)0x7fffffffffffLL / Dh || n_seq > (int64_t)0x7fffffffffffLL / (S * Dh)))
        return AK_ERR_SHAPE;
    if (!is_aligned(x, (size_t)dtype_bytes(dtype)) || !is_aligned(y, (size_t)dtype_bytes(dtype))) return AK_ERR_ALIGN;
    if (!(base > 0.0f) || !std::isfinite(base)) return AK_ERR_ARG;
    if (pos_offset < 0 || pos_offset > ((int64_t)1 << 52) - S) return AK_ERR_ARG;
    if (n_seq == 0 || S == 0) return AK_OK;
    return rope_dispatch(x, y, n_seq, S, Dh, base, pos_offset, dtype, static_cast<cudaStream_t>(cuda_stream));
}

int ak_xent_vp_nsplit(int64_t rows, int64_t V_local) {
    int ns = 1;
    if (rows > 0 && V_local > 0) xent_choose(rows, V_local, &ns);
    return ns;
}
size_t ak_xent_vp_partial_bytes(int64_t rows, int nsplit) {
    if (rows <= 0 || nsplit < 1) return 0;
    return (size_t)rows * (size_t)(nsplit + 1) * sizeof(float2);
}
int ak_xent_vp_partial(const void* logits_shard, const int64_t* targets, int64_t ignore_index,
                       int64_t vocab_start, int64_t V_total, void* partial, int64_t rows, int64_t V_local,
                       int nsplit, int dtype, void* cuda_stream) {
    if (!known_dtype(dtype)) return AK_ERR_ARG;
    if (rows != 0 && (!logits_shard || !targets || !partial)) return AK_ERR_NULL;
    if (int s = check_rows_cols(rows, V_local)) return s;
    if (vocab_start < 0 || V_total < V_local || vocab_start > V_total - V_local) return AK_ERR_SHAPE;
    if (!is_aligned(logits_shard, (size_t)dtype_bytes(dtype)) || !is_aligned(targets, 8) || !is_aligned(partial, 8))
        return AK_ERR_ALIGN;
    if (nsplit < 1 || nsplit > 64) return AK_ERR_ARG;
    if (rows > 2147483647LL) return AK_ERR_SHAPE;
    if (rows == 0) return AK_OK;
    return xent_vp_partial_launch(logits_shard, targets, ignore_index, vocab_start, V_total, partial, rows, V_local,
                                  nsplit, dtype, static_cast<cudaStream_t>(cuda_stream));
}
int ak_xent_vp_merge(const void* partials, int nranks, int nsplit, const int64_t* targets, int64_t ignore_index,
                     int64_t V_total, float* loss_rows, float* loss_mean, int64_t rows, void* cuda_stream) {
    if (rows != 0 && (!partials || !targets || !loss_rows)) return AK_ERR_NULL;
    if (rows < 0 || V_total <= 0) return AK_ERR_SHAPE;
    if (nranks < 1 || nranks > 4096 || nsplit < 1 || nsplit > 64) return AK_ERR_ARG;
    if (!is_aligned(partials, 8) || !is_aligned(targets, 8) || !is_aligned(loss_rows, 4) ||
        (loss_mean && !is_aligned(loss_mean, 4)))
        return AK_ERR_ALIGN;
    if (rows > 2147483647LL * 128) return AK_ERR_SHAPE;
    return xent_vp_merge_launch(partials, nranks, nsplit, targets, ignore_index, V_total, loss_rows, loss_mean, rows,
                                static_cast<cudaStream_t>(cuda_stream));
}

int ak_choose_path_dt(int op, int64_t rows, int64_t D, int aligned16, int dtype) {
    if (!known_dtype(dtype)) return -1;
    if (op == 0) return rmsnorm_choose(rows, D, aligned16 != 0, dtype);
    if (op == 1) return softmax_choose(rows, D, aligned16 != 0, dtype);
    if (op == 2) return layernorm_choose(rows, D, aligned16 != 0, dtype);
    return -1;
}

int ak_layernorm_fwd_path(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t D,
                          float eps, void* cuda_stream, int path) {
    if (int s = validate_rmsnorm(x, gamma, y, rows, D, eps)) return s;
    if (rows != 0 && !beta) return AK_ERR_NULL;
    if (!is_aligned(beta, 2)) return AK_ERR_ALIGN;
    if (path < AK_PATH_AUTO || path > AK_PATH_CLUSTER) return AK_ERR_ARG;
    if (rows == 0) return AK_OK;
    return layernorm_dispatch(x, gamma, beta, y, rows, D, eps, static_cast<cudaStream_t>(cuda_stream), path);
}
int ak_layernorm_fwd(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t D,
                     float eps, void* cuda_stream) {
    return ak_layernorm_fwd_path(x, gamma, beta, y, rows, D, eps, cuda_stream, AK_PATH_AUTO);
}

int ak_rowsum_fwd(const void* x, float* out, int64_t rows, int64_t D, void* cuda_stream) {
    if (rows != 0 && (!x || !out)) return AK_ERR_NULL;
    if (int s = check_rows_cols(rows, D)) return s;
    if (!is_aligned(x, 2) || !is_aligned(out, 4)) return AK_ERR_ALIGN;
    if (rows == 0) return AK_OK;
    return rowsum_dispatch(x, out, rows, D, static_cast<cudaStream_t>(cuda_stream));
}

int ak_softmax_fwd_path(const void* x, void* y, int64_t rows, int64_t D, void* cuda_stream, int path) {
    if (int s = validate_softmax(x, y, rows, D)) return s;
    if (path < AK_PATH_AUTO || path > AK_PATH_CLUSTER) return AK_ERR_ARG;
    if (rows == 0) return AK_OK;
    return softmax_dispatch(x, y, rows, D, static_cast<cudaStream_t>(cuda_stream), path);
}
int ak_softmax_fwd(const void* x, void* y, int64_t rows, int64_t D, void* cuda_stream) {
    return ak_softmax_fwd_path(x, y, rows, D, cuda_stream, AK_PATH_AUTO);
}

int ak_xent_fwd_path(const void* logits, const int64_t* targets, int64_t ignore_index,
                     float* loss_rows, float* loss_mean, int64_t rows, int64_t V,
                     void* cuda_stream, int path, int nsplit) {
    if (int s = validate_xent(logits, targets, loss_rows, loss_mean, rows, V)) return s;
    if (path < AK_XENT_AUTO || path > AK_XENT_SPLIT || nsplit < 0 || nsplit > 64) return AK_ERR_ARG;
    return xent_dispatch(logits, targets, ignore_index, loss_rows, loss_mean, rows, V, nullptr, 0, true,
                         static_cast<cudaStream_t>(cuda_stream), path, nsplit);
}
int ak_xent_fwd(const void* logits, const int64_t* targets, int64_t ignore_index,
                float* loss_rows, float* loss_mean, int64_t rows, int64_t V, void* cuda_stream) {
    return ak_xent_fwd_path(logits, targets, ignore_index, loss_rows, loss_mean, rows, V, cuda_stream,
                            AK_XENT_AUTO, 0);
}

size_t ak_xent_workspace_bytes(int64_t rows, int64_t V) {
    if (rows <= 0 || V <= 0) return 0;
    int ns = 1;
    if (xent_choose(rows, V, &ns) != AK_XENT_SPLIT) return 0;
    return (size_t)rows * (size_t)ns * sizeof(float2);
}

int ak_xent_fwd_ws(const void* logits, const int64_t* targets, int64_t ignore_index,
                   float* loss_rows, float* loss_mean, int64_t rows, int64_t V,
                   void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (int s = validate_xent(logits, targets, loss_rows, loss_mean, rows, V)) return s;
    const size_t need = ak_xent_workspace_bytes(rows, V);
    if (need > 0) {
        if (!workspace) return AK_ERR_NULL;
        if (!is_aligned(workspace, 8)) return AK_ERR_ALIGN;
        if (workspace_bytes < need) return AK_ERR_NOMEM;
    }
    return xent_dispatch(logits, targets, ignore_index, loss_rows, loss_mean, rows, V, workspace,
                         workspace_bytes, false, static_cast<cudaStream_t>(cuda_stream), AK_XENT_AUTO, 0);
}

int ak_xent_sum_count(const float* loss_rows, const int64_t* targets, int64_t ignore_index, int64_t rows,
                      double* sum_count, void* cuda_stream) {
    if (rows < 0) return AK_ERR_SHAPE;
    if (!sum_count || (rows != 0 && (!loss_rows || !targets))) return AK_ERR_NULL;  // an empty block may carry NULL data
    if (!is_aligned(loss_rows, 4) || !is_aligned(targets, 8) || !is_aligned(sum_count, 8)) return AK_ERR_ALIGN;
    return xent_sum_count_launch(loss_rows, targets, ignore_index, rows, sum_count,
                                 static_cast<cudaStream_t>(cuda_stream));
}

int ak_xent_mean_merge(const double* sum_count_pairs, int64_t n, float* loss_mean, void* cuda_stream) {
    if (n < 0) return AK_ERR_SHAPE;
    if (!loss_mean || (n != 0 && !sum_count_pairs)) return AK_ERR_NULL;  // no pairs: the mean is NaN
    if (!is_aligned(sum_count_pairs, 8) || !is_aligned(loss_mean, 4)) return AK_ERR_ALIGN;
    return xent_mean_merge_launch(sum_count_pairs, n, loss_mean, static_cast<cudaStream_t>(cuda_stream));
}

int ak_rmsnorm_choose_path(int64_t rows, int64_t D, int aligned16) {
    return rmsnorm_choose(rows, D, aligned16 != 0);
}
int ak_layernorm_choose_path(int64_t rows, int64_t D, int aligned16) {
    return layernorm_choose(rows, D, aligned16 != 0);
}
int ak_softmax_choose_path(int64_t rows, int64_t D, int aligned16) {
    return softmax_choose(rows, D, aligned16 != 0);
}
int ak_xent_choose_path(int64_t rows, int64_t V, int* nsplit_out) { return xent_choose(rows, V, nsplit_out); }

int64_t ak_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int ak_sm_count(void) { return sm_count(); }

int ak_wait_timeouts(void) {
    const int a = rmsnorm_wait_timeouts(), b = softmax_wait_timeouts(), c = layernorm_wait_timeouts();
    if (a < 0 || b < 0 || c < 0) return -1;
    return (a != 0) + (b != 0) + (c != 0);
}

const char* ak_status_string(int status) {
    switch (status) {
        case AK_OK: return "ok";
        case AK_ERR_NULL: return "a required pointer is NULL";
        case AK_ERR_SHAPE: return "bad shape (rows < 0, D <= 0, or size not supported by the requested path)";
        case AK_ERR_ALIGN: return "pointer not sufficiently aligned";
        case AK_ERR_ARG: return "bad scalar argument (eps, base, position offset, path id, nsplit or dtype)";
        case AK_ERR_CUDA: return "CUDA runtime error";
        case AK_ERR_NOMEM: return "scratch memory unavailable or workspace too small";
        case AK_ERR_CAPACITY: return "problem exceeds the fixed scratch of the no-allocation entry point (rows * nsplit * 8 bytes > 1 MiB or rows > 65535)";
        default: return "unknown status";
    }
}

int ak_version(void) { return 100; }

}  // extern "C"

// ======================================================================================
// Host-buffer variants.  Rows are independent, so the tensor is cut into row chunks that
// flow through kSlots lanes; lane i owns one stream and one pair of device staging
// buffers, and runs copy-in -> kernel -> copy-out for chunks i, i+kSlots, ...  Work in
// different lanes overlaps (both copy engines and the SMs stay busy); work in one lane is
// ordered by its stream, which also makes buffer reuse safe.
// ======================================================================================
namespace ak {
namespace {

constexpr int kSlots = 3;
constexpr size_t kChunkBytes = 16u << 20;  // staging bytes per lane and direction
constexpr int kMaxDevices = 64;

struct Arena {
    bool init = false;
    cudaStream_t st[kSlots] = {};
    void* in[kSlots] = {};
    void* out[kSlots] = {};
    size_t in_cap = 0, out_cap = 0;
    void* aux = nullptr;  // weights, or targets + loss rows + mean
    size_t aux_cap = 0;
};

std::mutex g_arena_mu;
Arena g_arena[kMaxDevices];

void arena_free(Arena& a) {
    for (int i = 0; i < kSlots; ++i) {
        if (a.in[i]) cudaFree(a.in[i]);
        if (a.out[i]) cudaFree(a.out[i]);
        if (a.st[i]) cudaStreamDestroy(a.st[i]);
        a.in[i] = a.out[i] = nullptr;
        a.st[i] = nullptr;
    }
    if (a.aux) cudaFree(a.aux);
    a = Arena{};
}

// Returns the arena of the current device with at least the requested capacities.
int arena_get(size_t in_bytes, size_t out_bytes, size_t aux_bytes, Arena** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return AK_ERR_CUDA;
    if (dev < 0 || dev >= kMaxDevices) return AK_ERR_CUDA;
    Arena& a = g_arena[dev];
    if (!a.init) {
        for (int i = 0; i < kSlots; ++i)
            if (cudaStreamCreateWithFlags(&a.st[i], cudaStreamNonBlocking) != cudaSuccess) {
                arena_free(a);
                return AK_ERR_CUDA;
            }
        a.init = true;
    }
    auto grow = [](void** p, size_t* cap, size_t need) -> bool {
        if (need <= *cap) return true;
        if (*p) cudaFree(*p);
        *p = nullptr;
        *cap = 0;
        if (cudaMalloc(p, need) != cudaSuccess) { (void)cudaGetLastError(); return false; }
        *cap = need;
        return true;
    };
    if (in_bytes > a.in_cap) {
        for (int i = 0; i < kSlots; ++i) {
            size_t cap = a.in_cap;
            if (!grow(&a.in[i], &cap, in_bytes)) { arena_free(a); return AK_ERR_NOMEM; }
        }
        a.in_cap = in_bytes;
    }
    if (out_bytes > a.out_cap) {
        for (int i = 0; i < kSlots; ++i) {
            size_t cap = a.out_cap;
            if (!grow(&a.out[i], &cap, out_bytes)) { arena_free(a); return AK_ERR_NOMEM; }
        }
        a.out_cap = out_bytes;
    }
    if (!grow(&a.aux, &a.aux_cap, aux_bytes)) { arena_free(a); return AK_ERR_NOMEM; }
    *out = &a;
    return AK_OK;
}

int64_t rows_per_chunk(int64_t rows, int64_t D) {
    int64_t r = (int64_t)(kChunkBytes / ((size_t)D * 2));
    if (r < 1) r = 1;
    return r < rows ? r : rows;
}

int sync_all(Arena& a) {
    int status = AK_OK;
    for (int i = 0; i < kSlots; ++i)
        if (cudaStreamSynchronize(a.st[i]) != cudaSuccess) status = AK_ERR_CUDA;
    return status;
}

#define AK_TRY_CUDA(expr)                         \
    do {                                          \
        if ((expr) != cudaSuccess) {              \
            (void)cudaGetLastError();             \
            sync_all(*a);                         \
            return AK_ERR_CUDA;                   \
        }                                         \
    } while (0)

}  // namespace
}  // namespace ak

extern "C" {

int ak_rmsnorm_fwd_host(const void* x_host, const void* w_host, void* y_host, int64_t rows, int64_t D,
                        float eps) {
    if (int s = validate_rmsnorm(x_host, w_host, y_host, rows, D, eps)) return s;
    if (rows == 0) return AK_OK;
    std::lock_guard<std::mutex> lock(g_arena_mu);
    const int64_t rc = rows_per_chunk(rows, D);
    const size_t chunk = (size_t)rc * (size_t)D * 2;
    Arena* a = nullptr;
    if (int s = arena_get(chunk, chunk, (size_t)D * 2, &a)) return s;
    AK_TRY_CUDA(cudaMemcpyAsync(a->aux, w_host, (size_t)D * 2, cudaMemcpyHostToDevice, a->st[0]));
    AK_TRY_CUDA(cudaStreamSynchronize(a->st[0]));  // weights visible to every lane
    const char* xs = static_cast<const char*>(x_host);
    char* ys = static_cast<char*>(y_host);
    int64_t c = 0;
    for (int64_t r0 = 0; r0 < rows; r0 += rc, ++c) {
        const int lane = (int)(c % kSlots);
        const int64_t nr = (rows - r0 < rc) ? rows - r0 : rc;
        const size_t bytes = (size_t)nr * (size_t)D * 2, off = (size_t)r0 * (size_t)D * 2;
        AK_TRY_CUDA(cudaMemcpyAsync(a->in[lane], xs + off, bytes, cudaMemcpyHostToDevice, a->st[lane]));
        if (int s = rmsnorm_dispatch(a->in[lane], a->aux, a->out[lane], nr, D, eps, a->st[lane], AK_PATH_AUTO)) {
            sync_all(*a);
            return s;
        }
        AK_TRY_CUDA(cudaMemcpyAsync(ys + off, a->out[lane], bytes, cudaMemcpyDeviceToHost, a->st[lane]));
    }
    return sync_all(*a);
}

int ak_softmax_fwd_host(const void* x_host, void* y_host, int64_t rows, int64_t D) {
    if (int s = validate_softmax(x_host, y_host, rows, D)) return s;
    if (rows == 0) return AK_OK;
    std::lock_guard<std::mutex> lock(g_arena_mu);
    const int64_t rc = rows_per_chunk(rows, D);
    const size_t chunk = (size_t)rc * (size_t)D * 2;
    Arena* a = nullptr;
    if (int s = arena_get(chunk, chunk, 0, &a)) return s;
    const char* xs = static_cast<const char*>(x_host);
    char* ys = static_cast<char*>(y_host);
    int64_t c = 0;
    for (int64_t r0 = 0; r0 < rows; r0 += rc, ++c) {
        const int lane = (int)(c % kSlots);
        const int64_t nr = (rows - r0 < rc) ? rows - r0 : rc;
        const size_t bytes = (size_t)nr * (size_t)D * 2, off = (size_t)r0 * (size_t)D * 2;
        AK_TRY_CUDA(cudaMemcpyAsync(a->in[lane], xs + off, bytes, cudaMemcpyHostToDevice, a->st[lane]));
        if (int s = softmax_dispatch(a->in[lane], a->out[lane], nr, D, a->st[lane], AK_PATH_AUTO)) {
            sync_all(*a);
            return s;
        }
        AK_TRY_CUDA(cudaMemcpyAsync(ys + off, a->out[lane], bytes, cudaMemcpyDeviceToHost, a->st[lane]));
    }
    return sync_all(*a);
}

int ak_xent_fwd_host(const void* logits_host, const int64_t* targets_host, int64_t ignore_index,
                     float* loss_rows_host, float* loss_mean_host, int64_t rows, int64_t V) {
    if (int s = validate_xent(logits_host, targets_host, loss_rows_host, loss_mean_host, rows, V)) return s;
    if (rows == 0) {
        if (loss_mean_host) *loss_mean_host = std::nanf("");
        return AK_OK;
    }
    std::lock_guard<std::mutex> lock(g_arena_mu);
    const int64_t rc = rows_per_chunk(rows, V);
    const size_t chunk = (size_t)rc * (size_t)V * 2;
    // per-lane scratch for the split-row path lives in the lane's `out` buffer: what a full chunk
    // and the last, shorter chunk need (nothing when both take one CTA per row)
    const int64_t tail_rows = rows % rc;
    size_t ws_bytes = ak_xent_workspace_bytes(rc, V);
    if (tail_rows > 0 && ak_xent_workspace_bytes(tail_rows, V) > ws_bytes) ws_bytes = ak_xent_workspace_bytes(tail_rows, V);
    // aux: targets [rows] int64 | loss rows [rows] fp32 | mean fp32 (8-byte slots)
    const size_t t_bytes = (size_t)rows * 8, l_bytes = ((size_t)rows * 4 + 7) & ~(size_t)7;
    Arena* a = nullptr;
    if (int s = arena_get(chunk, ws_bytes, t_bytes + l_bytes + 8, &a)) return s;
    int64_t* d_targets = static_cast<int64_t*>(a->aux);
    float* d_loss = reinterpret_cast<float*>(static_cast<char*>(a->aux) + t_bytes);
    float* d_mean = reinterpret_cast<float*>(static_cast<char*>(a->aux) + t_bytes + l_bytes);
    AK_TRY_CUDA(cudaMemcpyAsync(d_targets, targets_host, t_bytes, cudaMemcpyHostToDevice, a->st[0]));
    AK_TRY_CUDA(cudaStreamSynchronize(a->st[0]));
    const char* xs = static_cast<const char*>(logits_host);
    int64_t c = 0;
    for (int64_t r0 = 0; r0 < rows; r0 += rc, ++c) {
        const int lane = (int)(c % kSlots);
        const int64_t nr = (rows - r0 < rc) ? rows - r0 : rc;
        const size_t bytes = (size_t)nr * (size_t)V * 2, off = (size_t)r0 * (size_t)V * 2;
        AK_TRY_CUDA(cudaMemcpyAsync(a->in[lane], xs + off, bytes, cudaMemcpyHostToDevice, a->st[lane]));
        if (int s = xent_dispatch(a->in[lane], d_targets + r0, ignore_index, d_loss + r0, nullptr, nr, V,
                                  ws_bytes ? a->out[lane] : nullptr, ws_bytes ? a->out_cap : 0, false, a->st[lane],
                                  AK_XENT_AUTO, 0)) {
            sync_all(*a);
            return s;
        }
        AK_TRY_CUDA(cudaMemcpyAsync(loss_rows_host + r0, d_loss + r0, (size_t)nr * 4, cudaMemcpyDeviceToHost,
                                    a->st[lane]));
    }
    if (int s = sync_all(*a)) return s;
    if (loss_mean_host) {
        if (int s = xent_mean_launch(d_loss, d_targets, ignore_index, rows, d_mean, a->st[0])) return s;
        AK_TRY_CUDA(cudaMemcpyAsync(loss_mean_host, d_mean, 4, cudaMemcpyDeviceToHost, a->st[0]));
        AK_TRY_CUDA(cudaStreamSynchronize(a->st[0]));
    }
    return AK_OK;
}

int ak_host_arena_release(void) {
    std::lock_guard<std::mutex> lock(g_arena_mu);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AK_ERR_CUDA;
    arena_free(g_arena[dev]);
    return AK_OK;
}

}  // extern "C"
