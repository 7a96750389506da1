// Fused cross-entropy forward kernels (paper Table 3 "cross_ent": online log-sum-exp fused
// with the NLL gather; a single pass over the logits).
//
//   loss[r] = (m - x[r, t]) + log( sum_k exp(x[r, k] - m) ),  m = max_k x[r, k]
//
// Each thread streams 16-byte vectors of its row (or of its slice of the row) and keeps an
// online pair: the running maximum m (always a bf16 value) and s = sum 2^(x*log2e - mf)
// with mf = rn(m*log2e).  Rescaling by 2^(mf_old - mf_new) happens once per batch of
// vectors, only when the maximum moved.  Working in the rounded log2 domain is exact up to
// one per-row constant: x*log2e - m*log2e = (x*log2e - mf) - err with
// err = fma(m, log2e, -mf) (the rounding error of a product is representable), so
//   log sum exp(x - m) = ln2 * (log2(s) - err).
// The loss is assembled as (m - x_t) + that term: both parts are >= 0, and no large
// magnitude is ever added to a small one.
//
// Two layouts:
//   row    one CTA per row, loss written by the CTA itself
//   split  nsplit CTAs per row write partial (m, s) pairs to scratch; a merge kernel
//          combines them in split order (used for few rows or very long rows)
// followed by a single-CTA fixed-order fp64 mean.  Rows whose target is ignore_index are
// never read.  Any 2-byte alignment and any V are handled (scalar head and tail).
#include "ak_common.cuh"

namespace ak {
namespace {

constexpr uint32_t kNegInf2 = 0xFF80FF80u;
constexpr float kFloor2 = -1.0e30f;  // finite stand-in for "no maximum yet" in the log2 domain
constexpr int kThreads = 256;
constexpr int kUnroll = 4;

struct Online {
    float m;   // running maximum (bf16-valued, -inf when nothing finite seen)
    float mf;  // max(rn(m * log2e), kFloor2)
    float s;   // sum of 2^(x*log2e - mf)
};

__device__ __forceinline__ uint32_t max8(const uint4& v) {
    return bf16x2_max(bf16x2_max(v.x, v.y), bf16x2_max(v.z, v.w));
}
__device__ __forceinline__ float hmax_of(uint32_t m2) { return fmaxf(bf16lo(m2), bf16hi(m2)); }

__device__ __forceinline__ void raise_max(Online& o, float vm) {
    const float vmf = fmaxf(vm * kLog2e, kFloor2);
    if (vmf > o.mf) {
        o.s *= fast_exp2(o.mf - vmf);
        o.mf = vmf;
    }
    o.m = fmaxf(o.m, vm);
}

__device__ __forceinline__ float sumexp8(const uint4& v, float mf) {
    const float e0 = fast_exp2(fmaf(bf16lo(v.x), kLog2e, -mf));
    const float e1 = fast_exp2(fmaf(bf16hi(v.x), kLog2e, -mf));
    const float e2 = fast_exp2(fmaf(bf16lo(v.y), kLog2e, -mf));
    const float e3 = fast_exp2(fmaf(bf16hi(v.y), kLog2e, -mf));
    const float e4 = fast_exp2(fmaf(bf16lo(v.z), kLog2e, -mf));
    const float e5 = fast_exp2(fmaf(bf16hi(v.z), kLog2e, -mf));
    const float e6 = fast_exp2(fmaf(bf16lo(v.w), kLog2e, -mf));
    const float e7 = fast_exp2(fmaf(bf16hi(v.w), kLog2e, -mf));
    return ((e0 + e1) + (e2 + e3)) + ((e4 + e5) + (e6 + e7));
}

__device__ __forceinline__ void absorb_scalar(Online& o, float v) {
    raise_max(o, v);
    o.s += fast_exp2(fmaf(v, kLog2e, -o.mf));
}

// CTA-wide online (m, s) over elements [begin, end) of one row.  Returns, in every
// thread, the maximum M and the sum S relative to MF = max(rn(M*log2e), kFloor2).
// Uses both slot sets (max then sum), so consecutive calls need no extra barrier.
__device__ __forceinline__ void row_slice_lse(const uint16_t* __restrict__ xr, int64_t begin, int64_t end,
                                              float* slots, float& M, float& S) {
    Online o{-INFINITY, kFloor2, 0.0f};
    const uint16_t* p = xr + begin;
    const int64_t n = end - begin;
    int64_t head = (8 - (int)((reinterpret_cast<uintptr_t>(p) >> 1) & 7)) & 7;
    if (head > n) head = n;
    const int64_t nbody = (n - head) >> 3;
    const int64_t tail0 = head + (nbody << 3);
    const uint4* body = reinterpret_cast<const uint4*>(p + head);

    for (int64_t base = 0; base < nbody; base += (int64_t)kThreads * kUnroll) {
        uint4 q[kUnroll];
#pragma unroll
        for (int k = 0; k < kUnroll; ++k) {
            const int64_t i = base + threadIdx.x + (int64_t)k * kThreads;
            q[k] = (i < nbody) ? ld_stream(body + i) : make_uint4(kNegInf2, kNegInf2, kNegInf2, kNegInf2);
        }
        uint32_t mx = max8(q[0]);
#pragma unroll
        for (int k = 1; k < kUnroll; ++k) mx = bf16x2_max(mx, max8(q[k]));
        raise_max(o, hmax_of(mx));
        float acc = 0.0f;
#pragma unroll
        for (int k = 0; k < kUnroll; ++k) acc += sumexp8(q[k], o.mf);
        o.s += acc;
    }
    if ((int64_t)threadIdx.x < head) absorb_scalar(o, bf16_to_float(ld_stream_u16(p + threadIdx.x)));
    if (tail0 + threadIdx.x < n) absorb_scalar(o, bf16_to_float(ld_stream_u16(p + tail0 + threadIdx.x)));

    M = cta_max<kThreads>(o.m, slots, 0);
    const float MF = fmaxf(M * kLog2e, kFloor2);
    S = cta_sum<kThreads>(o.s * fast_exp2(o.mf - MF), slots, 1);
}

// loss from the row's (M, S) and the target logit.
__device__ __forceinline__ float finish_loss(float M, float S, float xt) {
    const float MF = fmaxf(M * kLog2e, kFloor2);
    const float err = fmaf(M, kLog2e, -MF);
    // The exact value is >= 0 (the maximum contributes 1 to the sum); the SFU's 2^-22
    // error can leave it a few 1e-8 below.  Clamp without swallowing a NaN.
    float lse = kLn2 * (log2f(S) - err);
    if (lse < 0.0f) lse = 0.0f;
    return (M - xt) + lse;
}

// ------------------------------------------------------------------ one CTA per row
__global__ void __launch_bounds__(kThreads)
xent_row_kernel(const uint16_t* __restrict__ logits, const int64_t* __restrict__ targets,
                int64_t ignore_index, float* __restrict__ loss_rows, int64_t V) {
    __shared__ float slots[2 * kWarp];
    const int64_t row = blockIdx.x;
    const int64_t t = targets[row];
    if (t == ignore_index || t < 0 || t >= V) {  // uniform across the CTA: nothing is read
        if (threadIdx.x == 0) loss_rows[row] = (t == ignore_index) ? 0.0f : __int_as_float(0x7fc00000);
        return;
    }
    const uint16_t* xr = logits + row * V;
    float M, S;
    row_slice_lse(xr, 0, V, slots, M, S);
    if (threadIdx.x == 0) loss_rows[row] = finish_loss(M, S, bf16_to_float(xr[t]));
}

// ------------------------------------------------------------------ split row, phase 1
// grid = (nsplit, rows).  Slice boundaries are multiples of 8 elements so an aligned row
// keeps aligned slices.
__global__ void __launch_bounds__(kThreads)
xent_split_kernel(const uint16_t* __restrict__ logits, const int64_t* __restrict__ targets,
                  int64_t ignore_index, float2* __restrict__ partial, int64_t V, int nsplit) {
    __shared__ float slots[2 * kWarp];
    const int64_t row = blockIdx.y;
    const int sp = blockIdx.x;
    const int64_t t = targets[row];
    if (t == ignore_index || t < 0 || t >= V) return;
    const int64_t groups = (V + 7) >> 3;
    int64_t begin = ((groups * sp) / nsplit) << 3;
    int64_t end = ((groups * (sp + 1)) / nsplit) << 3;
    if (end > V) end = V;
    float M, S;
    row_slice_lse(logits + row * V, begin, end, slots, M, S);
    if (threadIdx.x == 0) partial[row * nsplit + sp] = make_float2(M, S);
}

// ------------------------------------------------------------------ split row, phase 2
// One thread per row merges its nsplit partials in split order.
__global__ void __launch_bounds__(kThreads)
xent_merge_kernel(const uint16_t* __restrict__ logits, const int64_t* __restrict__ targets,
                  int64_t ignore_index, const float2* __restrict__ partial,
                  float* __restrict__ loss_rows, int64_t rows, int64_t V, int nsplit) {
    const int64_t row = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    if (row >= rows) return;
    const int64_t t = targets[row];
    if (t == ignore_index) { loss_rows[row] = 0.0f; return; }
    if (t < 0 || t >= V) { loss_rows[row] = __int_as_float(0x7fc00000); return; }
    const float2* pr = partial + row * nsplit;
    float M = -INFINITY;
    for (int i = 0; i < nsplit; ++i) M = fmaxf(M, pr[i].x);
    const float MF = fmaxf(M * kLog2e, kFloor2);
    float S = 0.0f;
    for (int i = 0; i < nsplit; ++i) {
        const float2 ps = pr[i];
        S += ps.y * fast_exp2(fmaxf(ps.x * kLog2e, kFloor2) - MF);
    }
    loss_rows[row] = finish_loss(M, S, bf16_to_float(logits[row * V + t]));
}

// ------------------------------------------------------------------ mean
// Single CTA, fixed order: thread i adds rows i, i+T, i+2T, ... in fp64, then a fixed
// tree over threads.  loss_mean = sum / count over rows whose target != ignore_index.
constexpr int kMeanThreads = 1024;

// out_mean != nullptr: write the fp32 mean.  out_pair != nullptr: write {sum, count} as two
// doubles (the per-rank contribution to a mean over row shards).
__global__ void __launch_bounds__(kMeanThreads)
xent_mean_kernel(const float* __restrict__ loss_rows, const int64_t* __restrict__ targets,
                 int64_t ignore_index, int64_t rows, float* __restrict__ out_mean,
                 double* __restrict__ out_pair) {
    __shared__ double ssum[kMeanThreads];
    __shared__ long long scnt[kMeanThreads];
    double acc = 0.0;
    long long cnt = 0;
    for (int64_t r = threadIdx.x; r < rows; r += kMeanThreads) {
        if (targets[r] != ignore_index) {
            acc += (double)loss_rows[r];
            ++cnt;
        }
    }
    ssum[threadIdx.x] = acc;
    scnt[threadIdx.x] = cnt;
    __syncthreads();
    for (int stride = kMeanThreads / 2; stride > 0; stride >>= 1) {
        if (threadIdx.x < stride) {
            ssum[threadIdx.x] += ssum[threadIdx.x + stride];
            scnt[threadIdx.x] += scnt[threadIdx.x + stride];
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        if (out_mean)
            out_mean[0] = (scnt[0] > 0) ? (float)(ssum[0] / (double)scnt[0]) : __int_as_float(0x7fc00000);
        if (out_pair) {
            out_pair[0] = ssum[0];
            out_pair[1] = (double)scnt[0];
        }
    }
}

// Mean over row shards: pairs[i] = {sum_i, count_i}; added in index order by one thread.
__global__ void xent_mean_merge_kernel(const double* __restrict__ pairs, int64_t n, float* __restrict__ out_mean) {
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    double total = 0.0, count = 0.0;
    for (int64_t i = 0; i < n; ++i) {
        total += pairs[2 * i];
        count += pairs[2 * i + 1];
    }
    out_mean[0] = (count > 0.0) ? (float)(total / count) : __int_as_float(0x7fc00000);
}

}  // namespace

// Split when one CTA per row cannot fill the machine (few rows) and the row is long
// enough for slices of at least 16 KiB.  Pure function of (rows, V).
int xent_choose(int64_t rows, int64_t V, int* nsplit) {
    constexpr int64_t kTargetCtas = 148 * 8;  // about two resident waves of 256-thread CTAs
    constexpr int64_t kMinSlice = 8192;       // elements
    int ns = 1;
    if (rows > 0 && rows < kTargetCtas) {
        int64_t want = (kTargetCtas + rows - 1) / rows;
        int64_t cap = V / kMinSlice;
        if (want > cap) want = cap;
        if (want > 64) want = 64;
        if (want > 1) ns = (int)want;
    }
    if (nsplit) *nsplit = ns;
    return ns > 1 ? AK_XENT_SPLIT : AK_XENT_ROW;
}

int xent_dispatch(const void* logits, const int64_t* targets, int64_t ignore_index,
                  float* loss_rows, float* loss_mean, int64_t rows, int64_t V,
                  void* workspace, size_t workspace_bytes, bool may_allocate,
                  cudaStream_t st, int path, int nsplit) {
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
    const uint16_t* lg = static_cast<const uint16_t*>(logits);

    if (rows == 0) {
        // nothing to stream; the mean of an empty batch is NaN
    } else if (path == AK_XENT_ROW) {
        xent_row_kernel<<<(unsigned)rows, kThreads, 0, st>>>(lg, targets, ignore_index, loss_rows, V);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return AK_ERR_CUDA;
    } else {
        if (rows > 65535) return AK_ERR_SHAPE;  // grid.y limit; the dispatcher never splits that many rows
        const size_t need = (size_t)rows * (size_t)nsplit * sizeof(float2);
        float2* partial = static_cast<float2*>(workspace);
        bool own = false;
        if (partial == nullptr || workspace_bytes < need) {
            if (!may_allocate) return AK_ERR_NOMEM;
            void* p = nullptr;
            if (cudaMallocAsync(&p, need, st) != cudaSuccess) {
                (void)cudaGetLastError();
                return AK_ERR_NOMEM;
            }
            partial = static_cast<float2*>(p);
            own = true;
        }
        xent_split_kernel<<<dim3((unsigned)nsplit, (unsigned)rows), kThreads, 0, st>>>(
            lg, targets, ignore_index, partial, V, nsplit);
        count_launch();
        cudaError_t e1 = cudaGetLastError();
        xent_merge_kernel<<<(unsigned)((rows + kThreads - 1) / kThreads), kThreads, 0, st>>>(
            lg, targets, ignore_index, partial, loss_rows, rows, V, nsplit);
        count_launch();
        cudaError_t e2 = cudaGetLastError();
        if (own) cudaFreeAsync(partial, st);
        if (e1 != cudaSuccess || e2 != cudaSuccess) return AK_ERR_CUDA;
    }
    if (loss_mean != nullptr) return xent_mean_launch(loss_rows, targets, ignore_index, rows, loss_mean, st);
    return AK_OK;
}

int xent_mean_launch(const float* loss_rows, const int64_t* targets, int64_t ignore_index, int64_t rows,
                     float* loss_mean, cudaStream_t st) {
    xent_mean_kernel<<<1, kMeanThreads, 0, st>>>(loss_rows, targets, ignore_index, rows, loss_mean, nullptr);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

int xent_sum_count_launch(const float* loss_rows, const int64_t* targets, int64_t ignore_index, int64_t rows,
                          double* sum_count, cudaStream_t st) {
    xent_mean_kernel<<<1, kMeanThreads, 0, st>>>(loss_rows, targets, ignore_index, rows, nullptr, sum_count);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

int xent_mean_merge_launch(const double* pairs, int64_t n, float* loss_mean, cudaStream_t st) {
    xent_mean_merge_kernel<<<1, 32, 0, st>>>(pairs, n, loss_mean);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

}  // namespace ak
