// Row-sum reduce (paper Table 3 "reduce"): out[r] = sum_j x[r, j], bf16 / fp16 / fp32 in, fp32
// accumulate and out.  Read-only streaming: one read of every element, 4 bytes per row back.
//
// A group of GROUP threads owns a row.  Rows need no alignment beyond the element's own: a few
// head elements bring the row to a 16-byte boundary, the body is read as 16-byte vectors
// (UNROLL independent loads in flight per thread) and a few tail elements finish it.  Every
// thread keeps eight lane accumulators (16-bit types: fed straight from the packed halves by
// the mixed-precision add; fp32: four of them, one per vector lane); the combine order (lanes
// pairwise, XOR butterfly over the warp, then over the group's warps) is fixed, so results
// are bitwise reproducible.
#include "ak_common.cuh"

namespace ak {
namespace {

template <int DT>
__device__ __forceinline__ float add_h(uint16_t x, float c) {   // x + c, x a 16-bit element (exact operand)
    float d;
    if constexpr (DT == AK_DTYPE_F16) asm("add.rn.f32.f16 %0, %1, %2;" : "=f"(d) : "h"(x), "f"(c));
    else asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(x), "f"(c));
    return d;
}
template <int DT>
__device__ __forceinline__ void acc_pair(uint32_t u, float& a, float& b) {
    uint16_t lo, hi;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(u));
    a = add_h<DT>(lo, a);
    b = add_h<DT>(hi, b);
}
template <int DT>
__device__ __forceinline__ void acc_v(const uint4& v, float (&a)[8]) {
    if constexpr (DT == AK_DTYPE_F32) {
        a[0] += __uint_as_float(v.x);
        a[1] += __uint_as_float(v.y);
        a[2] += __uint_as_float(v.z);
        a[3] += __uint_as_float(v.w);
    } else {
        acc_pair<DT>(v.x, a[0], a[1]);
        acc_pair<DT>(v.y, a[2], a[3]);
        acc_pair<DT>(v.z, a[4], a[5]);
        acc_pair<DT>(v.w, a[6], a[7]);
    }
}
template <int DT> struct RsElem { using type = uint16_t; };
template <> struct RsElem<AK_DTYPE_F32> { using type = float; };
template <int DT>
__device__ __forceinline__ float load_one(const typename RsElem<DT>::type* p) {
    if constexpr (DT == AK_DTYPE_F32) return __ldcs(p); else return Elem<DT>::to_float(ld_stream_u16(p));
}

// Adds the elements of one contiguous span p[0, n) that thread t of a group of GROUP threads
// owns into its lane accumulators: head elements up to the 16-byte boundary, aligned vectors
// (UNROLL in flight), tail elements.
template <int GROUP, int UNROLL, int DT>
__device__ __forceinline__ void span_sum(const typename RsElem<DT>::type* p, int64_t n, int t, float (&a)[8]) {
    constexpr int PV = Elem<DT>::kPerVec, LOG_PV = (PV == 8) ? 3 : 2, LOG_BYTES = (Elem<DT>::kBytes == 2) ? 1 : 2;
    static_assert(GROUP >= PV, "head and tail elements take one thread each");
    const int phase = (int)((reinterpret_cast<uintptr_t>(p) >> LOG_BYTES) & (PV - 1));
    int64_t head = (PV - phase) & (PV - 1);
    if (head > n) head = n;
    const int64_t nbody = (n - head) >> LOG_PV;
    const int64_t tail0 = head + (nbody << LOG_PV);
    const uint4* xb = reinterpret_cast<const uint4*>(p + head);
    int64_t i = t;
    for (; i + (int64_t)(UNROLL - 1) * GROUP < nbody; i += (int64_t)UNROLL * GROUP) {
        uint4 v[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) v[u] = ld_stream(xb + i + (int64_t)u * GROUP);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) acc_v<DT>(v[u], a);
    }
    for (; i < nbody; i += GROUP) acc_v<DT>(ld_stream(xb + i), a);
    if (t < head) a[0] += load_one<DT>(p + t);
    if (tail0 + t < n) a[1] += load_one<DT>(p + tail0 + t);
}

template <int THREADS, int GROUP, int UNROLL, int MINB, int DT>
__global__ void __launch_bounds__(THREADS, MINB)
rowsum_kernel(const typename RsElem<DT>::type* __restrict__ x, float* __restrict__ out, int64_t rows, int64_t D,
              int first_wave) {
    constexpr int GROUPS = THREADS / GROUP;
    constexpr int WARPS_PER_GROUP = GROUP / kWarp;
    static_assert(GROUP % kWarp == 0 && THREADS % GROUP == 0, "groups are whole warps");
    __shared__ float slots[THREADS / kWarp];
    {
        const int64_t r0 = (int64_t)blockIdx.x * GROUPS;
        const int64_t nr = rows - r0 < GROUPS ? rows - r0 : GROUPS;
        pdl_prologue(x + r0 * D, nr * D * (int64_t)sizeof(typename RsElem<DT>::type), first_wave);
    }
    const int g = threadIdx.x / GROUP;
    const int t = threadIdx.x % GROUP;
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * GROUPS + g;
    const bool live = row < rows;

    float a[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
    if (live) span_sum<GROUP, UNROLL, DT>(x + row * D, D, t, a);
    float s = ((a[0] + a[1]) + (a[2] + a[3])) + ((a[4] + a[5]) + (a[6] + a[7]));
    s = warp_sum(s);
    if constexpr (WARPS_PER_GROUP > 1) {
        float* sl = slots + g * WARPS_PER_GROUP;
        if (lane == 0) sl[t >> 5] = s;
        __syncthreads();
        s = warp_sum((lane < WARPS_PER_GROUP) ? sl[lane] : 0.0f);
    }
    if (live && t == 0) out[row] = s;
}

// ------------------------------------------------------------------ few, long rows (a vector sum is rows == 1)
// One CTA per row cannot fill the GPU when there are only a few rows: nsplit CTAs per row each
// sum a slice (boundaries on multiples of 8 elements) and write a partial; a second kernel,
// launched as a programmatic dependent, adds each row's partials in a fixed order (thread t takes
// partials t, t + 256, ... in turn, then the usual tree).  grid = (nsplit, rows).
constexpr int kRsSplitThreads = 256;

template <int UNROLL, int DT>
__global__ void __launch_bounds__(kRsSplitThreads)
rowsum_split_kernel(const typename RsElem<DT>::type* __restrict__ x, float* __restrict__ partial, int64_t D, int nsplit) {
    __shared__ float slots[2 * kWarp];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int64_t row = blockIdx.y;
    const int sp = blockIdx.x;
    const int64_t groups = (D + 7) >> 3;
    const int64_t begin = ((groups * sp) / nsplit) << 3;
    int64_t end = ((groups * (sp + 1)) / nsplit) << 3;
    if (end > D) end = D;
    float a[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
    if (end > begin) span_sum<kRsSplitThreads, UNROLL, DT>(x + row * D + begin, end - begin, (int)threadIdx.x, a);
    float s = ((a[0] + a[1]) + (a[2] + a[3])) + ((a[4] + a[5]) + (a[6] + a[7]));
    s = cta_sum<kRsSplitThreads>(s, slots, 0);
    if (threadIdx.x == 0) partial[row * nsplit + sp] = s;
}

__global__ void __launch_bounds__(kRsSplitThreads)
rowsum_finish_kernel(const float* __restrict__ partial, float* __restrict__ out, int nsplit) {
    __shared__ float slots[2 * kWarp];
    asm volatile("griddepcontrol.wait;" ::: "memory");   // the partials of the whole grid before are visible
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int64_t row = blockIdx.x;
    float s = 0.0f;
    for (int i = threadIdx.x; i < nsplit; i += kRsSplitThreads) s += __ldcg(partial + row * nsplit + i);
    s = cta_sum<kRsSplitThreads>(s, slots, 0);
    if (threadIdx.x == 0) out[row] = s;
}

// Split count: a pure function of (rows, D) and the device's SM count.  Enough CTAs for about one wave, more for very
// long rows (slices of about 64K elements), slices of at least 8192 elements, at most 8192 of them.
int rowsum_nsplit(int64_t rows, int64_t D) {
    const int64_t kTargetCtas = (int64_t)sm_count() * 8;   // 1184 on a full B200
    constexpr int64_t kMinSlice = 8192;
    if (rows <= 0 || rows >= kTargetCtas / 2) return 1;
    int64_t want = (kTargetCtas + rows - 1) / rows;
    if (want < D / 65536) want = D / 65536;
    const int64_t cap = D / kMinSlice;
    if (want > cap) want = cap;
    if (want > 8192) want = 8192;
    return want > 1 ? (int)want : 1;
}

template <int DT>
int launch_split(const void* x, float* out, int64_t rows, int64_t D, int nsplit, cudaStream_t st) {
    if (rows > 65535) return AK_ERR_SHAPE;   // grid.y; the split is only chosen for a few rows
    float* partial = nullptr;
    if (scratch_alloc(reinterpret_cast<void**>(&partial), (size_t)rows * nsplit * sizeof(float), st) != cudaSuccess) {
        (void)cudaGetLastError();
        return AK_ERR_NOMEM;
    }
    rowsum_split_kernel<4, DT><<<dim3((unsigned)nsplit, (unsigned)rows), kRsSplitThreads, 0, st>>>(
        static_cast<const typename RsElem<DT>::type*>(x), partial, D, nsplit);
    count_launch();
    int status = cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
    if (status == AK_OK) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)rows);
        cfg.blockDim = dim3(kRsSplitThreads);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const float* cpartial = partial;
        if (cudaLaunchKernelEx(&cfg, rowsum_finish_kernel, cpartial, out, nsplit) != cudaSuccess) status = AK_ERR_CUDA;
        count_launch();
    }
    cudaFreeAsync(partial, st);
    return status;
}

template <int DT, int THREADS, int GROUP, int UNROLL, int MINB>
int launch(const void* x, float* out, int64_t rows, int64_t D, cudaStream_t st) {
    constexpr int GROUPS = THREADS / GROUP;
    const int64_t grid = (rows + GROUPS - 1) / GROUPS;
    if (grid > 2147483647LL) return AK_ERR_SHAPE;
    auto kernel = rowsum_kernel<THREADS, GROUP, UNROLL, MINB, DT>;
    const cudaError_t e = launch_dependent(kernel, dim3((unsigned)grid), dim3(THREADS), 0, st,
                                           static_cast<const typename RsElem<DT>::type*>(x), out, rows, D,
                                           first_wave_ctas(kernel, THREADS, 0));
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

template <int DT>
int dispatch_t(const void* x, float* out, int64_t rows, int64_t D, cudaStream_t st) {
    const int64_t row_bytes = D * Elem<DT>::kBytes;
    const int nsplit = rowsum_nsplit(rows, D);
    if (nsplit > 1) return launch_split<DT>(x, out, rows, D, nsplit, st);
    if (row_bytes <= 2048) return launch<DT, 256, 32, 4, 4>(x, out, rows, D, st);    // a warp per row
    if (row_bytes <= 32768) return launch<DT, 128, 128, 4, 8>(x, out, rows, D, st);  // a 128-thread CTA per row
    return launch<DT, 256, 256, 8, 4>(x, out, rows, D, st);
}

}  // namespace

int rowsum_dispatch(const void* x, float* out, int64_t rows, int64_t D, cudaStream_t st, int dtype) {
    switch (dtype) {
        case AK_DTYPE_BF16: return dispatch_t<AK_DTYPE_BF16>(x, out, rows, D, st);
        case AK_DTYPE_F16: return dispatch_t<AK_DTYPE_F16>(x, out, rows, D, st);
        case AK_DTYPE_F32: return dispatch_t<AK_DTYPE_F32>(x, out, rows, D, st);
        default: return AK_ERR_ARG;
    }
}

}  // namespace ak
