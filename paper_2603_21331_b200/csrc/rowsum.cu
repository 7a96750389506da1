// Row-sum reduce (paper Table 3 "reduce"): out[r] = sum_j x[r, j], bf16 in, fp32 accumulate
// and out.  Read-only streaming: 2 bytes per element from HBM, 4 bytes per row back.
//
// A group of GROUP threads owns a row.  Rows need no alignment beyond 2 bytes: up to 7 head
// elements bring the row to a 16-byte boundary, the body is read as 16-byte vectors (UNROLL
// independent loads in flight per thread) and up to 7 tail elements finish it.  Every thread
// keeps eight lane accumulators fed straight from the bf16 halves by the mixed-precision add;
// the combine order (lanes pairwise, XOR butterfly over the warp, then over the group's warps)
// is fixed, so results are bitwise reproducible.
#include "ak_common.cuh"

namespace ak {
namespace {

__device__ __forceinline__ float add_bf16(uint16_t x, float c) {
    float d;
    asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(x), "f"(c));
    return d;
}
__device__ __forceinline__ void acc_pair(uint32_t u, float& a, float& b) {
    uint16_t lo, hi;
    asm("mov.b32 {%0, %1}, %2;" : "=h"(lo), "=h"(hi) : "r"(u));
    a = add_bf16(lo, a);
    b = add_bf16(hi, b);
}
__device__ __forceinline__ void acc8(const uint4& v, float (&a)[8]) {
    acc_pair(v.x, a[0], a[1]);
    acc_pair(v.y, a[2], a[3]);
    acc_pair(v.z, a[4], a[5]);
    acc_pair(v.w, a[6], a[7]);
}

template <int THREADS, int GROUP, int UNROLL, int MINB>
__global__ void __launch_bounds__(THREADS, MINB)
rowsum_kernel(const uint16_t* __restrict__ x, float* __restrict__ out, int64_t rows, int64_t D) {
    constexpr int GROUPS = THREADS / GROUP;
    constexpr int WARPS_PER_GROUP = GROUP / kWarp;
    static_assert(GROUP % kWarp == 0 && THREADS % GROUP == 0, "groups are whole warps");
    __shared__ float slots[THREADS / kWarp];
    const int g = threadIdx.x / GROUP;
    const int t = threadIdx.x % GROUP;
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * GROUPS + g;
    const bool live = row < rows;

    float a[8] = {0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f, 0.0f};
    if (live) {
        const uint16_t* xr = x + row * D;
        const int phase = (int)((reinterpret_cast<uintptr_t>(xr) >> 1) & 7);
        int64_t head = (8 - phase) & 7;
        if (head > D) head = D;
        const int64_t nbody = (D - head) >> 3;
        const int64_t tail0 = head + (nbody << 3);
        const uint4* xb = reinterpret_cast<const uint4*>(xr + head);
        int64_t i = t;
        for (; i + (int64_t)(UNROLL - 1) * GROUP < nbody; i += (int64_t)UNROLL * GROUP) {
            uint4 v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) v[u] = ld_stream(xb + i + (int64_t)u * GROUP);
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) acc8(v[u], a);
        }
        for (; i < nbody; i += GROUP) acc8(ld_stream(xb + i), a);
        if (t < head) a[0] = add_bf16(ld_stream_u16(xr + t), a[0]);
        if (tail0 + t < D) a[1] = add_bf16(ld_stream_u16(xr + tail0 + t), a[1]);
    }
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

template <int THREADS, int GROUP, int UNROLL, int MINB>
int launch(const void* x, float* out, int64_t rows, int64_t D, cudaStream_t st) {
    constexpr int GROUPS = THREADS / GROUP;
    const int64_t grid = (rows + GROUPS - 1) / GROUPS;
    if (grid > 2147483647LL) return AK_ERR_SHAPE;
    rowsum_kernel<THREADS, GROUP, UNROLL, MINB><<<(unsigned)grid, THREADS, 0, st>>>(
        static_cast<const uint16_t*>(x), out, rows, D);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

}  // namespace

int rowsum_dispatch(const void* x, float* out, int64_t rows, int64_t D, cudaStream_t st) {
    if (D <= 1024) return launch<256, 32, 4, 4>(x, out, rows, D, st);    // a warp per row
    if (D <= 16384) return launch<128, 128, 4, 8>(x, out, rows, D, st);  // a 128-thread CTA per row
    return launch<256, 256, 8, 4>(x, out, rows, D, st);
}

}  // namespace ak
