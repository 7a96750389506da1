// Shared device helpers for the row-reduction kernels (sm_100a).
// bf16 pack/unpack, streaming 16-byte loads/stores, fixed-order warp/CTA reductions.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "ak.h"

namespace ak {

constexpr int kWarp = 32;
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// ---------------------------------------------------------------- bf16 <-> fp32
// A 32-bit word holds two bf16: element 2i in the low half, 2i+1 in the high half.
__device__ __forceinline__ float bf16lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ float bf16_to_float(uint16_t b) { return __uint_as_float(((uint32_t)b) << 16); }

// Two floats -> packed bf16x2 with round-to-nearest-even (one cvt instruction).
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ uint16_t float_to_bf16(float v) {
    return (uint16_t)(pack_bf16x2(v, 0.0f) & 0xffffu);
}

// Packed bf16x2 max (exact; returns the non-NaN operand when one side is NaN).
__device__ __forceinline__ uint32_t bf16x2_max(uint32_t a, uint32_t b) {
    uint32_t r;
    asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// ---------------------------------------------------------------- packed f32x2 arithmetic
// sm_100 executes two fp32 operations per instruction on register pairs: half the issue
// slots (and the energy that goes with them) for the conversions' consumers.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// the two bf16 of a 32-bit word as a packed float pair (element 2i low, 2i+1 high)
__device__ __forceinline__ f32x2 widen2(uint32_t u) { return pack2(bf16lo(u), bf16hi(u)); }

// ---------------------------------------------------------------- element types
// The kernels are written once over 16-byte vectors and take the element type as a template
// parameter (an ak_dtype value): bf16 and fp16 put 8 elements in a vector (pairs packed in
// 32-bit words, element 2i in the low half), fp32 puts 4.  Elem<DT> holds what differs for the
// 16-bit types: widening (exact), rounding (nearest-even), the packed max and the packed -inf.
template <int DT> struct Elem;
template <> struct Elem<AK_DTYPE_BF16> {
    static constexpr int kBytes = 2, kPerVec = 8;
    static constexpr uint32_t kNegInf2 = 0xFF80FF80u;
    static constexpr uint16_t kNegInf = 0xFF80;
    static __device__ __forceinline__ float lo(uint32_t u) { return bf16lo(u); }
    static __device__ __forceinline__ float hi(uint32_t u) { return bf16hi(u); }
    static __device__ __forceinline__ float to_float(uint16_t b) { return bf16_to_float(b); }
    static __device__ __forceinline__ uint32_t pack(float l, float h) { return pack_bf16x2(l, h); }
    static __device__ __forceinline__ uint16_t from_float(float v) { return float_to_bf16(v); }
    static __device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) { return bf16x2_max(a, b); }
    static __device__ __forceinline__ uint32_t max2_nan(uint32_t a, uint32_t b) {
        uint32_t r;
        asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ float fma_h(uint16_t a, uint16_t b, float c) {  // a*b exact, + c, one rounding
        float d;
        asm("fma.rn.f32.bf16 %0, %1, %2, %3;" : "=f"(d) : "h"(a), "h"(b), "f"(c));
        return d;
    }
};
template <> struct Elem<AK_DTYPE_F16> {
    static constexpr int kBytes = 2, kPerVec = 8;
    static constexpr uint32_t kNegInf2 = 0xFC00FC00u;
    static constexpr uint16_t kNegInf = 0xFC00;
    static __device__ __forceinline__ float to_float(uint16_t b) {
        float f;
        asm("cvt.f32.f16 %0, %1;" : "=f"(f) : "h"(b));
        return f;
    }
    static __device__ __forceinline__ float lo(uint32_t u) { return to_float((uint16_t)(u & 0xffffu)); }
    static __device__ __forceinline__ float hi(uint32_t u) { return to_float((uint16_t)(u >> 16)); }
    static __device__ __forceinline__ uint32_t pack(float l, float h) {
        uint32_t r;
        asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(h), "f"(l));
        return r;
    }
    static __device__ __forceinline__ uint16_t from_float(float v) {
        uint16_t r;
        asm("cvt.rn.f16.f32 %0, %1;" : "=h"(r) : "f"(v));
        return r;
    }
    static __device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
        uint32_t r;
        asm("max.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ uint32_t max2_nan(uint32_t a, uint32_t b) {
        uint32_t r;
        asm("max.NaN.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ float fma_h(uint16_t a, uint16_t b, float c) {  // 11-bit x 11-bit: exact product
        float d;
        asm("fma.rn.f32.f16 %0, %1, %2, %3;" : "=f"(d) : "h"(a), "h"(b), "f"(c));
        return d;
    }
};
template <> struct Elem<AK_DTYPE_F32> {
    static constexpr int kBytes = 4, kPerVec = 4;
};
template <int DT>
__device__ __forceinline__ f32x2 widen2_t(uint32_t u) { return pack2(Elem<DT>::lo(u), Elem<DT>::hi(u)); }

// ---------------------------------------------------------------- memory
// Activations are touched exactly once: streaming (evict-first) loads and stores keep
// them from displacing the reusable weight vector in L2/L1.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) { __stcs(p, v); }
__device__ __forceinline__ uint16_t ld_stream_u16(const uint16_t* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream_u16(uint16_t* p, uint16_t v) { __stcs(p, v); }

// Ask for the 128-byte line at p to be brought into L2.  No data is returned and nothing is
// observed, so it may be issued where a load may not (before griddepcontrol.wait).
__device__ __forceinline__ void prefetch_l2(const void* p) { asm volatile("prefetch.global.L2 [%0];" ::"l"(p)); }

// blockIdx.x through an opaque read: the compiler cannot merge it with an earlier use of
// blockIdx.x, so values derived from the earlier one need not live across the code in between.
__device__ __forceinline__ unsigned cta_id_x() {
    unsigned r;
    asm volatile("mov.u32 %0, %%ctaid.x;" : "=r"(r));
    return r;
}

// exp2 on the SFU (max relative error 2^-22; ex2(-inf) = 0, ex2(NaN) = NaN).
__device__ __forceinline__ float fast_exp2(float t) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(t));
    return r;
}

// ---------------------------------------------------------------- reductions
// XOR butterflies: fp add / max are commutative, so at every level both partners compute
// the same bits and all lanes end with one identical value; the order of operations is
// fixed by the lane ids, hence run-to-run deterministic.
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// CTA-wide reductions with ONE barrier each.  `slots` points to 2 * 32 floats of shared
// memory; consecutive reductions must alternate `phase` (0/1): a warp can only pass the
// barrier of reduction k+1 after every warp has finished reading the slots of
// reduction k, so set k%2 is free again when reduction k+2 writes it.
template <int THREADS>
__device__ __forceinline__ float cta_sum(float v, float* slots, int phase) {
    constexpr int NW = THREADS / kWarp;
    v = warp_sum(v);
    if constexpr (NW == 1) return v;
    float* s = slots + phase * kWarp;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) s[warp] = v;
    __syncthreads();
    float t = (lane < NW) ? s[lane] : 0.0f;
    return warp_sum(t);
}
template <int THREADS>
__device__ __forceinline__ float cta_max(float v, float* slots, int phase) {
    constexpr int NW = THREADS / kWarp;
    v = warp_max(v);
    if constexpr (NW == 1) return v;
    float* s = slots + phase * kWarp;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) s[warp] = v;
    __syncthreads();
    float t = (lane < NW) ? s[lane] : -INFINITY;
    return warp_max(t);
}

// ---------------------------------------------------------------- bulk (TMA) copies into shared memory
// One elected thread asks the copy engine for a whole contiguous span (a row); the bytes
// land in shared memory without passing through registers and an mbarrier counts them in.
// Source, destination and size must be multiples of 16 bytes.  Every copy has one destination CTA.
__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, int arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(arrivals));
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(smem_dst)),
                 "l"(gmem_src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
// Set when a bounded wait gave up (never expected; a thread that sees it returns early and
// leaves its outputs unwritten rather than spinning).  The library is built without relocatable
// device code, so every translation unit that includes this header has its own copy of the flag;
// each of them that waits on mbarriers exports a reader (AK_DEFINE_WAIT_TIMEOUT_READER) and
// ak_wait_timeouts() adds them up.
static __device__ int g_wait_timeout;
// Host side: this translation unit's flag on the current device (-1 if it cannot be read).
static inline int read_wait_timeout_flag() {
    int v = 0;
    if (cudaMemcpyFromSymbol(&v, g_wait_timeout, sizeof(int)) != cudaSuccess) {
        (void)cudaGetLastError();
        return -1;
    }
    return v;
}
#define AK_DEFINE_WAIT_TIMEOUT_READER(name) \
    int name() { return read_wait_timeout_flag(); }
// Bounded wait for the phase with the given parity.  Returns false after ~2^20 polls.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (int it = 0; it < (1 << 20); ++it) {
        uint32_t ok;
        asm volatile(
            "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
            : "=r"(ok)
            : "r"(smem_addr(bar)), "r"(parity)
            : "memory");
        if (ok) return true;
    }
    atomicExch(&g_wait_timeout, 1);
    return false;
}

// Bring the fully-inside vectors k_lo .. k_hi - 1 of a phase-staged row (16-byte aligned in
// global and in shared memory) into the staging buffer with bulk copies of at most kStageChunk
// bytes, all counted in by one mbarrier.  Every thread of the CTA calls this (it contains a
// barrier); the caller fills the edge vectors, calls __syncthreads and then mbar_wait(bar, 0).
constexpr uint32_t kStageChunk = 32768;
__device__ __forceinline__ void stage_interior_bulk(unsigned char* smem_raw, const uint4* xa, int k_lo, int k_hi,
                                                    uint64_t* bar) {
    if (threadIdx.x == 0) mbar_init(bar, 1);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (k_hi > k_lo) {
            const uint32_t bytes = (uint32_t)(k_hi - k_lo) * 16u;
            mbar_expect_tx(bar, bytes);
            const unsigned char* src = reinterpret_cast<const unsigned char*>(xa + k_lo);
            unsigned char* dst = smem_raw + (size_t)k_lo * 16;
            for (uint32_t off = 0; off < bytes; off += kStageChunk)
                bulk_load(dst + off, src + off, min(kStageChunk, bytes - off), bar);
        } else {
            mbar_arrive(bar);
        }
    }
}

// ---------------------------------------------------------------- thread-block clusters
// A row split over the C CTAs of a cluster (C = 2, 4 or 8): every CTA stages its slice in its own
// shared memory, reduces it, and the per-CTA results meet through distributed shared memory.
// An exchange is a mailbox: `box` (C floats) plus an mbarrier in every CTA, armed once for
// C x 4 bytes.  CTA `rank` posts its value v (uniform over its threads) to slot `rank` of the box
// of EVERY CTA of the cluster with asynchronous remote stores that count their bytes in on the
// RECEIVER's mbarrier; each CTA then waits on its own barrier only.  No cluster-wide barrier or
// fence is on the path (a release / acquire cluster barrier per exchange stalled every warp on
// the fence: about a fifth of the kernel's time).  Every CTA combines box[0 .. C-1] in rank
// order, so all of them hold the same bits.  A mailbox serves one exchange per kernel.
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// The one cluster barrier of these kernels says "every CTA of the cluster runs and has armed its
// mailboxes" (the mbarrier initialisation is published by fence.mbarrier_init.release.cluster in
// mbar_init); it orders no other memory, so the arrival is relaxed, and it is split so that the
// row's load and first pass run between arrival and wait.
__device__ __forceinline__ void cluster_arrive_relaxed() {
    asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.aligned;" ::: "memory"); }
// by one thread, before the CTA's cluster_arrive_relaxed
__device__ __forceinline__ void mailbox_arm(uint64_t* xbar, int C) {
    mbar_init(xbar, 1);
    mbar_expect_tx(xbar, (uint32_t)C * 4u);
}
// by every thread of every CTA of the cluster; returns false if the bounded wait gave up
__device__ __forceinline__ bool mailbox_exchange(float v, float* box, uint64_t* xbar, int C, uint32_t rank) {
    if ((int)threadIdx.x < C) {
        uint32_t rbox, rbar;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbox) : "r"(smem_addr(box + rank)), "r"(threadIdx.x));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(smem_addr(xbar)), "r"(threadIdx.x));
        asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];" ::"r"(rbox),
                     "r"(__float_as_uint(v)), "r"(rbar)
                     : "memory");
    }
    return mbar_wait(xbar, 0);
}
// the same for a pair of values per CTA (`box`: C float2, 8-byte aligned; armed for C x 8 bytes)
__device__ __forceinline__ void mailbox_arm2(uint64_t* xbar, int C) {
    mbar_init(xbar, 1);
    mbar_expect_tx(xbar, (uint32_t)C * 8u);
}
__device__ __forceinline__ bool mailbox_exchange2(float a, float b, float2* box, uint64_t* xbar, int C, uint32_t rank) {
    if ((int)threadIdx.x < C) {
        uint32_t rbox, rbar;
        uint64_t v;
        asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(a), "f"(b));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbox) : "r"(smem_addr(box + rank)), "r"(threadIdx.x));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(smem_addr(xbar)), "r"(threadIdx.x));
        asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.b64 [%0], %1, [%2];" ::"r"(rbox), "l"(v),
                     "r"(rbar)
                     : "memory");
    }
    return mbar_wait(xbar, 0);
}
// One thread starts the bulk copies of a contiguous, 16-byte aligned span into shared memory
// (nothing to copy: a plain arrival, so the wait still completes).  The mbarrier must be
// initialised and that made visible (a CTA barrier) before.
__device__ __forceinline__ void bulk_load_span(unsigned char* smem_dst, const void* gmem_src, uint32_t bytes, uint64_t* bar) {
    if (bytes == 0) {
        mbar_arrive(bar);
        return;
    }
    mbar_expect_tx(bar, bytes);
    const unsigned char* src = static_cast<const unsigned char*>(gmem_src);
    for (uint32_t off = 0; off < bytes; off += kStageChunk) bulk_load(smem_dst + off, src + off, min(kStageChunk, bytes - off), bar);
}
constexpr int kMaxCluster = 8;   // portable cluster size limit

// Largest row (bytes) the shared-memory-staged kernels accept: 224 KiB of dynamic shared
// memory out of the 227 KiB a CTA may own (a few hundred bytes stay static).
constexpr int kMaxRowSmemBytes = 224 * 1024;

// ---------------------------------------------------------------- host-side plumbing
// Launch bookkeeping shared by the translation units (defined in ak_api.cu).
void count_launch(int n = 1);
// cudaMallocAsync from the library's own pool (free with cudaFreeAsync on the same stream)
cudaError_t scratch_alloc(void** p, size_t bytes, cudaStream_t st);
// CTAs per row of the cluster layout for aligned rows of `row_bytes` bytes: 1 = keep one CTA per
// row (or the row does not fit eight slices); otherwise 2, 4 or 8.  Pure function of its arguments.
int cluster_ctas(int64_t rows, int64_t row_bytes, int64_t split_from);
// rows longer than 64 KiB are always split (at exactly 64 KiB the one-CTA kernels are as fast or
// faster: softmax 16384 x 32768 317 us against 338 us in clusters of two)
constexpr int64_t kClusterFrom = 65536 + 16;
bool clusters_enabled();   // false when AK_DISABLE_CLUSTERS switches the cluster layouts off
int sm_count();  // SMs of the current device (cached per device)
// per translation unit: has a bounded mbarrier wait of its kernels ever given up on this device?
int rmsnorm_wait_timeouts();
int softmax_wait_timeouts();
int layernorm_wait_timeouts();
// Per-device memos, keyed by kernel (a process may drive several GPUs, and function attributes
// and occupancy belong to the device that is current at the call):
//   dyn_smem_configured  cudaFuncAttributeMaxDynamicSharedMemorySize = kMaxRowSmemBytes set once
//   resident_ctas_of     CTAs of this kernel the whole device holds at once (>= 1 per SM)
bool dyn_smem_configured(const void* kernel);
int resident_ctas_of(const void* kernel, int threads, size_t dyn_smem);
template <typename... A>
inline bool allow_big_smem(void (*kernel)(A...)) { return dyn_smem_configured(reinterpret_cast<const void*>(kernel)); }
template <typename... A>
inline int resident_ctas(void (*kernel)(A...), int threads, size_t dyn_smem) {
    return resident_ctas_of(reinterpret_cast<const void*>(kernel), threads, dyn_smem);
}
// CTAs of the first wave that prefetch before the wait (see pdl_prologue); 0 switches it off
bool first_wave_prefetch_enabled();
template <typename... A>
inline int first_wave_ctas(void (*kernel)(A...), int threads, size_t dyn_smem) {
    return first_wave_prefetch_enabled() ? resident_ctas(kernel, threads, dyn_smem) : 0;
}

// Per-op host dispatchers (each defined next to its kernels).  All arguments have been
// validated; `path` is a concrete path id or AUTO.  They return an ak_status.
int rmsnorm_dispatch(const void* x, const void* w, void* y, int64_t rows, int64_t D, float eps,
                     cudaStream_t st, int path, int dtype = AK_DTYPE_BF16);
int softmax_dispatch(const void* x, void* y, int64_t rows, int64_t D, cudaStream_t st, int path,
                     int dtype = AK_DTYPE_BF16);
int xent_dispatch(const void* logits, const int64_t* targets, int64_t ignore_index,
                  float* loss_rows, float* loss_mean, int64_t rows, int64_t V,
                  void* workspace, size_t workspace_bytes, bool may_allocate,
                  cudaStream_t st, int path, int nsplit, int dtype = AK_DTYPE_BF16);
// Fixed-order fp64 mean of loss_rows over rows whose target != ignore_index (one small launch).
// dependent: launch it as a programmatic dependent of the kernel enqueued just before, which must
// be one that lets its dependents in only after its own wait (the mean kernel reads the targets
// before it waits).
int xent_mean_launch(const float* loss_rows, const int64_t* targets, int64_t ignore_index, int64_t rows,
                     float* loss_mean, cudaStream_t st, bool dependent = false);
int xent_sum_count_launch(const float* loss_rows, const int64_t* targets, int64_t ignore_index, int64_t rows,
                          double* sum_count, cudaStream_t st);
// Vocabulary-parallel cross-entropy (defined in xent_vp.cu).
int xent_vp_partial_launch(const void* logits, const int64_t* targets, int64_t ignore_index, int64_t vocab_start,
                           int64_t V_total, void* part, int64_t rows, int64_t V_local, int nsplit, int dtype,
                           cudaStream_t st);
int xent_vp_merge_launch(const void* parts, int nranks, int nsplit, const int64_t* targets, int64_t ignore_index,
                         int64_t V_total, float* loss_rows, float* loss_mean, int64_t rows, cudaStream_t st);
int xent_mean_merge_launch(const double* pairs, int64_t n, float* loss_mean, cudaStream_t st);
int layernorm_dispatch(const void* x, const void* gamma, const void* beta, void* y, int64_t rows, int64_t D,
                       float eps, cudaStream_t st, int path, int dtype = AK_DTYPE_BF16);
int layernorm_choose(int64_t rows, int64_t D, bool aligned16, int dtype = AK_DTYPE_BF16);
int rope_dispatch(const void* x, void* y, int64_t n_seq, int64_t S, int64_t Dh, float base, int64_t pos_offset,
                  int dtype, cudaStream_t st);
int rowsum_dispatch(const void* x, float* out, int64_t rows, int64_t D, cudaStream_t st, int dtype = AK_DTYPE_BF16);
int rmsnorm_choose(int64_t rows, int64_t D, bool aligned16, int dtype = AK_DTYPE_BF16);
int softmax_choose(int64_t rows, int64_t D, bool aligned16, int dtype = AK_DTYPE_BF16);
int xent_choose(int64_t rows, int64_t V, int* nsplit);

// Argument checks shared by every cross-entropy entry point (pointers, shape limits, alignment).
int validate_xent(const void* logits, const int64_t* targets, float* loss_rows, float* loss_mean,
                  int64_t rows, int64_t V, size_t esize = 2);

inline int dtype_bytes(int dtype) { return dtype == AK_DTYPE_F32 ? 4 : 2; }
inline bool is_aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// Programmatic dependent launch: let the next kernel in the stream be scheduled while this
// grid is still running (it waits for our completion with pdl_wait before it reads).
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Prologue of a kernel launched as a programmatic dependent of whatever precedes it in the stream.
// Its CTAs may become resident while the grids before it still drain; nothing may be read or
// written until griddepcontrol.wait returns.  The CTAs of the first wave (blockIdx.x < first_wave
// = as many CTAs as the device holds at once) use that time to ask for the first 128 bytes per
// thread of their input span to be brought into L2: a prefetch reads nothing architecturally.
// Later CTAs start on a busy machine and skip it.  After the wait the kernel lets its own
// dependents in at once (they wait for this grid's completion in turn).
__device__ __forceinline__ void pdl_prologue(const void* span, int64_t span_bytes, int first_wave) {
    if ((int)blockIdx.x < first_wave) {
        const int64_t off = (int64_t)threadIdx.x * 128;
        if (off < span_bytes) prefetch_l2(static_cast<const char*>(span) + off);
    }
    pdl_wait();
    pdl_launch_dependents();
}

// ------------------------------------------------------------------ pre-shifted parameter vectors
// Rows of 2-byte elements that do not start on a 16-byte boundary are processed in their own
// phase (phase p = the row start's element offset inside its 16-byte group): vector k of such a
// row holds elements 8k - p .. 8k - p + 7.  Per-column parameters (the RMSNorm weight, the
// LayerNorm gamma and beta) are needed in the same shifted layout.  Rather than assembling them
// from 4-byte loads and funnel shifts for every output vector of every row, this kernel writes
// all eight shifts once per launch:
//     tab[(o * 8 + p) * nvp + k] = elements 8k - p .. 8k - p + 7 of parameter vector o
// (zero outside [0, D)), nvp = (D + 14) / 8 vectors; the row kernels, launched as programmatic
// dependents, read them with one 16-byte load each after pdl_wait.  p1 may be null (one vector).
constexpr int kShiftThreads = 128;
template <int UNUSED = 0>
__global__ void __launch_bounds__(kShiftThreads)
shift_params_kernel(const uint16_t* __restrict__ p0, const uint16_t* __restrict__ p1, int64_t D, int nvp,
                    uint4* __restrict__ tab) {
    pdl_launch_dependents();
    const int idx = blockIdx.x * kShiftThreads + threadIdx.x;
    const int total = (p1 ? 16 : 8) * nvp;
    if (idx >= total) return;
    const int k = idx % nvp;
    const int p = (idx / nvp) & 7;
    const uint16_t* src = (idx >= 8 * nvp) ? p1 : p0;
    uint32_t w[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
        const int64_t j = (int64_t)k * 8 - p + 2 * h;
        const uint32_t lo = (j >= 0 && j < D) ? (uint32_t)__ldg(src + j) : 0u;
        const uint32_t hi = (j + 1 >= 0 && j + 1 < D) ? (uint32_t)__ldg(src + j + 1) : 0u;
        w[h] = lo | (hi << 16);
    }
    tab[idx] = make_uint4(w[0], w[1], w[2], w[3]);
}

// Launch `kernel` in thread-block clusters of C CTAs along x (grid a multiple of C).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_cluster(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, int C,
                                  cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Both: clusters of C CTAs, launched as a programmatic dependent of the work before it.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_cluster_dependent(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem, int C,
                                            cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)C;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// Launch `kernel` as a programmatic dependent of the work before it in the stream.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

}  // namespace ak
