// Vocabulary-parallel cross-entropy: the logits' last dimension is sharded over ranks
// (tensor parallelism), rank k holding columns [vocab_start_k, vocab_start_k + V_local_k).
//
//   phase 1 (every rank, its own shard)  ak_xent_vp_partial: per row, nsplit slices' online
//           (max, sum-exp) pairs and the target logit if this shard owns the target column
//   exchange                             one all-gather of rows * (nsplit + 1) * 8 bytes per rank
//   phase 2 (every rank, identical bits) ak_xent_vp_merge: merge all ranks' pairs in
//           (rank, slice) order, add the owner's target logit, then the fixed-order mean
//
// This is the split-row layout of the single-GPU kernel with the slices living on different
// GPUs: the same slice_lse, the same merge arithmetic, the same loss assembly.  The exchange
// is 16 bytes per row against 2 * V_local bytes per row of local streaming (1 : 16000 at
// V_local = 128k), so it is latency-bound and there is no tile whose transfer could overlap
// the math; it goes through the communication library as one small collective.
#include "xent_kernels.cuh"

namespace ak {
namespace {

// grid = (rows, nsplit).  part[row * (nsplit + 1) + s] = (M, S) of slice s of this shard;
// part[row * (nsplit + 1) + nsplit] = (x_t, 1) if the shard owns column t, else (0, 0).
// Rows whose target is ignore_index or outside [0, V_total) are not read and their entries
// are not written (the merge never looks at them).
template <int UNROLL, int POLY, int MINB, int T, int DT, bool ONE_SLICE>
__global__ void __launch_bounds__(T, MINB)
xent_vp_partial_kernel(const typename XElem<DT>::type* __restrict__ logits, const int64_t* __restrict__ targets,
                       int64_t ignore_index, int64_t vocab_start, int64_t V_total, float2* __restrict__ part,
                       int64_t V_local, int nsplit, int first_wave) {
    __shared__ float slots[2 * kWarp];
    // launched as a programmatic dependent; with one slice per row the first wave prefetches the
    // head of its rows while the grids before drain (first_wave is 0 for split rows)
    pdl_prologue(logits + (int64_t)blockIdx.x * V_local, V_local * (int64_t)sizeof(typename XElem<DT>::type), first_wave);
    const int64_t row = cta_id_x();
    const int sp = blockIdx.y;
    const int64_t t = targets[row];
    if (t != ignore_index && t >= 0 && t < V_total) {   // (this form, not an early return, keeps the compiler from spilling)
        const typename XElem<DT>::type* xr = logits + row * V_local;
        int64_t begin = 0, end = V_local;
        if constexpr (!ONE_SLICE) {
            const int64_t groups = (V_local + 7) >> 3;
            begin = ((groups * sp) / nsplit) << 3;
            end = ((groups * (sp + 1)) / nsplit) << 3;
            if (end > V_local) end = V_local;
        }
        // slice 0 of the shard that owns the target's column fetches the target logit
        const int64_t tl = t - vocab_start;
        float M, S, xt = 0.0f;
        row_lse<UNROLL, POLY, T, DT, ONE_SLICE>(xr, begin, end, slots, M, S, [&] {   // (one slice: the pointer-loop form, which fits 64 registers here without a spill slot)
            if (sp == 0 && tl >= 0 && tl < V_local && threadIdx.x == 0) xt = xread<DT>(xr + tl);
        });
        if (threadIdx.x == 0) {
            // (row, slice and ownership are worked out again here rather than kept in registers
            // across the loop: at 64 registers the compiler would spill them)
            const int64_t row2 = cta_id_x();
            const int64_t tl2 = targets[row2] - vocab_start;
            float2* pr = part + row2 * (nsplit + 1);
            pr[sp] = make_float2(M, S);
            if (sp == 0) pr[nsplit] = (tl2 >= 0 && tl2 < V_local) ? make_float2(xt, 1.0f) : make_float2(0.0f, 0.0f);
        }
    }
}

// One thread per row: all ranks' slices in (rank, slice) order, exactly the arithmetic of the
// single-GPU split merge.  parts = [nranks][rows][nsplit + 1] pairs.
constexpr int kVpMergeThreads = 128;
constexpr int kVpBatch = 16;   // pairs (and ranks) per row held in registers by the merge
// the loss of row r from all ranks' pairs, in (rank, slice) order
__device__ __forceinline__ float vp_merge_row(const float2* __restrict__ parts, int nranks, int nsplit,
                                              const int64_t* __restrict__ targets, int64_t ignore_index, int64_t V_total,
                                              int64_t rows, int64_t r) {
    const int64_t t = targets[r];
    float loss;
    if (t == ignore_index) {
        loss = 0.0f;
    } else if (t < 0 || t >= V_total) {
        loss = __int_as_float(0x7fc00000);
    } else {
        const int64_t stride = (int64_t)rows * (nsplit + 1);
        const float2* pr = parts + r * (nsplit + 1);
        float M = -INFINITY, S = 0.0f, xt = 0.0f, owners = 0.0f;
        const int n = nranks * nsplit;
        if (n <= kVpBatch && nranks <= kVpBatch) {
            // the usual case (up to 16 pairs per row): every load of the row is issued before the
            // first use, so the thread waits for memory once, not once per pair; same order of
            // the arithmetic as the loops below
            float2 p[kVpBatch], own[kVpBatch];
#pragma unroll
            for (int q = 0; q < kVpBatch; ++q) {
                const int k = q / nsplit, i = q - k * nsplit;
                if (q < n) p[q] = __ldg(pr + k * stride + i);
                if (q < nranks) own[q] = __ldg(pr + q * stride + nsplit);
            }
#pragma unroll
            for (int q = 0; q < kVpBatch; ++q)
                if (q < n) M = fmaxf(M, p[q].x);
            const float MF = fmaxf(M * kLog2e, kFloor2);
#pragma unroll
            for (int q = 0; q < kVpBatch; ++q)
                if (q < n) S += p[q].y * fast_exp2(fmaxf(p[q].x * kLog2e, kFloor2) - MF);
#pragma unroll
            for (int q = 0; q < kVpBatch; ++q)
                if (q < nranks && own[q].y != 0.0f) { xt = own[q].x; owners += 1.0f; }
        } else {
            for (int k = 0; k < nranks; ++k)
                for (int i = 0; i < nsplit; ++i) M = fmaxf(M, __ldg(pr + k * stride + i).x);
            const float MF = fmaxf(M * kLog2e, kFloor2);
            for (int k = 0; k < nranks; ++k) {
                for (int i = 0; i < nsplit; ++i) {
                    const float2 ps = __ldg(pr + k * stride + i);
                    S += ps.y * fast_exp2(fmaxf(ps.x * kLog2e, kFloor2) - MF);
                }
                const float2 own = __ldg(pr + k * stride + nsplit);
                if (own.y != 0.0f) { xt = own.x; owners += 1.0f; }
            }
        }
        // exactly one shard owns a valid target when the shards tile [0, V_total)
        loss = (owners == 1.0f) ? finish_loss(M, S, xt) : __int_as_float(0x7fc00000);
    }
    return loss;
}

__global__ void __launch_bounds__(kVpMergeThreads)
xent_vp_merge_kernel(const float2* __restrict__ parts, int nranks, int nsplit, const int64_t* __restrict__ targets,
                     int64_t ignore_index, int64_t V_total, float* __restrict__ loss_rows, int64_t rows) {
    pdl_wait();                 // launched as a programmatic dependent of whatever precedes it
    pdl_launch_dependents();    // the mean kernel may take a slot now (it reads the targets, which are final)
    const int64_t r = (int64_t)blockIdx.x * kVpMergeThreads + threadIdx.x;
    if (r >= rows) return;
    loss_rows[r] = vp_merge_row(parts, nranks, nsplit, targets, ignore_index, V_total, rows, r);
}

// Merge and mean in ONE launch for batches of up to kVpFusedMaxRows rows (4096 x 16032 as one of eight
// ranks: 31.5 -> 27.6 us for partial + merge + mean; 1000 rows 14.4 -> 11.6 us; at 16384 rows the eight CTAs
// are too few and the two kernels are 3 us faster): a single cluster of eight
// CTAs of 512 threads.  The 1024 threads t < 128 of the eight CTAs are the 1024 virtual threads of
// the fixed-order mean (xent_finish_kernel): virtual thread v = 128 * rank + t owns rows v, v + 1024,
// v + 2048, ...  First every thread merges rows (group q = threadIdx.x / 128 of a CTA takes the rows
// v + 1024 * (q + 4 j)), writes them and leaves them in shared memory; then the threads of group 0 add
// their rows in increasing order in fp64, the four warps reduce as the finish kernel's warps do,
// and the 32 warp sums and the counts meet in rank 0 through its mailbox (asynchronous remote
// stores that count in on rank 0's mbarrier; the one cluster barrier says that it is armed), where
// warp 0 adds them in warp order.  Same losses and the same mean, bit for bit, as the two kernels.
constexpr int kVpFusedThreads = 512, kVpFusedCtas = 8, kVpFusedMaxRows = 8192;
constexpr int kVpFusedK = kVpFusedMaxRows / 1024;   // rows per virtual thread at most

__global__ void __launch_bounds__(kVpFusedThreads, 1)
xent_vp_merge_mean_kernel(const float2* __restrict__ parts, int nranks, int nsplit, const int64_t* __restrict__ targets,
                          int64_t ignore_index, int64_t V_total, float* __restrict__ loss_rows, float* __restrict__ out_mean,
                          int64_t rows) {
    __shared__ float sloss[kVpFusedK][128];
    __shared__ unsigned char scounted[kVpFusedK][128];
    __shared__ __align__(8) double box[32];        // rank 0: the 32 warp sums of the cluster
    __shared__ __align__(8) long long cnt[kVpFusedCtas];
    __shared__ uint64_t xbar;
    const uint32_t c = cluster_rank();
    const int t = threadIdx.x & 127, q = threadIdx.x >> 7;
    const int lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(&xbar, 1);
        mbar_expect_tx(&xbar, (uint32_t)kVpFusedCtas * (4u * 8u + 8u));
    }
    __syncthreads();
    cluster_arrive_relaxed();
    pdl_wait();                 // the partial buffers (and whatever else precedes) are complete
    pdl_launch_dependents();
    const int64_t v = (int64_t)c * 128 + t;
    for (int k = q; k < kVpFusedK; k += 4) {
        const int64_t r = (int64_t)k * 1024 + v;
        float loss = 0.0f;
        bool counted = false;
        if (r < rows) {
            loss = vp_merge_row(parts, nranks, nsplit, targets, ignore_index, V_total, rows, r);
            loss_rows[r] = loss;
            counted = targets[r] != ignore_index;
        }
        sloss[k][t] = loss;
        scounted[k][t] = counted ? 1 : 0;
    }
    __syncthreads();
    double acc = 0.0;
    long long n = 0;
    if (q == 0) {
#pragma unroll
        for (int k = 0; k < kVpFusedK; ++k)
            if (scounted[k][t]) {
                acc += (double)sloss[k][t];
                ++n;
            }
        acc = warp_sum_f64(acc);
        n = __reduce_add_sync(0xffffffffu, (int)n);
    }
    cluster_wait();   // rank 0 runs and its mailbox is armed
    // lane 0 of the four warps of group 0 posts its warp sum; thread 0 posts the CTA's count
    __shared__ long long ncta[4];
    if (q == 0 && lane == 0) ncta[t >> 5] = n;
    __syncthreads();
    if (q == 0 && lane == 0) {
        uint32_t rbox, rbar;
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbox) : "r"(smem_addr(box + 4 * c + (t >> 5))), "r"(0));
        asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rbar) : "r"(smem_addr(&xbar)), "r"(0));
        asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.b64 [%0], %1, [%2];" ::"r"(rbox),
                     "l"(__double_as_longlong(acc)), "r"(rbar)
                     : "memory");
        if (t == 0) {
            const long long nc = ncta[0] + ncta[1] + ncta[2] + ncta[3];
            uint32_t rcnt;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(rcnt) : "r"(smem_addr(cnt + c)), "r"(0));
            asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.b64 [%0], %1, [%2];" ::"r"(rcnt), "l"(nc),
                         "r"(rbar)
                         : "memory");
        }
    }
    if (c != 0 || threadIdx.x >= 32) return;
    if (!mbar_wait(&xbar, 0)) return;   // gave up (flag set, see ak_wait_timeouts): the mean is left unwritten
    const double total = warp_sum_f64(box[lane]);
    long long cc = (lane < kVpFusedCtas) ? cnt[lane] : 0;
    cc = __reduce_add_sync(0xffffffffu, (int)cc);
    if (lane == 0) {
        const double dn = (double)cc;
        out_mean[0] = (dn > 0.0) ? (float)(total / dn) : __int_as_float(0x7fc00000);
    }
}

template <int DT>
int partial_t(const void* logits, const int64_t* targets, int64_t ignore_index, int64_t vocab_start, int64_t V_total,
              float2* part, int64_t rows, int64_t V_local, int nsplit, cudaStream_t st) {
    using elem_t = typename XElem<DT>::type;
    const elem_t* lg = static_cast<const elem_t*>(logits);
    const dim3 grid((unsigned)rows, (unsigned)nsplit);
    // the single-GPU row layout: 128 threads x 8 vectors, 64 registers (fp32: no cap)
    constexpr int kMinCtas = (DT == AK_DTYPE_F32) ? 1 : 8;
    cudaError_t e;
    if (nsplit == 1) {
        auto kernel = xent_vp_partial_kernel<8, 2, kMinCtas, 128, DT, true>;
        e = launch_dependent(kernel, grid, dim3(128), 0, st, lg, targets, ignore_index, vocab_start, V_total, part,
                             V_local, nsplit, first_wave_ctas(kernel, 128, 0));
    } else {
        e = launch_dependent(xent_vp_partial_kernel<4, 2, 1, kXentThreads, DT, false>, grid, dim3(kXentThreads), 0, st, lg,
                             targets, ignore_index, vocab_start, V_total, part, V_local, nsplit, 0);
    }
    count_launch();
    return e == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}

}  // namespace

int xent_vp_partial_launch(const void* logits, const int64_t* targets, int64_t ignore_index, int64_t vocab_start,
                           int64_t V_total, void* part, int64_t rows, int64_t V_local, int nsplit, int dtype,
                           cudaStream_t st) {
    float2* p = static_cast<float2*>(part);
    switch (dtype) {
        case AK_DTYPE_BF16:
            return partial_t<AK_DTYPE_BF16>(logits, targets, ignore_index, vocab_start, V_total, p, rows, V_local, nsplit, st);
        case AK_DTYPE_F16:
            return partial_t<AK_DTYPE_F16>(logits, targets, ignore_index, vocab_start, V_total, p, rows, V_local, nsplit, st);
        case AK_DTYPE_F32:
            return partial_t<AK_DTYPE_F32>(logits, targets, ignore_index, vocab_start, V_total, p, rows, V_local, nsplit, st);
        default:
            return AK_ERR_ARG;
    }
}

int xent_vp_merge_launch(const void* parts, int nranks, int nsplit, const int64_t* targets, int64_t ignore_index,
                         int64_t V_total, float* loss_rows, float* loss_mean, int64_t rows, cudaStream_t st) {
    if (rows > 0 && rows <= kVpFusedMaxRows && loss_mean != nullptr && clusters_enabled()) {
        const cudaError_t e = launch_cluster_dependent(xent_vp_merge_mean_kernel, (unsigned)kVpFusedCtas, kVpFusedThreads, 0,
                                                       kVpFusedCtas, st, static_cast<const float2*>(parts), nranks, nsplit,
                                                       targets, ignore_index, V_total, loss_rows, loss_mean, rows);
        if (e == cudaSuccess) {
            count_launch();
            return AK_OK;
        }
        (void)cudaGetLastError();   // a device that cannot co-schedule the cluster: the two kernels below
    }
    if (rows > 0) {
        const unsigned grid = (unsigned)((rows + kVpMergeThreads - 1) / kVpMergeThreads);
        const cudaError_t e = launch_dependent(xent_vp_merge_kernel, dim3(grid), dim3(kVpMergeThreads), 0, st,
                                               static_cast<const float2*>(parts), nranks, nsplit, targets, ignore_index,
                                               V_total, loss_rows, rows);
        count_launch();
        if (e != cudaSuccess) return AK_ERR_CUDA;
    }
    if (loss_mean == nullptr) return AK_OK;
    return xent_mean_launch(loss_rows, targets, ignore_index, rows, loss_mean, st, rows > 0);
}

}  // namespace ak
