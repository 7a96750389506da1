// ak_xent_fwd_static: the split-row cross-entropy forward for callers that may not allocate.
//
// Some users of this library run where device memory cannot be asked for at call time: a
// serving process that handed its whole memory budget to its own arena at start-up, a job
// that shares the GPU under a hard quota, a latency-critical loop that must never enter
// the allocator (cudaMalloc can stall the whole device; stream-ordered allocation needs a
// memory pool that such hosts often switch off).  ak_xent_fwd may allocate scratch for its
// split-row path and ak_xent_fwd_ws needs a buffer the caller must have allocated; this
// entry point needs neither.  Its scratch - the per-slice (max, sum) pairs - lives in a
// fixed array inside the library's device image, 1 MiB per GPU that loads the library,
// held until the process exits.  Nothing in this file calls cudaMalloc, cudaFree or any
// allocating routine.
//
// The array's name is only a host-side handle for the device object: it is not a device
// address and must never be passed to a kernel.  The real address is looked up once per
// device with cudaGetSymbolAddress, with that device current, on the first call made on
// that device; that first call should therefore be made before any stream capture is
// begun.  All calls on a device share the one array and find in it whatever the previous
// call left: nothing in the algorithm needs it zeroed (every slot that is read is written
// earlier in the same call), but two calls whose kernels overlap on the GPU - different
// streams - race on it.  Serialise them, or use ak_xent_fwd_ws with separate buffers.
#include <mutex>

#include "xent_kernels.cuh"

namespace ak {
namespace {

constexpr size_t kStaticScratchBytes = 1u << 20;  // 131072 (max, sum) pairs
static __device__ __align__(256) unsigned char g_xent_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_scratch_mu;
float2* g_scratch_ptr[kMaxDevices] = {};

// Device address of the static scratch on the current device (looked up once per device).
int static_scratch(float2** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AK_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_scratch_mu);
    if (g_scratch_ptr[dev] == nullptr) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_xent_static_scratch);
        if (e != cudaSuccess || p == nullptr) {
            (void)cudaGetLastError();
            return AK_ERR_CUDA;
        }
        g_scratch_ptr[dev] = static_cast<float2*>(p);
    }
    *out = g_scratch_ptr[dev];
    return AK_OK;
}

}  // namespace
}  // namespace ak

using namespace ak;

extern "C" int ak_xent_fwd_static(const void* logits, const int64_t* targets, int64_t ignore_index,
                                  float* loss_rows, float* loss_mean, int64_t rows, int64_t V,
                                  void* cuda_stream) {
    if (int s = validate_xent(logits, targets, loss_rows, loss_mean, rows, V)) return s;
    int nsplit = 1;
    xent_choose(rows, V, &nsplit);  // same split count as the allocating entry point would use
    // capacity check before anything is launched: rows * nsplit pairs of 8 bytes
    if (rows > 65535 || (size_t)rows * (size_t)nsplit * sizeof(float2) > kStaticScratchBytes)
        return AK_ERR_CAPACITY;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    float2* scratch = nullptr;
    if (int s = static_scratch(&scratch)) return s;
    const uint16_t* lg = static_cast<const uint16_t*>(logits);
    if (rows > 0) {
        xent_split_kernel<4, 2><<<dim3((unsigned)nsplit, (unsigned)rows), kXentThreads, 0, st>>>(
            lg, targets, ignore_index, scratch, V, nsplit);
        count_launch();
        if (cudaGetLastError() != cudaSuccess) return AK_ERR_CUDA;
    } else if (loss_mean == nullptr) {
        return AK_OK;
    }
    // merge the slices in split order, write the losses, then the fixed-order mean
    if (rows >= kFinishSmallRows)
        xent_finish_kernel<AK_DTYPE_BF16, kFinishThreadsMany><<<1, kFinishThreadsMany, 0, st>>>(
            lg, targets, ignore_index, scratch, nsplit, loss_rows, rows, V, loss_mean, nullptr);
    else
        xent_finish_kernel<AK_DTYPE_BF16, kFinishThreads><<<1, kFinishThreads, 0, st>>>(
            lg, targets, ignore_index, scratch, rows > 0 ? nsplit : 0, loss_rows, rows, V, loss_mean, nullptr);
    count_launch();
    return cudaGetLastError() == cudaSuccess ? AK_OK : AK_ERR_CUDA;
}
