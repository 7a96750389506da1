/*
 * Calls libak through its C ABI from plain C (no Python, no PyTorch): device buffers from the
 * CUDA runtime, raw pointers and sizes into the entry points, status codes back.  Inputs are
 * rows with known closed forms, so the program checks itself:
 *   RMSNorm of a constant row c with weight w:   w * c / sqrt(c^2 + eps)
 *   softmax of an all-equal row of length D:     1 / D
 *   cross-entropy of all-equal logits:           log V   (and the mean over counted rows)
 *   row sum of a row of ones:                    D
 *
 *   gcc c_abi_demo.c -I<repo>/include -I/usr/local/cuda/include -L<dir of libak.so> -lak \
 *       -L/usr/local/cuda/lib64 -lcudart -lm -Wl,-rpath,<dir of libak.so> -o c_abi_demo
 */
#include <cuda_runtime_api.h>
#include <math.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "ak.h"

#define CHECK_CUDA(call)                                                                     \
    do {                                                                                     \
        cudaError_t e_ = (call);                                                             \
        if (e_ != cudaSuccess) {                                                             \
            fprintf(stderr, "CUDA error %s at line %d\n", cudaGetErrorString(e_), __LINE__); \
            return 2;                                                                        \
        }                                                                                    \
    } while (0)
#define CHECK_AK(call)                                                                   \
    do {                                                                                 \
        int s_ = (call);                                                                 \
        if (s_ != AK_OK) {                                                               \
            fprintf(stderr, "%s -> %s (line %d)\n", #call, ak_status_string(s_), __LINE__); \
            return 3;                                                                    \
        }                                                                                \
    } while (0)

/* round-to-nearest-even float -> bf16 bits, and back */
static uint16_t to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}
static float from_bf16(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, 4);
    return f;
}

int main(void) {
    const int64_t rows = 64, D = 4096, V = 32000;
    const float c = 2.0f, w = 1.5f, eps = 1e-6f;
    int failures = 0;
    cudaStream_t st;
    CHECK_CUDA(cudaStreamCreate(&st));

    /* ---- RMSNorm, softmax, row sum on [rows, D] */
    size_t nx = (size_t)rows * D;
    uint16_t* hx = (uint16_t*)malloc(nx * 2);
    uint16_t* hw = (uint16_t*)malloc((size_t)D * 2);
    uint16_t* hy = (uint16_t*)malloc(nx * 2);
    float* hs = (float*)malloc((size_t)rows * 4);
    for (size_t i = 0; i < nx; ++i) hx[i] = to_bf16(c);
    for (int64_t j = 0; j < D; ++j) hw[j] = to_bf16(w);
    void *dx, *dw, *dy;
    float* ds;
    CHECK_CUDA(cudaMalloc(&dx, nx * 2));
    CHECK_CUDA(cudaMalloc(&dw, (size_t)D * 2));
    CHECK_CUDA(cudaMalloc(&dy, nx * 2));
    CHECK_CUDA(cudaMalloc((void**)&ds, (size_t)rows * 4));
    CHECK_CUDA(cudaMemcpyAsync(dx, hx, nx * 2, cudaMemcpyHostToDevice, st));
    CHECK_CUDA(cudaMemcpyAsync(dw, hw, (size_t)D * 2, cudaMemcpyHostToDevice, st));

    CHECK_AK(ak_rmsnorm_fwd(dx, dw, dy, rows, D, eps, st));
    CHECK_CUDA(cudaMemcpyAsync(hy, dy, nx * 2, cudaMemcpyDeviceToHost, st));
    CHECK_CUDA(cudaStreamSynchronize(st));
    {
        const double want = (double)w * c / sqrt((double)c * c + (double)eps);
        for (size_t i = 0; i < nx; ++i)
            if (fabs(from_bf16(hy[i]) - want) > 1.6e-2 * fmax(1.0, fabs(want))) ++failures;
        printf("rmsnorm  constant row: got %.6f, closed form %.6f\n", from_bf16(hy[0]), want);
    }
    CHECK_AK(ak_softmax_fwd(dx, dy, rows, D, st));
    CHECK_CUDA(cudaMemcpyAsync(hy, dy, nx * 2, cudaMemcpyDeviceToHost, st));
    CHECK_CUDA(cudaStreamSynchronize(st));
    for (size_t i = 0; i < nx; ++i)
        if (fabs(from_bf16(hy[i]) - 1.0 / (double)D) > 1.6e-2) ++failures;
    printf("softmax  all-equal row: got %.9f, closed form %.9f\n", from_bf16(hy[0]), 1.0 / (double)D);

    for (size_t i = 0; i < nx; ++i) hx[i] = to_bf16(1.0f);
    CHECK_CUDA(cudaMemcpyAsync(dx, hx, nx * 2, cudaMemcpyHostToDevice, st));
    CHECK_AK(ak_rowsum_fwd(dx, ds, rows, D, st));
    CHECK_CUDA(cudaMemcpyAsync(hs, ds, (size_t)rows * 4, cudaMemcpyDeviceToHost, st));
    CHECK_CUDA(cudaStreamSynchronize(st));
    for (int64_t r = 0; r < rows; ++r)
        if (hs[r] != (float)D) ++failures;
    printf("rowsum   row of ones:   got %.1f, closed form %.1f\n", hs[0], (double)D);

    /* ---- cross-entropy on [rows, V]: all-equal logits, every fourth row ignored */
    size_t nl = (size_t)rows * V;
    uint16_t* hl = (uint16_t*)malloc(nl * 2);
    int64_t* ht = (int64_t*)malloc((size_t)rows * 8);
    float* hloss = (float*)malloc((size_t)rows * 4);
    float hmean = 0.0f;
    for (size_t i = 0; i < nl; ++i) hl[i] = to_bf16(-3.5f);
    for (int64_t r = 0; r < rows; ++r) ht[r] = (r % 4 == 3) ? -100 : (r * 997) % V;
    void* dl;
    int64_t* dt;
    float *dloss, *dmean;
    CHECK_CUDA(cudaMalloc(&dl, nl * 2));
    CHECK_CUDA(cudaMalloc((void**)&dt, (size_t)rows * 8));
    CHECK_CUDA(cudaMalloc((void**)&dloss, (size_t)rows * 4));
    CHECK_CUDA(cudaMalloc((void**)&dmean, 4));
    CHECK_CUDA(cudaMemcpyAsync(dl, hl, nl * 2, cudaMemcpyHostToDevice, st));
    CHECK_CUDA(cudaMemcpyAsync(dt, ht, (size_t)rows * 8, cudaMemcpyHostToDevice, st));
    CHECK_AK(ak_xent_fwd(dl, dt, -100, dloss, dmean, rows, V, st));
    CHECK_CUDA(cudaMemcpyAsync(hloss, dloss, (size_t)rows * 4, cudaMemcpyDeviceToHost, st));
    CHECK_CUDA(cudaMemcpyAsync(&hmean, dmean, 4, cudaMemcpyDeviceToHost, st));
    CHECK_CUDA(cudaStreamSynchronize(st));
    for (int64_t r = 0; r < rows; ++r) {
        const double want = (r % 4 == 3) ? 0.0 : log((double)V);
        if (fabs(hloss[r] - want) > 1e-5 * fmax(1.0, want)) ++failures;
    }
    if (fabs(hmean - log((double)V)) > 1e-5 * log((double)V)) ++failures;
    printf("xent     all-equal logits: loss %.6f, mean %.6f, closed form log V = %.6f\n", hloss[0], hmean,
           log((double)V));

    /* ---- argument errors come back as status codes */
    if (ak_rmsnorm_fwd(NULL, dw, dy, rows, D, eps, st) != AK_ERR_NULL) ++failures;
    if (ak_softmax_fwd(dx, dy, rows, 0, st) != AK_ERR_SHAPE) ++failures;

    printf("library version %d, %lld kernel launches, %d failures\n", ak_version(), (long long)ak_launch_count(),
           failures);
    cudaFree(dx); cudaFree(dw); cudaFree(dy); cudaFree(ds); cudaFree(dl); cudaFree(dt); cudaFree(dloss); cudaFree(dmean);
    free(hx); free(hw); free(hy); free(hs); free(hl); free(ht); free(hloss);
    cudaStreamDestroy(st);
    return failures ? 1 : 0;
}
