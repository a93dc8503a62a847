// Measured arithmetic peaks of the plain ALUs: the denominators of the compute side of the
// sparse roofline.
//
// The paper (arXiv 1905.00571) has no counterpart; Section 5 only reports latencies.  A pruned
// layer's multiply-adds run on the ordinary FP32 / integer lanes (unstructured sparsity is not a
// dense contraction), so the rate to compare a kernel with is what those lanes sustain on this
// device at the clock it actually holds, not a product of data-sheet numbers.  Each kernel
// below keeps 8 independent dependent chains of multiply-adds per thread (enough to cover the
// pipeline latency with 8 resident warps per scheduler) and nothing else in its loop.
#include <algorithm>
#include "cadnn_internal.h"

namespace {

const int kChains = 8;
const int kInner = 64;   // multiply-adds per chain per loop trip (unrolled)

__global__ void __launch_bounds__(256) ffma_peak_kernel(float *out, int trips, float a, float b)
{
    float v[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) v[c] = (float)(threadIdx.x + c);
    for (int t = 0; t < trips; ++t) {
#pragma unroll
        for (int i = 0; i < kInner; ++i)
#pragma unroll
            for (int c = 0; c < kChains; ++c) v[c] = fmaf(v[c], a, b);
    }
    float s = 0.0f;
#pragma unroll
    for (int c = 0; c < kChains; ++c) s += v[c];
    if (s == 123.456f) out[blockIdx.x * blockDim.x + threadIdx.x] = s;   // keeps the chains alive; practically never taken
}

__global__ void __launch_bounds__(256) imad_peak_kernel(int *out, int trips, int a, int b)
{
    int v[kChains];
#pragma unroll
    for (int c = 0; c < kChains; ++c) v[c] = (int)(threadIdx.x + c);
    for (int t = 0; t < trips; ++t) {
#pragma unroll
        for (int i = 0; i < kInner; ++i)
#pragma unroll
            for (int c = 0; c < kChains; ++c) v[c] = v[c] * a + b;
    }
    int s = 0;
#pragma unroll
    for (int c = 0; c < kChains; ++c) s ^= v[c];
    if (s == 0x7fffabcd) out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

}  // namespace

extern "C" cadnn_status cadnn_measure_alu_peak(int dtype, double *ops_per_second, void *stream)
{
    if (!ops_per_second) return CADNN_E_ARG;
    if (dtype != CADNN_F32 && dtype != CADNN_S8) return CADNN_E_DTYPE;
    cudaStream_t st = (cudaStream_t)stream;
    int dev = 0, sms = 0;
    CADNN_CUDA_TRY(cudaGetDevice(&dev));
    CADNN_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    const int blocks = sms * 8, threads = 256, trips = 512;
    void *buf = nullptr;
    CADNN_CUDA_TRY(cudaMalloc(&buf, (size_t)blocks * threads * 4));
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaEventCreate(&e0);
    cudaEventCreate(&e1);
    double best = 0.0;
    cadnn_status rs = CADNN_OK;
    for (int rep = 0; rep < 4 && rs == CADNN_OK; ++rep) {   // the first repetition warms up
        cudaEventRecord(e0, st);
        if (dtype == CADNN_F32) ffma_peak_kernel<<<blocks, threads, 0, st>>>((float *)buf, trips, 1.000001f, 1e-7f);
        else imad_peak_kernel<<<blocks, threads, 0, st>>>((int *)buf, trips, 3, 7);
        cudaEventRecord(e1, st);
        cudaError_t e = cudaStreamSynchronize(st);
        if (e == cudaSuccess) e = cudaGetLastError();
        if (e != cudaSuccess) { rs = cadnn_note_cuda(e); break; }
        float ms = 0.0f;
        cudaEventElapsedTime(&ms, e0, e1);
        const double ops = 2.0 * (double)blocks * threads * kChains * kInner * (double)trips;
        if (rep > 0 && ms > 0.0f) best = std::max(best, ops / (ms * 1e-3));
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    cudaFree(buf);
    if (rs == CADNN_OK) *ops_per_second = best;
    return rs;
}
