// On-box FP32 FFMA peak: a register-only fused-multiply-add loop on every SM, timed with CUDA
// events.  The strict-mode roofline is quoted against the nominal peak (SMs x 128 lanes x 2 x
// clock); this measured figure is printed beside it by the benchmark.  (Measurement plumbing;
// the paper has no counterpart.)
#include <cuda_runtime.h>

#include "../../include/mgn_attn.h"

namespace {

__global__ void __launch_bounds__(512)
ffma_loop_kernel(float* out, float a, float b, int iters)
{
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = static_cast<float>(threadIdx.x + i);
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int i = 0; i < 16; ++i) acc[i] = fmaf(acc[i], a, b);
    }
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 16; ++i) s += acc[i];
    if (s == 12345.678f) out[0] = s;      // keeps the loop alive without a store per thread
}

}  // namespace

extern "C" int mgn_measure_fp32_ffma_tflops(float* scratch, double* tflops, void* stream)
{
    if (!scratch || !tflops) return MGN_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return MGN_ERR_CUDA;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return MGN_ERR_CUDA;
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    if (cudaEventCreate(&e0) != cudaSuccess) return MGN_ERR_CUDA;
    if (cudaEventCreate(&e1) != cudaSuccess) { cudaEventDestroy(e0); return MGN_ERR_CUDA; }
    const int threads = 512, grid = sms * 4, iters = 4096;
    double best = 0.0;
    bool ok = true;
    for (int rep = 0; ok && rep < 4; ++rep) {     // first repetition warms up
        ok = cudaEventRecord(e0, st) == cudaSuccess;
        ffma_loop_kernel<<<grid, threads, 0, st>>>(scratch, 1.0001f, 0.5f, iters);
        ok = ok && cudaGetLastError() == cudaSuccess;          // a failed launch must not pass as 0 TFLOP/s
        ok = ok && cudaEventRecord(e1, st) == cudaSuccess && cudaEventSynchronize(e1) == cudaSuccess;
        float ms = 0.f;
        ok = ok && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess;
        const double fl = 2.0 * 16 * 8 * iters * static_cast<double>(grid) * threads;
        if (ok && rep > 0 && ms > 0.f && fl / ms / 1e9 > best) best = fl / ms / 1e9;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (!ok || best <= 0.0) { cudaGetLastError(); return MGN_ERR_CUDA; }
    *tflops = best;
    return MGN_OK;
}
