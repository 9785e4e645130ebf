// Measuring aid: the fp32 multiply-add rate and the exp2 (special-function unit) rate of the device, the two
// ceilings of the fused upsample + cross-entropy kernel, which is bound by plain arithmetic rather than by
// memory or tensor cores.  Each thread runs eight independent dependency chains in registers; nothing but the
// final value touches memory.  Not part of the method.
#include "../../include/shadowtutor.h"
#include "st_internal.h"

namespace {

constexpr int kChains = 8, kPeakThreads = 256;

__global__ void __launch_bounds__(kPeakThreads) fma_rate_kernel(float* out, int iters, float a, float b)
{
    float v[kChains];
#pragma unroll
    for (int k = 0; k < kChains; ++k) v[k] = (float)(threadIdx.x + k) * 1e-3f;
    for (int i = 0; i < iters; ++i)
#pragma unroll
        for (int k = 0; k < kChains; ++k) v[k] = fmaf(v[k], a, b);
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < kChains; ++k) s += v[k];
    if (s == 12345.678f) out[0] = s;          // keeps the chains alive; practically never taken
}

__global__ void __launch_bounds__(kPeakThreads) ex2_rate_kernel(float* out, int iters)
{
    float v[kChains];
#pragma unroll
    for (int k = 0; k < kChains; ++k) v[k] = (float)(threadIdx.x + k) * 1e-3f;
    for (int i = 0; i < iters; ++i)
#pragma unroll
        for (int k = 0; k < kChains; ++k) {            // x -> 2^(-x) maps [0, 1] into itself
            float y;
            asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(-v[k]));
            v[k] = y;
        }
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < kChains; ++k) s += v[k];
    if (s == 12345.678f) out[0] = s;
}

}  // namespace

extern "C" st_status st_measure_arithmetic_peaks(void* cuda_stream, double* fma_tflops, double* ex2_tops)
{
    cudaStream_t s = (cudaStream_t)cuda_stream;
    int dev = 0, n_sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return ST_ERR_CUDA;
    float* sink = nullptr;
    if (cudaMalloc((void**)&sink, sizeof(float)) != cudaSuccess) { cudaGetLastError(); return ST_ERR_OOM; }
    cudaEvent_t e0, e1;
    cudaEventCreate(&e0); cudaEventCreate(&e1);
    const int blocks = n_sms * 8, iters = 4096, reps = 5;
    st_status status = ST_OK;
    double best[2] = {0.0, 0.0};
    for (int which = 0; which < 2 && status == ST_OK; ++which)
        for (int r = 0; r < reps + 1; ++r) {            // the first launch warms up
            cudaEventRecord(e0, s);
            if (which == 0) fma_rate_kernel<<<blocks, kPeakThreads, 0, s>>>(sink, iters, 0.999f, 1e-3f);
            else ex2_rate_kernel<<<blocks, kPeakThreads, 0, s>>>(sink, iters);
            cudaEventRecord(e1, s);
            if (cudaEventSynchronize(e1) != cudaSuccess || cudaGetLastError() != cudaSuccess) { status = ST_ERR_CUDA; break; }
            float ms = 0.f;
            cudaEventElapsedTime(&ms, e0, e1);
            const double ops = (double)blocks * kPeakThreads * kChains * iters;
            const double rate = ops / (ms * 1e-3) / 1e12;      // tera-operations per second
            if (r > 0 && rate > best[which]) best[which] = rate;
        }
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    cudaFree(sink);
    if (status != ST_OK) return status;
    if (fma_tflops) *fma_tflops = 2.0 * best[0];          // a multiply-add counts as two operations
    if (ex2_tops) *ex2_tops = best[1];
    return ST_OK;
}
