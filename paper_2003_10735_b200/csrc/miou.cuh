// Mean IoU of a confusion matrix, shared by the kernels that finish an agreement measurement themselves.
#pragma once

#include <cuda_runtime.h>

namespace st {

// Mean IoU (Section 3.2): IoU_c = conf[c][c] / (row_c + col_c - conf[c][c]), averaged over the
// classes present in the label (row_c > 0).  Integer counts, double arithmetic, fixed order.
// Called by all 256 threads of a block; the value is returned to thread 0 only.  The counts are read past the L1
// cache: the caller may be the last block of a kernel whose other blocks have just added to them.  Matrices of up to kMiouStage classes
// are first copied to shared memory in one coalesced pass (one memory latency instead of one per row element).
constexpr int kMiouStage = 32;
// The copy to shared memory in two halves, for a caller that has other loads to issue while these are on their way:
// miou_fetch starts the thread's share (blocks of 256 threads, C <= kMiouStage), block_miou takes it over.
struct MiouFetch { unsigned long long v[kMiouStage * kMiouStage / 256]; };
__device__ __forceinline__ MiouFetch miou_fetch(const unsigned long long* conf_g, int C)
{
    MiouFetch f;
#pragma unroll
    for (int k = 0; k < kMiouStage * kMiouStage / 256; ++k) {
        const int e = threadIdx.x + 256 * k;
        f.v[k] = e < C * C ? __ldcg(conf_g + e) : 0ull;
    }
    return f;
}
__device__ __forceinline__ double block_miou(const unsigned long long* conf_g, int C, double* iou, int* present, const MiouFetch* fetched = nullptr)
{
    __shared__ unsigned long long staged[kMiouStage * kMiouStage];
    const unsigned long long* conf = conf_g;
    if (C <= kMiouStage) {                                 // block-uniform
        if (fetched) {
#pragma unroll
            for (int k = 0; k < kMiouStage * kMiouStage / 256; ++k) {
                const int e = threadIdx.x + 256 * k;
                if (e < C * C) staged[e] = fetched->v[k];
            }
        } else {
            for (int e = threadIdx.x; e < C * C; e += blockDim.x) staged[e] = __ldcg(conf_g + e);
        }
        __syncthreads();
        conf = staged;
    }
    const int c = threadIdx.x;
    double v = 0.0; int pr = 0;
    if (c < C) {
        unsigned long long row = 0, col = 0;
        for (int q = 0; q < C; ++q) { row += conf == staged ? conf[c * C + q] : __ldcg(conf + c * C + q); col += conf == staged ? conf[q * C + c] : __ldcg(conf + q * C + c); }
        if (row > 0) {
            const unsigned long long inter = conf == staged ? conf[c * C + c] : __ldcg(conf + c * C + c);
            v = (double)inter / (double)(row + col - inter);
            pr = 1;
        }
    }
    iou[c] = v; present[c] = pr;
    __syncthreads();
    double m = 0.0;
    if (c == 0) {
        double sum = 0.0; int n = 0;
        for (int k = 0; k < C; ++k) { sum += iou[k]; n += present[k]; }
        m = n ? sum / n : 0.0;
    }
    return m;
}


}  // namespace st
