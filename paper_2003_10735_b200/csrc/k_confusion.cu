// K6 — confusion matrix of two one-byte masks (ComputeMetric of Algorithm 1; Section 3.2:
// IoU_c needs |pred_c ∩ label_c| and |pred_c ∪ label_c|, all of which are sums of
// conf[l][q] = #{pixels with label l and prediction q}).
//
// Integer work, exact.  Each thread reads 16 pixels of both masks as 16-byte vectors.
// Counters are privatised per warp in shared memory when C*C is small enough; equal keys
// inside a warp are merged with __match_any_sync first, so spatially coherent masks (the
// usual case: neighbouring pixels share a class) cost one shared-memory atomic per distinct
// key per warp instead of 32 conflicting ones.  Blocks then add their counters to the
// 64-bit global matrix.  Pixels with a label or prediction >= C are skipped and counted.
#include "st_internal.h"
#include "miou.cuh"

namespace st {

constexpr int kConfThreads = 256;
constexpr int kConfWarps = kConfThreads / 32;

template <typename CounterT>
__device__ __forceinline__ void warp_count(CounterT* hist, int key, bool valid)
{
    unsigned active = __ballot_sync(0xffffffffu, valid);
    if (!valid) return;
    unsigned peers = __match_any_sync(active, key);
    int leader = __ffs(peers) - 1;
    if ((int)(threadIdx.x & 31) == leader) atomicAdd(&hist[key], (CounterT)__popc(peers));
}

// MODE 0: one shared-memory matrix per warp; 1: one per block; 2: no shared memory (C*C too large),
// warp-merged atomics go straight to the global matrix.
template <int MODE>
__global__ void __launch_bounds__(kConfThreads)
confusion_kernel(const uint8_t* __restrict__ label, const uint8_t* __restrict__ pred, int64_t P, int C,
                 unsigned long long* __restrict__ conf, unsigned int* __restrict__ bad, ConfusionFinish fin)
{
    extern __shared__ unsigned int hist_all[];
    const int CC = C * C;
    const int copies = MODE == 0 ? kConfWarps : (MODE == 1 ? 1 : 0);
    for (int i = threadIdx.x; i < CC * copies; i += kConfThreads) hist_all[i] = 0;
    __syncthreads();
    unsigned int* hist = hist_all + (MODE == 0 ? (threadIdx.x >> 5) * CC : 0);
    unsigned int n_bad = 0;

    const int64_t n_vec = P / 16;
    const bool aligned = (((uintptr_t)label | (uintptr_t)pred) % 16) == 0;
    const int64_t stride = (int64_t)gridDim.x * kConfThreads;
    if (aligned) {
        // the loop bound is rounded up to a whole warp so that every lane takes part in the votes
        const int64_t n_iter = (n_vec + 31) / 32 * 32;
        for (int64_t v = (int64_t)blockIdx.x * kConfThreads + threadIdx.x; v < n_iter; v += stride) {
            bool in = v < n_vec;
            uint4 a = make_uint4(0, 0, 0, 0), b = a;
            if (in) {
                a = __ldcs(reinterpret_cast<const uint4*>(label) + v);
                b = __ldcs(reinterpret_cast<const uint4*>(pred) + v);
            }
            uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                int l = (aw[k >> 2] >> (8 * (k & 3))) & 0xff;
                int q = (bw[k >> 2] >> (8 * (k & 3))) & 0xff;
                bool ok = in && l < C && q < C;
                n_bad += (in && !ok);
                if (MODE == 2) warp_count(conf, l * C + q, ok);
                else warp_count(hist, l * C + q, ok);
            }
        }
    }
    // tail (or everything, if the masks are not 16-byte aligned): one pixel per thread
    {
        const int64_t start = aligned ? n_vec * 16 : 0;
        const int64_t n_tail = P - start;
        const int64_t n_iter = (n_tail + 31) / 32 * 32;
        for (int64_t t = (int64_t)blockIdx.x * kConfThreads + threadIdx.x; t < n_iter; t += stride) {
            bool in = t < n_tail;
            int l = in ? label[start + t] : 0, q = in ? pred[start + t] : 0;
            bool ok = in && l < C && q < C;
            n_bad += (in && !ok);
            if (MODE == 2) warp_count(conf, l * C + q, ok);
            else warp_count(hist, l * C + q, ok);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < CC * (copies > 0); i += kConfThreads) {
        unsigned long long sum = 0;
        for (int k = 0; k < copies; ++k) sum += hist_all[k * CC + i];
        if (sum) atomicAdd(&conf[i], sum);
    }
    if (n_bad) atomicAdd(bad, n_bad);
    if (!fin.ticket) return;

    // ---- the last block to finish delivers the matrix and its mean IoU and leaves the counters at zero for the next launch
    __shared__ bool is_last;
    __shared__ double iou[kConfThreads];
    __shared__ int present[kConfThreads];
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) is_last = atomicAdd(fin.ticket, 1u) == gridDim.x - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const double m = block_miou(conf, C, iou, present);
    for (int i = threadIdx.x; i < CC; i += kConfThreads) {
        fin.result[i] = __ldcg(conf + i);
        conf[i] = 0;
    }
    if (threadIdx.x == 0) { *fin.miou = m; *fin.ticket = 0; }
}

void launch_confusion(const uint8_t* label, const uint8_t* pred, int64_t P, int C,
                      unsigned long long* conf, unsigned int* bad, cudaStream_t s, const ConfusionFinish* finish)
{
    ConfusionFinish fin = {nullptr, nullptr, nullptr};
    if (finish) fin = *finish;
    if (P <= 0 && !fin.ticket) return;
    if (P < 0) P = 0;
    const size_t one = (size_t)C * C * sizeof(unsigned int);
    int64_t work = (P / 16 + kConfThreads - 1) / kConfThreads;
    int blocks = (int)(work < 1 ? 1 : (work > 148 * 4 ? 148 * 4 : work));
    // dynamic shared memory stays below 36 KB: the kernel's static arrays (mean IoU of the last block) take 11 KB of
    // the 48 KB a block gets without opting in
    constexpr size_t kDynLimit = 36 * 1024;
    if (one * kConfWarps <= kDynLimit)
        confusion_kernel<0><<<blocks, kConfThreads, one * kConfWarps, s>>>(label, pred, P, C, conf, bad, fin);
    else if (one <= kDynLimit)
        confusion_kernel<1><<<blocks, kConfThreads, one, s>>>(label, pred, P, C, conf, bad, fin);
    else
        confusion_kernel<2><<<blocks, kConfThreads, 0, s>>>(label, pred, P, C, conf, bad, fin);
}

}  // namespace st
