// K6 — confusion matrix of two one-byte masks (ComputeMetric of Algorithm 1; Section 3.2:
// IoU_c needs |pred_c ∩ label_c| and |pred_c ∪ label_c|, all of which are sums of
// conf[l][q] = #{pixels with label l and prediction q}).
//
// Integer work, exact.  Each thread reads 16 pixels of both masks as 16-byte vectors, two vectors in flight.
// Counters are privatised per warp in shared memory when C*C is small enough.  Masks are spatially coherent (neighbouring
// pixels share a class), so the usual case is a thread whose 16 pixels carry one (label, prediction) pair: where that holds
// for every lane of a warp the equal pairs are merged with one __match_any_sync and counted with weight 16, one
// shared-memory atomic per distinct pair.  Warps with mixed threads (region boundaries, noisy masks) count pixel by
// pixel with plain shared-memory atomics: their pairs differ, so the atomics rarely collide.  Blocks then add their
// counters to the 64-bit global matrix.  Pixels with a label or prediction >= C are skipped and counted.
#include "st_internal.h"
#include "miou.cuh"

namespace st {

constexpr int kConfThreads = 256;
constexpr int kConfWarps = kConfThreads / 32;

template <typename CounterT>
__device__ __forceinline__ void warp_count(CounterT* hist, int key, bool valid, unsigned weight = 1u)
{
    unsigned active = __ballot_sync(0xffffffffu, valid);
    if (!valid) return;
    unsigned peers = __match_any_sync(active, key);
    int leader = __ffs(peers) - 1;
    const unsigned total = __reduce_add_sync(peers, weight);      // the lanes of a group may carry different weights
    if ((int)(threadIdx.x & 31) == leader) atomicAdd(&hist[key], (CounterT)total);
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
        for (int64_t v0 = (int64_t)blockIdx.x * kConfThreads + threadIdx.x; v0 < n_iter; v0 += 2 * stride) {
            uint4 a[2], b[2];
            bool in[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {                      // both vectors' loads are issued before either is used
                const int64_t v = v0 + u * stride;
                in[u] = v < n_vec;
                a[u] = make_uint4(0, 0, 0, 0); b[u] = a[u];
                if (in[u]) {
                    a[u] = __ldcs(reinterpret_cast<const uint4*>(label) + v);
                    b[u] = __ldcs(reinterpret_cast<const uint4*>(pred) + v);
                }
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if (v0 + u * stride >= n_iter) continue;       // warp-uniform: n_iter and the strides are multiples of 32
                const uint32_t aw[4] = {a[u].x, a[u].y, a[u].z, a[u].w}, bw[4] = {b[u].x, b[u].y, b[u].z, b[u].w};
                const int l0 = aw[0] & 0xff, q0 = bw[0] & 0xff;
                const bool same = aw[0] == (uint32_t)l0 * 0x01010101u && aw[1] == aw[0] && aw[2] == aw[0] && aw[3] == aw[0] &&
                                  bw[0] == (uint32_t)q0 * 0x01010101u && bw[1] == bw[0] && bw[2] == bw[0] && bw[3] == bw[0];
                if (__all_sync(0xffffffffu, same || !in[u])) {
                    const bool ok = in[u] && l0 < C && q0 < C;
                    n_bad += (in[u] && !ok) ? 16u : 0u;
                    if (MODE == 2) warp_count(conf, l0 * C + q0, ok, 16u);
                    else warp_count(hist, l0 * C + q0, ok, 16u);
                } else {
                    // mixed warp: every thread counts the pixels that share its first pixel's pair in one go (merged over
                    // the warp like above), and the few that differ one by one with plain atomics
                    uint32_t eq[4];
                    int n_eq = 0;
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        eq[w] = __vcmpeq4(aw[w], (uint32_t)l0 * 0x01010101u) & __vcmpeq4(bw[w], (uint32_t)q0 * 0x01010101u);
                        n_eq += __popc(eq[w]) >> 3;
                    }
                    const bool ok0 = in[u] && l0 < C && q0 < C;
                    n_bad += (in[u] && !ok0) ? (unsigned)n_eq : 0u;
                    if (MODE == 2) warp_count(conf, l0 * C + q0, ok0, (unsigned)n_eq);
                    else warp_count(hist, l0 * C + q0, ok0, (unsigned)n_eq);
                    if (in[u] && n_eq < 16) {
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            if ((eq[k >> 2] >> (8 * (k & 3))) & 1u) continue;
                            const int l = (aw[k >> 2] >> (8 * (k & 3))) & 0xff;
                            const int q = (bw[k >> 2] >> (8 * (k & 3))) & 0xff;
                            if (l < C && q < C) {
                                if (MODE == 2) atomicAdd(&conf[l * C + q], 1ull);
                                else atomicAdd(&hist[l * C + q], 1u);
                            } else {
                                ++n_bad;
                            }
                        }
                    }
                }
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
