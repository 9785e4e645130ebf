// Train of Algorithm 1: the assessment of a prediction, shared by the kernels that take it.
#pragma once

#include "st_internal.h"
#include "miou.cuh"

namespace st {

// Train (Algorithm 1), the assessment of prediction i: metric <- mIoU of the prediction; better = the metric is the best
// so far (best_student <- student); skip = the loop ends here or had ended before (no OptimStep).  It is taken either
// by one extra block of the first backward kernel, beside that kernel's own work (the update then reads the outcome),
// or, where no backward follows the prediction, by every block of the update itself (same counts, same arithmetic,
// same answer).  In three parts so that the loads overlap what else a kernel waits for: train_history reads what the
// previous assessment left (it may run before the kernel's predecessors have finished), train_fetch starts the loads of
// the prediction's confusion matrix (blocks of 256 threads), train_decision finishes.  Block-uniform; called by all
// threads of the block.  `writer` (one block per stream) records the history.
struct TrainHistory { bool ended; double prev_best; };
__device__ __forceinline__ TrainHistory train_history(const TrainCtl& t, int s)
{
    TrainHistory h;
    const int i = t.iter;
    h.ended = i > 0 && t.done[(int64_t)s * kCtlPitch + i] != 0;      // the loop had ended before this prediction
    h.prev_best = i > 0 ? t.best[(int64_t)s * kCtlPitch + i] : 0.0;
    return h;
}
__device__ __forceinline__ MiouFetch train_fetch(const TrainCtl& t, int s, const TrainHistory& h)
{
    if (!h.ended && t.C <= kMiouStage) return miou_fetch(t.conf + (int64_t)s * t.conf_stream_stride, t.C);
    return MiouFetch{};
}
__device__ __forceinline__ void train_decision(const TrainCtl& t, int s, bool writer, const TrainHistory& h, const MiouFetch* f,
                                               bool& skip, bool& better)
{
    __shared__ double iou[256];
    __shared__ int present[256];
    __shared__ double m_sh;
    const int i = t.iter;
    int* done = t.done + (int64_t)s * kCtlPitch;
    double* best = t.best + (int64_t)s * kCtlPitch;
    double* metric = t.metric + (int64_t)s * kCtlPitch;
    better = false;
    if (h.ended) {
        skip = true;
        if (writer && threadIdx.x == 0) { done[i + 1] = 1; best[i + 1] = h.prev_best; metric[i] = -1.0; t.better[(int64_t)s * kCtlPitch + i] = 0; }
        return;
    }
    const double m0 = block_miou(t.conf + (int64_t)s * t.conf_stream_stride, t.C, iou, present, f);
    if (threadIdx.x == 0) m_sh = m0;
    __syncthreads();
    const double m = m_sh;
    better = i == 0 || m > h.prev_best;
    const bool stop = i == 0 ? !(m < t.threshold) : (m > t.threshold);
    skip = stop || i >= t.max_updates;
    if (writer && threadIdx.x == 0) {
        metric[i] = m;
        best[i + 1] = better ? m : h.prev_best;
        done[i + 1] = skip ? 1 : 0;
        t.better[(int64_t)s * kCtlPitch + i] = better ? 1 : 0;
        t.n_updates[s] = i;                                      // overwritten by the next prediction if the loop goes on
        if (better) t.best_iter[s] = i;
    }
}

// The outcome as the extra block of the backward kernel left it
__device__ __forceinline__ void train_outcome(const TrainCtl& t, int s, bool& skip, bool& better)
{
    skip = t.done[(int64_t)s * kCtlPitch + t.iter + 1] != 0;
    better = t.better[(int64_t)s * kCtlPitch + t.iter] != 0;
}

}  // namespace st
