// Student mask and its agreement with the labels (ComputeMetric of Algorithm 1; IoU of Section 3.2):
// mask[Y][X] = arg-max over the classes of the bilinearly x4 upsampled logits (lowest class on ties), and,
// fused on request, the confusion matrix of (label, mask) with the mean IoU computed by the last block.
//
// Geometry as in the fused upsample + cross-entropy kernel: the frame pixels 4n+2 .. 4n+5 lie between node
// columns n and n+1 ("cell" n) with weights 1/8, 3/8, 5/8, 7/8 toward n+1, rows alike; cells -1 and w-1 / h-1
// are the clamped borders.  A block covers 4 cell rows x 32 cell columns with the logits of the 5 x 34 surrounding
// nodes in shared memory, borders replicated.  Two warps share a cell row: one lane per cell and half of its four
// frame rows, 8 pixels each (the kernel is latency-bound in a single wave, so more and shorter warps finish sooner).
// Per class a lane reads the cell's four corner logits and interpolates vertically, then horizontally, with one
// fused multiply-add per step.  No pixel is shared between cells, so blocks are independent.
#include "st_internal.h"

namespace st {

namespace {

constexpr int SM_WARPS = 4;                                              // cell rows per block
#ifndef ST_MASK_SPLIT
#define ST_MASK_SPLIT 2
#endif
constexpr int SM_SPLIT = ST_MASK_SPLIT, SM_RW = 4 / SM_SPLIT;           // warps per cell row, frame rows per warp
constexpr int SM_THREADS = SM_WARPS * SM_SPLIT * 32;
constexpr int SM_TH = SM_WARPS + 1, SM_TW = 40, SM_T = SM_TH * SM_TW;   // tile: 5 node rows x 40 columns (34 used, start at a multiple of 4)
constexpr int kMaxChunk = 32;                                            // classes held in shared memory at a time

template <typename CounterT>
__device__ __forceinline__ void warp_count(CounterT* hist, int key, bool valid, unsigned weight)
{
    const unsigned active = __ballot_sync(0xffffffffu, valid);
    if (!valid) return;
    const unsigned peers = __match_any_sync(active, key);
    if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[key], (CounterT)(__popc(peers) * weight));
}

template <bool MASK, bool CONF>
__global__ void __launch_bounds__(SM_THREADS)
student_mask_kernel(StudentMaskArgs a, int chunk)
{
    extern __shared__ __align__(16) float zs[];                   // [chunk][SM_TH][SM_TW]
    unsigned int* hist = reinterpret_cast<unsigned int*>(zs + chunk * SM_T);   // [C][C] (CONF)
    __shared__ bool is_last;
    const int C = a.C, h = a.h, w = a.w, H = h * kUp, W = w * kUp;
    const int64_t p = (int64_t)h * w;
    const int tid = threadIdx.x, wi = tid / (32 * SM_SPLIT), l = tid & 31;   // wi: cell row inside the block
    const int r0 = ((tid >> 5) % SM_SPLIT) * SM_RW;                 // this warp's frame rows of the cell: r0 .. r0 + SM_RW - 1
    const int ya = blockIdx.y * SM_WARPS - 1, xa = blockIdx.x * 32 - 4;   // node row / column of the tile's first element
    const int i = ya + wi, n = blockIdx.x * 32 - 1 + l;                   // cell row / column
    const bool cell_ok = i <= h - 1 && n <= w - 1;
    const int X0 = 4 * n + 2;
    const bool v01 = cell_ok && X0 >= 0 && X0 + 1 < W, v23 = cell_ok && X0 + 2 >= 0 && X0 + 3 < W;

    if (CONF) for (int e = tid; e < C * C; e += SM_THREADS) hist[e] = 0;
    // labels of the lane's 16 pixels, fetched before the sweep over the classes (two aligned 16-bit loads per row)
    uint32_t labw[SM_RW] = {};
    if (CONF) {
#pragma unroll
        for (int r = 0; r < SM_RW; ++r) {
            const int Y = 4 * i + 2 + r0 + r;
            if (Y >= 0 && Y < H) {
                uint32_t llo = 0, lhi = 0;
                if (v01) llo = __ldg(reinterpret_cast<const unsigned short*>(a.labels + (int64_t)Y * W + X0));
                if (v23) lhi = __ldg(reinterpret_cast<const unsigned short*>(a.labels + (int64_t)Y * W + X0 + 2));
                labw[r] = llo | (lhi << 16);
            }
        }
    }

    float best[4 * SM_RW];
    uint32_t arg[4 * SM_RW];
#pragma unroll
    for (int k = 0; k < 4 * SM_RW; ++k) { best[k] = -INFINITY; arg[k] = 0; }

    const bool vec_ok = (w % 4 == 0) && ((uintptr_t)a.z % 16 == 0);
    for (int c0 = 0; c0 < C; c0 += chunk) {                      // classes in chunks that fit shared memory
        const int nc = min(chunk, C - c0);
        __syncthreads();
        for (int e = tid; e < nc * (SM_T / 4); e += SM_THREADS) {
            const int c = e / (SM_T / 4), q = e % (SM_T / 4);
            const int yy = min(max(ya + q / (SM_TW / 4), 0), h - 1), xq = xa + 4 * (q % (SM_TW / 4));
            const float* row = a.z + (int64_t)(c0 + c) * p + (int64_t)yy * w;
            float4 t;
            if (vec_ok && xq >= 0 && xq + 3 < w) t = __ldg(reinterpret_cast<const float4*>(row + xq));
            else {
                t.x = __ldg(row + min(max(xq, 0), w - 1));     t.y = __ldg(row + min(max(xq + 1, 0), w - 1));
                t.z = __ldg(row + min(max(xq + 2, 0), w - 1)); t.w = __ldg(row + min(max(xq + 3, 0), w - 1));
            }
            reinterpret_cast<float4*>(zs)[e] = t;
        }
        __syncthreads();
        if (cell_ok) {
            const float* q = zs + wi * SM_TW + l + 3;            // node (i, n); the tile replicates the clamped borders
#pragma unroll 3
            for (int cc = 0; cc < nc; ++cc, q += SM_T) {
                const uint32_t c = c0 + cc;
                const float tl = q[0], bl = q[SM_TW], tr = q[1], br = q[SM_TW + 1];
                const float dl = bl - tl, dr = br - tr;
#pragma unroll
                for (int r = 0; r < SM_RW; ++r) {
                    const float ly = (float)(2 * (r0 + r) + 1) * 0.125f;
                    const float vl = fmaf(ly, dl, tl), vr = fmaf(ly, dr, tr), d = vr - vl;
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float u = fmaf((2 * k + 1) * 0.125f, d, vl);
                        if (u > best[4 * r + k]) { best[4 * r + k] = u; arg[4 * r + k] = c; }
                    }
                }
            }
        }
    }

    unsigned int n_bad = 0;
#pragma unroll
    for (int r = 0; r < SM_RW; ++r) {
        const int Y = 4 * i + 2 + r0 + r;
        const bool row_ok = Y >= 0 && Y < H;
        const uint32_t lo = arg[4 * r] | (arg[4 * r + 1] << 8), hi = arg[4 * r + 2] | (arg[4 * r + 3] << 8);
        if (MASK && row_ok) {
            if (v01) *reinterpret_cast<unsigned short*>(a.mask + (int64_t)Y * W + X0) = (unsigned short)lo;
            if (v23) *reinterpret_cast<unsigned short*>(a.mask + (int64_t)Y * W + X0 + 2) = (unsigned short)hi;
        }
        if (CONF) {
            const bool ok01 = row_ok && v01, ok23 = row_ok && v23;
            const uint32_t lw = labw[r], aw = lo | (hi << 16);
            // a row whose four pixels are inside the frame and share one (label, class) pair is counted at once
            const bool full = ok01 && ok23, same = full && lw == (lw & 0xffu) * 0x01010101u && aw == (aw & 0xffu) * 0x01010101u;
            if (__all_sync(0xffffffffu, same || !(ok01 || ok23))) {
                const int lab = lw & 0xffu;
                if (same && lab >= C) n_bad += 4;
                warp_count(hist, lab * C + (int)(aw & 0xffu), same && lab < C, 4u);
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const bool in = k < 2 ? ok01 : ok23;
                    const int lab = (lw >> (8 * k)) & 0xffu;
                    if (in && lab >= C) ++n_bad;
                    warp_count(hist, lab * C + (int)((aw >> (8 * k)) & 0xffu), in && lab < C, 1u);
                }
            }
        }
    }
    if (!CONF) return;
    __syncthreads();
    for (int e = tid; e < C * C; e += SM_THREADS)
        if (hist[e]) atomicAdd(&a.conf[e], (unsigned long long)hist[e]);
    if (n_bad) atomicAdd(a.bad, n_bad);
    if (!a.miou) return;

    // ---- the last block to finish turns the matrix into the mean IoU (integer counts, double arithmetic, fixed order)
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = atomicAdd(a.ticket, 1u) == gridDim.x * gridDim.y - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double* iou = reinterpret_cast<double*>(zs);                  // [C] then present [C] (the tile is no longer needed)
    int* present = reinterpret_cast<int*>(iou + C);
    // the matrix goes to shared memory in one coalesced pass if it fits behind them (the tile region is free now)
    unsigned long long* cm = reinterpret_cast<unsigned long long*>(present + C + (C & 1));
    const bool staged = (size_t)C * (sizeof(double) + sizeof(int)) + 8 + (size_t)C * C * 8 <= (size_t)chunk * SM_T * sizeof(float);
    if (staged) {
        for (int e = tid; e < C * C; e += SM_THREADS) cm[e] = __ldcg(&a.conf[e]);
        __syncthreads();
    }
    for (int c = tid; c < C; c += SM_THREADS) {
        unsigned long long row = 0, col = 0;
        for (int q = 0; q < C; ++q) {
            row += staged ? cm[c * C + q] : __ldcg(&a.conf[c * C + q]);
            col += staged ? cm[q * C + c] : __ldcg(&a.conf[q * C + c]);
        }
        double v = 0.0; int pr = 0;
        if (row > 0) {
            const unsigned long long inter = staged ? cm[c * C + c] : __ldcg(&a.conf[c * C + c]);
            v = (double)inter / (double)(row + col - inter);
            pr = 1;
        }
        iou[c] = v; present[c] = pr;
    }
    __syncthreads();
    if (a.conf_out) {                                             // deliver the matrix, leave the counters at zero
        for (int e = tid; e < C * C; e += SM_THREADS) {
            a.conf_out[e] = staged ? cm[e] : __ldcg(&a.conf[e]);
            a.conf[e] = 0;
        }
    }
    if (tid == 0) {
        double sum = 0.0; int cnt = 0;
        for (int k = 0; k < C; ++k) { sum += iou[k]; cnt += present[k]; }
        *a.miou = cnt ? sum / cnt : 0.0;
        *a.ticket = 0;                                            // ready for the next launch
    }
}

size_t mask_smem(int C, bool conf, int* chunk)
{
    *chunk = C < kMaxChunk ? C : kMaxChunk;
    size_t tile = (size_t)*chunk * SM_T * sizeof(float);
    const size_t tail = conf ? (size_t)C * C * sizeof(unsigned int) : 0;
    // the tile region is reused for C doubles + C ints by the last block
    const size_t need = (size_t)C * (sizeof(double) + sizeof(int));
    if (conf && tile < need) tile = (need + 15) / 16 * 16;
    return tile + tail;
}

}  // namespace

bool student_mask_fused_supported(int C)
{
    int chunk;
    return mask_smem(C, true, &chunk) <= 160 * 1024;
}

cudaError_t prepare_student_mask(int C)
{
    int chunk;
    cudaError_t e = cudaFuncSetAttribute(student_mask_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mask_smem(C, false, &chunk));
    if (e != cudaSuccess || !student_mask_fused_supported(C)) return e;
    const int smem = (int)mask_smem(C, true, &chunk);
    e = cudaFuncSetAttribute(student_mask_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(student_mask_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
}

void launch_student_mask(const StudentMaskArgs& a, cudaStream_t s)
{
    if (a.fused) { launch_student_eval(a, s); return; }
    int chunk;
    const bool conf = a.labels != nullptr;
    const size_t smem = mask_smem(a.C, conf, &chunk);
    dim3 grid((unsigned)((a.w + 1 + 31) / 32), (unsigned)((a.h + 1 + SM_WARPS - 1) / SM_WARPS));
    if (!conf) student_mask_kernel<true, false><<<grid, SM_THREADS, smem, s>>>(a, chunk);
    else if (a.mask) student_mask_kernel<true, true><<<grid, SM_THREADS, smem, s>>>(a, chunk);
    else student_mask_kernel<false, true><<<grid, SM_THREADS, smem, s>>>(a, chunk);
}

}  // namespace st
