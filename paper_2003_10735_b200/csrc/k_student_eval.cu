// Student mask and its agreement with the labels for a head that is one 1x1 classifier over bf16 features
// (ComputeMetric of Algorithm 1; IoU of Section 3.2), in ONE kernel: every block multiplies the logits of its own tile
// of feature-map nodes (Forward, fused_tile.cuh), takes the arg-max over the classes of the bilinearly x4 upsampled
// logits of its cells (lowest class on ties), optionally stores the mask, counts (label, class) pairs, and the last
// block to finish turns the counts into the mean IoU.  The logits never reach global memory.
//
// Geometry as in the fused upsample + cross-entropy kernel: a block owns 7 x 30 nodes and runs 8 warps; warp i owns
// cell row y0-1+i (the 4 x 4 frame pixels between node rows i and i+1), lane l owns the cell to the right of node
// column x0-1+l; a cell is counted by the block that owns its lower right node.  Arithmetic of the interpolation as in
// k_student_mask.cu (vertical, then horizontal, one fused multiply-add per step), so both kernels give the same mask
// from the same logits.
#include "st_internal.h"
#include "tc_common.cuh"
#include "fused_tile.cuh"
#include "miou.cuh"

#include <string.h>

namespace st {

namespace {

using fused::kOwnCols;
using fused::kOwnRows;
using fused::kThreads;
constexpr int TW = fused::kTileCols, TZ = fused::kTile;

template <int CB, bool MASK, bool CONF>
__global__ void __launch_bounds__(kThreads, 2)
student_eval_kernel(StudentMaskArgs a, const __grid_constant__ CUtensorMap x_map, const __grid_constant__ CUtensorMap w_map)
{
    extern __shared__ __align__(128) float smem_e[];
    float* zt = (float*)(((uintptr_t)smem_e + 1023) & ~(uintptr_t)1023);   // [CB][9][32] logits; the feature stages lie over it
    unsigned int* hist = (unsigned int*)(zt + CB * TZ);                    // [C][C] (CONF), under the stages as well
    __shared__ fused::Shared fsh;
    __shared__ bool is_last;
    __shared__ double iou[256];
    __shared__ int present[256];
    const int C = a.C, h = a.h, w = a.w, H = h * kUp, W = w * kUp;
    const int tid = threadIdx.x, wi = tid >> 5, l = tid & 31;
    const int x0 = blockIdx.x * kOwnCols, y0 = blockIdx.y * kOwnRows;
    const int i = y0 - 1 + wi, n = x0 - 1 + l;             // cell row / column
    const bool cell_valid = i <= h - 1 && l <= 30 && n <= w - 1;
    // the block that owns node (min(i+1, h-1), min(n+1, w-1)) counts the cell
    const int t_row = min(i + 1, h - 1), t_col = min(n + 1, w - 1);
    const bool own_cell = cell_valid && t_row >= y0 && t_row < y0 + kOwnRows && t_col >= x0 && t_col < x0 + kOwnCols;
    const int X0 = 4 * n + 2;
    const bool v01 = own_cell && X0 >= 0 && X0 + 1 < W, v23 = own_cell && X0 + 2 >= 0 && X0 + 3 < W;
    // clamped tile coordinates of the cell's corner nodes
    const int ry_top = min(max(i, 0), h - 1) - (y0 - 1), ry_bot = min(max(i + 1, 0), h - 1) - (y0 - 1);
    const int rx_l = min(max(n, 0), w - 1) - (x0 - 1), rx_r = min(max(n + 1, 0), w - 1) - (x0 - 1);

    uint32_t labw[4] = {0, 0, 0, 0};                       // labels of the lane's 16 pixels (two aligned 16-bit loads per row)
    if (CONF) {
#pragma unroll
        for (int r = 0; r < 4; ++r) {
            const int Y = 4 * i + 2 + r;
            if (Y >= 0 && Y < H) {
                uint32_t lo = 0, hi = 0;
                if (v01) lo = __ldg(reinterpret_cast<const unsigned short*>(a.labels + (int64_t)Y * W + X0));
                if (v23) hi = __ldg(reinterpret_cast<const unsigned short*>(a.labels + (int64_t)Y * W + X0 + 2));
                labw[r] = lo | (hi << 16);
            }
        }
    }

    fused::Args fa;
    fa.kblocks = a.kblocks; fa.x_early = 1;                // nothing that can still be running writes the features
    fa.skip = nullptr; fa.err = a.err; fa.bias = a.bias; fa.z_out = nullptr;
    fa.C = C; fa.h = h; fa.w = w;
    fa.spin_limit = tc::kSpinLimit; fa.stall_bytes = 0;
    auto after_mma = [&]() {
        if (CONF) for (int e = tid; e < C * C; e += kThreads) hist[e] = 0;
    };
    const fused::Tile tile = fused::logit_tile<CB>(fa, &x_map, &w_map, fsh, zt, a.stream, x0, y0, after_mma);
    if (!tile.ok) return;
    const uint32_t tmem = tile.tmem;

    float best[16];
    uint32_t arg[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) { best[k] = -INFINITY; arg[k] = 0; }
    if (own_cell) {
        const float* q = zt + ry_top * TW + rx_l;
        const int dq = (ry_bot - ry_top) * TW, dr = rx_r - rx_l;
#pragma unroll 3
        for (int c = 0; c < C; ++c, q += TZ) {
            const float tl = q[0], bl = q[dq], tr = q[dr], br = q[dq + dr];
            const float dl = bl - tl, dright = br - tr;
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float ly = (float)(2 * r + 1) * 0.125f;
                const float vl = fmaf(ly, dl, tl), vr = fmaf(ly, dright, tr), d = vr - vl;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float u = fmaf((2 * k + 1) * 0.125f, d, vl);
                    if (u > best[4 * r + k]) { best[4 * r + k] = u; arg[4 * r + k] = (uint32_t)c; }
                }
            }
        }
    }

    unsigned int n_bad = 0;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int Y = 4 * i + 2 + r;
        const bool row_ok = Y >= 0 && Y < H;
        const uint32_t lo = arg[4 * r] | (arg[4 * r + 1] << 8), hi = arg[4 * r + 2] | (arg[4 * r + 3] << 8);
        if (MASK && row_ok) {
            if (v01) *reinterpret_cast<unsigned short*>(a.mask + (int64_t)Y * W + X0) = (unsigned short)lo;
            if (v23) *reinterpret_cast<unsigned short*>(a.mask + (int64_t)Y * W + X0 + 2) = (unsigned short)hi;
        }
        if (CONF && row_ok) {
            const uint32_t lw = labw[r], aw = lo | (hi << 16);
            if (v01 && v23 && lw == (lw & 0xffu) * 0x01010101u && aw == (aw & 0xffu) * 0x01010101u) {
                // four pixels inside the frame with one (label, class) pair: counted at once
                const uint32_t lab = lw & 0xffu;
                if (lab < (uint32_t)C) atomicAdd(&hist[lab * C + (aw & 0xffu)], 4u);
                else n_bad += 4;
            } else {
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (!(k < 2 ? v01 : v23)) continue;
                    const uint32_t lab = (lw >> (8 * k)) & 0xffu;
                    if (lab < (uint32_t)C) atomicAdd(&hist[lab * C + ((aw >> (8 * k)) & 0xffu)], 1u);
                    else ++n_bad;
                }
            }
        }
    }
    __syncthreads();                                          // all counts are in; every warp has left the tile
    fused::free_tmem(tmem);
    if (!CONF) return;
    for (int e = tid; e < C * C; e += kThreads)
        if (hist[e]) atomicAdd(&a.conf[e], (unsigned long long)hist[e]);
    if (n_bad) atomicAdd(a.bad, n_bad);
    if (!a.miou) return;

    // ---- the last block to finish turns the matrix into the mean IoU (integer counts, double arithmetic, fixed order),
    // delivers the matrix and leaves the counters and the ticket at zero for the next launch
    __threadfence();
    __syncthreads();
    if (tid == 0) is_last = atomicAdd(a.ticket, 1u) == gridDim.x * gridDim.y - 1;
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const double m = block_miou(a.conf, C, iou, present);
    if (a.conf_out) {
        for (int e = tid; e < C * C; e += kThreads) {
            a.conf_out[e] = __ldcg(&a.conf[e]);
            a.conf[e] = 0;
        }
    }
    if (tid == 0) {
        *a.miou = m;
        *a.ticket = 0;
    }
}

template <int CB>
size_t eval_smem_bytes(int C) { return fused::smem_bytes(((size_t)CB * TZ + (size_t)C * C) * sizeof(float)); }

template <int CB>
cudaError_t prepare_cb(int C)
{
    const int smem = (int)eval_smem_bytes<CB>(C);
    cudaError_t e = cudaFuncSetAttribute(student_eval_kernel<CB, true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(student_eval_kernel<CB, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(student_eval_kernel<CB, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    return e;
}

template <int CB>
cudaError_t launch_cb(const StudentMaskArgs& a, cudaStream_t s)
{
    const dim3 grid((unsigned)((a.w + kOwnCols - 1) / kOwnCols), (unsigned)((a.h + kOwnRows - 1) / kOwnRows));
    const size_t smem = eval_smem_bytes<CB>(a.C);
    const bool conf = a.labels != nullptr;
    if (!conf) student_eval_kernel<CB, true, false><<<grid, kThreads, smem, s>>>(a, *a.x_map, *a.w_map);
    else if (a.mask) student_eval_kernel<CB, true, true><<<grid, kThreads, smem, s>>>(a, *a.x_map, *a.w_map);
    else student_eval_kernel<CB, false, true><<<grid, kThreads, smem, s>>>(a, *a.x_map, *a.w_map);
    return cudaGetLastError();
}

// class-count buckets: the two workload sizes exactly, multiples of eight otherwise
int bucket(int C)
{
    if (C == 19 || C == 21) return C;
    return (C + 7) / 8 * 8;
}

}  // namespace

#define ST_EVAL_DISPATCH(FN, C, ...)                 \
    switch (bucket(C)) {                             \
        case 8: return FN<8>(__VA_ARGS__);           \
        case 16: return FN<16>(__VA_ARGS__);         \
        case 19: return FN<19>(__VA_ARGS__);         \
        case 21: return FN<21>(__VA_ARGS__);         \
        case 24: return FN<24>(__VA_ARGS__);         \
        default: return FN<32>(__VA_ARGS__);         \
    }

cudaError_t prepare_student_eval(int C)
{
    if (C > kClassPad) return cudaSuccess;
    ST_EVAL_DISPATCH(prepare_cb, C, C)
}

cudaError_t launch_student_eval(const StudentMaskArgs& a, cudaStream_t s) { ST_EVAL_DISPATCH(launch_cb, a.C, a, s) }

}  // namespace st
