// K3, row-walking form (n_classes <= 32) — ComputeLoss and the first half of PartialBackward
// (Algorithm 1; loss of Section 5.2): bilinear x4 upsample of the low-resolution logits, per-pixel
// softmax cross-entropy against the labels, and the gradient of the mean loss with respect to the
// low-resolution logits.  Same result as the cell-per-thread kernel in k_upsample_ce.cu.
//
// Geometry.  With half-pixel centres and factor 4 the frame pixels 4n+2 .. 4n+5 lie between node
// columns n and n+1 ("cell" n) with weights 1/8, 3/8, 5/8, 7/8 toward n+1; rows alike.  Cells -1 and
// w-1 are the clamped borders (their outer node is the inner one).
// A block owns RN_Y rows x 30 columns of nodes and runs RN_Y+1 warps.  Warp i owns cell row y0-1+i (the 4 x 4
// frame pixels between node rows i and i+1); lane l owns node column x0-1+l and the 16 pixels of the cell to its
// right.  Warp 0, lane 0 and lane 31 are halo (recomputed by the neighbouring block) so that a block finishes its
// nodes alone, in a fixed summation order, without floating-point atomics.
// The block's logit tile (RN_Y+2 node rows x 36 columns x C classes) arrives by one TMA tile copy issued before
// anything else; rows and columns outside the map arrive as zeros and border blocks overwrite them with the clamped
// border values.  Shapes the tile map cannot describe are fetched with plain loads.
// Fast path (the usual case), class by class for all 16 pixels of the lane's cell at once: inside a cell the
// interpolated logit of a class is u(r,k) = A + B k + G r + D k r (r = frame row, k = pixel in the row), so its 16
// exponentials form geometric progressions: four exp2 (of A, B, G, D) and 12 multiplications (packed fp32x2) replace
// 16 exp2.  Pass 1 sums them per pixel; pass 2 forms them again (cheaper than keeping 16 x C registers alive),
// multiplies by the adjoint interpolation weights / Z and reduces them to the cell's pull on its upper and lower
// node row, both stored in shared memory.  Both sweeps are rolled loops over the classes.
// Slow path (a class changing by more than kFastRange log2-units between two corners of a cell, or a sum that
// underflows): the warp walks its four frame rows one by one with exact per-pixel maxima:
//   pass 1  each lane interpolates its own node column vertically, takes the right neighbour's by shuffle,
//           interpolates its four pixels horizontally, and sums exp2(u - max) over the classes (logits pre-scaled
//           by log2 e);
//   pass 2  the exponentials are formed again, multiplied by the adjoint interpolation weights / Z, the right-hand
//           part is handed to the next lane by shuffle, and the row is added into the two shared-memory slots.
// The "- onehot(label)" part of the gradient is exact in units of 1/64, so it is accumulated with integer
// shared-memory atomics (order-independent), one round per distinct label of a cell.  Pixels tagged for the loss
// weighting (bit 7 of the label byte) count with an integer weight in the loss, in 1/Z and in those integers.
// The epilogue adds, per node row, the own cell row's upper part, the lower part of the cell row above and the
// integer part, writes the bf16 (and on request the fp32) gradient, and reduces the block's bias-gradient partial by
// a lane reduce-scatter.  With CONF the student's class of every pixel (arg-max of the interpolated logits) is taken
// from pass 1's exponentials and counted against the label in a shared-memory confusion matrix.
#include "st_internal.h"
#include "tc_common.cuh"
#include "fused_tile.cuh"

#include <string.h>

namespace st {

namespace {

constexpr int RN_Y = fused::kOwnRows, RN_X = fused::kOwnCols;      // nodes a block owns: 7 rows x 30 columns
constexpr int R_WARPS = RN_Y + 1, R_THREADS = R_WARPS * 32;
constexpr int TZ_H = RN_Y + 2;
// Columns of a tile row (template parameter TW of everything below): 36 when the logits are fetched from global memory
// (32 used, starting at a multiple of 4 so that rows are whole 16-byte vectors), 32 when the block computes its logits
// itself (kTwFused).
constexpr int kTwLoad = 36, kTwFused = fused::kTileCols;
constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;
// Classes per iteration of the two fast-path class sweeps.  The sweeps are rolled loops: unrolled over all classes
// they were ~70 KB of straight-line code that every warp ran through once, and instruction fetch was the main stall.
#ifndef ST_K3_CLASS_UNROLL
#define ST_K3_CLASS_UNROLL 3
#endif
constexpr int kClassUnroll = ST_K3_CLASS_UNROLL;
// Largest change of a class's logit between two corners of a cell (in log2 units) for which the cell stays on the
// fast path.  All 16 products of the progressions are exponentials of the cell's own pixels (at most 1 after the
// shift), the step factors stay below 2^20, and the relative error of a product grows with the size of the exponent
// arguments: about 5e-6 at this limit, below the tolerance of the logit gradient.
#ifndef ST_K3_FAST_RANGE
#define ST_K3_FAST_RANGE 40.0f
#endif
constexpr float kFastRange = ST_K3_FAST_RANGE;

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ float rcp_approx(float x)
{
    float y;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Byte k: (row eighths) x (column eighths of pixel k toward the left node column: 7, 5, 3, 1; toward the right one:
// 1, 3, 5, 7) -- the integer adjoint weights (units of 1/64) of a row's four pixels for one corner node.
__host__ __device__ constexpr uint32_t corner_weights(int row_eighths, bool right)
{
    return right ? (uint32_t)(row_eighths * 1) | (uint32_t)(row_eighths * 3) << 8 | (uint32_t)(row_eighths * 5) << 16 | (uint32_t)(row_eighths * 7) << 24
                 : (uint32_t)(row_eighths * 7) | (uint32_t)(row_eighths * 5) << 8 | (uint32_t)(row_eighths * 3) << 16 | (uint32_t)(row_eighths * 1) << 24;
}

// A lane reads its cell's corner logits at clamped tile coordinates, so the clamped borders (node row -1 is row 0, node
// column w is column w-1, ...) need no copies in the tile.
struct RowCtx {
    const float* za;     // own (clamped) node column, upper (clamped) node row, class 0
    int dq;              // elements from there to the lower node row: the tile's row pitch, or 0 where both rows clamp to one
    int dr;              // ... to the right-hand node column: 1, or 0 at the right border
    float ly;            // weight toward the lower node row
    float M;             // warp-uniform shift
};

// interpolated, shifted logits of the lane's four pixels for class c
template <bool SHIFT, int TW>
__device__ __forceinline__ void pixel_logits(const RowCtx& rc, int c, const float (&sk)[4], float (&u)[4])
{
    constexpr int TZ = TZ_H * TW;
    const float a = rc.za[c * TZ], b = rc.za[c * TZ + rc.dq];
    const float vl = fmaf(fmaf(rc.ly, b - a, a), kLog2e, -rc.M);
    const float vr = __shfl_down_sync(0xffffffffu, vl, 1);
    const float d = vr - vl;
    u[0] = fmaf(0.125f, d, vl); u[1] = fmaf(0.375f, d, vl); u[2] = fmaf(0.625f, d, vl); u[3] = fmaf(0.875f, d, vl);
    if (SHIFT) {
#pragma unroll
        for (int k = 0; k < 4; ++k) u[k] -= sk[k];
    }
}

template <int CB, bool CONF, bool SHIFT, int TW>
__device__ __forceinline__ void pass1(const RowCtx& rc, const float (&sk)[4], float (&Zs)[4], uint32_t (&arg)[4])
{
    float best[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    Zs[0] = Zs[1] = Zs[2] = Zs[3] = 0.f;
#pragma unroll
    for (int c = 0; c < CB; ++c) {
        float u[4];
        pixel_logits<SHIFT, TW>(rc, c, sk, u);
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            if (CONF && !SHIFT) { if (u[k] > best[k]) { best[k] = u[k]; arg[k] = c; } }
            Zs[k] += ex2_approx(u[k]);
        }
    }
}

// The 16 exponentials exp2(u(r,k) - M) of one class inside the lane's cell, u bilinear between the four
// corner logits (own column: the two node rows from shared memory, dq elements apart; right column from the next lane).
// With ly_r = (2r+1)/8 and fr_k = (2k+1)/8:  u(r,k) = A + B k + G r + D k r, so the values are geometric
// progressions along k and r: 4 exp2 and 12 multiplications (8 of them packed: X01[k] = (E(0,k), E(1,k)),
// X23[k] = (E(2,k), E(3,k))).  Returns the largest corner difference
// in the logits' own units (the caller leaves the fast path if a class changes by more than kFastRange log2-units across
// the cell: the progressions would lose their small terms).  q points at raw logits; M is in log2 units.
// The four quantities everything else is a product of: X01[0] = (E(0,0), E(1,0)), X23[0] = (E(2,0), E(3,0)) and the
// per-row ratios between neighbouring pixels q01 = (q_0, q_1), q23 = (q_2, q_3), E(r,k) = E(r,0) q_r^k.
__device__ __forceinline__ float cell_bases(const float* q, int dq, float M, float2& x01, float2& x23, float2& q01, float2& q23)
{
    const float a = q[0], b = q[dq];
    const float ar = __shfl_down_sync(0xffffffffu, a, 1), br = __shfl_down_sync(0xffffffffu, b, 1);
    const float p = b - a, qq = br - ar, e0 = ar - a;
    const float qp = qq - p;
    const float wv = fmaf(qp, 0.125f, e0);
    const float A = fmaf(wv, 0.125f, fmaf(p, 0.125f, a));
    const float E00 = ex2_approx(fmaf(A, kLog2e, -M)), QB = ex2_approx((0.25f * kLog2e) * wv),
                TG = ex2_approx(fmaf(qp, 0.03125f * kLog2e, (0.25f * kLog2e) * p)), SD = ex2_approx((0.0625f * kLog2e) * qp);
    const float TG2 = TG * TG, SD2 = SD * SD;
    q01 = make_float2(QB, QB * SD);
    q23 = __fmul2_rn(q01, make_float2(SD2, SD2));
    x01 = make_float2(E00, E00 * TG);
    x23 = __fmul2_rn(x01, make_float2(TG2, TG2));
    return fmaxf(fabsf(p), fmaxf(fabsf(qq), fabsf(e0)));
}

__device__ __forceinline__ float cell_exponentials(const float* q, int dq, float M, float2 (&X01)[4], float2 (&X23)[4])
{
    const float a = q[0], b = q[dq];
    const float ar = __shfl_down_sync(0xffffffffu, a, 1), br = __shfl_down_sync(0xffffffffu, b, 1);
    const float p = b - a, qq = br - ar, e0 = ar - a;
    const float qp = qq - p;
    const float wv = fmaf(qp, 0.125f, e0);
    const float A = fmaf(wv, 0.125f, fmaf(p, 0.125f, a));
    const float E00 = ex2_approx(fmaf(A, kLog2e, -M)), QB = ex2_approx((0.25f * kLog2e) * wv),
                TG = ex2_approx(fmaf(qp, 0.03125f * kLog2e, (0.25f * kLog2e) * p)), SD = ex2_approx((0.0625f * kLog2e) * qp);
    // rows (0, 1) and (2, 3) ride in the two halves of packed fp32x2 registers: one multiply advances two rows
    const float TG2 = TG * TG, SD2 = SD * SD;
    const float2 q01 = make_float2(QB, QB * SD);
    const float2 q23 = __fmul2_rn(q01, make_float2(SD2, SD2));
    X01[0] = make_float2(E00, E00 * TG);
    X23[0] = __fmul2_rn(X01[0], make_float2(TG2, TG2));
#pragma unroll
    for (int k = 1; k < 4; ++k) {
        X01[k] = __fmul2_rn(X01[k - 1], q01);
        X23[k] = __fmul2_rn(X23[k - 1], q23);
    }
    return fmaxf(fabsf(p), fmaxf(fabsf(qq), fabsf(e0)));
}

// pass 2 of one row on the slow path: the exponentials are formed again, multiplied by the adjoint interpolation
// weights / Z, the right-hand part goes to the next lane, and the row is added into this thread's shared-memory
// slots of the upper and the lower node row
template <int CB, int TW>
__device__ __forceinline__ void pass2_slow(const RowCtx& rc, const float (&sk)[4], const float (&wl)[4], const float (&wr)[4],
                                           float tw, float bw, float2* my_acc, int C)
{
#pragma unroll
    for (int c = 0; c < CB; ++c) {
        float u[4];
        pixel_logits<true, TW>(rc, c, sk, u);
        const float e0 = ex2_approx(u[0]), e1 = ex2_approx(u[1]), e2 = ex2_approx(u[2]), e3 = ex2_approx(u[3]);
        const float aL = fmaf(wl[0], e0, fmaf(wl[1], e1, fmaf(wl[2], e2, wl[3] * e3)));
        const float aR = fmaf(wr[0], e0, fmaf(wr[1], e1, fmaf(wr[2], e2, wr[3] * e3)));
        const float hs = aL + __shfl_up_sync(0xffffffffu, aR, 1);
        if (c < C) {
            const float2 t = my_acc[c * 32];
            my_acc[c * 32] = make_float2(fmaf(tw, hs, t.x), fmaf(bw, hs, t.y));
        }
    }
}

template <int CB, bool CONF, int TW>
__global__ void __launch_bounds__(R_THREADS, 2)
upsample_ce_rows_kernel(UpsampleCeArgs a, const __grid_constant__ CUtensorMap z_map, const __grid_constant__ CUtensorMap x_map,
                        const __grid_constant__ CUtensorMap w_map)
{
    constexpr bool FUSED = TW == kTwFused;      // the block multiplies its own logit tile (Forward of Algorithm 1 for a 1x1 classifier)
    constexpr int TZ_W = TW, TZ = TZ_H * TW;
    extern __shared__ __align__(128) float smem_r[];
    const int C = a.C, h = a.h, w = a.w, H = h * kUp, W = w * kUp;
    // [CB][TZ_H][TW]  logits, borders replicated; classes >= C hold -1e30 (their exponentials are 0).  FUSED: the feature
    // stages and the classifier weights lie over this and the next two arrays until the multiplication has finished.
    float* zt = FUSED ? (float*)(((uintptr_t)smem_r + 1023) & ~(uintptr_t)1023) : smem_r;
    int* corr = (int*)(zt + CB * TZ);           // [C][TZ_H][TW]    -64 * (adjoint of onehot)
    float2* acc = (float2*)(corr + C * TZ);     // [R_WARPS][C][32] (x, y): the cell's pull on its upper / lower node row
    unsigned int* hist = (unsigned int*)(acc + R_WARPS * C * 32);   // [C][C] (CONF): the block's share of the confusion matrix
    __shared__ float red[R_WARPS], red_m[R_WARPS];
    __shared__ __align__(8) uint64_t tile_bar;
    __shared__ fused::Shared fsh;               // FUSED: barriers, tensor-memory slot, bias of the block's own forward

    // Launch order: the last block row first, then rows 0, 1, ...  Blocks at the frame border do extra work, and the
    // blocks that reach an SM first finish earlier than their later companions, so the border rows go first.
    const int by = blockIdx.y == 0 ? gridDim.y - 1 : blockIdx.y - 1;
    const int s = blockIdx.z, x0 = blockIdx.x * RN_X, y0 = by * RN_Y;
    const int blk = by * gridDim.x + blockIdx.x, n_blk = gridDim.x * gridDim.y;
    const int64_t p = (int64_t)h * w;
    const float* z = a.z + (int64_t)s * C * p;
    const uint8_t* labels = a.labels + (int64_t)s * H * W;
    const int tid = threadIdx.x, wi = tid >> 5, l = tid & 31;

    // ---- tile: node rows y0-1 .. y0+RN_Y, node columns xa .. xa+35 where xa = (x0-1) rounded down to a
    // multiple of 4 (so that rows are fetched as 16-byte vectors), clamped at the borders, scaled by
    // log2(e).  Fully unrolled: all of a thread's loads are in flight together.
    const bool vec_ok = !FUSED && (w % 4 == 0) && ((uintptr_t)z % 16 == 0);
    const int xa = vec_ok ? ((x0 - 1) & ~3) : x0 - 1;      // x0-1 >= -1; (-1 & ~3) = -4
    const int off = (x0 - 1) - xa;                         // column of node x0-1 inside the tile
    const int i = y0 - 1 + wi;                  // cell row: frame rows 4i+2 .. 4i+5, node rows (i, i+1)
    const int n = x0 - 1 + l;                   // own node column; cell n lies between node columns n and n+1
    const bool cell_row_valid = i <= h - 1;
    const bool cell_valid = l <= 30 && n >= -1 && n <= w - 1;
    const bool node_owned = l >= 1 && l <= RN_X && n < w;
    // tile coordinates of the (clamped) nodes this lane's pixels pull toward
    const int ry_top = min(max(i, 0), h - 1) - (y0 - 1), ry_bot = min(max(i + 1, 0), h - 1) - (y0 - 1);
    const int rx_l = min(max(n, 0), w - 1) - xa, rx_r = min(max(n + 1, 0), w - 1) - xa;

    // the block that owns node (min(i+1, h-1), min(n+1, w-1)) counts the cell's loss
    const int t_row = min(i + 1, h - 1), t_col = min(n + 1, w - 1);
    const bool own_cell = cell_row_valid && cell_valid && t_row >= y0 && t_row < y0 + RN_Y && t_col >= x0 && t_col < x0 + RN_X;
    // labels of the lane's 16 pixels (rows 4i+2 .. 4i+5, columns 4n+2 .. 4n+5), two aligned 16-bit loads per row;
    // bit 4r+k of vmask: pixel k of row r lies inside the frame
    uint32_t labw[4], vb[4], vmask = 0;      // vb: 0x01 in the byte of each pixel inside the frame
    const int X0 = 4 * n + 2;
    const bool v01 = cell_valid && X0 >= 0 && X0 + 1 < W, v23 = cell_valid && X0 + 2 >= 0 && X0 + 3 < W;
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int Y = 4 * i + 2 + r;
        uint32_t lo = 0, hi = 0;
        if (cell_row_valid && Y >= 0 && Y < H) {
            if (v01) { lo = __ldg(reinterpret_cast<const unsigned short*>(labels + (int64_t)Y * W + X0)); vmask |= 0x3u << (4 * r); }
            if (v23) { hi = __ldg(reinterpret_cast<const unsigned short*>(labels + (int64_t)Y * W + X0 + 2)); vmask |= 0xcu << (4 * r); }
        }
        labw[r] = lo | (hi << 16);
        vb[r] = (((vmask >> (4 * r)) & 0x3u) ? 0x00000101u : 0u) | (((vmask >> (4 * r)) & 0xcu) ? 0x01010000u : 0u);
    }
    // loss weighting (Section 5.2): bit 7 of a label byte marks a pixel near / within a non-background object
    uint32_t hv[4] = {0, 0, 0, 0};                         // 0x01 in the byte of each weighted pixel
    const int hw1 = a.heavy_w - 1;                         // what a weighted pixel counts on top of 1
    if (hw1 > 0) {                                         // block-uniform
#pragma unroll
        for (int r = 0; r < 4; ++r) { hv[r] = (labw[r] >> 7) & 0x01010101u; labw[r] &= 0x7f7f7f7fu; }
    }
    // Node rows above 0 / below h-1 and node columns left of 0 / right of w-1 repeat the border row / column (the tile
    // holds something else there: zeros from the tile copy, or the bare bias from the block's own multiplication).
    auto replicate_borders = [&]() {
        float4* zt4 = reinterpret_cast<float4*>(zt);
        const bool edge_rows = y0 == 0 || y0 + RN_Y > h - 1, edge_cols = xa < 0 || xa + TZ_W > w;
        if (edge_rows) {                                   // block-uniform: node rows above 0 / below h-1 repeat the border row
            const int j_lo = y0 == 0 ? 1 : 0;              // first tile row inside the map
            const int j_hi = min(TZ_H - 1, h - y0);        // last one
            const int n_out = TZ_H - (j_hi - j_lo + 1);    // rows to fill: 0 .. j_lo-1 and j_hi+1 .. TZ_H-1
            for (int e = tid; e < C * n_out * (TZ_W / 4); e += R_THREADS) {
                const int c = e / (n_out * (TZ_W / 4)), r = (e / (TZ_W / 4)) % n_out, x4 = e % (TZ_W / 4);
                const int j = r < j_lo ? r : j_hi + 1 + (r - j_lo);
                const int jc = j < j_lo ? j_lo : j_hi;
                zt4[(c * TZ + j * TZ_W) / 4 + x4] = zt4[(c * TZ + jc * TZ_W) / 4 + x4];
            }
            __syncthreads();
        }
        if (edge_cols) {                                   // node columns left of 0 / right of w-1 repeat the border column
            const int x_lo = xa < 0 ? -xa : 0;             // first tile column inside the map
            const int x_hi = min(TZ_W - 1, w - 1 - xa);    // last one
            const int n_out = TZ_W - (x_hi - x_lo + 1);
            for (int e = tid; e < C * TZ_H * n_out; e += R_THREADS) {
                const int row = e / n_out, r = e % n_out;  // row = c * TZ_H + j
                const int x = r < x_lo ? r : x_hi + 1 + (r - x_lo);
                zt[row * TZ_W + x] = zt[row * TZ_W + (x < x_lo ? x_lo : x_hi)];
            }
            __syncthreads();
        }
    };
    float m_loc = -INFINITY;                               // largest logit of this thread's share of the tile
    uint32_t tmem = 0;                                     // FUSED: the block's tensor memory (given back at the very end)
    if constexpr (FUSED) {
        // ---- Forward for a 1x1 classifier, inside the block (fused_tile.cuh)
        fused::Args fa;
        fa.kblocks = a.kblocks; fa.x_early = a.x_early;
        fa.skip = a.skip ? a.skip + (int64_t)s * a.skip_stride : nullptr;
        fa.err = a.err;
        fa.bias = a.theta + (int64_t)s * a.n_params + a.b_off;
        fa.z_out = a.z_out ? a.z_out + (int64_t)s * C * p : nullptr;
        fa.C = C; fa.h = h; fa.w = w;
        fa.spin_limit = a.test_stall ? (1u << 12) : tc::kSpinLimit; fa.stall_bytes = a.test_stall ? 16u : 0u;
        auto after_mma = [&]() {                        // the arrays the stages lay over get their initial contents
            for (int e = tid; e < C * TZ / 4; e += R_THREADS) reinterpret_cast<int4*>(corr)[e] = make_int4(0, 0, 0, 0);
            if (CONF) for (int e = tid; e < C * C; e += R_THREADS) hist[e] = 0;
        };
        const fused::Tile tile = fused::logit_tile<CB>(fa, &x_map, &w_map, fsh, zt, s, x0, y0, after_mma);
        if (!tile.ok) return;
        m_loc = tile.m_loc; tmem = tile.tmem;
    } else
    {
        // a thread keeps one 16-byte group of the tile plane (81 groups) and walks the classes three at a time
        constexpr int kQuads = TZ / 4, kPlanes = R_THREADS / kQuads;       // 81, 3
        constexpr int kIter = (CB + kPlanes - 1) / kPlanes;
        const int g = tid / kQuads, q = tid % kQuads;
        float4* zt4 = reinterpret_cast<float4*>(zt);
        if (a.has_map) {                                       // shared memory the tile copy does not write
            for (int e = tid; e < (CB - C) * kQuads; e += R_THREADS) zt4[C * kQuads + e] = make_float4(-1e30f, -1e30f, -1e30f, -1e30f);
            for (int e = tid; e < C * TZ / 4; e += R_THREADS) reinterpret_cast<int4*>(corr)[e] = make_int4(0, 0, 0, 0);
            if (CONF) for (int e = tid; e < C * C; e += R_THREADS) hist[e] = 0;
        }
        // The logits come from the previous kernel of the step; nothing before this line depends on them, so a launch that
        // started while that kernel was still running has used the time.
        pdl_wait();
        if (a.skip && a.skip[(int64_t)s * a.skip_stride]) return;     // this stream's training loop has ended (block-uniform)
        if (a.has_map && tid == 0) {                           // block-uniform flag (implies vec_ok)
            // one tile copy for the whole block, started before anything else that needs the logits: box {36 columns,
            // RN_Y + 2 node rows, C classes} at (xa, y0 - 1, s C).  Rows and columns outside the map arrive as zeros and
            // are replaced below by the clamped border values.
            const uint32_t bar = tc::smem_u32(&tile_bar);
            tc::mbar_init(bar, 1);
            tc::fence_barrier_init();
            tc::mbar_expect_tx(bar, (uint32_t)(C * TZ * sizeof(float)));
            tc::tma_load_3d(tc::smem_u32(zt), &z_map, bar, xa, y0 - 1, s * C);
        }
        if (a.has_map) {
            // ---- the tile copy is in flight
            const uint32_t bar = tc::smem_u32(&tile_bar);
            __syncthreads();                                   // the barrier's initialisation is visible to every waiter
            bool ok = false;
            for (uint32_t it = 0; it < 2 * tc::kSpinLimit && !ok; ++it) ok = tc::mbar_try_wait(bar, 0);
            if (!__syncthreads_and(ok)) {                    // block-uniform: the copy never arrived
                if (tid == 0) atomicCAS(a.err, 0u, (unsigned int)tc::kWaitFull | (blockIdx.x << 8));
                tc::drain_after_error();
                return;
            }
            replicate_borders();
#pragma unroll
            for (int it = 0; it < kIter; ++it) {
                const int c = g + it * kPlanes;
                if (g < kPlanes && c < C) {
                    const float4 t = zt4[c * kQuads + q];
                    m_loc = fmaxf(fmaxf(m_loc, fmaxf(t.x, t.y)), fmaxf(t.z, t.w));
                }
            }
        } else {
            // ---- plain loads (edge columns, any width and alignment), fully unrolled: all of a thread's loads are in
            // flight together
            const int yy = min(max(y0 - 1 + q / (TZ_W / 4), 0), h - 1), xq = xa + 4 * (q % (TZ_W / 4));
            const bool vec = vec_ok && xq >= 0 && xq + 3 < w;
            const float* row = z + (int64_t)yy * w;
            const int x_0 = min(max(xq, 0), w - 1), x_1 = min(max(xq + 1, 0), w - 1), x_2 = min(max(xq + 2, 0), w - 1),
                      x_3 = min(max(xq + 3, 0), w - 1);
            float4 v[kIter];
#pragma unroll
            for (int it = 0; it < kIter; ++it) {
                const int c = g + it * kPlanes;
                float4 t = make_float4(-1e30f, -1e30f, -1e30f, -1e30f);
                if (g < kPlanes && c < C) {
                    const float* rp = row + (int64_t)c * p;
                    if (vec) t = __ldg(reinterpret_cast<const float4*>(rp + xq));
                    else { t.x = __ldg(rp + x_0); t.y = __ldg(rp + x_1); t.z = __ldg(rp + x_2); t.w = __ldg(rp + x_3); }
                    m_loc = fmaxf(fmaxf(m_loc, fmaxf(t.x, t.y)), fmaxf(t.z, t.w));
                }
                v[it] = t;
            }
#pragma unroll
            for (int it = 0; it < kIter; ++it) {
                const int c = g + it * kPlanes;
                if (g < kPlanes && c < CB) zt4[c * kQuads + q] = v[it];
            }
            for (int e = tid; e < C * TZ / 4; e += R_THREADS) reinterpret_cast<int4*>(corr)[e] = make_int4(0, 0, 0, 0);
            if (CONF) for (int e = tid; e < C * C; e += R_THREADS) hist[e] = 0;
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m_loc = fmaxf(m_loc, __shfl_xor_sync(0xffffffffu, m_loc, o));
    if (l == 0) red_m[wi] = m_loc;
    __syncthreads();

    RowCtx rc;
    rc.za = zt + ry_top * TZ_W + rx_l;
    rc.dq = (ry_bot - ry_top) * TZ_W;
    rc.dr = rx_r - rx_l;
    rc.ly = 0.f;
    {
        // shift of the exponentials: the largest logit of the block's tile (a pixel whose own logits lie far below it
        // is caught by the underflow check and redone with its exact maximum)
        float m = red_m[0];
#pragma unroll
        for (int k = 1; k < R_WARPS; ++k) m = fmaxf(m, red_m[k]);
        rc.M = m * kLog2e;                                 // log2 units
    }

    float loss = 0.f;
    unsigned n_bad = 0;
    float2* my_acc = acc + (size_t)wi * C * 32 + l;            // this thread's slot of class c: my_acc[c * 32]

    // at the clamped left and right borders the outer node column is the inner one
    const bool fold_l = n == -1, fold_r = n == w - 1;

    // per pixel of one row: loss, 1/Z, the "- onehot" part of the adjoint (integer, exact), confusion; returns the
    // horizontal adjoint weights (already divided by Z) of the row's four pixels
    auto finish_row = [&](int r, const float (&Zs)[4], const float (&sk)[4], const uint32_t (&arg)[4], float (&wl)[4], float (&wr)[4]) {
        const float ly = (2 * r + 1) * 0.125f;
        const int wy1 = 2 * r + 1, wy0 = 8 - wy1;                // eighths toward node rows i+1 / i
        int lab[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            lab[k] = (labw[r] >> (8 * k)) & 0xff;
            const bool valid = (vmask >> (4 * r + k)) & 1u;
            const bool own = valid && own_cell;
            if (valid && lab[k] >= C) { if (own) n_bad++; lab[k] = -1; }
            if (!valid) lab[k] = -1;
            float rz = 0.f;
            const float wk = ((hv[r] >> (8 * k)) & 1u) ? (float)a.heavy_w : 1.0f;
            if (lab[k] >= 0) {
                rz = rcp_approx(Zs[k]) * wk;
                if (own) {
                    const float* q = rc.za + lab[k] * TZ;
                    const float vl = fmaf(ly, q[rc.dq] - q[0], q[0]), vr = fmaf(ly, q[rc.dq + rc.dr] - q[rc.dr], q[rc.dr]);
                    const float ul = fmaf(fmaf((2 * k + 1) * 0.125f, vr - vl, vl), kLog2e, -rc.M) - sk[k];
                    loss += wk * (__log2f(Zs[k]) - ul) * kLn2;
                    if (CONF) atomicAdd(&hist[lab[k] * C + arg[k]], 1u);
                }
            }
            const float fr = (2 * k + 1) * 0.125f;
            wl[k] = (fold_l ? 0.f : (fold_r ? 1.0f : 1.0f - fr)) * rz;
            wr[k] = (fold_r ? 0.f : (fold_l ? 1.0f : fr)) * rz;
        }
        // four valid pixels with one label (the usual case): their onehot parts add up to 16 eighths per side
        if (hw1 == 0 && lab[0] >= 0 && lab[0] == lab[1] && lab[1] == lab[2] && lab[2] == lab[3]) {
            int* cc = corr + lab[0] * TZ;
            atomicAdd(cc + ry_top * TZ_W + rx_l, -wy0 * 16);
            atomicAdd(cc + ry_top * TZ_W + rx_r, -wy0 * 16);
            atomicAdd(cc + ry_bot * TZ_W + rx_l, -wy1 * 16);
            atomicAdd(cc + ry_bot * TZ_W + rx_r, -wy1 * 16);
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k)
                if (lab[k] >= 0) {
                    const int iw = ((hv[r] >> (8 * k)) & 1u) ? a.heavy_w : 1;
                    const int wb = (2 * k + 1) * iw, wa = (7 - 2 * k) * iw;       // eighths toward node columns n+1 / n, times the weight
                    int* cc = corr + lab[k] * TZ;
                    atomicAdd(cc + ry_top * TZ_W + rx_l, -wy0 * wa);
                    atomicAdd(cc + ry_top * TZ_W + rx_r, -wy0 * wb);
                    atomicAdd(cc + ry_bot * TZ_W + rx_l, -wy1 * wa);
                    atomicAdd(cc + ry_bot * TZ_W + rx_r, -wy1 * wb);
                }
        }
    };

    if (cell_row_valid) {                                        // warp-uniform
        // ---------------- fast path, pass 1: sums of exponentials of the 16 pixels
        float2 Z01[4], Z23[4];                                       // Z01[k] = (Z(0,k), Z(1,k)), Z23[k] = (Z(2,k), Z(3,k))
#pragma unroll
        for (int k = 0; k < 4; ++k) Z01[k] = Z23[k] = make_float2(0.f, 0.f);
        float wmax = 0.f;
        // CONF: the student's class of each pixel rides on the same sweep.  The exponentials are positive and monotone
        // in the logits, so the largest one marks the arg-max; its bit pattern with the low five bits replaced by
        // 31 - c is compared as an integer (equal values: the lowest class wins).  Dropping five bits can only swap
        // classes whose logits differ by less than 3e-6 relative.
        uint32_t key[16];
#pragma unroll
        for (int j = 0; j < 16; ++j) key[j] = 0;
#pragma unroll kClassUnroll
        for (int c = 0; c < CB; ++c) {
            float2 X01[4], X23[4];
            wmax = fmaxf(wmax, cell_exponentials(rc.za + c * TZ, rc.dq, rc.M, X01, X23));
#pragma unroll
            for (int k = 0; k < 4; ++k) { Z01[k] = __fadd2_rn(Z01[k], X01[k]); Z23[k] = __fadd2_rn(Z23[k], X23[k]); }
            if (CONF) {
                const uint32_t tag = 31u - (uint32_t)c;
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    key[k] = max(key[k], (__float_as_uint(X01[k].x) & ~31u) | tag);
                    key[4 + k] = max(key[4 + k], (__float_as_uint(X01[k].y) & ~31u) | tag);
                    key[8 + k] = max(key[8 + k], (__float_as_uint(X23[k].x) & ~31u) | tag);
                    key[12 + k] = max(key[12 + k], (__float_as_uint(X23[k].y) & ~31u) | tag);
                }
            }
        }
        float Z[16];                                                 // Z[4r + k]
#pragma unroll
        for (int k = 0; k < 4; ++k) { Z[k] = Z01[k].x; Z[4 + k] = Z01[k].y; Z[8 + k] = Z23[k].x; Z[12 + k] = Z23[k].y; }
        bool bad = !(wmax <= kFastRange / kLog2e);
#pragma unroll
        for (int j = 0; j < 16; ++j) bad |= ((vmask >> j) & 1u) && !(Z[j] > 1e-18f);
        const bool slow = __any_sync(0xffffffffu, bad);
        if (!slow) {
            float wl[16], wr[16];
            const float zero4[4] = {0.f, 0.f, 0.f, 0.f};
            // pixels that count: inside the frame, label below n_classes
            uint32_t rem[4];
            const uint32_t C4 = (uint32_t)C * 0x01010101u;
            int n_ok = 0;
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                rem[r] = __vcmpltu4(labw[r], C4) & vb[r];
                n_ok += __popc(rem[r]) + hw1 * __popc(rem[r] & hv[r]);      // the weights of the pixels that count
                if (own_cell) n_bad += __popc(rem[r] ^ vb[r]);
            }
            if (CONF) {
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (own_cell && ((rem[j >> 2] >> (8 * (j & 3))) & 1u))
                        atomicAdd(&hist[((labw[j >> 2] >> (8 * (j & 3))) & 0xffu) * C + (31u - (key[j] & 31u))], 1u);
            }
            float lz = 0.f;
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const bool ok = (rem[j >> 2] >> (8 * (j & 3))) & 1u;
                const float fr = (2 * (j & 3) + 1) * 0.125f;
                const float wj = ((hv[j >> 2] >> (8 * (j & 3))) & 1u) ? (float)a.heavy_w : 1.0f;
                const float rz = ok ? rcp_approx(Z[j]) * wj : 0.f;
                lz += ok ? wj * __log2f(Z[j]) : 0.f;
                wl[j] = (fold_l ? 0.f : (fold_r ? 1.0f : 1.0f - fr)) * rz;
                wr[j] = (fold_r ? 0.f : (fold_l ? 1.0f : fr)) * rz;
            }
            // One round per distinct label of the cell (one round for most cells).  The pixels carrying the label pull
            // the four corner nodes with integer weights (row eighths x column eighths, summed by byte-wise dot products);
            // the same four sums weight the label's corner logits in the loss.
            int* c_tl = corr + ry_top * TZ_W + rx_l;
            const int d_tr = rx_r - rx_l, d_bl = (ry_bot - ry_top) * TZ_W;
            float lsum = 0.f;
            while (rem[0] | rem[1] | rem[2] | rem[3]) {
                const uint32_t wsel = rem[0] ? labw[0] : rem[1] ? labw[1] : rem[2] ? labw[2] : labw[3];
                const uint32_t rsel = rem[0] ? rem[0] : rem[1] ? rem[1] : rem[2] ? rem[2] : rem[3];
                const uint32_t cur = (wsel >> (__ffs(rsel) - 1)) & 0xffu;
                const uint32_t cur4 = cur * 0x01010101u;
                uint32_t tl = 0, tr = 0, bl = 0, br = 0;
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    const uint32_t eq = __vcmpeq4(labw[r], cur4) & rem[r];
                    rem[r] ^= eq;
                    const uint32_t ew = eq + (eq & hv[r]) * (uint32_t)hw1;          // each byte: the pixel's weight (1..5) or 0
                    tl = __dp4a(ew, corner_weights(7 - 2 * r, false), tl);
                    tr = __dp4a(ew, corner_weights(7 - 2 * r, true), tr);
                    bl = __dp4a(ew, corner_weights(2 * r + 1, false), bl);
                    br = __dp4a(ew, corner_weights(2 * r + 1, true), br);
                }
                int* cc = c_tl + cur * TZ;
                atomicAdd(cc, -(int)tl);
                atomicAdd(cc + d_tr, -(int)tr);
                atomicAdd(cc + d_bl, -(int)bl);
                atomicAdd(cc + d_bl + d_tr, -(int)br);
                if (own_cell) {
                    const float* q = zt + (c_tl - corr) + cur * TZ;
                    lsum = fmaf((float)tl, q[0], fmaf((float)tr, q[d_tr], fmaf((float)bl, q[d_bl], fmaf((float)br, q[d_bl + d_tr], lsum))));
                }
            }
            if (own_cell) loss += (lz - (lsum * (kLog2e / 64.0f) - (float)n_ok * rc.M)) * kLn2;
            // vertical weights of the rows toward the upper / lower node row (clamped borders fold into the inner row)
            float tw[4], bw[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float ly = (2 * r + 1) * 0.125f;
                tw[r] = i == -1 ? 0.f : (i == h - 1 ? 1.0f : 1.0f - ly);
                bw[r] = i == h - 1 ? 0.f : (i == -1 ? 1.0f : ly);
            }
            // ---------------- fast path, pass 2 (packed fp32x2: rows (0,1) and (2,3) side by side)
            float2 WL01[4], WL23[4], WR01[4], WR23[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                WL01[k] = make_float2(wl[k], wl[4 + k]); WL23[k] = make_float2(wl[8 + k], wl[12 + k]);
                WR01[k] = make_float2(wr[k], wr[4 + k]); WR23[k] = make_float2(wr[8 + k], wr[12 + k]);
            }
            const float2 tw01 = make_float2(tw[0], tw[1]), tw23 = make_float2(tw[2], tw[3]);
            const float2 bw01 = make_float2(bw[0], bw[1]), bw23 = make_float2(bw[2], bw[3]);
#pragma unroll kClassUnroll
            for (int c = 0; c < CB; ++c) {
                // a row's four exponentials are E(r,0) q_r^k, so the row's weighted sum is E(r,0) times a cubic in q_r
                // with the pixel weights as coefficients: Horner's rule, the progression itself is not formed again
                float2 x01, x23, q01, q23;
                cell_bases(rc.za + c * TZ, rc.dq, rc.M, x01, x23, q01, q23);
                float2 aL01 = WL01[3], aL23 = WL23[3], aR01 = WR01[3], aR23 = WR23[3];
#pragma unroll
                for (int k = 2; k >= 0; --k) {
                    aL01 = __ffma2_rn(aL01, q01, WL01[k]); aL23 = __ffma2_rn(aL23, q23, WL23[k]);
                    aR01 = __ffma2_rn(aR01, q01, WR01[k]); aR23 = __ffma2_rn(aR23, q23, WR23[k]);
                }
                aL01 = __fmul2_rn(aL01, x01); aL23 = __fmul2_rn(aL23, x23);
                aR01 = __fmul2_rn(aR01, x01); aR23 = __fmul2_rn(aR23, x23);
                // own cell's left part + left cell's right part, per row
                const float2 hs01 = __fadd2_rn(aL01, make_float2(__shfl_up_sync(0xffffffffu, aR01.x, 1), __shfl_up_sync(0xffffffffu, aR01.y, 1)));
                const float2 hs23 = __fadd2_rn(aL23, make_float2(__shfl_up_sync(0xffffffffu, aR23.x, 1), __shfl_up_sync(0xffffffffu, aR23.y, 1)));
                const float2 t2 = __ffma2_rn(hs23, tw23, __fmul2_rn(hs01, tw01));
                const float2 b2 = __ffma2_rn(hs23, bw23, __fmul2_rn(hs01, bw01));
                if (c < C) my_acc[c * 32] = make_float2(t2.x + t2.y, b2.x + b2.y);
            }
        } else {
            // ---------------- slow path: row by row, exact per-pixel maxima
            for (int c = 0; c < C; ++c) my_acc[c * 32] = make_float2(0.f, 0.f);
            for (int r = 0; r < 4; ++r) {
                const int Y = 4 * i + 2 + r;
                if (!(Y >= 0 && Y < H)) continue;                    // warp-uniform
                rc.ly = (2 * r + 1) * 0.125f;
                float ex[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
                const float zero4[4] = {0.f, 0.f, 0.f, 0.f};
                for (int c = 0; c < C; ++c) {
                    float u[4];
                    pixel_logits<false, TW>(rc, c, zero4, u);
#pragma unroll
                    for (int k = 0; k < 4; ++k) ex[k] = fmaxf(ex[k], u[k]);
                }
                float Zs[4];
                uint32_t ar4[4] = {0, 0, 0, 0};
                if (CONF) pass1<CB, true, false, TW>(rc, zero4, Zs, ar4);    // arg-max of the interpolated logits
                pass1<CB, false, true, TW>(rc, ex, Zs, ar4);
                float wl4[4], wr4[4];
                finish_row(r, Zs, ex, ar4, wl4, wr4);
                const float twr = i == -1 ? 0.f : (i == h - 1 ? 1.0f : 1.0f - rc.ly);
                const float bwr = i == h - 1 ? 0.f : (i == -1 ? 1.0f : rc.ly);
                pass2_slow<CB, TW>(rc, ex, wl4, wr4, twr, bwr, my_acc, C);
            }
        }
    } else {
        for (int c = 0; c < C; ++c) my_acc[c * 32] = make_float2(0.f, 0.f);
    }
    // loss of the block, fixed order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
    if (l == 0) red[wi] = loss;
    if (n_bad) atomicAdd(a.bad, n_bad);
    __syncthreads();
    pdl_launch_dependents();                     // only the epilogue is left: the next kernel of the step may set itself up
    if (CONF) {                                  // one global update per non-empty counter of the block
        for (int e = tid; e < C * C; e += R_THREADS)
            if (hist[e]) atomicAdd(a.conf + (int64_t)s * a.conf_stream_stride + e, (unsigned long long)hist[e]);
    }

    // ---- node row y0-1+wi (warps 1..RN_Y): own upper part + lower part of the warp above + onehot part.
    // All shared-memory reads of the 21 classes are issued before the first store.
    const float invP = 1.0f / ((float)H * (float)W);
    const int y = i;
    const bool node_ok = wi >= 1 && y < h && node_owned;
    constexpr int CP = 32;                       // classes padded to the warp width for the lane reduce-scatter
    float v[CP];
    {
        int cr[CB];
        float2 up[CB], lo[CB];
#pragma unroll
        for (int c = 0; c < CB; ++c) {
            cr[c] = 0; up[c] = lo[c] = make_float2(0.f, 0.f);
            if (c < C && node_ok) {
                cr[c] = corr[c * TZ + wi * TZ_W + off + l];
                up[c] = acc[(wi * C + c) * 32 + l];
                lo[c] = acc[((wi - 1) * C + c) * 32 + l];
            }
        }
#pragma unroll
        for (int c = 0; c < CB; ++c) v[c] = (up[c].x + lo[c].y + (float)cr[c] * (1.0f / 64.0f)) * invP;
#pragma unroll
        for (int c = CB; c < CP; ++c) v[c] = 0.f;
    }
    if (node_ok) {
        if (a.dz) {
            float* dzp = a.dz + (int64_t)s * C * p + (int64_t)y * w + n;
#pragma unroll
            for (int c = 0; c < CB; ++c)
                if (c < C) dzp[(int64_t)c * p] = v[c];
        }
        if (a.dz_bf16) {
            bf16* dzb = a.dz_bf16 + (int64_t)s * kClassPad * a.dz_bf16_pitch + (int64_t)y * w + n;
#pragma unroll
            for (int c = 0; c < CB; ++c)
                if (c < C) dzb[(int64_t)c * a.dz_bf16_pitch] = __float2bfloat16_rn(v[c]);
        }
    }
    // bias-gradient partial of the block: sum of the block's gradient values per class.  Lane reduce-scatter inside
    // each warp (31 exchanges for 32 classes: at distance o a lane keeps the half of its values whose class has bit o
    // equal to its own lane bit and adds the partner's), after which lane c holds class c; then the warps' sums are
    // added in warp order.  Fixed order throughout.
#pragma unroll
    for (int o = CP / 2; o > 0; o >>= 1) {
        const bool hi = l & o;
#pragma unroll
        for (int j = 0; j < o; ++j) {
            const float send = hi ? v[j] : v[j + o];
            const float keep = hi ? v[j + o] : v[j];
            v[j] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
    }
    float* wsum = zt;                            // [R_WARPS][32] (the tile is no longer read)
    wsum[wi * 32 + l] = v[0];
    __syncthreads();
    if (tid < C) {
        float t = 0.f;
#pragma unroll
        for (int k = 1; k < R_WARPS; ++k) t += wsum[k * 32 + tid];
        a.db_part[((int64_t)s * n_blk + blk) * C + tid] = t;
    }
    if (tid == 32) {
        float t = 0.f;
        for (int k = 0; k < R_WARPS; ++k) t += red[k];
        a.loss_part[(int64_t)s * n_blk + blk] = t;
    }
    if constexpr (FUSED) fused::free_tmem(tmem);     // every warp's reads of tensor memory ended before the barriers above
}

template <int CB, int TW>
size_t rows_smem_bytes(int C, bool conf)
{
    constexpr size_t TZ = (size_t)TZ_H * TW;
    const size_t plain = ((size_t)CB * TZ + (size_t)C * TZ + (size_t)R_WARPS * C * 32 * 2 + (conf ? (size_t)C * C : 0)) * sizeof(float) + 128;
    if (TW != kTwFused) return plain;
    return fused::smem_bytes(plain);      // the feature stages and the weights lie over the kernel's arrays
}

template <int CB>
cudaError_t prepare_cb(int C)
{
    cudaError_t e = cudaFuncSetAttribute(upsample_ce_rows_kernel<CB, false, kTwLoad>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rows_smem_bytes<CB, kTwLoad>(C, false));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(upsample_ce_rows_kernel<CB, true, kTwLoad>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rows_smem_bytes<CB, kTwLoad>(C, true));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(upsample_ce_rows_kernel<CB, false, kTwFused>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rows_smem_bytes<CB, kTwFused>(C, false));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(upsample_ce_rows_kernel<CB, true, kTwFused>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rows_smem_bytes<CB, kTwFused>(C, true));
    return e;
}

template <int CB>
cudaError_t launch_cb(const UpsampleCeArgs& a, const CUtensorMap& z_map, const CUtensorMap& x_map, const CUtensorMap& w_map, cudaStream_t s)
{
    dim3 grid((unsigned)((a.w + RN_X - 1) / RN_X), (unsigned)((a.h + RN_Y - 1) / RN_Y), (unsigned)a.S);
    const bool early = a.chain_early != 0 || a.x_early != 0;
    if (a.fused) {
        if (a.conf) return launch_chain(early, upsample_ce_rows_kernel<CB, true, kTwFused>, grid, dim3(R_THREADS), rows_smem_bytes<CB, kTwFused>(a.C, true), s, a, z_map, x_map, w_map);
        return launch_chain(early, upsample_ce_rows_kernel<CB, false, kTwFused>, grid, dim3(R_THREADS), rows_smem_bytes<CB, kTwFused>(a.C, false), s, a, z_map, x_map, w_map);
    }
    if (a.conf) return launch_chain(early, upsample_ce_rows_kernel<CB, true, kTwLoad>, grid, dim3(R_THREADS), rows_smem_bytes<CB, kTwLoad>(a.C, true), s, a, z_map, x_map, w_map);
    return launch_chain(early, upsample_ce_rows_kernel<CB, false, kTwLoad>, grid, dim3(R_THREADS), rows_smem_bytes<CB, kTwLoad>(a.C, false), s, a, z_map, x_map, w_map);
}

// class-count buckets: the two workload sizes exactly, multiples of four otherwise
int bucket(int C)
{
    if (C == 19 || C == 21) return C;
    return (C + 3) / 4 * 4;
}

}  // namespace

bool upsample_ce_rows_supported(int C) { return C <= 32; }

int upsample_ce_rows_blocks(int h, int w) { return ((h + RN_Y - 1) / RN_Y) * ((w + RN_X - 1) / RN_X); }

#define ST_ROWS_DISPATCH(FN, C, ...)                 \
    switch (bucket(C)) {                             \
        case 4: return FN<4>(__VA_ARGS__);           \
        case 8: return FN<8>(__VA_ARGS__);           \
        case 12: return FN<12>(__VA_ARGS__);         \
        case 16: return FN<16>(__VA_ARGS__);         \
        case 19: return FN<19>(__VA_ARGS__);         \
        case 20: return FN<20>(__VA_ARGS__);         \
        case 21: return FN<21>(__VA_ARGS__);         \
        case 24: return FN<24>(__VA_ARGS__);         \
        case 28: return FN<28>(__VA_ARGS__);         \
        default: return FN<32>(__VA_ARGS__);         \
    }

cudaError_t prepare_upsample_ce_rows(int C) { ST_ROWS_DISPATCH(prepare_cb, C, C) }

cudaError_t launch_rows_dispatch(const UpsampleCeArgs& a, const CUtensorMap& z_map, const CUtensorMap& x_map, const CUtensorMap& w_map, cudaStream_t s)
{
    ST_ROWS_DISPATCH(launch_cb, a.C, a, z_map, x_map, w_map, s)
}

void launch_upsample_ce_rows(const UpsampleCeArgs& a, const CUtensorMap* z_map, cudaStream_t s, const CUtensorMap* x_map, const CUtensorMap* w_map)
{
    CUtensorMap none;
    memset(&none, 0, sizeof(none));
    UpsampleCeArgs b = a;
    if (b.fused && !(x_map && w_map && fused_forward_supported(b.C, b.h, b.w, b.kblocks * 64))) b.fused = 0;
    if (b.fused) { b.has_map = 0; launch_rows_dispatch(b, none, *x_map, *w_map, s); return; }
    b.x_early = 0;
    if (!(b.has_map && z_map)) b.has_map = 0;
    launch_rows_dispatch(b, b.has_map ? *z_map : none, none, none, s);
}

// The block multiplies its own logits when the classifier is a 1x1 layer over at most 256 channels (a multiple of 64)
// and the feature map is at least one tile large.
bool fused_forward_supported(int C, int h, int w, int c_in)
{
    return upsample_ce_rows_supported(C) && c_in >= 64 && c_in % 64 == 0 && c_in / 64 <= fused::kMaxKBlocks && w >= fused::kTileCols && h >= fused::kTileRows;
}

bool make_logit_tile_map(CUtensorMap* m, const float* z, int S, int C, int h, int w)
{
    if (!upsample_ce_rows_supported(C) || w % 4 != 0 || w < kTwLoad || h < TZ_H || ((uintptr_t)z & 15u)) return false;
    const uint64_t dims[3] = {(uint64_t)w, (uint64_t)h, (uint64_t)S * C};
    const uint64_t strides[2] = {(uint64_t)w * sizeof(float), (uint64_t)h * w * sizeof(float)};
    const uint32_t box[3] = {(uint32_t)kTwLoad, (uint32_t)TZ_H, (uint32_t)C};
    char err[128];
    return encode_tensor_map(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, CU_TENSOR_MAP_SWIZZLE_NONE, z, 3, dims, strides, box, err,
                             sizeof(err), "logit tile");
}

bool make_feature_tile_map(CUtensorMap* m, const bf16* x, int S, int c_in, int h, int w)
{
    if (c_in % 64 != 0 || w < kTwFused || h < TZ_H || ((uintptr_t)x & 15u)) return false;
    const uint64_t c = (uint64_t)c_in;
    const uint64_t dims[4] = {c, (uint64_t)w, (uint64_t)h, (uint64_t)S};
    const uint64_t strides[3] = {c * 2, (uint64_t)w * c * 2, (uint64_t)h * w * c * 2};
    const uint32_t box[4] = {64, (uint32_t)kTwFused, (uint32_t)TZ_H, 1};
    char err[128];
    return encode_tensor_map(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, x, 4, dims, strides, box, err,
                             sizeof(err), "feature tile");
}

}  // namespace st
