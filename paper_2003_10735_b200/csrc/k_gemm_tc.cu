// bf16 tensor-core GEMMs of the head (gemm_precision 1): Forward and PartialBackward of Algorithm 1
// for the trainable back part (Section 4.2), as TMA-fed tcgen05 kernels with fp32 accumulators in
// tensor memory.  Operands are bf16 (cached features, bf16 copies of the weights, rounded
// gradients); every accumulation is fp32.
//
//   fwd 1x1   z[c][pix]       = b[c] + sum_k A[pix][k] W[c][k]                 A = features or hidden
//   fwd 3x3   Hd[pix][co]     = ReLU(b1[co] + sum_{tap,ci} X[pix+tap][ci] W1[tap][co][ci])
//   wgrad 1x1 dW[c][k]        = sum_pix dz[c][pix] A[pix][k]                   split over pixel ranges
//   dgrad     dHd[pix][k]     = [Hd[pix][k] > 0] sum_c dz[c][pix] W2[c][k]     (bf16 out)
//   wgrad 3x3 dW1[tap][co][ci]= sum_pix dHd[pix][co] X[pix+tap][ci]            split over pixel ranges
//
// Pixel-major activations [pix][channel] are K-major operands when the GEMM reduces over channels
// (forward) and MN-major operands when it reduces over pixels (weight gradients); both forms are
// read straight from the same TMA 128-byte-swizzled tiles, no transposing pass exists.
// The zero padding of the 3x3 convolution is TMA's out-of-bounds fill: taps are plain box loads at
// shifted (x, y) coordinates of a [channel][x][y][stream] tensor map.
#include "st_internal.h"
#include "tc_common.cuh"
#include "train_ctl.cuh"

#include <cstdio>
#include <cstring>

namespace st {

using namespace tc;

namespace {

constexpr int kThreadsTc = 128;          // 4 warps: TMEM lanes 32w .. 32w+31 belong to warp w
constexpr int kBlockK = 64;              // bf16 elements per 128-byte swizzled row
constexpr int kTileM = 128;              // UMMA M
constexpr int kChunkPix = 64;            // pixels per pipeline stage of the weight-gradient GEMMs
constexpr int kTileW = 32, kTileH = 4;   // 3x3 forward: 128 pixels = 4 rows x 32 columns
constexpr int kChunkW = 32, kChunkH = 2; // 3x3 wgrad: 64 pixels = 2 rows x 32 columns
constexpr int kSmemAlign = 1024;
constexpr int kMaxKBlocks = 16;
#ifndef ST_WG1_STAGES
#define ST_WG1_STAGES 3
#endif
constexpr int kWg1Stages = ST_WG1_STAGES;   // pipeline depth of the 1x1 weight gradient (20 KB per stage at 128 channels per block)

__device__ __forceinline__ uint8_t* align_smem(uint8_t* p)
{
    return (uint8_t*)(((uintptr_t)p + kSmemAlign - 1) & ~(uintptr_t)(kSmemAlign - 1));
}

// ------------------------------------------------------------------------------------------------
// fwd 1x1: one 128-pixel tile per block; the whole K extent is loaded at once (one barrier per
// 64-channel block so that the MMAs start while later blocks are still in flight).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreadsTc)
tc_fwd1x1_kernel(const __grid_constant__ CUtensorMap tmA,   // {K, p, S}  box {64, 128, 1}
                 const __grid_constant__ CUtensorMap tmB,   // {K, 32, S} box {64, 32, 1}
                 const float* __restrict__ theta, int64_t n_params, int64_t b_off,
                 float* __restrict__ z, int C, int p, int kblocks, unsigned int* err, const int* __restrict__ skip, int64_t skip_stride,
                 int a_early, uint32_t spin_limit, uint32_t stall_bytes)
{
    // spin_limit / stall_bytes: kSpinLimit and 0 in normal use.  A test of the give-up path lowers the limit and makes
    // the first barrier expect stall_bytes more than its copies deliver, so that the wait on it runs out: every copy
    // that was issued still lands, the kernel records where it gave up, writes nothing, frees its tensor memory and
    // returns.
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_smem(smem_raw);
    const uint32_t a_base = smem_u32(smem);
    const uint32_t b_base = a_base + kblocks * (kTileM * 128);
    __shared__ __align__(8) uint64_t bars[kMaxKBlocks + 1];
    __shared__ uint32_t tmem_slot, gave_up;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int s = blockIdx.y, pix0 = blockIdx.x * kTileM;

    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 32);
    if (tid == 0) {
        for (int i = 0; i <= kblocks; ++i) mbar_init(smem_u32(&bars[i]), 1);
        gave_up = 0;
        fence_barrier_init();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    // a_early: the kernel before this one on the stream (the previous iteration's parameter update) writes the weights
    // but not the activations, and this kernel was launched to start while that one still runs: the activation tile
    // is fetched now, the weights after the wait.  Each barrier expects both parts.
    if (a_early && tid == 0) {
        for (int kb = 0; kb < kblocks; ++kb) {
            const uint32_t bar = smem_u32(&bars[kb]);
            mbar_expect_tx(bar, kTileM * 128 + kClassPad * 128 + (kb == 0 ? stall_bytes : 0u));
            tma_load_3d(a_base + kb * (kTileM * 128), &tmA, bar, kb * kBlockK, pix0, s);
        }
    }
    pdl_wait();                  // the weights (and, without a_early, the activations) come from the previous kernel
    if (skip && skip[(int64_t)blockIdx.y * skip_stride]) {     // this stream's training loop has ended (block-uniform; the flag
        tc_fence_before_sync();                                 // comes from an earlier kernel, so it is read after the wait)
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, 32);
        return;
    }
    const uint32_t done_bar = smem_u32(&bars[kblocks]);
    bool ok = true;

    if (tid == 0) {
        for (int kb = 0; kb < kblocks; ++kb) {
            const uint32_t bar = smem_u32(&bars[kb]);
            if (!a_early) {
                mbar_expect_tx(bar, kTileM * 128 + kClassPad * 128 + (kb == 0 ? stall_bytes : 0u));
                tma_load_3d(a_base + kb * (kTileM * 128), &tmA, bar, kb * kBlockK, pix0, s);
            }
            tma_load_3d(b_base + kb * (kClassPad * 128), &tmB, bar, kb * kBlockK, 0, s);
        }
    } else if (tid == 32) {
        constexpr uint32_t idesc = instr_desc(kTileM, kClassPad, 0, 0);
        for (int kb = 0; kb < kblocks; ++kb) {
            ok = mbar_wait(smem_u32(&bars[kb]), 0, err, kWaitFull, spin_limit);
            if (!ok) { gave_up = 1; break; }
            tc_fence_after_sync();
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint64_t da = smem_desc(a_base + kb * (kTileM * 128) + k * 32, 16, 1024);
                const uint64_t db = smem_desc(b_base + kb * (kClassPad * 128) + k * 32, 16, 1024);
                umma(tmem, da, db, idesc, (kb | k) != 0);
            }
        }
        umma_commit(done_bar);
    }
    __syncwarp();
    ok = mbar_wait(done_bar, 0, err, kWaitDone);
    pdl_launch_dependents();     // only the epilogue is left
    tc_fence_after_sync();
    __syncthreads();
    if (gave_up) ok = false;     // the issuing thread ran out of patience: nothing was multiplied, nothing is written
    if (ok) {
        float v[32];
        tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16), v);
        const int pix = pix0 + tid;
        if (pix < p) {
            const float* bias = theta + (int64_t)s * n_params + b_off;
            float* dst = z + (int64_t)s * C * p + pix;
#pragma unroll
            for (int c = 0; c < kClassPad; ++c)
                if (c < C) dst[(int64_t)c * p] = v[c] + __ldg(bias + c);
        }
    } else {
        drain_after_error();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 32);
}

// ------------------------------------------------------------------------------------------------
// wgrad 1x1: D[k][c] += sum over this block's pixel chunks of A[pix][k] * dz[c][pix].
// A (pixel-major activations) is the MN-major operand with M = channel; dz rows are K-major.
// ------------------------------------------------------------------------------------------------
template <int STAGES>
__global__ void __launch_bounds__(kThreadsTc)
tc_wgrad1x1_kernel(const __grid_constant__ CUtensorMap tmA,   // {K, p, S}      box {64, 64, 1}
                   const __grid_constant__ CUtensorMap tmB,   // {p, 32, S}     box {64, 32, 1}
                   float* __restrict__ partials,              // [S][n_split][32][K]
                   int K, int n_chunks, int chunks_per_block, int m_split, int tmem_cols, unsigned int* err,
                   const int* __restrict__ skip, int64_t skip_stride, int a_early, int has_ctl, const TrainCtl ctl)
{
    // Train: the block after the last one of the weight gradient assesses the prediction (metric, best so far, break)
    // while the others multiply; it takes no part in anything below
    if (has_ctl && blockIdx.x == gridDim.x - 1) {
        const int s = blockIdx.y;
        const TrainHistory hist = train_history(ctl, s);
        pdl_wait();
        bool stop, better;
        train_decision(ctl, s, true, hist, nullptr, stop, better);
        pdl_launch_dependents();
        return;
    }
    const int n_blocks_x = (int)gridDim.x - (has_ctl ? 1 : 0);
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_smem(smem_raw);
    // m_split blocks share a pixel range, each with its own 128-channel accumulators: with the channels divided the
    // pixel ranges are longer and fewer, and the update has that many fewer partial sums to add per weight
    const int m_all = (K + kTileM - 1) / kTileM;     // accumulators (128 channels each) of the whole layer
    const int m_tiles = m_all / m_split;             // ... of this block
    const int m0 = ((int)blockIdx.x % m_split) * m_tiles;
    const int a_blocks = m_tiles * 2;                // 64-channel blocks loaded per stage (absent ones are zero-filled)
    const uint32_t a_stage_bytes = a_blocks * (kChunkPix * 128);
    const uint32_t stage_bytes = a_stage_bytes + kClassPad * 128;
    const uint32_t base = smem_u32(smem);
    __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES], done;
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int s = blockIdx.y, split = (int)blockIdx.x / m_split, n_split = n_blocks_x / m_split;
    const int c_begin = split * chunks_per_block;
    const int c_end = min(n_chunks, c_begin + chunks_per_block);

    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), tmem_cols);
    if (tid == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(smem_u32(&full[i]), 1); mbar_init(smem_u32(&empty[i]), 1); }
        mbar_init(smem_u32(&done), 1);
        fence_barrier_init();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    // a_early: the activations are the frozen features, which no kernel of the loop writes, and this kernel may have been
    // launched while its predecessor (which produces the logit gradient) is still running: the activation part of the
    // first stages is fetched now, the gradient part after the wait.  Each barrier expects both parts.
    const int n_pre = a_early ? min(STAGES, c_end - c_begin) : 0;
    if (tid == 0)
        for (int it = 0; it < n_pre; ++it) {
            const uint32_t bar = smem_u32(&full[it]), sa = base + it * stage_bytes;
            mbar_expect_tx(bar, stage_bytes);
            for (int cb = 0; cb < a_blocks; ++cb)
                tma_load_3d(sa + cb * (kChunkPix * 128), &tmA, bar, (2 * m0 + cb) * kBlockK, (c_begin + it) * kChunkPix, s);
        }
    pdl_wait();                  // inputs come from the previous kernel of the step
    if (skip && skip[(int64_t)blockIdx.y * skip_stride]) {     // this stream's training loop has ended (block-uniform; the flag
        tc_fence_before_sync();                                 // comes from an earlier kernel, so it is read after the wait)
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, tmem_cols);
        return;
    }
    bool ok = true;

    if (tid == 0) {
        for (int i = c_begin; i < c_end; ++i) {
            const int it = i - c_begin, st = it % STAGES;
            if (it >= STAGES) ok = mbar_wait(smem_u32(&empty[st]), ((it / STAGES) - 1) & 1, err, kWaitEmpty);
            if (!ok) break;
            const uint32_t bar = smem_u32(&full[st]);
            const uint32_t sa = base + st * stage_bytes;
            if (it >= n_pre) {
                mbar_expect_tx(bar, stage_bytes);
                for (int cb = 0; cb < a_blocks; ++cb)
                    tma_load_3d(sa + cb * (kChunkPix * 128), &tmA, bar, (2 * m0 + cb) * kBlockK, i * kChunkPix, s);
            }
            tma_load_3d(sa + a_stage_bytes, &tmB, bar, i * kChunkPix, 0, s);
        }
    } else if (tid == 32) {
        constexpr uint32_t idesc = instr_desc(kTileM, kClassPad, 1, 0);
        for (int i = c_begin; i < c_end; ++i) {
            const int it = i - c_begin, st = it % STAGES;
            ok = mbar_wait(smem_u32(&full[st]), (it / STAGES) & 1, err, kWaitFull);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t sa = base + st * stage_bytes, sb = sa + a_stage_bytes;
            for (int m = 0; m < m_tiles; ++m)
#pragma unroll
                for (int j = 0; j < kChunkPix / 16; ++j) {
                    const uint64_t da = smem_desc(sa + (2 * m) * (kChunkPix * 128) + j * (16 * 128), kChunkPix * 128, 1024);
                    const uint64_t db = smem_desc(sb + j * 32, 16, 1024);
                    umma(tmem + m * kClassPad, da, db, idesc, (it | j) != 0);
                }
            umma_commit(smem_u32(&empty[st]));
        }
        umma_commit(smem_u32(&done));
    }
    __syncwarp();
    ok = mbar_wait(smem_u32(&done), 0, err, kWaitDone);
    pdl_launch_dependents();     // only the epilogue is left
    tc_fence_after_sync();
    if (ok) {
        float* dst = partials + ((int64_t)s * n_split + split) * kClassPad * K;
        const bool any = c_end > c_begin;
        for (int m = 0; m < m_tiles; ++m) {
            float v[32];
            tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + m * kClassPad, v);
            const int k = (m0 + m) * kTileM + tid;
            if (k < K)
#pragma unroll
                for (int c = 0; c < kClassPad; ++c) dst[(int64_t)c * K + k] = any ? v[c] : 0.f;
        }
    } else {
        drain_after_error();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, tmem_cols);
}

// ------------------------------------------------------------------------------------------------
// fwd 3x3 (+bias, ReLU), persistent: one block per SM walks the tiles (4 rows x 32 columns of pixels,
// N = Ch output channels; K loop = 9 taps x Cin/64 channel blocks).  Three roles: warp 0 feeds a ring of
// shared-memory stages by TMA across tile boundaries (the pipeline never drains), warp 1 issues the
// MMAs into one of two tensor-memory accumulators, warps 2-5 drain the other accumulator (bias, ReLU,
// bf16, ReLU bit mask) while the next tile is being multiplied.
// ------------------------------------------------------------------------------------------------
constexpr int kFwd3Threads = 192;

__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// ------------------------------------------------------------------------------------------------
// fwd 1x1, persistent: gridDim.x blocks per stream walk the stream's 128-pixel tiles.  Three roles as in the 3x3
// forward: one thread feeds a ring of shared-memory stages by TMA across tile boundaries (one 128-pixel x 64-channel
// block per stage, 128 KB in flight), one thread issues the MMAs into one of two tensor-memory accumulators, the
// epilogue warps drain the other one (bias, fp32 logits, planar) meanwhile.  The classifier weights are loaded once
// per block.
// ------------------------------------------------------------------------------------------------
#ifndef ST_F1_STAGES
#define ST_F1_STAGES 8
#endif
constexpr int kF1Threads = 192, kF1Stages = ST_F1_STAGES;
constexpr uint32_t kF1StageBytes = kTileM * 128;

__global__ void __launch_bounds__(kF1Threads)
tc_fwd1x1p_kernel(const __grid_constant__ CUtensorMap tmA,   // {K, p, S}  box {64, 128, 1}
                  const __grid_constant__ CUtensorMap tmB,   // {K, 32, S} box {64, 32, 1}
                  const float* __restrict__ theta, int64_t n_params, int64_t b_off,
                  float* __restrict__ z, int C, int p, int kblocks, unsigned int* err,
                  const int* __restrict__ skip, int64_t skip_stride)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_smem(smem_raw);
    const uint32_t a_base = smem_u32(smem);
    const uint32_t b_base = a_base + kF1Stages * kF1StageBytes;
    __shared__ __align__(8) uint64_t full[kF1Stages], empty[kF1Stages], b_full, acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int s = blockIdx.y;
    const int n_items = (p + kTileM - 1) / kTileM;

    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 2 * kClassPad);
    if (tid == 0) {
        for (int i = 0; i < kF1Stages; ++i) { mbar_init(smem_u32(&full[i]), 1); mbar_init(smem_u32(&empty[i]), 1); }
        mbar_init(smem_u32(&b_full), 1);
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&acc_full[i]), 1); mbar_init(smem_u32(&acc_empty[i]), 4); }
        fence_barrier_init();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    pdl_wait();                  // inputs come from the previous kernel of the step
    if (skip && skip[(int64_t)blockIdx.y * skip_stride]) {     // this stream's training loop has ended (block-uniform; the flag
        tc_fence_before_sync();                                 // comes from an earlier kernel, so it is read after the wait)
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, 2 * kClassPad);
        return;
    }
    bool ok = true;

    if (tid == 0) {
        // ---- producer
        const uint32_t bb = smem_u32(&b_full);
        mbar_expect_tx(bb, (uint32_t)kblocks * kClassPad * 128);
        for (int kb = 0; kb < kblocks; ++kb) tma_load_3d(b_base + kb * (kClassPad * 128), &tmB, bb, kb * kBlockK, 0, s);
        int g = 0;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            for (int kb = 0; kb < kblocks; ++kb, ++g) {
                const int st = g % kF1Stages;
                if (g >= kF1Stages) ok = mbar_wait(smem_u32(&empty[st]), ((g / kF1Stages) - 1) & 1, err, kWaitEmpty);
                if (!ok) break;
                const uint32_t bar = smem_u32(&full[st]);
                mbar_expect_tx(bar, kF1StageBytes);
                tma_load_3d(a_base + st * kF1StageBytes, &tmA, bar, kb * kBlockK, it * kTileM, s);
            }
        }
        pdl_launch_dependents();     // every load is issued: the next kernel of the step may set itself up
    } else if (tid == 32) {
        // ---- MMA issuer
        constexpr uint32_t idesc = instr_desc(kTileM, kClassPad, 0, 0);
        ok = mbar_wait(smem_u32(&b_full), 0, err, kWaitFull);
        int g = 0, j = 0;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++j) {
            const int buf = j & 1;
            if (j >= 2) ok = mbar_wait(smem_u32(&acc_empty[buf]), ((j >> 1) - 1) & 1, err, kWaitEmpty);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t acc = tmem + buf * kClassPad;
            for (int kb = 0; kb < kblocks; ++kb, ++g) {
                const int st = g % kF1Stages;
                ok = mbar_wait(smem_u32(&full[st]), (g / kF1Stages) & 1, err, kWaitFull);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t sa = a_base + st * kF1StageBytes, sb = b_base + kb * (kClassPad * 128);
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma(acc, smem_desc(sa + k * 32, 16, 1024), smem_desc(sb + k * 32, 16, 1024), idesc, (kb | k) != 0);
                umma_commit(smem_u32(&empty[st]));
            }
            if (ok) umma_commit(smem_u32(&acc_full[buf]));
        }
    } else if (warp >= 2) {
        // ---- epilogue warps: TMEM lanes 32*(warp % 4) .. +31 = pixels of the tile
        const int q = warp & 3;
        const float* bias = theta + (int64_t)s * n_params + b_off;
        int j = 0;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++j) {
            const int buf = j & 1;
            ok = mbar_wait(smem_u32(&acc_full[buf]), (j >> 1) & 1, err, kWaitDone);
            if (!ok) break;
            tc_fence_after_sync();
            float v[32];
            tmem_ld_32x32(tmem + ((uint32_t)(q * 32) << 16) + buf * kClassPad, v);
            const int pix = it * kTileM + q * 32 + lane;
            if (pix < p) {
                float* dst = z + (int64_t)s * C * p + pix;
#pragma unroll
                for (int c = 0; c < kClassPad; ++c)
                    if (c < C) dst[(int64_t)c * p] = v[c] + __ldg(bias + c);
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));
        }
    }
    if (!ok) drain_after_error();
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 2 * kClassPad);
}

// MODE 0: the layer's forward (bias, ReLU, bf16 output, one ReLU bit per output value).
// MODE 1: the gradient passed back through the layer to the block before it: the same tile walk over the layer's output
//         gradient with the weights transposed and their taps mirrored (prepared by the update kernel); the epilogue
//         applies the ReLU mask of the receiving block, writes bf16 and emits per-tile channel sums of the unrounded
//         values (the receiving block's bias gradient).
// The K loop runs over 9 taps x (kblocks1 + kblocks2) channel blocks: the first kblocks1 come from tmA (the previous
// block's output, or the frozen part's), the others from tmA2 (the block's skip input): the concatenation of
// Section 5.2 is never materialised.
template <int STAGES, int MODE>
__global__ void __launch_bounds__(kFwd3Threads)
tc_fwd3x3_kernel(const __grid_constant__ CUtensorMap tmA,   // {C1, w, h, S}     box {64, 32, 4, 1}
                 const __grid_constant__ CUtensorMap tmA2,  // {C2, w, h, S}     box {64, 32, 4, 1} (unused if kblocks2 == 0)
                 int kblocks1, int kblocks2,
                 const __grid_constant__ CUtensorMap tmB,   // {C1+C2, 9*Ch, S}  box {64, Ch, 1}
                 const __grid_constant__ CUtensorMap tmBq,  // same tensor, box {64, 64, 1}: one block of 64 output channels
                 int tail_split,                             // the tiles of the last, partly filled round are cut into this many
                                                             // ranges of output channels (1, 2 or 4), one work item each
                 const float* __restrict__ theta, int64_t n_params, int64_t b_off,   // MODE 0: bias
                 bf16* __restrict__ out,                     // [S][p][Ch]
                 uint32_t* __restrict__ relu_bits,           // [S][p][Ch/32]: bit k of word j = out[32j + k] > 0 (MODE 0: written;
                                                             //   MODE 1: the receiving block's bits, read)
                 float* __restrict__ b_partials,             // MODE 1: [S][tiles per stream][Ch] channel sums of each tile
                 int Ch, int h, int w, int n_tiles_total, int acc_cols, unsigned int* err, const int* __restrict__ skip, int64_t skip_stride)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_smem(smem_raw);
    const uint32_t base = smem_u32(smem);
    const uint32_t a_bytes = kTileM * 128, b_bytes = (uint32_t)Ch * 128, stage_bytes = a_bytes + b_bytes;
    __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_slot;
    __shared__ float part[MODE == 1 ? 4 * 256 : 1];             // MODE 1: per-warp channel sums of the tile
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int tiles_x = (w + kTileW - 1) / kTileW, tiles_y = (h + kTileH - 1) / kTileH;
    const int tiles_per_stream = tiles_x * tiles_y;
    const int kblocks = kblocks1 + kblocks2, n_iter = 9 * kblocks;
    // Work items: whole tiles while every block has one, then the remaining tiles in tail_split pieces each, so that
    // the last round is short instead of leaving most blocks idle for a full tile's time.
    const int n_full = tail_split > 1 ? (n_tiles_total / (int)gridDim.x) * (int)gridDim.x : n_tiles_total;
    const int n_items = n_full + (n_tiles_total - n_full) * tail_split;
    struct Item { int tile, ch0, chn; };
    auto item_of = [&](int wi) {
        Item it;
        if (wi < n_full) { it.tile = wi; it.ch0 = 0; it.chn = Ch; }
        else { const int q = wi - n_full; it.tile = n_full + q / tail_split; it.chn = Ch / tail_split; it.ch0 = (q % tail_split) * it.chn; }
        return it;
    };

    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), 2 * acc_cols);
    if (tid == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(smem_u32(&full[i]), 1); mbar_init(smem_u32(&empty[i]), 1); }
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&acc_full[i]), 1); mbar_init(smem_u32(&acc_empty[i]), 4); }
        fence_barrier_init();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    pdl_wait();                  // inputs come from the previous kernel of the step
    bool ok = true;

    if (tid == 0) {
        // ---- producer: the ring index runs on across tiles
        int g = 0;
        for (int wi = blockIdx.x; wi < n_items && ok; wi += gridDim.x) {
            const Item im = item_of(wi);
            const int s = im.tile / tiles_per_stream, tt = im.tile % tiles_per_stream;
            if (skip && skip[(int64_t)s * skip_stride]) continue;     // all three roles leave out the same items
            const int x0 = (tt % tiles_x) * kTileW, y0 = (tt / tiles_x) * kTileH;
            // One stage: wait for its slot, then the activation block (from `src`, whose tensor map is fixed at each of
            // the two places this is expanded: a map chosen at run time costs every copy a slow look-up) and the weights.
#define ST_FWD3_STAGE(src, a_coord)                                                                                       \
            {                                                                                                             \
                const int st = g % STAGES;                                                                                \
                if (g >= STAGES) ok = mbar_wait(smem_u32(&empty[st]), ((g / STAGES) - 1) & 1, err, kWaitEmpty);          \
                if (!ok) break;                                                                                           \
                const uint32_t bar = smem_u32(&full[st]), sa = base + st * stage_bytes;                                   \
                mbar_expect_tx(bar, a_bytes + (uint32_t)im.chn * 128);                                                    \
                tma_load_4d(sa, &(src), bar, (a_coord), x0 + tap % 3 - 1, y0 + tap / 3 - 1, s);                          \
                if (im.chn == Ch) tma_load_3d(sa + a_bytes, &tmB, bar, kb * kBlockK, tap * Ch, s);                        \
                else                                                                                                      \
                    for (int j = 0; j < im.chn / 64; ++j)        /* 64 weight rows per copy, laid out like the single copy */ \
                        tma_load_3d(sa + a_bytes + j * (64 * 128), &tmBq, bar, kb * kBlockK, tap * Ch + im.ch0 + j * 64, s); \
                ++g;                                                                                                      \
            }
            for (int tap = 0; tap < 9 && ok; ++tap) {
                int kb = 0;
                for (; kb < kblocks1; ++kb) ST_FWD3_STAGE(tmA, kb * kBlockK)
                for (; kb < kblocks && ok; ++kb) ST_FWD3_STAGE(tmA2, (kb - kblocks1) * kBlockK)
            }
#undef ST_FWD3_STAGE
        }
        pdl_launch_dependents();     // every load is issued: the next kernel of the step may set itself up
    } else if (tid == 32) {
        // ---- MMA issuer
        int g = 0, j = 0;
        for (int wi = blockIdx.x; wi < n_items && ok; wi += gridDim.x) {
            const Item im = item_of(wi);
            if (skip && skip[(int64_t)(im.tile / tiles_per_stream) * skip_stride]) continue;
            const uint32_t idesc = instr_desc(kTileM, im.chn, 0, 0);
            const int buf = j & 1;
            if (j >= 2) ok = mbar_wait(smem_u32(&acc_empty[buf]), ((j >> 1) - 1) & 1, err, kWaitEmpty);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t acc = tmem + buf * acc_cols;
            for (int it = 0; it < n_iter; ++it, ++g) {
                const int st = g % STAGES;
                ok = mbar_wait(smem_u32(&full[st]), (g / STAGES) & 1, err, kWaitFull);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t sa = base + st * stage_bytes, sb = sa + a_bytes;
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    umma(acc, smem_desc(sa + k * 32, 16, 1024), smem_desc(sb + k * 32, 16, 1024), idesc, (it | k) != 0);
                umma_commit(smem_u32(&empty[st]));
            }
            if (ok) umma_commit(smem_u32(&acc_full[buf]));
            ++j;                                                       // j counts the tiles this block works on
        }
    } else if (warp >= 2) {
        // ---- epilogue warps: TMEM lanes 32*(warp % 4) .. +31 = pixel rows of the tile
        const int q = warp & 3, row = q * 32 + lane;
        int j = 0;
        for (int wi = blockIdx.x; wi < n_items && ok; wi += gridDim.x) {
            const Item im = item_of(wi);
            const int s = im.tile / tiles_per_stream, tt = im.tile % tiles_per_stream;
            if (skip && skip[(int64_t)s * skip_stride]) continue;
            const int buf = j & 1;
            const int x = (tt % tiles_x) * kTileW + row % kTileW, y = (tt / tiles_x) * kTileH + row / kTileW;
            ok = mbar_wait(smem_u32(&acc_full[buf]), (j >> 1) & 1, err, kWaitDone);
            if (MODE == 1) {                                           // the four epilogue warps stay together: they share `part`
                int all_ok;
                asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 p, %1, 0;\n\tbarrier.cta.red.and.pred q, 1, 128, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                             : "=r"(all_ok) : "r"((int)ok) : "memory");
                ok = all_ok != 0;
            }
            if (!ok) break;
            tc_fence_after_sync();
            const bool in = y < h && x < w;
            const int64_t pixel = (int64_t)s * h * w + (int64_t)y * w + x;
            bf16* dst = out + pixel * Ch + im.ch0;
            const float* bias = theta + (int64_t)s * n_params + b_off + im.ch0;
            for (int n0 = 0; n0 < im.chn; n0 += 32) {
                float v[32];
                tmem_ld_32x32(tmem + ((uint32_t)(q * 32) << 16) + buf * acc_cols + n0, v);
                if (MODE == 0) {
                    if (in) {
                        uint4 o4[4];
                        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(o4);
                        uint32_t bits = 0;
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            const float a = fmaxf(v[2 * k] + __ldg(bias + n0 + 2 * k), 0.f), b = fmaxf(v[2 * k + 1] + __ldg(bias + n0 + 2 * k + 1), 0.f);
                            o2[k] = __floats2bfloat162_rn(a, b);
                            // the mask is taken on the stored (rounded) activation, the value the next layer sees
                            bits |= (__low2float(o2[k]) > 0.f ? 1u : 0u) << (2 * k);
                            bits |= (__high2float(o2[k]) > 0.f ? 1u : 0u) << (2 * k + 1);
                        }
                        store_256(dst + n0, reinterpret_cast<const uint32_t*>(o4));            // 32 channels = 64 bytes
                        store_256(dst + n0 + 16, reinterpret_cast<const uint32_t*>(o4) + 8);
                        relu_bits[pixel * (Ch / 32) + (im.ch0 + n0) / 32] = bits;
                    }
                } else {
                    if (in) {
                        const uint32_t bits = __ldg(relu_bits + pixel * (Ch / 32) + (im.ch0 + n0) / 32);
                        uint4 o4[4];
                        __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(o4);
#pragma unroll
                        for (int k = 0; k < 16; ++k) {
                            if (!((bits >> (2 * k)) & 1u)) v[2 * k] = 0.f;
                            if (!((bits >> (2 * k + 1)) & 1u)) v[2 * k + 1] = 0.f;
                            o2[k] = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
                        }
                        store_256(dst + n0, reinterpret_cast<const uint32_t*>(o4));
                        store_256(dst + n0 + 16, reinterpret_cast<const uint32_t*>(o4) + 8);
                    } else {
#pragma unroll
                        for (int k = 0; k < 32; ++k) v[k] = 0.f;
                    }
                    // sums over the warp's 32 pixels in a fixed order: a reduce-scatter over the lanes, after which lane c
                    // holds the sum of channel n0 + c
#pragma unroll
                    for (int half = 16; half >= 1; half >>= 1) {
                        const bool up = (lane & half) != 0;
#pragma unroll
                        for (int k = 0; k < half; ++k) {
                            const float keep = up ? v[k + half] : v[k];
                            const float send = up ? v[k] : v[k + half];
                            v[k] = keep + __shfl_xor_sync(0xffffffffu, send, half);
                        }
                    }
                    part[q * 256 + n0 + lane] = v[0];
                }
            }
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&acc_empty[buf]));     // this warp's quarter of the accumulator is free
            if (MODE == 1) {
                asm volatile("barrier.cta.sync 1, 128;" ::: "memory");
                const int e = (warp - 2) * 32 + lane;                  // 0..127 over the four epilogue warps
                for (int k = e; k < im.chn; k += 128)
                    b_partials[((int64_t)s * tiles_per_stream + tt) * Ch + im.ch0 + k] =
                        (part[k] + part[256 + k]) + (part[512 + k] + part[768 + k]);
                asm volatile("barrier.cta.sync 1, 128;" ::: "memory");
            }
            ++j;
        }
    }
    if (!ok) drain_after_error();
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, 2 * acc_cols);
}

// ------------------------------------------------------------------------------------------------
// wgrad 3x3: for one tap, D[ci][co] += sum over this block's pixel chunks of X[pix+tap][ci] * dHd[pix][co].
// Both operands are MN-major (pixel-major activations, reduction over pixels).  A block keeps
// ceil(Cin/128) accumulators of Ch columns (all input channels of one tap) so that the dHd tile of a
// stage is shared by all of them.
// ------------------------------------------------------------------------------------------------
template <int STAGES>
__global__ void __launch_bounds__(kThreadsTc)
tc_wgrad3x3_kernel(const __grid_constant__ CUtensorMap tmA,   // previous output {C1, w, h, S} box {64, 32, 2, 1}
                   const __grid_constant__ CUtensorMap tmA2,  // skip input      {C2, w, h, S} box {64, 32, 2, 1} (unused if C2 == 0)
                   int blocks1,                                // C1 / 64: input-channel blocks that come from tmA
                   const __grid_constant__ CUtensorMap tmB,   // dHd {Ch,  w, h, S} box {64, 32, 2, 1}
                   float* __restrict__ partials,              // [S][n_split][9][Ch][Cin]
                   int Cin, int Ch, int h, int w, int n_chunks, int chunks_per_block, int n_split,
                   int tmem_cols, unsigned int* err, const int* __restrict__ skip, int64_t skip_stride)
{
    // Cin = C1 + C2: the layer's input is the concatenation (previous output, skip input), read from its two sources
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_smem(smem_raw);
    const uint32_t base = smem_u32(smem);
    const int m_tiles = (Cin + kTileM - 1) / kTileM;
    const int a_blocks = m_tiles * 2, b_blocks = Ch / kBlockK;
    const uint32_t blk_bytes = kChunkPix * 128;
    const uint32_t a_bytes = a_blocks * blk_bytes, stage_bytes = a_bytes + b_blocks * blk_bytes;
    __shared__ __align__(8) uint64_t full[STAGES], empty[STAGES], done;
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int tap = blockIdx.x % 9, split = blockIdx.x / 9, s = blockIdx.y;
    const int chunks_x = (w + kChunkW - 1) / kChunkW;
    const int c_begin = split * chunks_per_block, c_end = min(n_chunks, c_begin + chunks_per_block);

    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), tmem_cols);
    if (tid == 0) {
        for (int i = 0; i < STAGES; ++i) { mbar_init(smem_u32(&full[i]), 1); mbar_init(smem_u32(&empty[i]), 1); }
        mbar_init(smem_u32(&done), 1);
        fence_barrier_init();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    pdl_wait();                  // inputs come from the previous kernel of the step
    if (skip && skip[(int64_t)blockIdx.y * skip_stride]) {     // this stream's training loop has ended (block-uniform; the flag
        tc_fence_before_sync();                                 // comes from an earlier kernel, so it is read after the wait)
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, tmem_cols);
        return;
    }
    bool ok = true;

    if (tid == 0) {
        for (int i = c_begin; i < c_end; ++i) {
            const int it = i - c_begin, st = it % STAGES;
            if (it >= STAGES) ok = mbar_wait(smem_u32(&empty[st]), ((it / STAGES) - 1) & 1, err, kWaitEmpty);
            if (!ok) break;
            const int x0 = (i % chunks_x) * kChunkW, y0 = (i / chunks_x) * kChunkH;
            const uint32_t bar = smem_u32(&full[st]), sa = base + st * stage_bytes;
            mbar_expect_tx(bar, stage_bytes);
            // blocks past the last channel arrive as zeros (out-of-range fill); two loops, each with its own tensor map
            // (a map chosen at run time costs every copy a slow look-up)
            const int n_first = blocks1 * kBlockK == Cin ? a_blocks : blocks1;
            int cb = 0;
            for (; cb < n_first; ++cb)
                tma_load_4d(sa + cb * blk_bytes, &tmA, bar, cb * kBlockK, x0 + tap % 3 - 1, y0 + tap / 3 - 1, s);
            for (; cb < a_blocks; ++cb)
                tma_load_4d(sa + cb * blk_bytes, &tmA2, bar, (cb - blocks1) * kBlockK, x0 + tap % 3 - 1, y0 + tap / 3 - 1, s);
            for (int cb = 0; cb < b_blocks; ++cb)
                tma_load_4d(sa + a_bytes + cb * blk_bytes, &tmB, bar, cb * kBlockK, x0, y0, s);
        }
    } else if (tid == 32) {
        const uint32_t idesc = instr_desc(kTileM, Ch, 1, 1);
        for (int i = c_begin; i < c_end; ++i) {
            const int it = i - c_begin, st = it % STAGES;
            ok = mbar_wait(smem_u32(&full[st]), (it / STAGES) & 1, err, kWaitFull);
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t sa = base + st * stage_bytes, sb = sa + a_bytes;
            for (int m = 0; m < m_tiles; ++m)
#pragma unroll
                for (int j = 0; j < kChunkPix / 16; ++j) {
                    const uint64_t da = smem_desc(sa + (2 * m) * blk_bytes + j * (16 * 128), blk_bytes, 1024);
                    const uint64_t db = smem_desc(sb + j * (16 * 128), blk_bytes, 1024);
                    umma(tmem + m * Ch, da, db, idesc, (it | j) != 0);
                }
            umma_commit(smem_u32(&empty[st]));
        }
        umma_commit(smem_u32(&done));
    }
    __syncwarp();
    ok = mbar_wait(smem_u32(&done), 0, err, kWaitDone);
    pdl_launch_dependents();     // only the epilogue is left
    tc_fence_after_sync();
    if (ok) {
        float* dst = partials + (((int64_t)s * n_split + split) * 9 + tap) * Ch * Cin;
        const bool any = c_end > c_begin;
        for (int m = 0; m < m_tiles; ++m) {
            const int ci = m * kTileM + tid;
            for (int n0 = 0; n0 < Ch; n0 += 32) {
                float v[32];
                tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + m * Ch + n0, v);
                if (ci < Cin)
#pragma unroll
                    for (int c = 0; c < 32; ++c) dst[(int64_t)(n0 + c) * Cin + ci] = any ? v[c] : 0.f;
            }
        }
    } else {
        drain_after_error();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, tmem_cols);
}

// ------------------------------------------------------------------------------------------------
// dgrad through the 1x1 output layer with the ReLU mask of the hidden activation:
//   dHd[pix][k] = [Hd[pix][k] > 0] * sum_c dz[c][pix] * W2[c][k]
// One 128-pixel tile per block, N = Ch, K = 32 class rows (rows >= C are zero in both operands).
// dz rows [c][pix] and weight rows [c][k] are both contiguous along the non-reduced index, so both are
// MN-major operands.  The epilogue applies the mask, writes bf16 (a GEMM operand next) and emits the
// block's sums over pixels of the unrounded result: the bias gradient of the 3x3 layer.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreadsTc)
tc_dgrad_kernel(const __grid_constant__ CUtensorMap tmA,   // dz  {p, 32, S}  box {64, 32, 1}
                const __grid_constant__ CUtensorMap tmB,   // W2  {Ch, 32, S} box {64, 32, 1}
                const uint32_t* __restrict__ relu_bits,     // [S][p][Ch/32]
                bf16* __restrict__ dhidden,                 // [S][p][Ch]
                float* __restrict__ b1_partials,            // [S][n_blocks][Ch]
                int Ch, int p, int tmem_cols, unsigned int* err, const int* __restrict__ skip, int64_t skip_stride)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_smem(smem_raw);
    const uint32_t a_base = smem_u32(smem);
    const uint32_t blk_bytes = kClassPad * 128;                 // 32 class rows x 64 elements
    const uint32_t b_base = a_base + 2 * blk_bytes;
    // gridDim.z blocks share a pixel tile, each with its own range of Ch / gridDim.z hidden channels (more and
    // shorter blocks: the kernel's time is the latency of one block's epilogue)
    const int Chb = Ch / (int)gridDim.z, ch0 = (int)blockIdx.z * Chb;
    const int b_blocks = Chb / kBlockK;
    __shared__ float part[4 * 256];                             // per-warp channel sums
    __shared__ __align__(8) uint64_t full, done;
    __shared__ uint32_t tmem_slot;
    const int tid = threadIdx.x, warp = tid >> 5;
    const int s = blockIdx.y, pix0 = blockIdx.x * kTileM;

    if (warp == 0) tmem_alloc(smem_u32(&tmem_slot), tmem_cols);
    if (tid == 0) {
        mbar_init(smem_u32(&full), 1); mbar_init(smem_u32(&done), 1);
        fence_barrier_init();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem = tmem_slot;
    pdl_wait();                  // inputs come from the previous kernel of the step
    if (skip && skip[(int64_t)blockIdx.y * skip_stride]) {     // this stream's training loop has ended (block-uniform; the flag
        tc_fence_before_sync();                                 // comes from an earlier kernel, so it is read after the wait)
        __syncthreads();
        if (warp == 0) tmem_dealloc(tmem, tmem_cols);
        return;
    }
    bool ok = true;

    if (tid == 0) {
        const uint32_t bar = smem_u32(&full);
        mbar_expect_tx(bar, (2 + b_blocks) * blk_bytes);
        tma_load_3d(a_base, &tmA, bar, pix0, 0, s);
        tma_load_3d(a_base + blk_bytes, &tmA, bar, pix0 + 64, 0, s);
        for (int cb = 0; cb < b_blocks; ++cb) tma_load_3d(b_base + cb * blk_bytes, &tmB, bar, ch0 + cb * kBlockK, 0, s);
    } else if (tid == 32) {
        const uint32_t idesc = instr_desc(kTileM, Chb, 1, 1);
        ok = mbar_wait(smem_u32(&full), 0, err, kWaitFull);
        if (ok) {
            tc_fence_after_sync();
#pragma unroll
            for (int j = 0; j < kClassPad / 16; ++j)
                umma(tmem, smem_desc(a_base + j * (16 * 128), blk_bytes, 1024), smem_desc(b_base + j * (16 * 128), blk_bytes, 1024),
                     idesc, j != 0);
        }
        umma_commit(smem_u32(&done));
    }
    __syncwarp();
    // the ReLU mask of this thread's pixel (one bit per hidden channel), fetched while the MMAs run
    const int pix = pix0 + tid;
    const bool in = pix < p;
    uint32_t mbits[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    if (in) {
        const uint32_t* mp = relu_bits + ((int64_t)s * p + pix) * (Ch / 32);
#pragma unroll
        for (int j = 0; j < 8; ++j) if (j < Chb / 32) mbits[j] = __ldg(mp + ch0 / 32 + j);
    }
    ok = mbar_wait(smem_u32(&done), 0, err, kWaitDone);
    pdl_launch_dependents();             // only the epilogue is left
    tc_fence_after_sync();
    ok = __syncthreads_and(ok);          // the epilogue below synchronises the block: all or none
    if (ok) {
        const int64_t row = ((int64_t)s * p + (in ? pix : 0)) * Ch;
        for (int n0 = 0; n0 < Chb; n0 += 32) {
            float v[32];
            tmem_ld_32x32(tmem + ((uint32_t)(warp * 32) << 16) + n0, v);
            if (in) {
                uint4 out[4];
                __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(out);
                uint32_t bits = 0;
#pragma unroll
                for (int j = 0; j < 8; ++j) if (j == n0 / 32) bits = mbits[j];
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    if (!((bits >> (2 * k)) & 1u)) v[2 * k] = 0.f;
                    if (!((bits >> (2 * k + 1)) & 1u)) v[2 * k + 1] = 0.f;
                    o2[k] = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
                }
                store_256(dhidden + row + ch0 + n0, reinterpret_cast<const uint32_t*>(out));
                store_256(dhidden + row + ch0 + n0 + 16, reinterpret_cast<const uint32_t*>(out) + 8);
            } else {
#pragma unroll
                for (int k = 0; k < 32; ++k) v[k] = 0.f;
            }
            // sums over the warp's 32 pixels, fixed order: a reduce-scatter over the lanes (lanes whose bit
            // is set keep the upper half of the channels), after which lane c holds the sum of channel n0 + c
            const int lane = tid & 31;
#pragma unroll
            for (int half = 16; half >= 1; half >>= 1) {
                const bool up = (lane & half) != 0;
#pragma unroll
                for (int k = 0; k < half; ++k) {
                    const float keep = up ? v[k + half] : v[k];
                    const float send = up ? v[k] : v[k + half];
                    v[k] = keep + __shfl_xor_sync(0xffffffffu, send, half);
                }
            }
            part[warp * 256 + n0 + lane] = v[0];
        }
        __syncthreads();
        for (int k = tid; k < Chb; k += kThreadsTc)
            b1_partials[((int64_t)s * gridDim.x + blockIdx.x) * Ch + ch0 + k] =
                (part[k] + part[256 + k]) + (part[512 + k] + part[768 + k]);
    } else {
        drain_after_error();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, tmem_cols);
}

// ---- host side -------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (fn) return fn;
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &q) != cudaSuccess || !ptr) return nullptr;
    fn = (EncodeTiledFn)ptr;
    return fn;
}

// bf16 tensor, innermost dimension first; strides (bytes) for dimensions 1..rank-1; 128-byte swizzle.
bool make_map(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides,
              const uint32_t* box, char* err, size_t err_len, const char* what)
{
    return encode_tensor_map(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, base, rank, dims, strides, box,
                             err, err_len, what);
}

int pow2_cols(int n) { int c = 32; while (c < n) c <<= 1; return c; }

void split_geometry(int n_chunks, int target_blocks, int* per, int* n_split)
{
    int pb = (n_chunks + target_blocks - 1) / target_blocks;
    if (pb < 1) pb = 1;
    *per = pb;
    *n_split = (n_chunks + pb - 1) / pb;
    if (*n_split < 1) *n_split = 1;
}

}  // namespace

bool encode_tensor_map(CUtensorMap* m, CUtensorMapDataType dtype, CUtensorMapSwizzle swizzle, const void* base, int rank,
                       const uint64_t* dims, const uint64_t* strides, const uint32_t* box, char* err, size_t err_len,
                       const char* what)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) { snprintf(err, err_len, "cuTensorMapEncodeTiled is not available"); return false; }
    cuuint64_t d[5], st[4];
    cuuint32_t b[5], es[5];
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; b[i] = box[i]; es[i] = 1; }
    for (int i = 0; i + 1 < rank; ++i) st[i] = strides[i];
    CUresult r = fn(m, dtype, (cuuint32_t)rank, const_cast<void*>(base), d, st, b, es, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                    CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { snprintf(err, err_len, "tensor map for %s rejected (CUresult %d)", what, (int)r); return false; }
    return true;
}

// the instantiation of a 3x3 kernel with a given pipeline depth (all depths share one function type)
template <int MODE>
static decltype(&tc_fwd3x3_kernel<4, MODE>) fwd3_kernel(int stages)
{
    return stages >= 8 ? tc_fwd3x3_kernel<8, MODE> : (stages >= 6 ? tc_fwd3x3_kernel<6, MODE> : tc_fwd3x3_kernel<4, MODE>);
}
static decltype(&tc_wgrad3x3_kernel<3>) wgrad3_kernel(int stages)
{
    return stages >= 5 ? tc_wgrad3x3_kernel<5> : (stages >= 4 ? tc_wgrad3x3_kernel<4> : tc_wgrad3x3_kernel<3>);
}

struct TcBlockPlan {
    CUtensorMap in_fwd, skip_fwd;    // the block's two inputs {C, w, h, S}, box {64, 32, 4, 1} (forward tiles)
    CUtensorMap in_wg, skip_wg;      // same tensors, box {64, 32, 2, 1} (weight-gradient chunks)
    CUtensorMap w_map, w_map_q;      // {c_tot, 9*c_out, S}, boxes {64, c_out, 1} and {64, 64, 1}
    CUtensorMap wt_map, wt_map_q;    // mirrored, transposed weights {c_out, 9*c_prev, S}, boxes {64, c_prev, 1} and {64, 64, 1}
    CUtensorMap dout_fwd;            // the block's output gradient {c_out, w, h, S}, box {64, 32, 4, 1} (A operand when passed back)
    CUtensorMap dout_wg;             // same tensor, box {64, 32, 2, 1} (B operand of the weight gradient)
    int cols_wg;                     // tensor-memory columns of the weight gradient
    int stages_fwd, stages_back, stages_wg;   // pipeline depths of the three kernels of this block
    size_t smem_fwd, smem_back, smem_wg;
};

struct TcPlan {
    TcBuffers b;
    int p, p_pad, c_last;
    CUtensorMap act_fwd;     // last-layer input {c_last, p, S} box {64, 128, 1}
    CUtensorMap act_wg;      // same tensor, box {64, 64, 1}
    CUtensorMap w2_map;      // {c_last, 32, S} box {64, 32, 1}
    CUtensorMap dz_map;      // {p, 32, S} box {64, 32, 1}
    TcBlockPlan blk[kMaxBlocks];
    int split2, chunks2, per2, cols2, msplit2;
    int split1, chunks1, per1;          // pixel chunks of the 3x3 weight gradients (the same for every block)
    size_t smem_fwd1, smem_fwd1p, smem_wg1, smem_dgrad;
    bool fwd1_persistent;
    int n_sms;
    bool test_stall;         // test of the give-up path (environment ST_TEST_STALL_FWD1X1=1 when the plan is made)
};

// blocks per pixel range of the 1x1 weight gradient: one per 128-channel accumulator
static int wgrad1x1_m_split(int c_last) { const int m = (c_last + kTileM - 1) / kTileM; return m < 1 ? 1 : m; }

int tc_wgrad_splits(int layer, int c_last, int h, int w)
{
    int per, n;
    if (layer == 2) {
        const int64_t p = (int64_t)h * w;
        split_geometry((int)((p + kChunkPix - 1) / kChunkPix), 148 / wgrad1x1_m_split(c_last), &per, &n);
    } else {
        const int chunks = ((w + kChunkW - 1) / kChunkW) * ((h + kChunkH - 1) / kChunkH);
        split_geometry(chunks, 148 / 9, &per, &n);
    }
    return n;
}

int tc_b1_partials(int h, int w) { return (int)(((int64_t)h * w + kTileM - 1) / kTileM); }

int tc_tile3_count(int h, int w) { return ((w + kTileW - 1) / kTileW) * ((h + kTileH - 1) / kTileH); }

int tc_dz_pitch(int h, int w) { return (int)((((int64_t)h * w + 63) / 64) * 64); }

TcPlan* tc_plan_create(const TcBuffers& b, char* err, size_t err_len)
{
    TcPlan* P = new TcPlan();
    memset((void*)P, 0, sizeof *P);
    P->b = b;
    P->p = b.h * b.w; P->p_pad = tc_dz_pitch(b.h, b.w);
    {
        int dev = 0;
        cudaGetDevice(&dev);
        if (cudaDeviceGetAttribute(&P->n_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || P->n_sms < 1) P->n_sms = 148;
    }
    const int nb = b.n_blocks;
    P->c_last = nb ? b.blk[nb - 1].c_out : b.c_in;
    const uint64_t S = (uint64_t)b.S, p = (uint64_t)P->p, cl = (uint64_t)P->c_last;
    const bf16* act = nb ? b.blk[nb - 1].out : b.x;
    bool ok = true;
    {
        uint64_t dims[3] = {cl, p, S}, str[2] = {cl * 2, p * cl * 2};
        uint32_t box_f[3] = {64, 128, 1}, box_w[3] = {64, 64, 1};
        ok = ok && make_map(&P->act_fwd, act, 3, dims, str, box_f, err, err_len, "last-layer input (forward)");
        ok = ok && make_map(&P->act_wg, act, 3, dims, str, box_w, err, err_len, "last-layer input (wgrad)");
    }
    if (ok) {
        uint64_t dims[3] = {cl, (uint64_t)kClassPad, S}, str[2] = {cl * 2, (uint64_t)kClassPad * cl * 2};
        uint32_t box[3] = {64, (uint32_t)kClassPad, 1};
        ok = make_map(&P->w2_map, b.w2, 3, dims, str, box, err, err_len, "1x1 weight");
    }
    if (ok) {
        uint64_t dims[3] = {p, (uint64_t)kClassPad, S}, str[2] = {(uint64_t)P->p_pad * 2, (uint64_t)kClassPad * P->p_pad * 2};
        uint32_t box[3] = {64, (uint32_t)kClassPad, 1};
        ok = make_map(&P->dz_map, b.dz_bf16, 3, dims, str, box, err, err_len, "logit gradient");
    }
    const size_t lim = 227 * 1024;
    for (int i = 0; ok && i < nb; ++i) {
        const TcBlock& k = b.blk[i];
        TcBlockPlan& q = P->blk[i];
        const uint64_t w = (uint64_t)b.w, h = (uint64_t)b.h, c1 = (uint64_t)k.c_prev, c2 = (uint64_t)k.c_skip, co = (uint64_t)k.c_out,
                       ct = c1 + c2;
        const uint32_t bf[4] = {64, (uint32_t)kTileW, (uint32_t)kTileH, 1}, bw[4] = {64, (uint32_t)kChunkW, (uint32_t)kChunkH, 1};
        auto act_maps = [&](const bf16* base, uint64_t c, CUtensorMap* fwd, CUtensorMap* wg, const char* what) {
            uint64_t d[4] = {c, w, h, S}, st[3] = {c * 2, w * c * 2, h * w * c * 2};
            bool r = true;
            if (fwd) r = r && make_map(fwd, base, 4, d, st, bf, err, err_len, what);
            if (wg) r = r && make_map(wg, base, 4, d, st, bw, err, err_len, what);
            return r;
        };
        ok = ok && act_maps(k.in_prev, c1, &q.in_fwd, &q.in_wg, "block input");
        if (c2) ok = ok && act_maps(k.in_skip, c2, &q.skip_fwd, &q.skip_wg, "skip input");
        else { q.skip_fwd = q.in_fwd; q.skip_wg = q.in_wg; }
        ok = ok && act_maps(k.dout, co, &q.dout_fwd, &q.dout_wg, "block output gradient");
        {
            uint64_t dw[3] = {ct, 9 * co, S}, sw[2] = {ct * 2, 9 * co * ct * 2};
            uint32_t bwt[3] = {64, (uint32_t)co, 1}, bwq[3] = {64, 64, 1};
            ok = ok && make_map(&q.w_map, k.w, 3, dw, sw, bwt, err, err_len, "3x3 weight");
            ok = ok && make_map(&q.w_map_q, k.w, 3, dw, sw, bwq, err, err_len, "3x3 weight (64 rows)");
        }
        if (ok && k.pass_back) {
            uint64_t dw[3] = {co, 9 * c1, S}, sw[2] = {co * 2, 9 * c1 * co * 2};
            uint32_t bwt[3] = {64, (uint32_t)c1, 1}, bwq[3] = {64, 64, 1};
            ok = ok && make_map(&q.wt_map, k.w_t, 3, dw, sw, bwt, err, err_len, "3x3 weight, transposed");
            ok = ok && make_map(&q.wt_map_q, k.w_t, 3, dw, sw, bwq, err, err_len, "3x3 weight, transposed (64 rows)");
        }
        const int m_in = ((int)ct + kTileM - 1) / kTileM;
        q.cols_wg = pow2_cols(m_in * k.c_out);
        // pipeline depth: as many stages as fit in about 208 KB (a stage of a narrow layer is small, and with only four
        // of them in flight the copies' latency, not the tensor pipe, sets the pace)
        auto pick = [](size_t stage_bytes, int lo, int mid, int hi) {
            const size_t fit = ((size_t)208 * 1024) / stage_bytes;
            return fit >= (size_t)hi ? hi : (fit >= (size_t)mid ? mid : lo);
        };
        const size_t st_fwd = (size_t)kTileM * 128 + (size_t)k.c_out * 128, st_back = (size_t)kTileM * 128 + (size_t)k.c_prev * 128,
                     st_wg = (size_t)(m_in * 2 + k.c_out / kBlockK) * kChunkPix * 128;
        q.stages_fwd = pick(st_fwd, 4, 6, 8); q.stages_back = pick(st_back, 4, 6, 8); q.stages_wg = pick(st_wg, 3, 4, 5);
        q.smem_fwd = q.stages_fwd * st_fwd + kSmemAlign;
        q.smem_back = q.stages_back * st_back + kSmemAlign;
        q.smem_wg = q.stages_wg * st_wg + kSmemAlign;
        if (ok && q.cols_wg > 512) {
            snprintf(err, err_len, "a block with %d input and %d output channels needs %d TMEM columns (> 512)", (int)ct, k.c_out, q.cols_wg);
            ok = false;
        }
        if (ok && (q.smem_fwd > lim || q.smem_wg > lim || (k.pass_back && (q.smem_back > lim || k.c_prev > 256)))) {
            snprintf(err, err_len, "shared memory per block exceeds 227 KB for these channel counts");
            ok = false;
        }
    }
    if (!ok) { delete P; return nullptr; }

    const int m_last = (P->c_last + kTileM - 1) / kTileM;
    P->chunks2 = (P->p + kChunkPix - 1) / kChunkPix;
    P->msplit2 = wgrad1x1_m_split(P->c_last);
    split_geometry(P->chunks2, 148 / P->msplit2, &P->per2, &P->split2);
    P->cols2 = pow2_cols((m_last / P->msplit2) * kClassPad);
    P->smem_fwd1 = (size_t)(P->c_last / kBlockK) * (kTileM * 128 + kClassPad * 128) + kSmemAlign;
    P->smem_fwd1p = (size_t)kF1Stages * kF1StageBytes + (size_t)(P->c_last / kBlockK) * kClassPad * 128 + kSmemAlign;
    {
        // The persistent form wins where every block has many tiles to stream (16 streams at 720p: 90 us against
        // 110 us, 0.93 of the HBM copy bandwidth); with about three tiles per SM (one 720p stream) its partly filled
        // last round costs more than the one-tile blocks' second wave.  ST_FWD1X1_PERSISTENT=0/1 forces a choice.
        const int64_t tiles = (int64_t)((P->p + kTileM - 1) / kTileM) * b.S;
        bool use = tiles >= (int64_t)6 * 148;
        if (const char* e = getenv("ST_FWD1X1_PERSISTENT")) { if (e[0] == '0') use = false; else if (e[0] == '1') use = true; }
        if (const char* e = getenv("ST_TEST_STALL_FWD1X1")) if (e[0] == '1') { P->test_stall = true; use = false; }
        // the one-tile form keeps the whole channel extent of its tile in shared memory: beyond 704 channels it no
        // longer fits, and the persistent form (a ring of eight stages, whatever the channel count) takes over
        if (P->smem_fwd1 > (size_t)227 * 1024) use = true;
        P->fwd1_persistent = use && P->smem_fwd1p <= (size_t)227 * 1024;
    }
    P->smem_wg1 = kWg1Stages * ((size_t)(m_last / P->msplit2) * 2 * kChunkPix * 128 + kClassPad * 128) + kSmemAlign;
    if (nb) {
        P->chunks1 = ((b.w + kChunkW - 1) / kChunkW) * ((b.h + kChunkH - 1) / kChunkH);
        split_geometry(P->chunks1, 148 / 9, &P->per1, &P->split1);
        P->smem_dgrad = (size_t)(2 + P->c_last / kBlockK) * kClassPad * 128 + kSmemAlign;
    }
    if (P->c_last / kBlockK > kMaxKBlocks || (!P->fwd1_persistent && P->smem_fwd1 > lim) || P->smem_wg1 > lim || P->smem_dgrad > lim) {
        snprintf(err, err_len, "shared memory per block exceeds 227 KB for these channel counts");
        delete P; return nullptr;
    }
    // Raise a kernel's shared-memory allowance to what this plan launches it with, never lower it: the attribute belongs
    // to the function, not to a plan, and an earlier plan with larger layers may still be in use.
    auto allow = [&](const void* fn, size_t need) -> cudaError_t {
        cudaFuncAttributes at;
        cudaError_t r = cudaFuncGetAttributes(&at, fn);
        if (r != cudaSuccess) return r;
        if (need <= (size_t)at.maxDynamicSharedSizeBytes) return cudaSuccess;
        return cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)need);
    };
    cudaError_t e = cudaSuccess;
    if (!P->fwd1_persistent) e = allow((const void*)tc_fwd1x1_kernel, P->smem_fwd1);
    if (e == cudaSuccess && P->fwd1_persistent) e = allow((const void*)tc_fwd1x1p_kernel, P->smem_fwd1p);
    if (e == cudaSuccess) e = allow((const void*)tc_wgrad1x1_kernel<kWg1Stages>, P->smem_wg1);
    for (int i = 0; i < nb; ++i) {
        const TcBlockPlan& q = P->blk[i];
        if (e == cudaSuccess) e = allow((const void*)fwd3_kernel<0>(q.stages_fwd), q.smem_fwd);
        if (e == cudaSuccess && b.blk[i].pass_back) e = allow((const void*)fwd3_kernel<1>(q.stages_back), q.smem_back);
        if (e == cudaSuccess) e = allow((const void*)wgrad3_kernel(q.stages_wg), q.smem_wg);
    }
    if (nb && e == cudaSuccess) e = allow((const void*)tc_dgrad_kernel, P->smem_dgrad);
    if (e != cudaSuccess) { snprintf(err, err_len, "shared-memory attribute: %s", cudaGetErrorString(e)); delete P; return nullptr; }
    return P;
}

void tc_plan_destroy(TcPlan* P) { delete P; }

static bool fwd1_early_enabled()     // ST_FWD1_EARLY=0 switches the early activation fetch off
{
    static const bool on = [] { const char* e = getenv("ST_FWD1_EARLY"); return !(e && e[0] == '0'); }();
    return on;
}

static const char* const kFwd3Names[kMaxBlocks] = {"tc_fwd3x3", "tc_fwd3x3#2"};
static const char* const kWg3Names[kMaxBlocks] = {"tc_wgrad3x3", "tc_wgrad3x3#2"};

// the tile walk of a 3x3 layer over `total` tiles: grid size and how the tiles of a partly filled last round are cut
static void tile_walk(const TcPlan* P, int total, int n_out, int* grid, int* tail_split)
{
    *grid = total < P->n_sms ? total : P->n_sms;
    // the tiles of a partly filled last round are cut into 4 or 2 ranges of output channels if that lets every
    // piece have its own block (pieces are multiples of 64 channels)
    const int tail = total > *grid ? total % *grid : 0;
    *tail_split = 1;
    if (tail > 0) {
        if (n_out % 256 == 0 && tail * 4 <= *grid) *tail_split = 4;
        else if (n_out % 128 == 0 && tail * 2 <= *grid) *tail_split = 2;
    }
}

int tc_forward_blocks(const TcPlan* P, int first, int last, cudaStream_t s, StageTimer* t, const int* skip, int64_t skip_stride)
{
    const TcBuffers& b = P->b;
    int n = 0;
    const int total = tc_tile3_count(b.h, b.w) * b.S;
    for (int i = first; i < last; ++i) {
        const TcBlock& k = b.blk[i];
        const TcBlockPlan& q = P->blk[i];
        int grid, tail_split;
        tile_walk(P, total, k.c_out, &grid, &tail_split);
        ST_REPEAT(t) launch_chain(b.chain_early != 0, fwd3_kernel<0>(q.stages_fwd), dim3(grid), dim3(kFwd3Threads), q.smem_fwd, s,
            q.in_fwd, q.skip_fwd, k.c_prev / kBlockK, k.c_skip / kBlockK, q.w_map, q.w_map_q, tail_split, b.theta, b.n_params, k.b_off,
            k.out, k.relu_bits, (float*)nullptr, k.c_out, b.h, b.w, total, pow2_cols(k.c_out), b.err, skip, skip_stride);
        if (t) t->mark(kFwd3Names[i], s, st_repeats(t));
        n += st_repeats(t);
    }
    return n;
}

int tc_forward(const TcPlan* P, cudaStream_t s, StageTimer* t, const int* skip, int64_t skip_stride, bool after_update, int first_block)
{
    const TcBuffers& b = P->b;
    int n = tc_forward_blocks(P, first_block, b.n_blocks, s, t, skip, skip_stride);
    const int tiles1 = (P->p + kTileM - 1) / kTileM;
    if (P->fwd1_persistent) {
        int gx = P->n_sms / b.S;
        if (gx < 1) gx = 1;
        if (gx > tiles1) gx = tiles1;
        ST_REPEAT(t) launch_chain(b.chain_early != 0, tc_fwd1x1p_kernel, dim3(gx, b.S), dim3(kF1Threads), P->smem_fwd1p, s,
            P->act_fwd, P->w2_map, b.theta, b.n_params, b.b2_off, b.z, b.C, P->p, P->c_last / kBlockK, b.err, skip, skip_stride);
    } else {
        // one-layer head, no per-stream skip flags to wait for, not a timing run: the activations are the frozen
        // features, which no kernel of the loop writes
        const bool a_early = after_update && !b.n_blocks && !skip && !t && fwd1_early_enabled();
        ST_REPEAT(t) launch_early(a_early || b.chain_early, tc_fwd1x1_kernel, dim3(tiles1, b.S), dim3(kThreadsTc), P->smem_fwd1, s,
            P->act_fwd, P->w2_map, b.theta, b.n_params, b.b2_off, b.z, b.C, P->p, P->c_last / kBlockK, b.err, skip, skip_stride,
            a_early ? 1 : 0, P->test_stall ? (1u << 12) : kSpinLimit, P->test_stall ? 16u : 0u);
    }
    if (t) t->mark("tc_fwd1x1", s, st_repeats(t));
    return n + st_repeats(t);
}

int tc_backward(const TcPlan* P, cudaStream_t s, StageTimer* t, const int* skip, int64_t skip_stride, const TrainCtl* ctl)
{
    const TcBuffers& b = P->b;
    int n = 0;
    // one-layer head: the activations are the frozen features, which no kernel of the loop writes
    const int a_early = (!b.n_blocks && !skip && !t && b.chain_early) ? 1 : 0;
    TrainCtl no_ctl;
    memset(&no_ctl, 0, sizeof no_ctl);
    ST_REPEAT(t) launch_chain(b.chain_early != 0, tc_wgrad1x1_kernel<kWg1Stages>, dim3(P->split2 * P->msplit2 + (ctl ? 1 : 0), b.S), dim3(kThreadsTc),
        P->smem_wg1, s, P->act_wg, P->dz_map, b.w2_partials, P->c_last, P->chunks2, P->per2, P->msplit2, P->cols2, b.err, skip, skip_stride,
        a_early, ctl ? 1 : 0, ctl ? *ctl : no_ctl);
    if (t) t->mark("tc_wgrad1x1", s, st_repeats(t));
    n += st_repeats(t);
    const int nb = b.n_blocks;
    if (!nb || !b.blk[nb - 1].trained) return n;          // nothing is passed back into a frozen block (Section 4.2)
    {
        const TcBlock& k = b.blk[nb - 1];
        const int blocks = tc_b1_partials(b.h, b.w);
        const int n_ch_split = (k.c_out % 128 == 0) ? 2 : 1;      // each block: a multiple of 64 channels (four ways measured no better)
        ST_REPEAT(t) launch_chain(b.chain_early != 0, tc_dgrad_kernel, dim3(blocks, b.S, n_ch_split), dim3(kThreadsTc), P->smem_dgrad, s,
            P->dz_map, P->w2_map, k.relu_bits, k.dout, k.b_partials, k.c_out, P->p, pow2_cols(k.c_out / n_ch_split), b.err, skip, skip_stride);
        if (t) t->mark("tc_dgrad", s, st_repeats(t));
        n += st_repeats(t);
    }
    const int total = tc_tile3_count(b.h, b.w) * b.S;
    for (int i = nb - 1; i >= 0 && b.blk[i].trained; --i) {
        const TcBlock& k = b.blk[i];
        const TcBlockPlan& q = P->blk[i];
        ST_REPEAT(t) launch_chain(b.chain_early != 0, wgrad3_kernel(q.stages_wg), dim3(9 * P->split1, b.S), dim3(kThreadsTc), q.smem_wg, s,
            q.in_wg, q.skip_wg, k.c_prev / kBlockK, q.dout_wg, k.w_partials, k.c_prev + k.c_skip, k.c_out, b.h, b.w, P->chunks1, P->per1,
            P->split1, q.cols_wg, b.err, skip, skip_stride);
        if (t) t->mark(kWg3Names[i], s, st_repeats(t));
        n += st_repeats(t);
        if (k.pass_back) {
            // gradient with respect to the previous block's output: the tile walk of the forward over this block's
            // output gradient, with the mirrored and transposed weights; masked by the previous block's ReLU bits
            const TcBlock& r = b.blk[i - 1];
            int grid, tail_split;
            tile_walk(P, total, k.c_prev, &grid, &tail_split);
            ST_REPEAT(t) launch_chain(b.chain_early != 0, fwd3_kernel<1>(q.stages_back), dim3(grid), dim3(kFwd3Threads), q.smem_back, s,
                q.dout_fwd, q.dout_fwd, k.c_out / kBlockK, 0, q.wt_map, q.wt_map_q, tail_split, (const float*)nullptr, (int64_t)0, (int64_t)0,
                r.dout, r.relu_bits, r.b_partials, k.c_prev, b.h, b.w, total, pow2_cols(k.c_prev), b.err, skip, skip_stride);
            if (t) t->mark("tc_dgrad3x3", s, st_repeats(t));
            n += st_repeats(t);
        }
    }
    return n;
}

}  // namespace st
