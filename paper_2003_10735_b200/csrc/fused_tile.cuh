// Forward of a 1x1 classifier inside a block that needs the logits of a tile of feature-map nodes (Forward of
// Algorithm 1 for the trainable back part of Section 4.2 when that part is one 1x1 layer): shared by the fused
// upsample + cross-entropy kernel and by the student-mask kernel.
//
// z[pix][c] = b[c] + sum_k X[pix][k] W[c][k] for the kTileRows x kTileCols nodes of the tile (node rows y0-1 .. y0+7,
// node columns x0-1 .. x0+30: the 7 x 30 nodes a block owns and the ring around them).  The feature tile arrives in
// 64-channel slices (one 4-d tile copy each; rows and columns outside the map arrive as zeros) through a ring of two
// stages, the classifier weights in one barrier's worth of copies; one thread issues three 128 x 32 x 16 tcgen05
// multiplications per 16 channels (pixel rows 288 .. 383 of the third one read whatever follows the stage: their
// results are never looked at), the accumulators (fp32, in tensor memory) are drained into the logit tile
// [class][row][column] in shared memory by all eight warps.  Tile entries outside the frame hold the bare bias: readers
// take their logits at clamped coordinates and never look at them.
#pragma once

#include "st_internal.h"
#include "tc_common.cuh"

namespace st {
namespace fused {

constexpr int kOwnRows = 7, kOwnCols = 30;                   // nodes a block owns
constexpr int kTileRows = kOwnRows + 2, kTileCols = 32, kTile = kTileRows * kTileCols;
constexpr int kThreads = (kOwnRows + 1) * 32;                // eight warps
constexpr uint32_t kStageBytes = kTile * 128, kWeightBytes = kClassPad * 128;   // one 64-channel slice of the tile / of the weights
constexpr int kStages = 2, kTmemCols = 128, kMaxKBlocks = 4, kBars = 2 * kStages + 2;
// bytes from the (1024-aligned) start of the ring that the copies and the multiplications touch
constexpr size_t kRingBytes = (size_t)kStages * kStageBytes + (size_t)kMaxKBlocks * kWeightBytes;
constexpr size_t kReachBytes = (size_t)(kStages - 1) * kStageBytes + 384 * 128;

struct Args {
    int kblocks;             // 64-channel slices of the classifier's input
    int x_early;             // the features are not written by the kernel just before this one: fetch them before waiting for it
    const int* skip;         // nullptr, or the flag of this block's stream: non-zero = the block returns at once
    unsigned int* err;       // device word: first wait that gave up
    const float* bias;       // the classifier's bias of this block's stream (fp32 master parameters)
    float* z_out;            // nullptr, or the stream's logits [C][h][w]: the block's own nodes are written there as well
    int C, h, w;
    // tc::kSpinLimit and 0 in normal use.  A test of the give-up path lowers the limit and makes the first barrier expect
    // stall_bytes more than its copy delivers, so that the wait on it runs out: every copy that was issued still lands,
    // the block records where it gave up, writes nothing, frees its tensor memory and returns.
    uint32_t spin_limit, stall_bytes;
};

// What the block keeps in static shared memory for this
struct Shared {
    alignas(8) uint64_t bar[kBars];   // full[2], empty[2], weights, done
    uint32_t tmem_slot, gave_up;
    float bias[kClassPad];
};

// Called by all kFused threads of the block.  `zt` (1024-byte aligned) receives the tile; the ring and the weights lie
// over it and the kRingBytes behind its start until the multiplication has finished, then `after_mma()` is called (the
// caller gives the arrays under the ring their initial contents there) and the tile is written.  `tmem` is the block's
// tensor memory, which the caller frees at its very end (free_tmem).  m_loc: the largest logit this thread has written
// for a node inside the frame.  ok = false: the block has to return at once (its stream is flagged, or a wait gave
// up); the tensor memory is then already freed.
struct Tile { bool ok; float m_loc; uint32_t tmem; };
template <int CB, class AfterMma>
__device__ __forceinline__ Tile logit_tile(const Args& a, const CUtensorMap* x_map, const CUtensorMap* w_map, Shared& sh, float* zt,
                                           int s, int x0, int y0, AfterMma after_mma)
{
    float m_loc = -INFINITY;
    uint32_t tmem;
    constexpr int TW = kTileCols, TZ = kTile, RN_Y = kOwnRows, RN_X = kOwnCols;
    const int tid = threadIdx.x, wi = tid >> 5, l = tid & 31;
    const int C = a.C, h = a.h, w = a.w;
    const int64_t p = (int64_t)h * w;
    const uint32_t ring = tc::smem_u32(zt), w_base = ring + kStages * kStageBytes;
    const uint32_t bar0 = tc::smem_u32(&sh.bar[0]);
    auto full_bar = [&](int st) { return bar0 + 8u * (uint32_t)st; };
    auto empty_bar = [&](int st) { return bar0 + 8u * (uint32_t)(kStages + st); };
    const uint32_t w_bar = bar0 + 8u * (2 * kStages), done_bar = w_bar + 8u;
    if (wi == 0) tc::tmem_alloc(tc::smem_u32(&sh.tmem_slot), kTmemCols);
    if (tid == 0) {
        for (int k = 0; k < kBars; ++k) tc::mbar_init(bar0 + 8u * (uint32_t)k, 1);
        sh.gave_up = 0;
        tc::fence_barrier_init();
    }
    tc::tc_fence_before_sync();
    __syncthreads();
    tc::tc_fence_after_sync();
    tmem = sh.tmem_slot;
    const int kblocks = a.kblocks;
    const int n_pre = a.x_early ? min(kStages, kblocks) : 0;
    if (tid == 0)
        for (int kb = 0; kb < n_pre; ++kb) {
            tc::mbar_expect_tx(full_bar(kb), kStageBytes + (kb == 0 ? a.stall_bytes : 0u));
            tc::tma_load_4d(ring + kb * kStageBytes, x_map, full_bar(kb), kb * 64, x0 - 1, y0 - 1, s);
        }
    pdl_wait();                                        // the weights come from the previous kernel of the stream
    if (a.skip && *a.skip) {                           // this stream's training loop has ended (block-uniform)
        if (tid == 0)                                   // copies already on their way land before shared memory is given back
            for (int kb = 0; kb < n_pre; ++kb) tc::mbar_wait(full_bar(kb), 0, a.err, tc::kWaitFull);
        tc::tc_fence_before_sync();
        __syncthreads();
        if (wi == 0) tc::tmem_dealloc(tmem, kTmemCols);
        return Tile{false, m_loc, 0u};
    }
    if (tid < kClassPad) sh.bias[tid] = tid < C ? a.bias[tid] : 0.f;
    bool ok = true;
    if (tid == 0) {
        tc::mbar_expect_tx(w_bar, (uint32_t)kblocks * kWeightBytes);
        for (int kb = 0; kb < kblocks; ++kb) tc::tma_load_3d(w_base + kb * kWeightBytes, w_map, w_bar, kb * 64, 0, s);
        for (int kb = n_pre; kb < kblocks && ok; ++kb) {
            const int st = kb % kStages;
            if (kb >= kStages) ok = tc::mbar_wait(empty_bar(st), ((kb / kStages) - 1) & 1, a.err, tc::kWaitEmpty);
            if (ok) {
                tc::mbar_expect_tx(full_bar(st), kStageBytes + (kb == 0 ? a.stall_bytes : 0u));
                tc::tma_load_4d(ring + st * kStageBytes, x_map, full_bar(st), kb * 64, x0 - 1, y0 - 1, s);
            }
        }
    } else if (tid == 32) {
        constexpr uint32_t idesc = tc::instr_desc(128, kClassPad, 0, 0);
        ok = tc::mbar_wait(w_bar, 0, a.err, tc::kWaitFull);
        for (int kb = 0; kb < kblocks && ok; ++kb) {
            const int st = kb % kStages;
            ok = tc::mbar_wait(full_bar(st), (kb / kStages) & 1, a.err, tc::kWaitFull, a.spin_limit);
            if (!ok) break;
            tc::tc_fence_after_sync();
#pragma unroll
            for (int m = 0; m < 3; ++m)
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    tc::umma(tmem + m * kClassPad, tc::smem_desc(ring + st * kStageBytes + m * (128 * 128) + k * 32, 16, 1024),
                             tc::smem_desc(w_base + kb * kWeightBytes + k * 32, 16, 1024), idesc, (kb | k) != 0);
            tc::umma_commit(empty_bar(st));
        }
        if (!ok) sh.gave_up = 1;
        tc::umma_commit(done_bar);
    }
    __syncwarp();
    ok = tc::mbar_wait(done_bar, 0, a.err, tc::kWaitDone);
    tc::tc_fence_after_sync();
    if (!__syncthreads_and(ok) || sh.gave_up) {          // block-uniform: a wait ran out; nothing is written
        tc::drain_after_error();
        tc::tc_fence_before_sync();
        __syncthreads();
        if (wi == 0) tc::tmem_dealloc(tmem, kTmemCols);
        return Tile{false, m_loc, 0u};
    }
    after_mma();                                        // the stages are dead
    {
        float4* zt4 = reinterpret_cast<float4*>(zt);    // classes the caller pads to: their exponentials are 0, they never win an arg-max
        for (int e = tid; e < (CB - C) * (TZ / 4); e += kThreads) zt4[C * (TZ / 4) + e] = make_float4(-1e30f, -1e30f, -1e30f, -1e30f);
    }
    // accumulator m holds tile rows 4m .. 4m+3 (one row of 32 nodes per 32 lanes of tensor memory, and a warp reaches
    // the lanes 32 (warp % 4) ..): warps 0-3 drain rows 0-3, warps 4-7 rows 4-7, warps 0 and 4 half of the classes of
    // row 8 each
    auto put_row = [&](const float* v, int n_cols, int c0, int j) {     // v[i]: class c0 + i of node (row j, column l)
        const int ny = y0 - 1 + j, nx = x0 - 1 + l;
        const bool in_frame = ny >= 0 && ny < h && nx >= 0 && nx < w;
        // the block's own nodes go to global memory as well where the caller wants the logits kept
        const bool keep = a.z_out && in_frame && j >= 1 && j <= RN_Y && l >= 1 && l <= RN_X;
        float* dst = zt + c0 * TZ + j * TW + l;
        float* zo = a.z_out + (int64_t)c0 * p + (int64_t)ny * w + nx;
#pragma unroll
        for (int i = 0; i < 32; ++i)
            if (i < n_cols && c0 + i < C) {
                const float t = v[i] + sh.bias[c0 + i];
                dst[i * TZ] = t;
                if (in_frame) m_loc = fmaxf(m_loc, t);
                if (keep) zo[(int64_t)i * p] = t;
            }
    };
    {
        float v[32];
        tc::tmem_ld_32x32(tmem + ((uint32_t)((wi & 3) * 32) << 16) + (wi >> 2) * kClassPad, v);
        put_row(v, 32, 0, wi);
    }
    if ((wi & 3) == 0) {
        const int c0 = wi ? 16 : 0;
        float v[32];
        tc::tmem_ld_32x16(tmem + 2 * kClassPad + c0, reinterpret_cast<float(&)[16]>(v));
        put_row(v, 16, c0, 8);
    }
    tc::tc_fence_before_sync();
    __syncthreads();                                   // the tile is complete
    return Tile{true, m_loc, tmem};
}

// at the very end of the kernel, after a block-wide barrier that follows every warp's last read of tensor memory
__device__ __forceinline__ void free_tmem(uint32_t tmem)
{
    if ((threadIdx.x >> 5) == 0) {
        __syncwarp();
        tc::tc_fence_after_sync();
        tc::tmem_dealloc(tmem, kTmemCols);
    }
}

// dynamic shared memory a kernel needs for the ring (on top of its own arrays, which the ring lies over), including the
// slack for aligning the ring's start
__host__ __device__ constexpr size_t smem_bytes(size_t own)
{
    size_t need = own;
    if (kRingBytes > need) need = kRingBytes;
    if (kReachBytes > need) need = kReachBytes;
    return need + 1024;
}

}  // namespace fused
}  // namespace st
