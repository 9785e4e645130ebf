// K3 — ComputeLoss and the first half of PartialBackward (Algorithm 1; loss of Section 5.2),
// fused: bilinear x4 upsample of the head's low-resolution logits z to frame resolution,
// per-pixel softmax cross-entropy against the one-byte labels, and the gradient of the mean
// loss with respect to z (the transpose of the upsample applied to softmax - onehot), without
// ever writing a frame-resolution tensor.
//
// Geometry.  With half-pixel centres and factor 4, the frame pixels between four neighbouring
// low-resolution nodes (i,j),(i,j+1),(i+1,j),(i+1,j+1) form a 4x4 "cell": rows 4i+2..4i+5,
// columns 4j+2..4j+5, with weights 1/8, 3/8, 5/8, 7/8 toward the lower/right node.  Cells
// i = -1 and i = h-1 (same for j) are the clamped borders: their outer node coincides with the
// inner one.  A block owns a tile of NY x NX nodes and evaluates the (NY+1) x (NX+1) cells that
// touch it (the halo cells are recomputed by the neighbouring block too, so every block can
// finish its nodes alone, in a fixed summation order, without atomics).
//
// One thread per cell, three sweeps over the classes with z held in shared memory:
//   1. per-pixel maximum (and arg-max, for the optional confusion matrix);
//   2. per-pixel sum of exponentials -> log-partition, loss, 1/Z;
//   3. softmax - onehot, reduced inside the thread to the cell's four corner contributions.
// Then every node adds the four corner values of its four cells.
#include "st_internal.h"

namespace st {

constexpr int NY = 8, NX = 16;
constexpr int kCells = (NY + 1) * (NX + 1);
constexpr int kThreads = 160;
constexpr int ZT_H = NY + 2, ZT_W = NX + 2;

int upsample_ce_blocks(int h, int w, int C)
{
    if (upsample_ce_rows_supported(C)) return upsample_ce_rows_blocks(h, w);
    return ((h + NY - 1) / NY) * ((w + NX - 1) / NX);
}

__device__ __forceinline__ float lerp_f(float a, float b, float t) { return fmaf(t, b - a, a); }

// classes per chunk of sweep 3 (limited by shared memory)
static int chunk_classes(int C, size_t* smem_bytes)
{
    const size_t zt = (size_t)C * ZT_H * ZT_W * sizeof(float);
    const size_t per_class = (size_t)kCells * 4 * sizeof(float) + (size_t)NY * NX * sizeof(float);
    const size_t budget = 200 * 1024;
    size_t avail = budget > zt ? budget - zt : 0;
    int chunk = (int)(avail / per_class);
    if (chunk > C) chunk = C;
    if (chunk < 1) chunk = 1;
    *smem_bytes = zt + per_class * chunk + 64;
    return chunk;
}

template <bool CONF>
__global__ void __launch_bounds__(kThreads)
upsample_ce_kernel(UpsampleCeArgs a, int chunk)
{
    extern __shared__ __align__(16) float smem[];
    const int C = a.C, h = a.h, w = a.w, H = h * kUp, W = w * kUp;
    float* zt = smem;                                   // [C][ZT_H][ZT_W]
    float* acc = zt + (size_t)C * ZT_H * ZT_W;          // [chunk][kCells][4]
    float* dzt = acc + (size_t)chunk * kCells * 4;      // [chunk][NY*NX]
    __shared__ float red[kThreads / 32];

    const int s = blockIdx.z;
    const int x0 = blockIdx.x * NX, y0 = blockIdx.y * NY;
    const int blk = blockIdx.y * gridDim.x + blockIdx.x, n_blk = gridDim.x * gridDim.y;
    const int64_t p = (int64_t)h * w;
    const float* z = a.z + (int64_t)s * C * p;
    const uint8_t* labels = a.labels + (int64_t)s * H * W;
    const int tid = threadIdx.x;
    pdl_wait();
    pdl_launch_dependents();
    if (a.skip && a.skip[(int64_t)s * a.skip_stride]) return;     // this stream's training loop has ended (block-uniform)

    // ---- z tile with replicated borders
    for (int idx = tid; idx < C * ZT_H * ZT_W; idx += kThreads) {
        int c = idx / (ZT_H * ZT_W), r = idx % (ZT_H * ZT_W);
        int ry = r / ZT_W, rx = r % ZT_W;
        int yy = min(max(y0 - 1 + ry, 0), h - 1), xx = min(max(x0 - 1 + rx, 0), w - 1);
        zt[idx] = __ldg(z + (int64_t)c * p + (int64_t)yy * w + xx);
    }
    __syncthreads();

    const int ci = tid / (NX + 1), cj = tid % (NX + 1);
    const int i = y0 - 1 + ci, j = x0 - 1 + cj;
    const bool cell_ok = tid < kCells && i <= h - 1 && j <= w - 1;

    float m[16], Zs[16];
    uint32_t lab[16];
    uint32_t arg[16];
    float loss = 0.f;
    unsigned n_bad = 0;
    uint32_t owned_mask = 0;       // bit per pixel: valid and owned by this block's node tile

    if (cell_ok) {
        const float* zc = zt + ci * ZT_W + cj;
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int ay = k >> 2, bx = k & 3;
            const int Y = 4 * i + 2 + ay, X = 4 * j + 2 + bx;
            const bool valid = Y >= 0 && Y < H && X >= 0 && X < W;
            uint32_t l = 255;
            if (valid) l = labels[(int64_t)Y * W + X];
            const int gy = (Y >> 2) - y0, gx = (X >> 2) - x0;
            const bool own = valid && gy >= 0 && gy < NY && gx >= 0 && gx < NX;
            if (own) owned_mask |= 1u << k;
            if (valid && l >= (uint32_t)C) { if (own) n_bad++; l = 255; }
            lab[k] = valid ? l : 255;
            m[k] = -INFINITY; Zs[k] = 0.f; arg[k] = 0;
        }
        // ---- sweep 1: maximum (and arg-max, lowest class on ties)
        for (int c = 0; c < C; ++c) {
            const float* q = zc + c * (ZT_H * ZT_W);
            const float z00 = q[0], z01 = q[1], z10 = q[ZT_W], z11 = q[ZT_W + 1];
#pragma unroll
            for (int bx = 0; bx < 4; ++bx) {
                const float lx = (2 * bx + 1) * 0.125f;
                const float top = lerp_f(z00, z01, lx), bot = lerp_f(z10, z11, lx);
#pragma unroll
                for (int ay = 0; ay < 4; ++ay) {
                    const float u = lerp_f(top, bot, (2 * ay + 1) * 0.125f);
                    const int k = ay * 4 + bx;
                    if (u > m[k]) { m[k] = u; if (CONF) arg[k] = c; }
                }
            }
        }
        // ---- sweep 2: sum of exponentials
        for (int c = 0; c < C; ++c) {
            const float* q = zc + c * (ZT_H * ZT_W);
            const float z00 = q[0], z01 = q[1], z10 = q[ZT_W], z11 = q[ZT_W + 1];
#pragma unroll
            for (int bx = 0; bx < 4; ++bx) {
                const float lx = (2 * bx + 1) * 0.125f;
                const float top = lerp_f(z00, z01, lx), bot = lerp_f(z10, z11, lx);
#pragma unroll
                for (int ay = 0; ay < 4; ++ay) {
                    const float u = lerp_f(top, bot, (2 * ay + 1) * 0.125f);
                    const int k = ay * 4 + bx;
                    Zs[k] += __expf(u - m[k]);
                }
            }
        }
        // ---- per pixel: loss, 1/Z (0 for pixels that carry no gradient)
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const int ay = k >> 2, bx = k & 3;
            if (lab[k] < 255) {
                const float* q = zc + lab[k] * (ZT_H * ZT_W);
                const float lx = (2 * bx + 1) * 0.125f;
                const float ul = lerp_f(lerp_f(q[0], q[1], lx), lerp_f(q[ZT_W], q[ZT_W + 1], lx),
                                        (2 * ay + 1) * 0.125f);
                if (owned_mask & (1u << k)) loss += logf(Zs[k]) + (m[k] - ul);
                Zs[k] = 1.0f / Zs[k];
            } else {
                Zs[k] = 0.f;
            }
        }
    }

    // ---- optional confusion of label vs arg-max (owned pixels only, so each pixel counts once)
    if (CONF) {
        if (cell_ok) {
            unsigned long long* conf = a.conf + (int64_t)s * a.conf_stream_stride;
#pragma unroll
            for (int k = 0; k < 16; ++k)
                if ((owned_mask & (1u << k)) && lab[k] < 255)
                    atomicAdd(&conf[lab[k] * C + arg[k]], 1ull);
        }
    }

    // ---- loss partial of this block (fixed order)
    {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
        if ((tid & 31) == 0) red[tid >> 5] = loss;
        if (n_bad) atomicAdd(a.bad, n_bad);
    }

    // ---- sweep 3 in chunks of classes: corner contributions, then node sums
    const float invP = 1.0f / ((float)H * (float)W);
    for (int c0 = 0; c0 < C; c0 += chunk) {
        const int nc = min(chunk, C - c0);
        __syncthreads();     // acc/dzt free (previous chunk consumed); red[] written
        if (tid < kCells) {
            for (int cc = 0; cc < nc; ++cc) {
                float t0 = 0.f, t1 = 0.f, b0 = 0.f, b1 = 0.f;
                if (cell_ok) {
                    const int c = c0 + cc;
                    const float* q = zt + ci * ZT_W + cj + c * (ZT_H * ZT_W);
                    const float z00 = q[0], z01 = q[1], z10 = q[ZT_W], z11 = q[ZT_W + 1];
                    float r0[4] = {0.f, 0.f, 0.f, 0.f}, r1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int bx = 0; bx < 4; ++bx) {
                        const float lx = (2 * bx + 1) * 0.125f;
                        const float top = lerp_f(z00, z01, lx), bot = lerp_f(z10, z11, lx);
#pragma unroll
                        for (int ay = 0; ay < 4; ++ay) {
                            const int k = ay * 4 + bx;
                            const float u = lerp_f(top, bot, (2 * ay + 1) * 0.125f);
                            float g = __expf(u - m[k]) * Zs[k];
                            if (lab[k] == (uint32_t)c) g -= 1.0f;
                            r0[ay] = fmaf(1.0f - lx, g, r0[ay]);
                            r1[ay] = fmaf(lx, g, r1[ay]);
                        }
                    }
#pragma unroll
                    for (int ay = 0; ay < 4; ++ay) {
                        const float ly = (2 * ay + 1) * 0.125f;
                        t0 = fmaf(1.0f - ly, r0[ay], t0); t1 = fmaf(1.0f - ly, r1[ay], t1);
                        b0 = fmaf(ly, r0[ay], b0);        b1 = fmaf(ly, r1[ay], b1);
                    }
                    // clamped borders: the outer node coincides with the inner one
                    if (i == -1)    { b0 += t0; b1 += t1; t0 = 0.f; t1 = 0.f; }
                    if (i == h - 1) { t0 += b0; t1 += b1; b0 = 0.f; b1 = 0.f; }
                    if (j == -1)    { t1 += t0; b1 += b0; t0 = 0.f; b0 = 0.f; }
                    if (j == w - 1) { t0 += t1; b0 += b1; t1 = 0.f; b1 = 0.f; }
                }
                reinterpret_cast<float4*>(acc)[cc * kCells + tid] = make_float4(t0, t1, b0, b1);
            }
        }
        __syncthreads();
        for (int idx = tid; idx < nc * NY * NX; idx += kThreads) {
            const int cc = idx / (NY * NX), r = idx % (NY * NX);
            const int ny = r / NX, nx = r % NX;
            const int y = y0 + ny, x = x0 + nx;
            float v = 0.f;
            if (y < h && x < w) {
                const float4* A = reinterpret_cast<const float4*>(acc) + cc * kCells;
                const float4 ul = A[ny * (NX + 1) + nx];            // cell up-left: this node is its lower-right corner
                const float4 ur = A[ny * (NX + 1) + nx + 1];        // up-right: lower-left corner
                const float4 ll = A[(ny + 1) * (NX + 1) + nx];      // low-left: upper-right corner
                const float4 lr = A[(ny + 1) * (NX + 1) + nx + 1];  // low-right: upper-left corner
                v = ((ul.w + ur.z) + (ll.y + lr.x)) * invP;
                const int c = c0 + cc;
                if (a.dz) a.dz[((int64_t)s * C + c) * p + (int64_t)y * w + x] = v;
                if (a.dz_bf16)
                    a.dz_bf16[((int64_t)s * kClassPad + c) * a.dz_bf16_pitch + (int64_t)y * w + x] = __float2bfloat16_rn(v);
            }
            dzt[idx] = v;
        }
        __syncthreads();
        for (int cc = tid; cc < nc; cc += kThreads) {
            float sum = 0.f;
            for (int r = 0; r < NY * NX; ++r) sum += dzt[cc * NY * NX + r];
            a.db_part[((int64_t)s * n_blk + blk) * C + c0 + cc] = sum;
        }
    }
    if (tid == 0) {
        float t = 0.f;
        for (int k = 0; k < kThreads / 32; ++k) t += red[k];
        a.loss_part[(int64_t)s * n_blk + blk] = t;
    }
}

cudaError_t prepare_upsample_ce(int C)
{
    if (upsample_ce_rows_supported(C)) return prepare_upsample_ce_rows(C);
    size_t smem = 0;
    chunk_classes(C, &smem);
    cudaError_t e = cudaFuncSetAttribute(upsample_ce_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(upsample_ce_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

void launch_upsample_ce(const UpsampleCeArgs& a, const CUtensorMap* z_map, cudaStream_t s, const CUtensorMap* x_map, const CUtensorMap* w_map)
{
    if (upsample_ce_rows_supported(a.C)) { launch_upsample_ce_rows(a, z_map, s, x_map, w_map); return; }
    size_t smem = 0;
    const int chunk = chunk_classes(a.C, &smem);
    dim3 grid((unsigned)((a.w + NX - 1) / NX), (unsigned)((a.h + NY - 1) / NY), (unsigned)a.S);
    if (a.conf) launch_chain(a.chain_early != 0, upsample_ce_kernel<true>, grid, dim3(kThreads), smem, s, a, chunk);
    else launch_chain(a.chain_early != 0, upsample_ce_kernel<false>, grid, dim3(kThreads), smem, s, a, chunk);
}

}  // namespace st
