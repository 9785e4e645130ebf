// K3, register-resident form (n_classes <= 32) — ComputeLoss and the first half of PartialBackward
// (Algorithm 1; loss of Section 5.2): bilinear x4 upsample of the low-resolution logits, per-pixel
// softmax cross-entropy against the labels, and the gradient of the mean loss with respect to the
// low-resolution logits.  Same result as the cell-per-thread kernel in k_upsample_ce.cu, organised
// so that every exponential is evaluated once.
//
// A block owns 7 rows x 30 columns of feature-map nodes and runs 8 warps (two per scheduler, so that each
// thread may hold the exponentials of four pixels x all classes in registers).  Warp i handles "cell row"
// y0-1+i: the four frame rows between node rows (y0-1+i, y0+i); lane l handles the four frame pixels
// of node column x0-1+l in each of those rows.  (Warp 0 and lanes 0/31 are the halo: their pixels are
// recomputed by the neighbouring block, so that a block finishes its nodes alone, in a fixed order.)
// Per frame row a thread
//   A. interpolates the logits of its four pixels class by class (logits pre-scaled by log2 e in shared
//      memory), exponentiates against an upper bound of the maximum (the largest logit of the six
//      nodes it reads; the pixel is redone with its exact maximum if the sum underflows), keeps the
//      exponentials in registers and sums them;
//   B. forms softmax * (adjoint interpolation weights) toward its left/own/right node column, trades
//      the side parts with the neighbouring lanes by shuffle, and adds the row into two per-class
//      accumulators: toward the upper and the lower node row.
// The "- onehot(label)" part of the gradient is exact in units of 1/64 (products of the eighths
// weights), so it is accumulated with integer shared-memory atomics, order-independent.
// At the end warp i adds its upper accumulator to the lower accumulator of warp i-1 (through shared
// memory) and writes node row y0-1+i: one 120-byte run per class.
#include "st_internal.h"

namespace st {

namespace {

constexpr int RN_Y = 7, RN_X = 30;
constexpr int R_WARPS = RN_Y + 1, R_THREADS = R_WARPS * 32;
constexpr int TZ_H = RN_Y + 2, TZ_W = RN_X + 4, TZ = TZ_H * TZ_W;
constexpr float kLog2e = 1.4426950408889634f, kLn2 = 0.6931471805599453f;

__device__ __forceinline__ float lerp_r(float a, float b, float t) { return fmaf(t, b - a, a); }
__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

template <int CB, bool CONF>
__global__ void __launch_bounds__(R_THREADS, 1)
upsample_ce_rows_kernel(UpsampleCeArgs a)
{
    extern __shared__ __align__(16) float smem_r[];
    const int C = a.C, h = a.h, w = a.w, H = h * kUp, W = w * kUp;
    float* zt = smem_r;                         // [CB][TZ_H][TZ_W] logits * log2(e), borders replicated;
                                                //                  classes >= C hold -1e30 (their exponentials are 0),
                                                //                  which keeps the class loops free of branches
    float* nmax = zt + CB * TZ;                 // [TZ_H][TZ_W]     max over classes
    int* corr = (int*)(nmax + TZ);              // [C][TZ_H][TZ_W]  -64 * (adjoint of onehot)
    float* bsh = (float*)(corr + C * TZ);       // [R_WARPS][C][32] lower-row accumulators
    float* dbs = bsh + R_WARPS * C * 32;        // [R_WARPS][C]
    __shared__ float red[R_WARPS];

    const int s = blockIdx.z, x0 = blockIdx.x * RN_X, y0 = blockIdx.y * RN_Y;
    const int blk = blockIdx.y * gridDim.x + blockIdx.x, n_blk = gridDim.x * gridDim.y;
    const int64_t p = (int64_t)h * w;
    const float* z = a.z + (int64_t)s * C * p;
    const uint8_t* labels = a.labels + (int64_t)s * H * W;
    const int tid = threadIdx.x, wi = tid >> 5, l = tid & 31;

    const int i = y0 - 1 + wi;                  // cell row: frame rows 4i+2 .. 4i+5, nodes (i, i+1)
    const int xg = x0 - 1 + l;                  // node column whose four frame pixels this lane handles
    const bool lane_valid = xg >= 0 && xg < w;

    // ---- tile: nodes y0-1 .. y0+RN_Y, x0-2 .. x0+31 (clamped), scaled; zeroed corrections; per-node maximum
    // (fully unrolled: all of a thread's loads are in flight together, one memory latency for the whole tile)
    {
        constexpr int kIter = (CB * TZ + R_THREADS - 1) / R_THREADS;
        float v[kIter];
#pragma unroll
        for (int it = 0; it < kIter; ++it) {
            const int e = tid + it * R_THREADS;
            const int c = e / TZ, n = e % TZ;
            const int ry = n / TZ_W, rx = n % TZ_W;
            const int yy = min(max(y0 - 1 + ry, 0), h - 1), xx = min(max(x0 - 2 + rx, 0), w - 1);
            v[it] = (e < CB * TZ && c < C) ? __ldg(z + (int64_t)c * p + (int64_t)yy * w + xx) * kLog2e : -1e30f;
        }
#pragma unroll
        for (int it = 0; it < kIter; ++it) {
            const int e = tid + it * R_THREADS;
            if (e < CB * TZ) zt[e] = v[it];
        }
    }
    for (int e = tid; e < C * TZ; e += R_THREADS) corr[e] = 0;
    __syncthreads();
    for (int e = tid; e < TZ; e += R_THREADS) {
        float m = -INFINITY;
        for (int c = 0; c < C; ++c) m = fmaxf(m, zt[c * TZ + e]);
        nmax[e] = m;
    }
    __syncthreads();

    const bool lane_owned = lane_valid && l >= 1 && l <= RN_X;
    const bool cell_row_valid = i <= h - 1;
    const float* zp = zt + wi * TZ_W + l;       // node (i, xg-1) of class 0
    // tile coordinates of the (clamped) nodes this thread's pixels pull toward
    const int ry_top = min(max(i, 0), h - 1) - (y0 - 1), ry_bot = min(max(i + 1, 0), h - 1) - (y0 - 1);
    const int rx_l = min(max(xg - 1, 0), w - 1) - (x0 - 2), rx_c = min(max(xg, 0), w - 1) - (x0 - 2),
              rx_r = min(max(xg + 1, 0), w - 1) - (x0 - 2);

    float top[CB], bot[CB];
#pragma unroll
    for (int c = 0; c < CB; ++c) { top[c] = 0.f; bot[c] = 0.f; }
    float loss = 0.f;
    unsigned n_bad = 0;

    for (int r = 0; r < 4; ++r) {
        const int Y = 4 * i + 2 + r;
        const bool row_valid = cell_row_valid && Y >= 0 && Y < H;     // warp-uniform
        if (!row_valid) continue;
        const float ly = (2 * r + 1) * 0.125f;
        const bool row_owned = (Y >> 2) >= y0 && (Y >> 2) < y0 + RN_Y;
        uint32_t lw = 0xffffffffu;
        if (lane_valid) lw = __ldg(reinterpret_cast<const uint32_t*>(labels + (int64_t)Y * W + 4 * xg));
        int lab[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            lab[k] = (lw >> (8 * k)) & 0xff;
            if (lab[k] >= C) { if (lane_valid && row_owned && lane_owned) n_bad++; lab[k] = -1; }
        }
        float mk[4];
        {
            const float* nm = nmax + wi * TZ_W + l;
            const float m = fmaxf(fmaxf(fmaxf(nm[0], nm[1]), fmaxf(nm[2], nm[TZ_W])), fmaxf(nm[TZ_W + 1], nm[TZ_W + 2]));
            mk[0] = mk[1] = mk[2] = mk[3] = m;
        }
        float ev[4][CB], Zs[4];
        uint32_t arg[4] = {0, 0, 0, 0};
        for (int attempt = 0; attempt < 2; ++attempt) {
            Zs[0] = Zs[1] = Zs[2] = Zs[3] = 0.f;
            float best[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int c = 0; c < CB; ++c) {
                const float* q = zp + c * TZ;
                const float vl = lerp_r(q[0], q[TZ_W], ly), vc = lerp_r(q[1], q[TZ_W + 1], ly), vr = lerp_r(q[2], q[TZ_W + 2], ly);
                const float dl = vc - vl, dr = vr - vc;
                float u[4] = {fmaf(0.625f, dl, vl), fmaf(0.875f, dl, vl), fmaf(0.125f, dr, vc), fmaf(0.375f, dr, vc)};
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (CONF && attempt == 0) { if (u[k] > best[k]) { best[k] = u[k]; arg[k] = c; } }
                    const float e = ex2_approx(u[k] - mk[k]);
                    ev[k][c] = e;
                    Zs[k] += e;
                }
            }
            // the bound can sit far above a pixel's true maximum only for wildly varying logits; then redo exactly
            const bool under = !(Zs[0] > 1e-30f) || !(Zs[1] > 1e-30f) || !(Zs[2] > 1e-30f) || !(Zs[3] > 1e-30f);
            if (!under || attempt == 1) break;
            float ex[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
            for (int c = 0; c < C; ++c) {
                const float* q = zp + c * TZ;
                const float vl = lerp_r(q[0], q[TZ_W], ly), vc = lerp_r(q[1], q[TZ_W + 1], ly), vr = lerp_r(q[2], q[TZ_W + 2], ly);
                const float dl = vc - vl, dr = vr - vc;
                ex[0] = fmaxf(ex[0], fmaf(0.625f, dl, vl)); ex[1] = fmaxf(ex[1], fmaf(0.875f, dl, vl));
                ex[2] = fmaxf(ex[2], fmaf(0.125f, dr, vc)); ex[3] = fmaxf(ex[3], fmaf(0.375f, dr, vc));
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) mk[k] = ex[k];
        }

        // ---- per pixel: loss, 1/Z, the "- onehot" part of the adjoint (integer, exact), confusion
        float rz[4];
        const int wy1 = 2 * r + 1, wy0 = 8 - wy1;                // eighths toward node rows i+1 / i
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            rz[k] = 0.f;
            if (lane_valid && lab[k] >= 0) {
                rz[k] = 1.0f / Zs[k];
                const float* q = zp + lab[k] * TZ;
                const float vl = lerp_r(q[0], q[TZ_W], ly), vc = lerp_r(q[1], q[TZ_W + 1], ly), vr = lerp_r(q[2], q[TZ_W + 2], ly);
                const float ul = k == 0 ? fmaf(0.625f, vc - vl, vl) : k == 1 ? fmaf(0.875f, vc - vl, vl)
                               : k == 2 ? fmaf(0.125f, vr - vc, vc) : fmaf(0.375f, vr - vc, vc);
                if (row_owned && lane_owned) {
                    loss += (__log2f(Zs[k]) + (mk[k] - ul)) * kLn2;
                    if (CONF) atomicAdd(a.conf + (int64_t)s * a.conf_stream_stride + lab[k] * C + arg[k], 1ull);
                }
                // horizontal eighths: k = 0,1 pull toward (xg-1, xg) with (3,5), (1,7); k = 2,3 toward (xg, xg+1) with (7,1), (5,3)
                const int wa = k == 0 ? 3 : k == 1 ? 1 : k == 2 ? 7 : 5, wb = 8 - wa;
                const int ca = k < 2 ? rx_l : rx_c, cb = k < 2 ? rx_c : rx_r;
                int* cc = corr + lab[k] * TZ;
                atomicAdd(cc + ry_top * TZ_W + ca, -wy0 * wa);
                atomicAdd(cc + ry_top * TZ_W + cb, -wy0 * wb);
                atomicAdd(cc + ry_bot * TZ_W + ca, -wy1 * wa);
                atomicAdd(cc + ry_bot * TZ_W + cb, -wy1 * wb);
            }
        }
        // ---- B: softmax part of the adjoint
        // at the clamped left/right border the outer node is the inner one: its weight joins the centre weight
        const bool fold_l = xg == 0, fold_r = xg == w - 1;
        const float w0l = fold_l ? 0.f : 0.375f * rz[0], w0c = (fold_l ? 1.0f : 0.625f) * rz[0];
        const float w1l = fold_l ? 0.f : 0.125f * rz[1], w1c = (fold_l ? 1.0f : 0.875f) * rz[1];
        const float w2r = fold_r ? 0.f : 0.125f * rz[2], w2c = (fold_r ? 1.0f : 0.875f) * rz[2];
        const float w3r = fold_r ? 0.f : 0.375f * rz[3], w3c = (fold_r ? 1.0f : 0.625f) * rz[3];
#pragma unroll
        for (int c = 0; c < CB; ++c) {
            const float aL = fmaf(w0l, ev[0][c], w1l * ev[1][c]);
            const float aR = fmaf(w2r, ev[2][c], w3r * ev[3][c]);
            const float aC = fmaf(w0c, ev[0][c], fmaf(w1c, ev[1][c], fmaf(w2c, ev[2][c], w3c * ev[3][c])));
            const float hsum = aC + __shfl_up_sync(0xffffffffu, aR, 1) + __shfl_down_sync(0xffffffffu, aL, 1);
            top[c] = fmaf(1.0f - ly, hsum, top[c]);
            bot[c] = fmaf(ly, hsum, bot[c]);
        }
    }
    // clamped borders in y
    if (i == -1) {
#pragma unroll
        for (int c = 0; c < CB; ++c) bot[c] += top[c];
    }
    if (i == h - 1) {
#pragma unroll
        for (int c = 0; c < CB; ++c) { top[c] += bot[c]; bot[c] = 0.f; }
    }
#pragma unroll
    for (int c = 0; c < CB; ++c)
        if (c < C) bsh[(wi * C + c) * 32 + l] = bot[c];
    // loss of the block, fixed order
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, o);
    if (l == 0) red[wi] = loss;
    if (n_bad) atomicAdd(a.bad, n_bad);
    __syncthreads();

    // ---- node row y0-1+wi (warps 1..RN_Y): own upper part + lower part of the warp above + onehot part
    const float invP = 1.0f / ((float)H * (float)W);
    const int y = i;
    const bool node_ok = wi >= 1 && y < h && lane_owned;
#pragma unroll
    for (int c = 0; c < CB; ++c) {
        if (c < C) {
            float v = 0.f;
            if (node_ok) {
                const int cr = corr[c * TZ + (y - (y0 - 1)) * TZ_W + (xg - (x0 - 2))];
                v = (top[c] + bsh[((wi - 1) * C + c) * 32 + l] + (float)cr * (1.0f / 64.0f)) * invP;
                a.dz[((int64_t)s * C + c) * p + (int64_t)y * w + xg] = v;
                if (a.dz_bf16)
                    a.dz_bf16[((int64_t)s * kClassPad + c) * a.dz_bf16_pitch + (int64_t)y * w + xg] = __float2bfloat16_rn(v);
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (l == 0) dbs[wi * C + c] = v;
        }
    }
    __syncthreads();
    for (int c = tid; c < C; c += R_THREADS) {
        float t = 0.f;
        for (int k = 1; k < R_WARPS; ++k) t += dbs[k * C + c];
        a.db_part[((int64_t)s * n_blk + blk) * C + c] = t;
    }
    if (tid == 0) {
        float t = 0.f;
        for (int k = 0; k < R_WARPS; ++k) t += red[k];
        a.loss_part[(int64_t)s * n_blk + blk] = t;
    }
}

template <int CB>
size_t rows_smem_bytes(int C)
{
    return ((size_t)(CB + C) * TZ + TZ + (size_t)R_WARPS * C * 32 + (size_t)R_WARPS * C) * sizeof(float) + 16;
}

template <int CB>
cudaError_t prepare_cb(int C)
{
    cudaError_t e = cudaFuncSetAttribute(upsample_ce_rows_kernel<CB, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rows_smem_bytes<CB>(C));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(upsample_ce_rows_kernel<CB, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rows_smem_bytes<CB>(C));
}

template <int CB>
void launch_cb(const UpsampleCeArgs& a, cudaStream_t s)
{
    dim3 grid((unsigned)((a.w + RN_X - 1) / RN_X), (unsigned)((a.h + RN_Y - 1) / RN_Y), (unsigned)a.S);
    if (a.conf) upsample_ce_rows_kernel<CB, true><<<grid, R_THREADS, rows_smem_bytes<CB>(a.C), s>>>(a);
    else upsample_ce_rows_kernel<CB, false><<<grid, R_THREADS, rows_smem_bytes<CB>(a.C), s>>>(a);
}

}  // namespace

bool upsample_ce_rows_supported(int C) { return C <= 32; }

int upsample_ce_rows_blocks(int h, int w) { return ((h + RN_Y - 1) / RN_Y) * ((w + RN_X - 1) / RN_X); }

cudaError_t prepare_upsample_ce_rows(int C)
{
    switch ((C + 3) / 4) {
        case 1: return prepare_cb<4>(C);
        case 2: return prepare_cb<8>(C);
        case 3: return prepare_cb<12>(C);
        case 4: return prepare_cb<16>(C);
        case 5: return prepare_cb<20>(C);
        case 6: return prepare_cb<24>(C);
        case 7: return prepare_cb<28>(C);
        default: return prepare_cb<32>(C);
    }
}

void launch_upsample_ce_rows(const UpsampleCeArgs& a, cudaStream_t s)
{
    switch ((a.C + 3) / 4) {
        case 1: launch_cb<4>(a, s); break;
        case 2: launch_cb<8>(a, s); break;
        case 3: launch_cb<12>(a, s); break;
        case 4: launch_cb<16>(a, s); break;
        case 5: launch_cb<20>(a, s); break;
        case 6: launch_cb<24>(a, s); break;
        case 7: launch_cb<28>(a, s); break;
        default: launch_cb<32>(a, s); break;
    }
}

}  // namespace st
