// fp32 CUDA-core convolutions of the head (gemm_precision 0): forward, weight/bias gradients and
// the gradient passed from the 1x1 output layer to the hidden activation.  Planar [C][h][w].
// These state Algorithm 1's Forward / PartialBackward for the trainable back part in plain FMA
// arithmetic with fixed-order reductions (bit-reproducible run to run).  The bf16 tensor-core path
// replaces them when gemm_precision is 1.
#include "st_internal.h"

namespace st {

constexpr int kCoT = 8;   // output channels per thread

// Internal order of a conv weight: [tap][cout][cin] (for a 1x1 layer this is [cout][cin]).
__device__ __forceinline__ int64_t weight_index(int co, int ci, int tap, int Cout, int Cin, int /*taps*/)
{
    return ((int64_t)tap * Cout + co) * Cin + ci;
}

// out[co][y][x] = b[co] + sum_{ci,ky,kx} W[co][ci][ky][kx] * in[ci][y+ky-r][x+kx-r]  (zero padding);
// W is stored tap-major, see weight_index.
template <int KS>
__global__ void __launch_bounds__(128)
conv_fwd_f32_kernel(const float* __restrict__ in, int Cin, int h, int w, const float* __restrict__ Wt,
                    const float* __restrict__ b, int Cout, int relu, float* __restrict__ out,
                    int64_t in_stride, int64_t w_stride, int64_t b_stride, int64_t out_stride)
{
    const int s = blockIdx.z;
    in += s * in_stride; Wt += s * w_stride; b += s * b_stride; out += s * out_stride;
    const int64_t p = (int64_t)h * w;
    const int64_t pix = (int64_t)blockIdx.x * 128 + threadIdx.x;
    const int co0 = blockIdx.y * kCoT;
    if (pix >= p) return;
    const int y = (int)(pix / w), x = (int)(pix % w);
    constexpr int R = KS / 2;
    float acc[kCoT];
#pragma unroll
    for (int k = 0; k < kCoT; ++k) acc[k] = 0.f;
    for (int ci = 0; ci < Cin; ++ci) {
        const float* plane = in + (int64_t)ci * p;
#pragma unroll
        for (int ky = 0; ky < KS; ++ky) {
            int yy = y + ky - R;
#pragma unroll
            for (int kx = 0; kx < KS; ++kx) {
                int xx = x + kx - R;
                float v = (yy >= 0 && yy < h && xx >= 0 && xx < w) ? __ldg(plane + (int64_t)yy * w + xx) : 0.f;
#pragma unroll
                for (int k = 0; k < kCoT; ++k) {
                    int co = co0 + k;
                    float wv = co < Cout ? __ldg(Wt + weight_index(co, ci, ky * KS + kx, Cout, Cin, KS * KS)) : 0.f;
                    acc[k] = fmaf(wv, v, acc[k]);
                }
            }
        }
    }
#pragma unroll
    for (int k = 0; k < kCoT; ++k) {
        int co = co0 + k;
        if (co < Cout) {
            float v = acc[k] + __ldg(b + co);
            if (relu) v = v > 0.f ? v : 0.f;
            out[(int64_t)co * p + pix] = v;
        }
    }
}

void launch_conv_fwd_f32(const float* in, int Cin, int h, int w, const float* Wt, const float* b,
                         int Cout, int ks, bool relu, float* out, int S, int64_t in_stride,
                         int64_t w_stride, int64_t b_stride, int64_t out_stride, cudaStream_t s)
{
    int64_t p = (int64_t)h * w;
    dim3 grid((unsigned)((p + 127) / 128), (unsigned)((Cout + kCoT - 1) / kCoT), (unsigned)S);
    if (ks == 1)
        conv_fwd_f32_kernel<1><<<grid, 128, 0, s>>>(in, Cin, h, w, Wt, b, Cout, relu, out, in_stride, w_stride, b_stride, out_stride);
    else
        conv_fwd_f32_kernel<3><<<grid, 128, 0, s>>>(in, Cin, h, w, Wt, b, Cout, relu, out, in_stride, w_stride, b_stride, out_stride);
}

// dW[co][ci][ky][kx] = sum_{y,x} dout[co][y][x] * in[ci][y+ky-r][x+kx-r].
// One block per (ci, tile of kCoT output channels, stream); threads stride over pixels, then a
// fixed-order block reduction (shuffle tree inside a warp, warps added in index order).
template <int KS>
__global__ void __launch_bounds__(256)
conv_wgrad_f32_kernel(const float* __restrict__ in, const float* __restrict__ dout, int Cin, int Cout,
                      int h, int w, float* __restrict__ dW, int64_t in_stride, int64_t dout_stride,
                      int64_t dw_stride)
{
    constexpr int T = KS * KS, R = KS / 2;
    const int s = blockIdx.z;
    in += s * in_stride; dout += s * dout_stride; dW += s * dw_stride;
    const int ci = blockIdx.x, co0 = blockIdx.y * kCoT;
    const int64_t p = (int64_t)h * w;
    const float* plane = in + (int64_t)ci * p;
    float acc[kCoT][T];
#pragma unroll
    for (int k = 0; k < kCoT; ++k)
#pragma unroll
        for (int t = 0; t < T; ++t) acc[k][t] = 0.f;
    for (int64_t pix = threadIdx.x; pix < p; pix += 256) {
        const int y = (int)(pix / w), x = (int)(pix % w);
        float xv[T];
#pragma unroll
        for (int ky = 0; ky < KS; ++ky)
#pragma unroll
            for (int kx = 0; kx < KS; ++kx) {
                int yy = y + ky - R, xx = x + kx - R;
                xv[ky * KS + kx] = (yy >= 0 && yy < h && xx >= 0 && xx < w) ? __ldg(plane + (int64_t)yy * w + xx) : 0.f;
            }
#pragma unroll
        for (int k = 0; k < kCoT; ++k) {
            int co = co0 + k;
            float d = co < Cout ? __ldg(dout + (int64_t)co * p + pix) : 0.f;
#pragma unroll
            for (int t = 0; t < T; ++t) acc[k][t] = fmaf(d, xv[t], acc[k][t]);
        }
    }
    __shared__ float red[8][kCoT * T];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int k = 0; k < kCoT; ++k)
#pragma unroll
        for (int t = 0; t < T; ++t) {
            float v = acc[k][t];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if (lane == 0) red[warp][k * T + t] = v;
        }
    __syncthreads();
    for (int i = threadIdx.x; i < kCoT * T; i += 256) {
        float v = 0.f;
        for (int wv = 0; wv < 8; ++wv) v += red[wv][i];
        int k = i / T, t = i % T, co = co0 + k;
        if (co < Cout) dW[weight_index(co, ci, t, Cout, Cin, T)] = v;
    }
}

void launch_conv_wgrad_f32(const float* in, const float* dout, int Cin, int Cout, int h, int w, int ks,
                           float* dW, int S, int64_t in_stride, int64_t dout_stride,
                           int64_t dw_stride, cudaStream_t s)
{
    dim3 grid((unsigned)Cin, (unsigned)((Cout + kCoT - 1) / kCoT), (unsigned)S);
    if (ks == 1)
        conv_wgrad_f32_kernel<1><<<grid, 256, 0, s>>>(in, dout, Cin, Cout, h, w, dW, in_stride, dout_stride, dw_stride);
    else
        conv_wgrad_f32_kernel<3><<<grid, 256, 0, s>>>(in, dout, Cin, Cout, h, w, dW, in_stride, dout_stride, dw_stride);
}

// db[c] = sum_p d[c][p]; one block per (channel, stream), fixed-order reduction.
__global__ void __launch_bounds__(256)
bias_grad_f32_kernel(const float* __restrict__ d, int64_t p, float* __restrict__ db, int64_t d_stride,
                     int64_t db_stride)
{
    const int c = blockIdx.x, s = blockIdx.y;
    const float* src = d + s * d_stride + (int64_t)c * p;
    float v = 0.f;
    for (int64_t i = threadIdx.x; i < p; i += 256) v += __ldg(src + i);
    __shared__ float red[8];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    if (threadIdx.x == 0) {
        float t = 0.f;
        for (int k = 0; k < 8; ++k) t += red[k];
        db[s * db_stride + c] = t;
    }
}

void launch_bias_grad_f32(const float* d, int C, int64_t p, float* db, int S, int64_t d_stride,
                          int64_t db_stride, cudaStream_t s)
{
    bias_grad_f32_kernel<<<dim3((unsigned)C, (unsigned)S), 256, 0, s>>>(d, p, db, d_stride, db_stride);
}

// dH[k][p] = [Hact[k][p] > 0] * sum_c W2[c][k] * dz[c][p]
__global__ void __launch_bounds__(128)
conv1x1_dgrad_relu_f32_kernel(const float* __restrict__ W2, const float* __restrict__ dz,
                              const float* __restrict__ Hact, int C, int Ch, int64_t p,
                              float* __restrict__ dH, int64_t w_stride, int64_t dz_stride, int64_t h_stride)
{
    const int s = blockIdx.z;
    W2 += s * w_stride; dz += s * dz_stride; Hact += s * h_stride; dH += s * h_stride;
    const int64_t pix = (int64_t)blockIdx.x * 128 + threadIdx.x;
    const int k0 = blockIdx.y * kCoT;
    if (pix >= p) return;
    float acc[kCoT];
#pragma unroll
    for (int k = 0; k < kCoT; ++k) acc[k] = 0.f;
    for (int c = 0; c < C; ++c) {
        float d = __ldg(dz + (int64_t)c * p + pix);
#pragma unroll
        for (int k = 0; k < kCoT; ++k) {
            float wv = (k0 + k) < Ch ? __ldg(W2 + (int64_t)c * Ch + k0 + k) : 0.f;
            acc[k] = fmaf(wv, d, acc[k]);
        }
    }
#pragma unroll
    for (int k = 0; k < kCoT; ++k)
        if (k0 + k < Ch) {
            int64_t i = (int64_t)(k0 + k) * p + pix;
            dH[i] = Hact[i] > 0.f ? acc[k] : 0.f;
        }
}

void launch_conv1x1_dgrad_relu_f32(const float* W2, const float* dz, const float* Hact, int C, int Ch,
                                   int64_t p, float* dH, int S, int64_t w_stride, int64_t dz_stride,
                                   int64_t h_stride, cudaStream_t s)
{
    dim3 grid((unsigned)((p + 127) / 128), (unsigned)((Ch + kCoT - 1) / kCoT), (unsigned)S);
    conv1x1_dgrad_relu_f32_kernel<<<grid, 128, 0, s>>>(W2, dz, Hact, C, Ch, p, dH, w_stride, dz_stride, h_stride);
}

}  // namespace st
