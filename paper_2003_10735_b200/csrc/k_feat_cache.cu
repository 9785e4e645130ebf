// K8 — cache the frozen front part's output once per key frame (Section 4.2: the frozen layers'
// outputs do not change while the back part is trained, so they are laid out once in the form
// the head's GEMMs read): fp32 [Cin][p] planar -> bf16 [p][Cin] (pixel-major, channels contiguous),
// round-to-nearest-even.
//
// A dtype/layout change: Cin*p*4 bytes in, Cin*p*2 bytes out.  Tiles of 64 channels x 64 pixels go
// through shared memory so that both the reads (along pixels) and the writes (along channels) are
// full 128-byte lines: reads are 16-byte vectors of 4 pixels, writes 16-byte vectors of 8 channels.
#include "st_internal.h"

namespace st {

constexpr int kTileC = 64, kTileP = 64;

__global__ void __launch_bounds__(256)
feat_to_bf16_nhwc_kernel(const float* __restrict__ in, int Cin, int64_t p, bf16* __restrict__ out)
{
    __shared__ float tile[kTileC][kTileP + 1];
    const int64_t p0 = (int64_t)blockIdx.x * kTileP;
    const int c0 = blockIdx.y * kTileC;
    const bool vec_in = (p % 4 == 0) && ((uintptr_t)in % 16 == 0);
    // load: 64 channels x 16 quads
    for (int i = threadIdx.x; i < kTileC * (kTileP / 4); i += 256) {
        int c = i / (kTileP / 4), q = i % (kTileP / 4);
        int64_t pp = p0 + q * 4;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c0 + c < Cin) {
            const float* src = in + (int64_t)(c0 + c) * p + pp;
            if (vec_in && pp + 3 < p) v = __ldcs(reinterpret_cast<const float4*>(src));
            else {
                if (pp + 0 < p) v.x = src[0];
                if (pp + 1 < p) v.y = src[1];
                if (pp + 2 < p) v.z = src[2];
                if (pp + 3 < p) v.w = src[3];
            }
        }
        tile[c][q * 4 + 0] = v.x; tile[c][q * 4 + 1] = v.y; tile[c][q * 4 + 2] = v.z; tile[c][q * 4 + 3] = v.w;
    }
    __syncthreads();
    // store: 64 pixels x 8 groups of 8 channels
    const bool vec_out = (Cin % 8 == 0) && ((uintptr_t)out % 16 == 0);
    for (int i = threadIdx.x; i < kTileP * (kTileC / 8); i += 256) {
        int px = i / (kTileC / 8), g = i % (kTileC / 8);
        int64_t pp = p0 + px;
        if (pp >= p) continue;
        int c = c0 + g * 8;
        if (vec_out && c + 7 < Cin) {
            __nv_bfloat162 h[4];
#pragma unroll
            for (int k = 0; k < 4; ++k)
                h[k] = __floats2bfloat162_rn(tile[g * 8 + 2 * k][px], tile[g * 8 + 2 * k + 1][px]);
            *reinterpret_cast<uint4*>(out + pp * Cin + c) = *reinterpret_cast<uint4*>(h);
        } else {
            for (int k = 0; k < 8; ++k)
                if (c + k < Cin) out[pp * Cin + c + k] = __float2bfloat16_rn(tile[g * 8 + k][px]);
        }
    }
}

void launch_feat_to_bf16_nhwc(const float* feat_chw, int Cin, int64_t p, bf16* out, cudaStream_t s)
{
    dim3 grid((unsigned)((p + kTileP - 1) / kTileP), (unsigned)((Cin + kTileC - 1) / kTileC));
    feat_to_bf16_nhwc_kernel<<<grid, 256, 0, s>>>(feat_chw, Cin, p, out);
}

// Verification helper: bf16 [p][C] -> fp32 [C][p].  Not on the hot path.
__global__ void nhwc_bf16_to_chw_kernel(const bf16* __restrict__ in, int C, int64_t p, float* __restrict__ out)
{
    int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= (int64_t)C * p) return;
    int c = (int)(i / p);
    int64_t pp = i % p;
    out[i] = __bfloat162float(in[pp * C + c]);
}

void launch_nhwc_bf16_to_chw(const bf16* in, int C, int64_t p, float* out, cudaStream_t s)
{
    int64_t n = (int64_t)C * p;
    nhwc_bf16_to_chw_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(in, C, p, out);
}

}  // namespace st
