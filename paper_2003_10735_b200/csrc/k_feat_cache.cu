// K8 — cache the frozen front part's output once per key frame (Section 4.2: the frozen layers'
// outputs do not change while the back part is trained, so they are laid out once in the form
// the head's GEMMs read): fp32 [Cin][p] planar -> bf16 [p][Cin] (pixel-major, channels contiguous),
// round-to-nearest-even.
//
// A dtype/layout change: Cin*p*4 bytes in, Cin*p*2 bytes out.  A thread owns one pixel and 16 consecutive channels:
// it reads 16 planes (each warp 128 contiguous bytes per plane, all 16 loads in flight) and writes one full 32-byte
// sector of the pixel-major output with a single 256-bit store.  Neighbouring lanes' outputs lie Cin*2 bytes apart, so
// a sector written as two 16-byte halves reaches L2 as two partial writes: 18.5 us at 720p, against 14.5 us with the
// one store (a version that transposed 64 x 64 tiles through shared memory took 20.4 us).  No shared memory, no
// barrier.  The tensor-core path only exists for channel counts that are multiples of 64, so 16 always divides Cin.
#include "st_internal.h"

namespace st {

constexpr int kFeatGroup = 16;

__global__ void __launch_bounds__(256)
feat_to_bf16_nhwc_kernel(const float* __restrict__ in, int Cin, int64_t p, bf16* __restrict__ out)
{
    const int64_t pix = (int64_t)blockIdx.x * 256 + threadIdx.x;
    const int c0 = blockIdx.y * kFeatGroup;
    if (pix >= p) return;
    float v[kFeatGroup];
#pragma unroll
    for (int k = 0; k < kFeatGroup; ++k) v[k] = (c0 + k < Cin) ? __ldcs(in + (int64_t)(c0 + k) * p + pix) : 0.f;
    if (c0 + kFeatGroup <= Cin && ((uintptr_t)(out + pix * Cin + c0) % 32 == 0)) {
        uint32_t h[kFeatGroup / 2];
#pragma unroll
        for (int k = 0; k < kFeatGroup / 2; ++k) {
            __nv_bfloat162 two = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
            h[k] = *reinterpret_cast<uint32_t*>(&two);
        }
        store_256(out + pix * Cin + c0, h);
    } else {                                   // ragged channel count or unaligned output: element by element
        for (int k = 0; k < kFeatGroup; ++k)
            if (c0 + k < Cin) out[pix * Cin + c0 + k] = __float2bfloat16_rn(v[k]);
    }
}

void launch_feat_to_bf16_nhwc(const float* feat_chw, int Cin, int64_t p, bf16* out, cudaStream_t s)
{
    dim3 grid((unsigned)((p + 255) / 256), (unsigned)((Cin + kFeatGroup - 1) / kFeatGroup));
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
