// Loss weighting against class imbalance (Section 5.2): pixels near and within non-background objects weigh more.
// Computed once per key frame (the labels do not change over the K steps): a pixel is "near" if a pixel within
// `radius` rows and columns of it (square window, cut at the frame border) carries a label other than the
// background class.  Two passes (columns within a row, then rows) over one temporary byte map; the result is the
// label map again with bit 7 set on the weighted pixels, which is what the fused loss kernel reads, so that the
// weighting costs the step no extra memory traffic.  Labels above 126 cannot be tagged and become 127.
#include "st_internal.h"

namespace st {

namespace {

__global__ void near_rows_kernel(const uint8_t* __restrict__ lab, int H, int W, int background, int radius, uint8_t* __restrict__ tmp)
{
    const int x = blockIdx.x * blockDim.x + threadIdx.x, y = blockIdx.y;
    if (x >= W) return;
    const uint8_t* row = lab + (int64_t)y * W;
    int near = 0;
    for (int xx = max(x - radius, 0); xx <= min(x + radius, W - 1); ++xx) near |= row[xx] != background;
    tmp[(int64_t)y * W + x] = (uint8_t)near;
}

__global__ void near_cols_tag_kernel(const uint8_t* __restrict__ lab, const uint8_t* __restrict__ tmp, int H, int W, int radius,
                                     uint8_t* __restrict__ out)
{
    const int x = blockIdx.x * blockDim.x + threadIdx.x, y = blockIdx.y;
    if (x >= W) return;
    int near = 0;
    for (int yy = max(y - radius, 0); yy <= min(y + radius, H - 1); ++yy) near |= tmp[(int64_t)yy * W + x];
    const int64_t i = (int64_t)y * W + x;
    const int l = lab[i];
    out[i] = (uint8_t)((l > 126 ? 127 : l) | (near ? 0x80 : 0));
}

}  // namespace

void launch_object_weight_tags(const uint8_t* labels, int H, int W, int background, int radius, uint8_t* tmp, uint8_t* tagged,
                               cudaStream_t s)
{
    const dim3 grid((unsigned)((W + 255) / 256), (unsigned)H, 1);
    near_rows_kernel<<<grid, 256, 0, s>>>(labels, H, W, background, radius, tmp);
    near_cols_tag_kernel<<<grid, 256, 0, s>>>(labels, tmp, H, W, radius, tagged);
}

}  // namespace st
