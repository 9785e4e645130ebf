// K5 — OptimStep of Algorithm 1 ("most simply gradient descent", Section 4.1.4) with heavy-ball
// momentum:  v <- mu*v + g ;  theta <- theta - lr*v   (mu = 0: plain gradient descent),
// on the fp32 master parameters; the bf16 copies read by the tensor-core GEMMs are refreshed in
// the same pass.  The kernel also finishes the reductions the step left open, always in a fixed
// order so that results are bit-reproducible: split-K partial sums of the weight gradients,
// per-block partial sums of the bias gradients, and the per-block loss partials.
// K7 — UpdatedPart(student) (Algorithm 3): the packed fp32 buffer of all trainable tensors.
#include "st_internal.h"
#include "miou.cuh"
#include "train_ctl.cuh"

#include <cstdlib>

namespace st {

bool pdl_enabled()
{
    static const bool on = [] { const char* e = getenv("ST_PDL"); return !(e && e[0] == '0'); }();
    return on;
}

constexpr int kUpdThreads = 256;

// bf16 copies of weight element e (internal order [tap][cout][cin]) of a layer: the one the forward and the weight
// gradient read, and, for a 3x3 layer whose gradient is passed back, the mirrored and transposed one
__device__ __forceinline__ void write_shadows(const LayerUpdate& ly, int s, int64_t e, float value)
{
    const bf16 v = __float2bfloat16_rn(value);
    if (ly.shadow) ly.shadow[(int64_t)s * ly.shadow_stream_stride + e] = v;
    if (ly.shadow_t) {
        const int ci = (int)(e % ly.cin);
        if (ci < ly.c_take) {
            const int64_t r = e / ly.cin;
            const int co = (int)(r % ly.cout), tap = (int)(r / ly.cout);
            ly.shadow_t[(int64_t)s * ly.shadow_t_stream_stride + ((int64_t)(ly.taps - 1 - tap) * ly.c_take + ci) * ly.cout + co] = v;
        }
    }
}

// Bias corrections of Adam's step t: (1 - b1^t, 1 - b2^t), t = steps taken before this call + position in the call.
struct AdamCorr { double c1, c2; };
template <bool ADAM>
__device__ __forceinline__ AdamCorr adam_corrections(const UpdateArgs& a, int s)
{
    AdamCorr c = {1.0, 1.0};
    if (ADAM) {
        const double t = (double)(a.step_base[s] + a.loss_slot + 1);
        c.c1 = 1.0 - exp(t * a.ln_b1);
        c.c2 = 1.0 - exp(t * a.ln_b2);
    }
    return c;
}

// OptimStep on one parameter.  Gradient descent with momentum: v <- mu v + g; theta <- theta - lr v.
// Adam (each element in double, stored as fp32): m <- b1 m + (1 - b1) g; v <- b2 v + (1 - b2) g^2;
// theta <- theta - lr (m / c1) / (sqrt(v / c2) + eps).
// The state of one parameter (value, momentum or first moment, second moment), which the gradient kernels before the
// update never write: it can be fetched before their results are waited for.
struct ParamState { float theta, vel, vel2; };
template <bool ADAM>
__device__ __forceinline__ ParamState load_state(const UpdateArgs& a, int64_t gi)
{
    ParamState p;
    p.theta = a.theta[gi]; p.vel = a.vel[gi]; p.vel2 = ADAM ? a.vel2[gi] : 0.f;
    return p;
}

template <bool ADAM>
__device__ __forceinline__ float apply_update(const UpdateArgs& a, int64_t gi, float g, const AdamCorr& k, const ParamState& p)
{
    a.grad[gi] = g;
    if (ADAM) {
        const double gd = (double)g;
        const double m = a.b1 * (double)p.vel + (1.0 - a.b1) * gd;
        const double v = a.b2 * (double)p.vel2 + (1.0 - a.b2) * gd * gd;
        a.vel[gi] = (float)m;
        a.vel2[gi] = (float)v;
        const float t = (float)((double)p.theta - (double)a.lr * (m / k.c1) / (sqrt(v / k.c2) + a.eps));
        a.theta[gi] = t;
        return t;
    }
    float v = fmaf(a.mu, p.vel, g);
    a.vel[gi] = v;
    const float t = fmaf(-a.lr, v, p.theta);
    a.theta[gi] = t;
    return t;
}
template <bool ADAM>
__device__ __forceinline__ float apply_update(const UpdateArgs& a, int64_t gi, float g, const AdamCorr& k)
{
    return apply_update<ADAM>(a, gi, g, k, load_state<ADAM>(a, gi));
}

// Parameter blocks: a block covers kUpdThreads / G consecutive parameters; the G thread groups of a
// block each sum every G-th split-K partial of "their" parameter (coalesced along the parameters),
// the group sums are added in group order through shared memory, and group 0 applies the update.
template <int G, int E, bool ADAM>
__global__ void __launch_bounds__(kUpdThreads)
sgd_update_kernel(UpdateArgs a, int n_param_blocks, int64_t range_begin)
{
    constexpr int kRow = kUpdThreads / G;      // consecutive parameters covered by one thread group
    constexpr int kPer = kRow * E;             // parameters per block
    __shared__ float part[G][kPer];
    const int s = blockIdx.y;
    const int64_t base = (int64_t)s * a.n_params;
    const bool param_block = (int)blockIdx.x < n_param_blocks;
    const int col = threadIdx.x % kRow, g = threadIdx.x / kRow;
    int layer[E];
    bool is_weight[E], has_partials[E];
    ParamState state[E];
    // which parameters this thread looks after, and (first thread group) their current state: none of it comes from the
    // kernels just before this one, so it is done before their completion is waited for
    if (param_block) {
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int64_t i = range_begin + (int64_t)blockIdx.x * kPer + e * kRow + col;
            layer[e] = -1; is_weight[e] = false; has_partials[e] = false;
            state[e].theta = state[e].vel = state[e].vel2 = 0.f;
            if (i < a.n_params) {
                for (int L = 0; L < a.n_layers; ++L) {
                    const LayerUpdate& ly = a.layer[L];
                    const int64_t nw = (int64_t)ly.cout * ly.cin * ly.taps;
                    if (i >= ly.w_off && i < ly.w_off + nw && !ly.streamed) { layer[e] = L; is_weight[e] = true; }
                    if (i >= ly.b_off && i < ly.b_off + ly.cout) { layer[e] = L; is_weight[e] = false; }
                }
            }
            if (g == 0 && layer[e] >= 0 && (is_weight[e] || !a.layer[layer[e]].b_partials)) state[e] = load_state<ADAM>(a, base + i);
        }
    }
    TrainHistory hist{};
    if (a.has_ctl) hist = train_history(a.ctl, s);
    pdl_wait();
    pdl_launch_dependents();
    bool skip = a.skip && a.skip[(int64_t)s * a.skip_stride];   // block-uniform
    bool better = false;                                         // Train: this prediction is the best so far
    MiouFetch fetched{};
    const bool decide_here = a.has_ctl == 1;                     // 2: the backward before this kernel has assessed the prediction
    if (decide_here) fetched = train_fetch(a.ctl, s, hist);      // on their way while the partial sums are fetched and added
    if (a.has_ctl == 2 && !hist.ended) train_outcome(a.ctl, s, skip, better);
    float* best_theta = a.has_ctl ? a.ctl.best_theta : nullptr;
    const AdamCorr corr = adam_corrections<ADAM>(a, s);
    if (param_block) {
        if (a.has_ctl && hist.ended) {                  // nothing to assess, nothing to update: the history goes on
            if (decide_here) train_decision(a.ctl, s, blockIdx.x == 0, hist, &fetched, skip, better);
            return;
        }
        if (skip && !decide_here && !better) return;
        float sum[E];
        // E parameters per thread, all of their split-K loads issued before any is consumed
#pragma unroll
        for (int e = 0; e < E; ++e) {
            const int64_t i = range_begin + (int64_t)blockIdx.x * kPer + e * kRow + col;
            sum[e] = 0.f;
            if (layer[e] >= 0 && is_weight[e] && a.layer[layer[e]].w_partials) {
                const LayerUpdate& ly = a.layer[layer[e]];
                has_partials[e] = true;
                const float* src = ly.w_partials + (int64_t)s * ly.w_stream_stride + (i - ly.w_off);
                // batches of 8 predicated loads: all in flight together, no one-at-a-time remainder loop
                float t = 0.f;
                for (int k0 = g; k0 < ly.n_split; k0 += 8 * G) {
                    float v[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int k = k0 + j * G;
                        v[j] = k < ly.n_split ? __ldg(src + (int64_t)k * ly.w_split_stride) : 0.f;
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) t += v[j];
                }
                sum[e] = t;
            }
        }
#pragma unroll
        for (int e = 0; e < E; ++e) part[g][e * kRow + col] = sum[e];
        if (decide_here) train_decision(a.ctl, s, blockIdx.x == 0, hist, &fetched, skip, better);
        __syncthreads();
        if (g != 0 || (skip && !better)) return;
#pragma unroll
        for (int e = 0; e < E; ++e) {
            if (layer[e] < 0) continue;
            const int64_t i = range_begin + (int64_t)blockIdx.x * kPer + e * kRow + col;
            const LayerUpdate& ly = a.layer[layer[e]];
            if (is_weight[e]) {
                float gr;
                if (has_partials[e]) {
                    gr = 0.f;
#pragma unroll
                    for (int k = 0; k < G; ++k) gr += part[k][e * kRow + col];
                } else {
                    gr = a.grad[base + i];
                }
                if (better) best_theta[base + i] = state[e].theta;
                if (!skip) write_shadows(ly, s, i - ly.w_off, apply_update<ADAM>(a, base + i, gr, corr, state[e]));
            } else if (!ly.b_partials) {
                if (better) best_theta[base + i] = state[e].theta;
                if (!skip) apply_update<ADAM>(a, base + i, a.grad[base + i], corr, state[e]);
            }   // biases with partial sums are finished by the reduction warps below
        }
        return;
    }
    // ---- reduction warps: one warp per bias element that has partial sums, plus one for the loss
    if (decide_here) train_decision(a.ctl, s, blockIdx.x == 0, hist, &fetched, skip, better);
    else if (a.has_ctl && hist.ended) skip = true;
    const int warp = ((int)blockIdx.x - n_param_blocks) * (kUpdThreads / 32) + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    int item = warp;
    for (int L = 0; L < a.n_layers; ++L) {
        const LayerUpdate& ly = a.layer[L];
        if (!ly.b_partials) continue;
        if (item < ly.cout) {
            const float* src = ly.b_partials + (int64_t)s * ly.n_bpart * ly.cout + item;
            float g = 0.f;
            for (int k0 = lane; k0 < ly.n_bpart; k0 += 8 * 32) {
                float v[8];
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    const int k = k0 + j * 32;
                    v[j] = k < ly.n_bpart ? __ldg(src + (int64_t)k * ly.cout) : 0.f;
                }
#pragma unroll
                for (int j = 0; j < 8; ++j) g += v[j];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) g += __shfl_xor_sync(0xffffffffu, g, o);
            if (lane == 0) {
                if (better) best_theta[base + ly.b_off + item] = a.theta[base + ly.b_off + item];
                if (!skip) apply_update<ADAM>(a, base + ly.b_off + item, g, corr);
            }
            return;
        }
        item -= ly.cout;
    }
    if (item == 0 && a.loss_part) {
        double t = 0.0;
        for (int k0 = lane; k0 < a.n_loss_part; k0 += 8 * 32) {
            float v[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int k = k0 + j * 32;
                v[j] = k < a.n_loss_part ? __ldg(a.loss_part + (int64_t)s * a.n_loss_part + k) : 0.f;
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) t += (double)v[j];
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (lane == 0) {
            if (a.loss_slot >= 0 && a.loss_slot < kMaxSteps)
                a.loss_buf[(int64_t)s * kMaxSteps + a.loss_slot] = (float)(t * a.inv_P);
        }
    }
}

// A large weight tensor with a moderate number of split-K partials (the 3x3 layer): a pure stream.
// Each thread owns VEC consecutive weights and reads them from every partial with all loads in flight.
template <int VEC, bool ADAM>
__global__ void __launch_bounds__(256)
sgd_update_stream_kernel(UpdateArgs a, int L)
{
    pdl_wait();
    pdl_launch_dependents();
    const LayerUpdate& ly = a.layer[L];
    const int s = blockIdx.y;
    bool skip = a.skip && a.skip[(int64_t)s * a.skip_stride], better = false;
    if (a.has_ctl) {                                                   // the grouped kernel's block 0 writes the history
        const TrainHistory hist = train_history(a.ctl, s);
        if (a.has_ctl == 1) { const MiouFetch f = train_fetch(a.ctl, s, hist); train_decision(a.ctl, s, false, hist, &f, skip, better); }
        else if (hist.ended) skip = true;
        else train_outcome(a.ctl, s, skip, better);
    }
    if (skip && !better) return;
    const int64_t nw = (int64_t)ly.cout * ly.cin * ly.taps;
    const int64_t e = ((int64_t)blockIdx.x * 256 + threadIdx.x) * VEC;
    if (e >= nw) return;
    const float* src = ly.w_partials + (int64_t)s * ly.w_stream_stride + e;
    float g[VEC];
#pragma unroll
    for (int j = 0; j < VEC; ++j) g[j] = 0.f;
    for (int k0 = 0; k0 < ly.n_split; k0 += 8) {
        if (VEC == 4) {
            float4 t[8];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                t[j] = k0 + j < ly.n_split ? __ldg(reinterpret_cast<const float4*>(src + (int64_t)(k0 + j) * ly.w_split_stride))
                                           : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j = 0; j < 8; ++j) { g[0] += t[j].x; g[1] += t[j].y; g[2] += t[j].z; g[3] += t[j].w; }
        } else {
            float t[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) t[j] = k0 + j < ly.n_split ? __ldg(src + (int64_t)(k0 + j) * ly.w_split_stride) : 0.f;
#pragma unroll
            for (int j = 0; j < 8; ++j) g[0] += t[j];
        }
    }
    const int64_t gi = (int64_t)s * a.n_params + ly.w_off + e;
    const AdamCorr corr = adam_corrections<ADAM>(a, s);
#pragma unroll
    for (int j = 0; j < VEC; ++j) {
        if (better) a.ctl.best_theta[gi + j] = a.theta[gi + j];
        if (!skip) write_shadows(ly, s, e + j, apply_update<ADAM>(a, gi + j, g[j], corr));
    }
}

template <bool ADAM>
static int launch_sgd_update_t(const UpdateArgs& a, cudaStream_t s)
{
    int n_launches = 1;
    // large layers with partial sums go through the streaming kernel; everything else (small layers, biases,
    // loss) through the grouped kernel, which then starts after the streamed range
    int64_t range_begin = a.param_begin;
    UpdateArgs g = a;                    // what the grouped kernel gets: streamed layers lose their partial sums there
    for (int L = 0; L < a.n_layers; ++L) {
        const LayerUpdate& ly = a.layer[L];
        const int64_t nw = (int64_t)ly.cout * ly.cin * ly.taps;
        if (ly.w_partials && nw >= 65536) {
            const bool vec = nw % 4 == 0 && ly.w_split_stride % 4 == 0 && ly.w_stream_stride % 4 == 0 &&
                             ((uintptr_t)ly.w_partials % 16 == 0);
            if (vec) launch_chain(a.chain_early != 0, sgd_update_stream_kernel<4, ADAM>, dim3((unsigned)((nw / 4 + 255) / 256), (unsigned)a.S), dim3(256), 0, s, a, L);
            else launch_chain(a.chain_early != 0, sgd_update_stream_kernel<1, ADAM>, dim3((unsigned)((nw + 255) / 256), (unsigned)a.S), dim3(256), 0, s, a, L);
            if (ly.w_off == range_begin) range_begin = ly.w_off + nw;     // the grouped kernel starts behind leading streamed layers
            g.layer[L].streamed = 1;                                       // ... and leaves the weights of later ones alone
            ++n_launches;
        }
    }
    int items = 1, max_split = 1;
    for (int L = 0; L < a.n_layers; ++L) {
        if (a.layer[L].b_partials) items += a.layer[L].cout;
        if (a.layer[L].w_partials && !g.layer[L].streamed && a.layer[L].n_split > max_split) max_split = a.layer[L].n_split;
    }
    const int n_red_blocks = (items + kUpdThreads / 32 - 1) / (kUpdThreads / 32);
    const int64_t n_rest = a.n_params - range_begin;
    const bool big = n_rest > 65536;
    // many partial sums per parameter: 16 thread groups, so that a group's share fits one batch of loads
    const int G = max_split <= 1 ? 1 : (max_split > 64 && !big ? 16 : 8), E = big ? 4 : 1;
    const int per = kUpdThreads / G * E;
    const int n_param_blocks = (int)((n_rest + per - 1) / per);
    const dim3 grid((unsigned)(n_param_blocks + n_red_blocks), (unsigned)a.S);
    const dim3 blk(kUpdThreads);
    if (G == 1 && E == 1) launch_chain(a.chain_early != 0, sgd_update_kernel<1, 1, ADAM>, grid, blk, 0, s, g, n_param_blocks, range_begin);
    else if (G == 1) launch_chain(a.chain_early != 0, sgd_update_kernel<1, 4, ADAM>, grid, blk, 0, s, g, n_param_blocks, range_begin);
    else if (G == 16) launch_chain(a.chain_early != 0, sgd_update_kernel<16, 1, ADAM>, grid, blk, 0, s, g, n_param_blocks, range_begin);
    else if (E == 1) launch_chain(a.chain_early != 0, sgd_update_kernel<8, 1, ADAM>, grid, blk, 0, s, g, n_param_blocks, range_begin);
    else launch_chain(a.chain_early != 0, sgd_update_kernel<8, 4, ADAM>, grid, blk, 0, s, g, n_param_blocks, range_begin);
    return n_launches;
}

int launch_sgd_update(const UpdateArgs& a, cudaStream_t s)
{
    return a.adam ? launch_sgd_update_t<true>(a, s) : launch_sgd_update_t<false>(a, s);
}

__global__ void step_tick_kernel(long long* step_base, int S, int add, const int* add_per_stream)
{
    const int s = threadIdx.x;
    if (s < S) step_base[s] += add_per_stream ? add_per_stream[s] : add;
}

void launch_step_tick(long long* step_base, int S, int add, const int* add_per_stream, cudaStream_t s)
{
    for (int s0 = 0; s0 < S; s0 += 256)
        step_tick_kernel<<<1, 256, 0, s>>>(step_base + s0, S - s0 < 256 ? S - s0 : 256, add, add_per_stream ? add_per_stream + s0 : nullptr);
}

__global__ void refresh_shadow_kernel(UpdateArgs a)
{
    const int s = blockIdx.y;
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= a.n_params) return;
    for (int L = 0; L < a.n_layers; ++L) {
        const LayerUpdate& ly = a.layer[L];
        const int64_t nw = (int64_t)ly.cout * ly.cin * ly.taps;
        if (i >= ly.w_off && i < ly.w_off + nw) write_shadows(ly, s, i - ly.w_off, a.theta[(int64_t)s * a.n_params + i]);
    }
}

void launch_refresh_shadow(const UpdateArgs& a, cudaStream_t s)
{
    refresh_shadow_kernel<<<dim3((unsigned)((a.n_params + 255) / 256), (unsigned)a.S), 256, 0, s>>>(a);
}

__global__ void __launch_bounds__(256) miou_kernel(const unsigned long long* __restrict__ conf, int C, double* out)
{
    __shared__ double iou[256];
    __shared__ int present[256];
    const double m = block_miou(conf, C, iou, present);
    if (threadIdx.x == 0) *out = m;
}

// ---- Algorithm 1, the lines after "metric <- ComputeMetric(prediction, label)" ------------------------
// One launch per prediction; blockIdx.y = stream.  Every block computes the stream's mean IoU from the confusion
// matrix of the prediction (same arithmetic as miou_kernel), all blocks together copy the parameters into
// best_student if the metric is a new best, and block 0 records the decisions:
//   prediction 0 (the incoming student):  best_metric <- metric; the loop is entered iff best_metric < THRESHOLD
//   prediction i > 0 (after i updates):   if metric > best_metric: best_metric, best_student <- metric, student;
//                                         if metric > THRESHOLD: break;  the loop also ends at i = MAX_UPDATES.
__global__ void __launch_bounds__(256) train_commit_kernel(const float* __restrict__ best_theta, float* __restrict__ theta, int64_t n_params,
                                                           int64_t begin)
{
    const int64_t base = (int64_t)blockIdx.y * n_params;
    for (int64_t e = begin + (int64_t)blockIdx.x * 256 + threadIdx.x; e < n_params; e += (int64_t)gridDim.x * 256) theta[base + e] = best_theta[base + e];
}

void launch_miou(const unsigned long long* conf, int C, double* out, cudaStream_t s)
{
    miou_kernel<<<1, 256, 0, s>>>(conf, C, out);
}

static unsigned copy_blocks(int64_t n_params)
{
    const int64_t b = (n_params + 256 * 8 - 1) / (256 * 8);      // about 8 values per thread
    return (unsigned)(b < 1 ? 1 : (b > 592 ? 592 : b));
}

void launch_train_commit(const TrainCtl& t, float* theta, cudaStream_t s)
{
    train_commit_kernel<<<dim3(copy_blocks(t.n_params - t.param_begin), (unsigned)t.S), 256, 0, s>>>(t.best_theta, theta, t.n_params, t.param_begin);
}

// ---- pack / unpack ---------------------------------------------------------------------------------
template <bool TO_PACKED>
__global__ void pack_kernel(const float* __restrict__ src, float* __restrict__ dst, PackLayout L, int64_t begin, int64_t count)
{
    const int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;   // index in the packed buffer
    if (q >= count) return;
    const int64_t i = begin + q;                                         // the parameter's index in packed order
    const int64_t base = (int64_t)blockIdx.y * L.n_params;
    int64_t j = i;                                                       // its index in internal order
    for (int k = 0; k < L.n_layers; ++k) {
        const int64_t nw = (int64_t)L.cout[k] * L.cin[k] * L.taps[k];
        if (i >= L.w_off[k] && i < L.w_off[k] + nw) {
            const int64_t e = i - L.w_off[k];
            const int tap = (int)(e % L.taps[k]);
            const int64_t r = e / L.taps[k];
            const int ci = (int)(r % L.cin[k]), co = (int)(r / L.cin[k]);
            j = L.w_off[k] + ((int64_t)tap * L.cout[k] + co) * L.cin[k] + ci;
        }
    }
    if (TO_PACKED) dst[(int64_t)blockIdx.y * count + q] = src[base + j];
    else dst[base + j] = src[(int64_t)blockIdx.y * count + q];
}

void launch_pack(const float* internal, float* packed, const PackLayout& L, int64_t begin, int64_t count, int n_bufs, cudaStream_t s)
{
    if (count <= 0) return;
    pack_kernel<true><<<dim3((unsigned)((count + 255) / 256), (unsigned)n_bufs), 256, 0, s>>>(internal, packed, L, begin, count);
}

void launch_unpack(const float* packed, float* internal, const PackLayout& L, int64_t begin, int64_t count, int n_bufs, cudaStream_t s)
{
    if (count <= 0) return;
    pack_kernel<false><<<dim3((unsigned)((count + 255) / 256), (unsigned)n_bufs), 256, 0, s>>>(packed, internal, L, begin, count);
}

}  // namespace st
