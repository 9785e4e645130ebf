// C-ABI layer of the key-frame partial-distillation library: context, host-side validation and the
// order in which the kernels of one step are enqueued (Algorithm 1's loop body; Algorithm 3's
// label and UpdatedPart).  See include/shadowtutor.h for the contract of every entry point.
#include "../../include/shadowtutor.h"
#include "st_internal.h"

#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <map>
#include <tuple>
#include <new>
#include <string>
#include <vector>

using namespace st;

namespace {
thread_local std::string g_init_error;

// A replayable graph: n_steps plain iterations (train = false), or Train with MAX_UPDATES = n_steps and the
// threshold whose bit pattern is `thr` (train = true).
struct GraphKey {
    int n_steps; bool conf; bool train; uint64_t thr;
    bool operator<(const GraphKey& o) const { return std::tie(n_steps, conf, train, thr) < std::tie(o.n_steps, o.conf, o.train, o.thr); }
};
}  // namespace

struct st_ctx {
    st_head_desc d;
    cudaStream_t stream = nullptr;
    int device = 0;
    int S = 0, C = 0, Cin = 0, Ch = 0, h = 0, w = 0, H = 0, W = 0;
    int64_t p = 0, P = 0, n_params = 0;
    bool bf16_mode = false;
    PackLayout layout;

    float *theta = nullptr, *vel = nullptr, *grad = nullptr;
    float* vel2 = nullptr;                  // Adam's second moment
    long long* step_base = nullptr;         // [S] optimisation steps taken so far (Adam's bias correction)
    bool adam = false;
    double b1 = 0.9, b2 = 0.999, eps = 1e-8;
    float* x_f32 = nullptr;
    bf16* x_bf16 = nullptr;
    uint8_t* labels = nullptr;
    uint8_t* labels_tagged = nullptr;       // [S][P] labels with bit 7 = near / within an object (loss weighting on)
    int heavy_w = 1, heavy_radius = 0, background = 0;
    float *z = nullptr, *dz = nullptr;
    bf16* dz_bf16 = nullptr;
    int64_t dz_pitch = 0;
    float *hid_f32 = nullptr, *dhid_f32 = nullptr;
    // student blocks in front of the classifier (bf16 tensor-core path): the head with one hidden layer is one block
    // without a skip input
    int n_blocks = 0, first_trained = 0;    // blocks before first_trained are frozen (Section 4.2)
    struct Block {
        int c_prev = 0, c_skip = 0, c_out = 0;
        bf16 *skip = nullptr, *out = nullptr, *dout = nullptr, *w = nullptr, *w_t = nullptr;
        uint32_t* relu_bits = nullptr;
        float *w_partials = nullptr, *b_partials = nullptr;
        int n_bpart = 0;
        std::vector<char> has_skip;
    } blk[kMaxBlocks];
    bool prefix_current = false;            // the frozen blocks' outputs belong to the current features and skip inputs
    int64_t trained_begin = 0, n_trained = 0;   // where the trained layers start in one stream's parameters; how many values
    bf16* w2_shadow = nullptr;
    float* w2_partials = nullptr;
    int n_split1 = 0, n_split2 = 0;
    float *loss_part = nullptr, *db_part = nullptr;
    int n_k3_blocks = 0;
    CUtensorMap k3_map;        // tile map of z for the fused upsample + cross-entropy kernel
    int k3_has_map = 0;
    CUtensorMap fx_map, fw_map; // tile maps of the features and of the bf16 classifier weights: the loss kernel multiplies its own logits
    int fused_fwd = 0;          //   (one-layer head with bf16 GEMMs; ST_FUSED_FORWARD=0 switches it off)
    int test_stall_fused = 0;   // test of the give-up path inside that kernel (environment ST_TEST_STALL_FUSED=1 at context creation)
    float* loss_buf = nullptr;              // [S][kMaxSteps]
    unsigned long long* conf_buf = nullptr; // [S][kMaxSteps][C][C], allocated on first use
    // Train (Algorithm 1), allocated on first use
    float* best_theta = nullptr;            // [S][n_params] best_student
    int* ctl_done = nullptr;                // [S][kCtlPitch]
    double* ctl_best = nullptr;             // [S][kCtlPitch]
    double* ctl_metric = nullptr;           // [S][kCtlPitch]
    int* ctl_n_updates = nullptr;           // [S]
    int* ctl_best_iter = nullptr;           // [S]
    int* ctl_better = nullptr;              // [S][kCtlPitch]
    unsigned int* bad = nullptr;            // [3]: labels >= C met by a step / by st_agreement; [2] = first device wait that gave up
    uint8_t* mask_tmp = nullptr;            // [P]
    uint8_t* mask_tmp2 = nullptr;           // [P]
    unsigned long long* conf_tmp = nullptr; // [C][C]
    double* miou_tmp = nullptr;             // status block on the device: [0] mean IoU, then the four words of `bad`
    double* status_host = nullptr;          // pinned copy of the status block (32 bytes)
    float* read_tmp = nullptr; size_t read_tmp_bytes = 0;
    void* staging = nullptr; size_t staging_bytes = 0;
    std::vector<char> has_feat, has_labels;
    // inputs of the next key frame, copied from host memory on a stream of the library's own while the current key
    // frame is trained (st_prefetch_key_frame); all created on first use
    cudaStream_t copy_stream = nullptr;
    struct Prefetch { float* feat = nullptr; float* logits = nullptr; cudaEvent_t copied = nullptr, consumed = nullptr; bool pending = false, used_once = false; };
    std::vector<Prefetch> prefetch;
    bool z_current = false;                 // z holds the forward of the current parameters and features of every stream
    bool z_unkept = false;                  // the last call multiplied its logits inside the loss kernel and kept none of them
    TcPlan* plan = nullptr;
    struct StepGraph { cudaGraphExec_t exec; int64_t n_launches; };
    std::map<GraphKey, StepGraph> graphs;
    bool use_graphs = true;
    bool chain_early = false;               // kernels of a step may start while their predecessor drains (one-layer heads)
    std::string err;
    int64_t launches = 0;
    std::vector<void*> allocs;
};

namespace {

st_status fail(st_ctx* ctx, st_status code, const char* fmt, ...)
{
    char buf[512];
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(buf, sizeof buf, fmt, ap);
    va_end(ap);
    if (ctx) ctx->err = buf; else g_init_error = buf;
    return code;
}

#define ST_CUDA(ctx, call)                                                                        \
    do {                                                                                          \
        cudaError_t e_ = (call);                                                                  \
        if (e_ != cudaSuccess)                                                                    \
            return fail(ctx, e_ == cudaErrorMemoryAllocation ? ST_ERR_OOM : ST_ERR_CUDA,          \
                        "%s failed: %s", #call, cudaGetErrorString(e_));                          \
    } while (0)

template <typename T>
cudaError_t dev_alloc(st_ctx* ctx, T** ptr, size_t count, bool zero = true)
{
    void* q = nullptr;
    size_t bytes = count * sizeof(T);
    if (bytes == 0) bytes = 16;
    cudaError_t e = cudaMalloc(&q, bytes);
    if (e != cudaSuccess) return e;
    ctx->allocs.push_back(q);
    if (zero) {
        e = cudaMemsetAsync(q, 0, bytes, ctx->stream);
        if (e != cudaSuccess) return e;
    }
    *ptr = (T*)q;
    return cudaSuccess;
}

bool is_device_ptr(const void* q)
{
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, q) != cudaSuccess) { cudaGetLastError(); return false; }
    return at.type == cudaMemoryTypeDevice || at.type == cudaMemoryTypeManaged;
}

st_status ensure_staging(st_ctx* ctx, size_t bytes)
{
    if (ctx->staging_bytes >= bytes) return ST_OK;
    // the old buffer may still be read by enqueued work
    ST_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    if (ctx->staging) cudaFree(ctx->staging);
    ctx->staging = nullptr; ctx->staging_bytes = 0;
    ST_CUDA(ctx, cudaMalloc(&ctx->staging, bytes));
    ctx->staging_bytes = bytes;
    return ST_OK;
}

// Bring `bytes` of a host-or-device source into device memory; *dev receives a device pointer
// (the source itself if it already is one).
st_status to_device(st_ctx* ctx, const void* src, size_t bytes, const void** dev)
{
    if (is_device_ptr(src)) { *dev = src; return ST_OK; }
    st_status st = ensure_staging(ctx, bytes);
    if (st != ST_OK) return st;
    ST_CUDA(ctx, cudaMemcpyAsync(ctx->staging, src, bytes, cudaMemcpyHostToDevice, ctx->stream));
    *dev = ctx->staging;
    return ST_OK;
}

st_status check_stream_index(st_ctx* ctx, int32_t s)
{
    if (!ctx) return ST_ERR_INVALID_ARG;
    if (s < 0 || s >= ctx->S) return fail(ctx, ST_ERR_INVALID_ARG, "stream index %d outside [0, %d)", s, ctx->S);
    return ST_OK;
}

st_status check_launch(st_ctx* ctx, const char* what)
{
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ctx, ST_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
    return ST_OK;
}

// Arguments of the update kernels.  `all_layers`: every layer including the frozen ones (refreshing the bf16 copies);
// otherwise the layers behind the freeze boundary only.
UpdateArgs make_update_args(st_ctx* c, int slot, const int* skip = nullptr, int64_t skip_stride = 0, bool all_layers = false)
{
    UpdateArgs u;
    memset(&u, 0, sizeof u);
    u.theta = c->theta; u.vel = c->vel; u.grad = c->grad;
    u.n_params = c->n_params; u.S = c->S; u.lr = c->d.lr; u.mu = c->d.momentum;
    const int n_all = c->layout.n_layers, first = all_layers ? 0 : (c->bf16_mode ? c->first_trained : 0);
    u.n_layers = n_all - first;
    u.param_begin = all_layers ? 0 : c->trained_begin;
    for (int L = first; L < n_all; ++L) {
        LayerUpdate& ly = u.layer[L - first];
        ly.w_off = c->layout.w_off[L]; ly.b_off = c->layout.b_off[L];
        ly.cout = c->layout.cout[L]; ly.cin = c->layout.cin[L]; ly.taps = c->layout.taps[L];
        const bool last = (L == n_all - 1);
        if (last) { ly.b_partials = c->db_part; ly.n_bpart = c->n_k3_blocks; }
        if (c->bf16_mode) {
            if (last) {
                ly.w_partials = c->w2_partials; ly.n_split = c->n_split2;
                ly.w_split_stride = (int64_t)kClassPad * ly.cin;
                ly.w_stream_stride = ly.w_split_stride * c->n_split2;
                ly.shadow = c->w2_shadow; ly.shadow_stream_stride = (int64_t)kClassPad * ly.cin;
            } else {
                const st_ctx::Block& k = c->blk[L];
                ly.w_partials = k.w_partials; ly.n_split = c->n_split1;
                ly.w_split_stride = (int64_t)9 * ly.cout * ly.cin;
                ly.w_stream_stride = ly.w_split_stride * c->n_split1;
                ly.shadow = k.w; ly.shadow_stream_stride = (int64_t)9 * ly.cout * ly.cin;
                ly.shadow_t = k.w_t; ly.shadow_t_stream_stride = (int64_t)9 * k.c_prev * ly.cout; ly.c_take = k.c_prev;
                ly.b_partials = k.b_partials; ly.n_bpart = k.n_bpart;
            }
        }
    }
    u.loss_part = c->loss_part; u.n_loss_part = c->n_k3_blocks;
    u.loss_buf = c->loss_buf; u.loss_slot = slot;
    u.inv_P = 1.0 / (double)c->P;
    u.skip = skip; u.skip_stride = skip_stride;
    u.adam = c->adam ? 1 : 0; u.vel2 = c->vel2; u.step_base = c->step_base;
    u.b1 = c->b1; u.b2 = c->b2; u.eps = c->eps; u.ln_b1 = log(c->b1); u.ln_b2 = log(c->b2);
    u.chain_early = c->chain_early ? 1 : 0;
    return u;
}

// The outputs of the frozen blocks do not change while the blocks behind them are trained (Section 4.2): they are
// computed once per key frame, outside the replayed step.
st_status ensure_prefix(st_ctx* c)
{
    if (!c->bf16_mode || c->prefix_current) return ST_OK;
    const int n = c->first_trained < c->n_blocks ? c->first_trained : c->n_blocks;
    if (n > 0) {
        c->launches += tc_forward_blocks(c->plan, 0, n, c->stream);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return ST_ERR_CUDA;
    }
    c->prefix_current = true;
    return ST_OK;
}

// Forward of the trainable part for all streams: z (and the hidden activation).
// `skip` (tensor-core kernels only): per-stream flags, see tc_forward.
st_status enqueue_forward(st_ctx* c, StageTimer* t = nullptr, const int* skip = nullptr, int64_t skip_stride = 0,
                          bool after_update = false, bool loss_follows = false)
{
    cudaStream_t s = c->stream;
    if (c->fused_fwd && loss_follows) return ST_OK;      // the loss kernel multiplies the logits itself (and writes them)
    if (c->bf16_mode) {
        c->launches += tc_forward(c->plan, s, t, skip, skip_stride, after_update, c->first_trained < c->n_blocks ? c->first_trained : c->n_blocks);
    } else if (c->Ch == 0) {
        ST_REPEAT(t) launch_conv_fwd_f32(c->x_f32, c->Cin, c->h, c->w, c->theta + c->layout.w_off[0], c->theta + c->layout.b_off[0],
                            c->C, 1, false, c->z, c->S, (int64_t)c->Cin * c->p, c->n_params, c->n_params,
                            (int64_t)c->C * c->p, s);
        if (t) t->mark("conv1x1_fwd_f32", s, st_repeats(t));
        c->launches += st_repeats(t);
    } else {
        ST_REPEAT(t) launch_conv_fwd_f32(c->x_f32, c->Cin, c->h, c->w, c->theta + c->layout.w_off[0], c->theta + c->layout.b_off[0],
                            c->Ch, 3, true, c->hid_f32, c->S, (int64_t)c->Cin * c->p, c->n_params, c->n_params,
                            (int64_t)c->Ch * c->p, s);
        if (t) t->mark("conv3x3_fwd_f32", s, st_repeats(t));
        ST_REPEAT(t) launch_conv_fwd_f32(c->hid_f32, c->Ch, c->h, c->w, c->theta + c->layout.w_off[1], c->theta + c->layout.b_off[1],
                            c->C, 1, false, c->z, c->S, (int64_t)c->Ch * c->p, c->n_params, c->n_params,
                            (int64_t)c->C * c->p, s);
        if (t) t->mark("conv1x1_fwd_f32", s, st_repeats(t));
        c->launches += 2 * st_repeats(t);
    }
    return check_launch(c, "head forward");
}

// Arguments of the fused upsample + cross-entropy kernel.  With bf16 GEMMs the weight gradient and the dgrad read the
// bf16 copy of the logit gradient only, so the fp32 copy is not written during a step (st_read_tensor produces it on
// demand by running the kernel once more on the same logits and labels).
// With the loss weighting on, the per-key-frame pass that marks the pixels near / within non-background objects.
st_status tag_labels(st_ctx* c, int32_t stream)
{
    if (c->heavy_w <= 1) return ST_OK;
    launch_object_weight_tags(c->labels + (int64_t)stream * c->P, c->H, c->W, c->background, c->heavy_radius, c->mask_tmp,
                              c->labels_tagged + (int64_t)stream * c->P, c->stream);
    c->launches += 2;
    return check_launch(c, "object weights");
}

UpsampleCeArgs k3_args(st_ctx* c, bool fp32_grad, bool bf16_grad, unsigned long long* conf, const int* skip = nullptr,
                       int64_t skip_stride = 0)
{
    UpsampleCeArgs k3;
    k3.z = c->z; k3.labels = c->heavy_w > 1 ? c->labels_tagged : c->labels;
    k3.heavy_w = c->heavy_w;
    k3.dz = fp32_grad ? c->dz : nullptr;
    k3.dz_bf16 = bf16_grad ? c->dz_bf16 : nullptr;
    k3.dz_bf16_pitch = c->dz_pitch;
    k3.loss_part = c->loss_part; k3.db_part = c->db_part;
    k3.conf = conf;
    k3.conf_stream_stride = (int64_t)kMaxSteps * c->C * c->C;
    k3.bad = c->bad; k3.err = c->bad + 2;
    k3.S = c->S; k3.C = c->C; k3.h = c->h; k3.w = c->w;
    k3.has_map = c->k3_has_map;
    k3.skip = skip; k3.skip_stride = skip_stride;
    k3.chain_early = c->chain_early ? 1 : 0;
    k3.fused = 0; k3.x_early = 0; k3.kblocks = 0; k3.theta = nullptr; k3.n_params = 0; k3.b_off = 0; k3.z_out = nullptr; k3.test_stall = 0;
    return k3;
}

// ComputeLoss and the first half of PartialBackward: loss partials, logit gradient, optionally the confusion matrix
// of this prediction.
st_status enqueue_loss(st_ctx* c, unsigned long long* conf, StageTimer* t = nullptr, const int* skip = nullptr, int64_t skip_stride = 0,
                       bool after_update = false, bool keep_logits = true)
{
    cudaStream_t s = c->stream;
    UpsampleCeArgs k3 = k3_args(c, !c->bf16_mode, c->bf16_mode, conf, skip, skip_stride);
    if (c->fused_fwd) {
        // Forward as well: the features are frozen, so after a parameter update (which writes weights only) their tiles
        // may be fetched while that update is still running
        k3.fused = 1; k3.x_early = after_update && !t ? 1 : 0; k3.kblocks = c->Cin / 64;
        k3.theta = c->theta; k3.n_params = c->n_params; k3.b_off = c->layout.b_off[c->layout.n_layers - 1];
        k3.z_out = keep_logits ? c->z : nullptr;         // logits that the next iteration overwrites unread stay on the chip
        k3.test_stall = c->test_stall_fused;
    }
    ST_REPEAT(t) launch_upsample_ce(k3, &c->k3_map, s, &c->fx_map, &c->fw_map);
    if (t) t->mark(k3.fused ? "fwd1x1_upsample_ce" : "upsample_ce", s, st_repeats(t));
    c->launches += st_repeats(t);
    return check_launch(c, "upsample + cross-entropy");
}

// The rest of PartialBackward: gradients of the head's tensors (as split-K partial sums with bf16 GEMMs).
st_status enqueue_backward(st_ctx* c, StageTimer* t = nullptr, const int* skip = nullptr, int64_t skip_stride = 0, const TrainCtl* ctl = nullptr)
{
    cudaStream_t s = c->stream;
    if (c->bf16_mode) {
        c->launches += tc_backward(c->plan, s, t, skip, skip_stride, ctl);
    } else if (c->Ch == 0) {
        ST_REPEAT(t) launch_conv_wgrad_f32(c->x_f32, c->dz, c->Cin, c->C, c->h, c->w, 1, c->grad + c->layout.w_off[0], c->S,
                              (int64_t)c->Cin * c->p, (int64_t)c->C * c->p, c->n_params, s);
        if (t) t->mark("conv1x1_wgrad_f32", s, st_repeats(t));
        c->launches += st_repeats(t);
    } else {
        const int64_t hs = (int64_t)c->Ch * c->p;
        launch_conv_wgrad_f32(c->hid_f32, c->dz, c->Ch, c->C, c->h, c->w, 1, c->grad + c->layout.w_off[1], c->S,
                              hs, (int64_t)c->C * c->p, c->n_params, s);
        launch_conv1x1_dgrad_relu_f32(c->theta + c->layout.w_off[1], c->dz, c->hid_f32, c->C, c->Ch, c->p,
                                      c->dhid_f32, c->S, c->n_params, (int64_t)c->C * c->p, hs, s);
        launch_conv_wgrad_f32(c->x_f32, c->dhid_f32, c->Cin, c->Ch, c->h, c->w, 3, c->grad + c->layout.w_off[0], c->S,
                              (int64_t)c->Cin * c->p, hs, c->n_params, s);
        launch_bias_grad_f32(c->dhid_f32, c->Ch, c->p, c->grad + c->layout.b_off[0], c->S, hs, c->n_params, s);
        if (t) t->mark("backward_f32", s, 4);
        c->launches += 4;
    }
    return check_launch(c, "head backward");
}

// OptimStep, and the loss of this prediction into loss_buf[slot].  `skip`: per-stream flags (see UpdateArgs).
st_status enqueue_update(st_ctx* c, int slot, const int* skip, int64_t skip_stride, StageTimer* t = nullptr, const TrainCtl* ctl = nullptr,
                         int ctl_mode = 1)
{
    UpdateArgs u = make_update_args(c, slot, skip, skip_stride);
    // Train: the update assesses the prediction itself (1), or reads what the backward before it has found (2)
    if (ctl) { u.has_ctl = ctl_mode; u.ctl = *ctl; u.skip = nullptr; }
    c->launches += launch_sgd_update(u, c->stream);
    if (t) t->mark("sgd_update", c->stream, 1);
    return check_launch(c, "sgd update");
}

st_status enqueue_step(st_ctx* c, int slot, bool want_conf, StageTimer* t = nullptr, bool last = true)
{
    // iterations after the first follow the previous iteration's update directly
    st_status st = enqueue_forward(c, t, nullptr, 0, slot > 0 && !t, true);
    if (st == ST_OK) st = enqueue_loss(c, want_conf ? c->conf_buf + (int64_t)slot * c->C * c->C : nullptr, t, nullptr, 0, slot > 0, last);
    if (st == ST_OK) st = enqueue_backward(c, t);
    if (st == ST_OK) st = enqueue_update(c, slot, nullptr, 0, t);
    return st;
}

// One 32-byte device-to-host copy and one wait: the mean IoU of the last st_agreement and the error words.
st_status fetch_status(st_ctx* c)
{
    ST_CUDA(c, cudaMemcpyAsync(c->status_host, c->miou_tmp, 32, cudaMemcpyDeviceToHost, c->stream));
    ST_CUDA(c, cudaStreamSynchronize(c->stream));
    return ST_OK;
}

// Turn the error words of the fetched status block into a status code, clearing what is reported.
st_status report_status(st_ctx* c, bool agreement_call)
{
    const unsigned int* host_bad = reinterpret_cast<const unsigned int*>(c->status_host + 1);
    const unsigned int gave_up = host_bad[2], bad_step = host_bad[0], bad_agree = host_bad[1];
    if (!gave_up && !bad_step && !(agreement_call && bad_agree)) return ST_OK;
    cudaMemsetAsync(c->bad, 0, 4 * sizeof(unsigned int), c->stream);
    if (gave_up)
        return fail(c, ST_ERR_CUDA, "a tensor-core kernel gave up waiting (code %u, block %u); results of that step are invalid",
                    gave_up & 0xffu, gave_up >> 8);
    if (agreement_call && bad_agree)
        return fail(c, ST_ERR_INVALID_ARG, "%u pixel(s) with a label or prediction >= n_classes were skipped (st_agreement)", bad_agree);
    return fail(c, ST_ERR_INVALID_ARG, "%u pixel(s) with a label >= n_classes were skipped (an earlier st_distill_step)", bad_step);
}

st_status report_bad_labels(st_ctx* c, int which, const char* what)
{
    (void)what;
    st_status st = fetch_status(c);
    if (st != ST_OK) return st;
    return report_status(c, which == 1);
}

}  // namespace

extern "C" {

size_t st_param_count(int32_t c_in, int32_t c_hidden, int32_t n_classes)
{
    if (c_in <= 0 || n_classes <= 0 || c_hidden < 0) return 0;
    if (c_hidden == 0) return (size_t)n_classes * c_in + n_classes;
    return (size_t)c_hidden * c_in * 9 + c_hidden + (size_t)n_classes * c_hidden + n_classes;
}

st_status st_head_param_counts(const st_head_desc* d, size_t* n_all, size_t* n_trained)
{
    if (!d || d->c_in < 1 || d->n_classes < 1 || d->c_hidden < 0) return ST_ERR_INVALID_ARG;
    size_t all = 0, frozen = 0;
    int prev = d->c_in;
    if (d->n_blocks != 0) {
        if (d->n_blocks < 0 || d->n_blocks > kMaxBlocks || d->c_hidden != 0 || d->first_trained < 0 || d->first_trained > d->n_blocks)
            return ST_ERR_INVALID_ARG;
        for (int i = 0; i < d->n_blocks; ++i) {
            if (d->block_c_out[i] < 1 || d->block_c_skip[i] < 0) return ST_ERR_INVALID_ARG;
            all += (size_t)d->block_c_out[i] * (prev + d->block_c_skip[i]) * 9 + d->block_c_out[i];
            if (i < d->first_trained) frozen = all;
            prev = d->block_c_out[i];
        }
    } else if (d->c_hidden > 0) {
        all += (size_t)d->c_hidden * prev * 9 + d->c_hidden;
        prev = d->c_hidden;
    }
    all += (size_t)d->n_classes * prev + d->n_classes;
    if (n_all) *n_all = all;
    if (n_trained) *n_trained = all - frozen;
    return ST_OK;
}

const char* st_status_name(st_status s)
{
    switch (s) {
        case ST_OK: return "ST_OK";
        case ST_ERR_INVALID_ARG: return "ST_ERR_INVALID_ARG";
        case ST_ERR_BAD_STATE: return "ST_ERR_BAD_STATE";
        case ST_ERR_BUFFER_TOO_SMALL: return "ST_ERR_BUFFER_TOO_SMALL";
        case ST_ERR_UNSUPPORTED: return "ST_ERR_UNSUPPORTED";
        case ST_ERR_OOM: return "ST_ERR_OOM";
        case ST_ERR_CUDA: return "ST_ERR_CUDA";
    }
    return "ST_ERR_?";
}

const char* st_last_error(const st_ctx* ctx) { return ctx ? ctx->err.c_str() : g_init_error.c_str(); }

int64_t st_launch_count(const st_ctx* ctx) { return ctx ? ctx->launches : 0; }

void st_destroy(st_ctx* ctx)
{
    if (!ctx) return;
    cudaStreamSynchronize(ctx->stream);
    for (auto& g : ctx->graphs) cudaGraphExecDestroy(g.second.exec);
    if (ctx->plan) tc_plan_destroy(ctx->plan);
    for (void* q : ctx->allocs) cudaFree(q);
    if (ctx->staging) cudaFree(ctx->staging);
    if (ctx->copy_stream) cudaStreamSynchronize(ctx->copy_stream);
    for (auto& pf : ctx->prefetch) {
        if (pf.feat) cudaFree(pf.feat);
        if (pf.logits) cudaFree(pf.logits);
        if (pf.copied) cudaEventDestroy(pf.copied);
        if (pf.consumed) cudaEventDestroy(pf.consumed);
    }
    if (ctx->copy_stream) cudaStreamDestroy(ctx->copy_stream);
    if (ctx->read_tmp) cudaFree(ctx->read_tmp);
    if (ctx->status_host) cudaFreeHost(ctx->status_host);
    delete ctx;
}

st_status st_init_head(const st_head_desc* desc, const float* init_params, st_ctx** out)
{
    if (!desc || !init_params || !out) return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: NULL argument");
    *out = nullptr;
    const st_head_desc& d = *desc;
    if (d.n_streams < 1 || d.c_in < 1 || d.c_hidden < 0 || d.feat_h < 1 || d.feat_w < 1)
        return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: n_streams, c_in, feat_h, feat_w must be >= 1 and c_hidden >= 0");
    if (d.n_classes < 2 || d.n_classes > 255)
        return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: n_classes %d outside 2..255", d.n_classes);
    if (!(d.lr >= 0.f) || !(d.momentum >= 0.f) || !(d.momentum < 1.f))
        return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: lr must be >= 0 and momentum in [0, 1)");
    if (d.optimizer != 0 && d.optimizer != 1)
        return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: optimizer must be 0 (gradient descent) or 1 (Adam)");
    const double ab1 = d.adam_beta1 == 0.0 ? 0.9 : d.adam_beta1, ab2 = d.adam_beta2 == 0.0 ? 0.999 : d.adam_beta2;
    const double aeps = d.adam_eps == 0.0 ? 1e-8 : d.adam_eps;
    if (d.optimizer == 1 && (!(ab1 > 0.0 && ab1 < 1.0) || !(ab2 > 0.0 && ab2 < 1.0) || !(aeps > 0.0)))
        return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: Adam needs beta1, beta2 in (0, 1) and eps > 0");
    if (d.object_weight > 1) {
        if (d.object_radius < 0 || d.background_class < 0 || d.background_class >= d.n_classes)
            return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: loss weighting needs object_radius >= 0 and a background class below n_classes");
        if (d.object_weight > 5 || d.object_radius > 64 || !upsample_ce_rows_supported(d.n_classes))
            return fail(nullptr, ST_ERR_UNSUPPORTED, "st_init_head: loss weighting covers weights 2..5, radii up to 64 and at most 32 classes");
    }
    if (d.gemm_precision != 0 && d.gemm_precision != 1)
        return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: gemm_precision must be 0 or 1");
    if (d.up != kUp) return fail(nullptr, ST_ERR_UNSUPPORTED, "st_init_head: up must be 4");
    if ((int64_t)d.feat_h * d.feat_w * 16 > (int64_t)1 << 30)
        return fail(nullptr, ST_ERR_UNSUPPORTED, "st_init_head: frame larger than 2^30 pixels");
    if (d.gemm_precision == 1) {
        if (d.c_in % 64 != 0 || d.c_hidden % 64 != 0 || d.c_hidden > 256 || d.c_in > 1024 || d.n_classes > kClassPad)
            return fail(nullptr, ST_ERR_UNSUPPORTED,
                        "st_init_head: the bf16 tensor-core path needs c_in and c_hidden multiples of 64, "
                        "c_hidden <= 256, c_in <= 1024 and n_classes <= %d", kClassPad);
    }
    // the back part as a stack of student blocks (n_blocks > 0), or the head given by c_hidden (n_blocks == 0)
    int n_blocks = 0, first_trained = 0, blk_out[kMaxBlocks] = {0}, blk_skip[kMaxBlocks] = {0};
    if (d.n_blocks != 0) {
        if (d.n_blocks < 0 || d.n_blocks > kMaxBlocks || d.c_hidden != 0 || d.first_trained < 0 || d.first_trained > d.n_blocks)
            return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: n_blocks must be 0..%d with c_hidden 0, and first_trained 0..n_blocks", kMaxBlocks);
        if (d.gemm_precision != 1)
            return fail(nullptr, ST_ERR_UNSUPPORTED, "st_init_head: a stack of blocks needs gemm_precision 1 (bf16 tensor cores)");
        int prev = d.c_in;
        for (int i = 0; i < d.n_blocks; ++i) {
            const int co = d.block_c_out[i], cs = d.block_c_skip[i];
            if (co < 1 || cs < 0) return fail(nullptr, ST_ERR_INVALID_ARG, "st_init_head: block %d needs c_out >= 1 and c_skip >= 0", i);
            const int tot = prev + cs;
            if (co % 64 != 0 || cs % 64 != 0 || prev % 64 != 0 || co > 256 || prev > 256 || ((tot + 127) / 128) * co > 512)
                return fail(nullptr, ST_ERR_UNSUPPORTED,
                            "st_init_head: block %d: channel counts must be multiples of 64, at most 256 for the block's output and for "
                            "the previous output it reads, and ceil((c_prev + c_skip) / 128) * c_out at most 512", i);
            blk_out[i] = co; blk_skip[i] = cs; prev = co;
        }
        n_blocks = d.n_blocks; first_trained = d.first_trained;
    } else if (d.c_hidden > 0 && d.gemm_precision == 1) {
        if (((d.c_in + 127) / 128) * d.c_hidden > 512)
            return fail(nullptr, ST_ERR_UNSUPPORTED, "st_init_head: ceil(c_in / 128) * c_hidden must be at most 512 on the bf16 path");
        n_blocks = 1; blk_out[0] = d.c_hidden;
    }

    st_ctx* c = new (std::nothrow) st_ctx();
    if (!c) return fail(nullptr, ST_ERR_OOM, "st_init_head: host allocation failed");
    c->d = d;
    c->stream = (cudaStream_t)d.cuda_stream;
    cudaGetDevice(&c->device);
    c->S = d.n_streams; c->C = d.n_classes; c->Cin = d.c_in;
    c->Ch = n_blocks ? blk_out[n_blocks - 1] : d.c_hidden;      // channels in front of the classifier (0: the features themselves)
    c->h = d.feat_h; c->w = d.feat_w; c->H = d.feat_h * kUp; c->W = d.feat_w * kUp;
    c->p = (int64_t)c->h * c->w; c->P = (int64_t)c->H * c->W;
    c->bf16_mode = d.gemm_precision == 1;
    c->n_blocks = n_blocks; c->first_trained = first_trained;
    for (int i = 0, prev = d.c_in; i < n_blocks; ++i) {
        c->blk[i].c_prev = prev; c->blk[i].c_skip = blk_skip[i]; c->blk[i].c_out = blk_out[i];
        c->blk[i].has_skip.assign(d.n_streams, blk_skip[i] ? 0 : 1);
        prev = blk_out[i];
    }
    c->adam = d.optimizer == 1; c->b1 = ab1; c->b2 = ab2; c->eps = aeps;
    c->heavy_w = d.object_weight > 1 ? d.object_weight : 1; c->heavy_radius = d.object_radius; c->background = d.background_class;
    c->has_feat.assign(c->S, 0); c->has_labels.assign(c->S, 0);
    // The legacy default stream cannot be captured: steps are then enqueued kernel by kernel.
    c->use_graphs = c->stream != nullptr && c->stream != cudaStreamLegacy && c->stream != cudaStreamPerThread;
    if (const char* e = getenv("ST_NO_GRAPH")) if (e[0] == '1') c->use_graphs = false;
    // Programmatic dependent launch along the step's chain: with the one-layer head every kernel has something to do
    // before its predecessor's results are needed (label fetch, feature tiles) and the step is 2 us shorter; the
    // two-layer head's kernels fill the SMs to the end and gain nothing (measured: 1 us slower).  ST_PDL=0 / 1 force it.
    c->chain_early = pdl_enabled() && c->Ch == 0;
    if (const char* e = getenv("ST_PDL")) if (e[0] == '1') c->chain_early = true;

    // layers in forward order: the 3x3 layers (blocks, or the fp32 path's hidden layer), then the classifier
    PackLayout& L = c->layout;
    memset(&L, 0, sizeof L);
    {
        int64_t off = 0;
        int n = 0, prev = c->Cin;
        const int n3 = c->bf16_mode ? n_blocks : (d.c_hidden ? 1 : 0);
        for (int i = 0; i < n3; ++i, ++n) {
            const int co = c->bf16_mode ? blk_out[i] : d.c_hidden, ci = prev + (c->bf16_mode ? blk_skip[i] : 0);
            L.cout[n] = co; L.cin[n] = ci; L.taps[n] = 9; L.w_off[n] = off; off += (int64_t)co * ci * 9;
            L.b_off[n] = off; off += co;
            if (i < first_trained) c->trained_begin = off;
            prev = co;
        }
        L.cout[n] = c->C; L.cin[n] = prev; L.taps[n] = 1; L.w_off[n] = off; off += (int64_t)c->C * prev;
        L.b_off[n] = off; off += c->C;
        L.n_layers = n + 1;
        L.n_params = c->n_params = off;
        c->n_trained = off - c->trained_begin;
    }

    const int S = c->S;
    const int c_last = c->Ch ? c->Ch : c->Cin;
    c->n_k3_blocks = upsample_ce_blocks(c->h, c->w, c->C);
    cudaError_t e = cudaSuccess;
#define ALLOC(ptr, count) if (e == cudaSuccess) e = dev_alloc(c, &c->ptr, (size_t)(count))
    ALLOC(theta, S * c->n_params); ALLOC(vel, S * c->n_params); ALLOC(grad, S * c->n_params);
    ALLOC(step_base, S);
    if (c->adam) ALLOC(vel2, S * c->n_params);
    ALLOC(labels, S * c->P);
    if (c->heavy_w > 1) ALLOC(labels_tagged, S * c->P);
    ALLOC(z, S * c->C * c->p); ALLOC(dz, S * c->C * c->p);
    ALLOC(loss_part, S * c->n_k3_blocks); ALLOC(db_part, (size_t)S * c->n_k3_blocks * c->C);
    ALLOC(loss_buf, S * kMaxSteps);
    ALLOC(miou_tmp, 4); ALLOC(mask_tmp, c->P); ALLOC(mask_tmp2, c->P); ALLOC(conf_tmp, 2 * c->C * c->C + 1);   // counters (zero between calls), the block counter, the delivered matrix
    if (e == cudaSuccess) { c->bad = reinterpret_cast<unsigned int*>(c->miou_tmp + 1); e = cudaHostAlloc((void**)&c->status_host, 32, cudaHostAllocDefault); }
    if (c->bf16_mode) {
        ALLOC(x_bf16, S * c->p * c->Cin);
        c->dz_pitch = tc_dz_pitch(c->h, c->w);
        ALLOC(dz_bf16, (size_t)S * kClassPad * c->dz_pitch);
        ALLOC(w2_shadow, (size_t)S * kClassPad * c_last);
        c->n_split2 = tc_wgrad_splits(2, c_last, c->h, c->w);
        ALLOC(w2_partials, (size_t)S * c->n_split2 * kClassPad * c_last);
        c->n_split1 = n_blocks ? tc_wgrad_splits(1, 0, c->h, c->w) : 0;
        for (int i = 0; i < n_blocks; ++i) {
            st_ctx::Block& k = c->blk[i];
            const size_t tot = (size_t)k.c_prev + k.c_skip;
            const bool trained = i >= first_trained;
            if (k.c_skip) ALLOC(blk[i].skip, S * c->p * k.c_skip);
            ALLOC(blk[i].out, S * c->p * k.c_out);
            ALLOC(blk[i].relu_bits, S * c->p * (k.c_out / 32));
            ALLOC(blk[i].w, (size_t)S * 9 * k.c_out * tot);
            if (trained) {
                ALLOC(blk[i].dout, S * c->p * k.c_out);
                ALLOC(blk[i].w_partials, (size_t)S * c->n_split1 * 9 * k.c_out * tot);
                // the block in front of the classifier gets its gradient from the 128-pixel tiles of the 1x1 layer's
                // kernel, the others from the 4 x 32 tiles of the 3x3 tile walk
                k.n_bpart = i == n_blocks - 1 ? tc_b1_partials(c->h, c->w) : tc_tile3_count(c->h, c->w);
                ALLOC(blk[i].b_partials, (size_t)S * k.n_bpart * k.c_out);
                if (i > first_trained) ALLOC(blk[i].w_t, (size_t)S * 9 * k.c_prev * k.c_out);
            }
        }
    } else {
        ALLOC(x_f32, S * c->Cin * c->p);
        if (c->Ch) { ALLOC(hid_f32, S * c->Ch * c->p); ALLOC(dhid_f32, S * c->Ch * c->p); }
    }
#undef ALLOC
    if (e == cudaSuccess) e = prepare_upsample_ce(c->C);
    if (e == cudaSuccess) c->k3_has_map = make_logit_tile_map(&c->k3_map, c->z, S, c->C, c->h, c->w) ? 1 : 0;
    if (e == cudaSuccess) e = prepare_student_mask(c->C);
    if (e != cudaSuccess) {
        st_status code = fail(nullptr, e == cudaErrorMemoryAllocation ? ST_ERR_OOM : ST_ERR_CUDA,
                              "st_init_head: device allocation failed: %s", cudaGetErrorString(e));
        cudaGetLastError();
        st_destroy(c);
        return code;
    }

    // parameters: packed order -> internal order (the momentum buffer serves as scratch, then is zeroed)
    const size_t pbytes = (size_t)S * c->n_params * sizeof(float);
    e = cudaMemcpyAsync(c->vel, init_params, pbytes, cudaMemcpyDefault, c->stream);
    if (e == cudaSuccess) { launch_unpack(c->vel, c->theta, c->layout, 0, c->n_params, S, c->stream); e = cudaGetLastError(); }
    if (e == cudaSuccess) e = cudaMemsetAsync(c->vel, 0, pbytes, c->stream);
    if (e == cudaSuccess && c->bf16_mode) {
        TcBuffers b;
        memset(&b, 0, sizeof b);
        b.S = S; b.c_in = c->Cin; b.C = c->C; b.h = c->h; b.w = c->w;
        b.x = c->x_bf16; b.w2 = c->w2_shadow; b.theta = c->theta; b.n_params = c->n_params;
        b.b2_off = L.b_off[L.n_layers - 1]; b.w2_off = L.w_off[L.n_layers - 1];
        b.err = c->bad + 2;
        b.chain_early = c->chain_early ? 1 : 0;
        b.z = c->z; b.dz = c->dz; b.dz_bf16 = c->dz_bf16; b.w2_partials = c->w2_partials;
        b.n_blocks = n_blocks;
        for (int i = 0; i < n_blocks; ++i) {
            const st_ctx::Block& k = c->blk[i];
            TcBlock& q = b.blk[i];
            q.c_prev = k.c_prev; q.c_skip = k.c_skip; q.c_out = k.c_out;
            q.in_prev = i ? c->blk[i - 1].out : c->x_bf16; q.in_skip = k.skip;
            q.w = k.w; q.w_t = k.w_t; q.b_off = L.b_off[i];
            q.out = k.out; q.relu_bits = k.relu_bits; q.dout = k.dout;
            q.w_partials = k.w_partials; q.b_partials = k.b_partials;
            q.trained = i >= first_trained ? 1 : 0; q.pass_back = i > first_trained ? 1 : 0;
        }
        char msg[256] = {0};
        c->plan = tc_plan_create(b, msg, sizeof msg);
        if (!c->plan) {
            st_status code = fail(nullptr, ST_ERR_CUDA, "st_init_head: tensor-core plan: %s", msg);
            st_destroy(c);
            return code;
        }
        launch_refresh_shadow(make_update_args(c, -1, nullptr, 0, true), c->stream);
        e = cudaGetLastError();
        const char* off = getenv("ST_FUSED_FORWARD");
        if (n_blocks == 0 && !(off && off[0] == '0') && fused_forward_supported(c->C, c->h, c->w, c->Cin)) {
            const uint64_t ci = (uint64_t)c->Cin;
            const uint64_t dims[3] = {ci, (uint64_t)kClassPad, (uint64_t)S}, str[2] = {ci * 2, (uint64_t)kClassPad * ci * 2};
            const uint32_t box[3] = {64, (uint32_t)kClassPad, 1};
            c->fused_fwd = make_feature_tile_map(&c->fx_map, c->x_bf16, S, c->Cin, c->h, c->w) &&
                           encode_tensor_map(&c->fw_map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, CU_TENSOR_MAP_SWIZZLE_128B, c->w2_shadow, 3,
                                             dims, str, box, msg, sizeof msg, "1x1 weight") &&
                           prepare_student_eval(c->C) == cudaSuccess;
            if (const char* ts = getenv("ST_TEST_STALL_FUSED")) c->test_stall_fused = ts[0] == '1' ? 1 : 0;
        }
    }
    if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);   // init_params may be released on return
    if (e != cudaSuccess) {
        st_status code = fail(nullptr, ST_ERR_CUDA, "st_init_head: %s", cudaGetErrorString(e));
        st_destroy(c);
        return code;
    }
    c->launches += 2;
    *out = c;
    return ST_OK;
}

st_status st_set_frozen_features(st_ctx* ctx, int32_t stream, const float* feat_chw)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    if (!feat_chw) return fail(ctx, ST_ERR_INVALID_ARG, "st_set_frozen_features: NULL features");
    const size_t bytes = (size_t)ctx->Cin * ctx->p * sizeof(float);
    if (ctx->bf16_mode) {
        const void* src = nullptr;
        st = to_device(ctx, feat_chw, bytes, &src);
        if (st != ST_OK) return st;
        launch_feat_to_bf16_nhwc((const float*)src, ctx->Cin, ctx->p, ctx->x_bf16 + (int64_t)stream * ctx->p * ctx->Cin, ctx->stream);
        ctx->launches += 1;
        st = check_launch(ctx, "feature cache");
        if (st != ST_OK) return st;
    } else {
        ST_CUDA(ctx, cudaMemcpyAsync(ctx->x_f32 + (int64_t)stream * ctx->Cin * ctx->p, feat_chw, bytes, cudaMemcpyDefault, ctx->stream));
    }
    ctx->has_feat[stream] = 1;
    ctx->z_current = false;
    ctx->prefix_current = false;
    return ST_OK;
}

st_status st_set_skip_features(st_ctx* ctx, int32_t stream, int32_t block, const float* feat_chw)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    if (block < 0 || block >= ctx->n_blocks || ctx->blk[block].c_skip == 0)
        return fail(ctx, ST_ERR_INVALID_ARG, "st_set_skip_features: block %d has no skip input", block);
    if (!feat_chw) return fail(ctx, ST_ERR_INVALID_ARG, "st_set_skip_features: NULL features");
    st_ctx::Block& k = ctx->blk[block];
    const void* src = nullptr;
    st = to_device(ctx, feat_chw, (size_t)k.c_skip * ctx->p * sizeof(float), &src);
    if (st != ST_OK) return st;
    launch_feat_to_bf16_nhwc((const float*)src, k.c_skip, ctx->p, k.skip + (int64_t)stream * ctx->p * k.c_skip, ctx->stream);
    ctx->launches += 1;
    st = check_launch(ctx, "skip feature cache");
    if (st != ST_OK) return st;
    k.has_skip[stream] = 1;
    ctx->z_current = false;
    ctx->prefix_current = false;
    return ST_OK;
}

st_status st_teacher_labels(st_ctx* ctx, int32_t stream, const float* logits_chw, uint8_t* labels_out)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    if (!logits_chw) return fail(ctx, ST_ERR_INVALID_ARG, "st_teacher_labels: NULL logits");
    const void* src = nullptr;
    st = to_device(ctx, logits_chw, (size_t)ctx->C * ctx->P * sizeof(float), &src);
    if (st != ST_OK) return st;
    uint8_t* dst = ctx->labels + (int64_t)stream * ctx->P;
    launch_argmax_u8((const float*)src, ctx->C, ctx->P, dst, ctx->stream);
    ctx->launches += 1;
    st = check_launch(ctx, "teacher argmax");
    if (st != ST_OK) return st;
    if (labels_out) ST_CUDA(ctx, cudaMemcpyAsync(labels_out, dst, (size_t)ctx->P, cudaMemcpyDefault, ctx->stream));
    ctx->has_labels[stream] = 1;
    return tag_labels(ctx, stream);
}

st_status st_prefetch_key_frame(st_ctx* ctx, int32_t stream, const float* feat_chw, const float* logits_chw)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    if (!feat_chw || !logits_chw) return fail(ctx, ST_ERR_INVALID_ARG, "st_prefetch_key_frame: NULL input");
    if (ctx->prefetch.empty()) ctx->prefetch.resize(ctx->S);
    st_ctx::Prefetch& pf = ctx->prefetch[stream];
    const size_t fbytes = (size_t)ctx->Cin * ctx->p * sizeof(float), lbytes = (size_t)ctx->C * ctx->P * sizeof(float);
    if (!ctx->copy_stream) ST_CUDA(ctx, cudaStreamCreateWithFlags(&ctx->copy_stream, cudaStreamNonBlocking));
    if (!pf.feat) {
        ST_CUDA(ctx, cudaMalloc((void**)&pf.feat, fbytes));
        ST_CUDA(ctx, cudaMalloc((void**)&pf.logits, lbytes));
        ST_CUDA(ctx, cudaEventCreateWithFlags(&pf.copied, cudaEventDisableTiming));
        ST_CUDA(ctx, cudaEventCreateWithFlags(&pf.consumed, cudaEventDisableTiming));
    }
    // the kernels that read the previous contents of the two buffers must have run before they are overwritten
    if (pf.used_once) ST_CUDA(ctx, cudaStreamWaitEvent(ctx->copy_stream, pf.consumed, 0));
    ST_CUDA(ctx, cudaMemcpyAsync(pf.feat, feat_chw, fbytes, cudaMemcpyDefault, ctx->copy_stream));
    ST_CUDA(ctx, cudaMemcpyAsync(pf.logits, logits_chw, lbytes, cudaMemcpyDefault, ctx->copy_stream));
    ST_CUDA(ctx, cudaEventRecord(pf.copied, ctx->copy_stream));
    pf.pending = true;
    return ST_OK;
}

st_status st_use_prefetched_key_frame(st_ctx* ctx, int32_t stream, uint8_t* labels_out)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    if (ctx->prefetch.empty() || !ctx->prefetch[stream].pending)
        return fail(ctx, ST_ERR_BAD_STATE, "st_use_prefetched_key_frame: stream %d has no prefetched key frame", stream);
    st_ctx::Prefetch& pf = ctx->prefetch[stream];
    ST_CUDA(ctx, cudaStreamWaitEvent(ctx->stream, pf.copied, 0));      // the device waits for the copy, the host does not
    st = st_set_frozen_features(ctx, stream, pf.feat);
    if (st == ST_OK) st = st_teacher_labels(ctx, stream, pf.logits, labels_out);
    if (st != ST_OK) return st;
    ST_CUDA(ctx, cudaEventRecord(pf.consumed, ctx->stream));
    pf.pending = false;
    pf.used_once = true;
    return ST_OK;
}

st_status st_set_labels(st_ctx* ctx, int32_t stream, const uint8_t* labels)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    if (!labels) return fail(ctx, ST_ERR_INVALID_ARG, "st_set_labels: NULL labels");
    ST_CUDA(ctx, cudaMemcpyAsync(ctx->labels + (int64_t)stream * ctx->P, labels, (size_t)ctx->P, cudaMemcpyDefault, ctx->stream));
    ctx->has_labels[stream] = 1;
    return tag_labels(ctx, stream);
}

namespace {
// every stream has its features (and skip inputs) and, if asked for, its labels; the frozen blocks' outputs are current
st_status ready_to_run(st_ctx* ctx, const char* who, bool need_labels)
{
    for (int s = 0; s < ctx->S; ++s) {
        if (!ctx->has_feat[s]) return fail(ctx, ST_ERR_BAD_STATE, "%s: stream %d has no frozen features yet", who, s);
        for (int b = 0; b < ctx->n_blocks; ++b)
            if (!ctx->blk[b].has_skip[s]) return fail(ctx, ST_ERR_BAD_STATE, "%s: stream %d has no skip input for block %d yet", who, s, b);
        if (need_labels && !ctx->has_labels[s]) return fail(ctx, ST_ERR_BAD_STATE, "%s: stream %d has no labels yet", who, s);
    }
    if (ensure_prefix(ctx) != ST_OK) return fail(ctx, ST_ERR_CUDA, "%s: forward of the frozen blocks failed", who);
    return ST_OK;
}
}  // namespace

st_status st_distill_step(st_ctx* ctx, int32_t n_steps, float* loss_out, int64_t* conf_out)
{
    if (!ctx) return ST_ERR_INVALID_ARG;
    if (n_steps < 1 || n_steps > kMaxSteps)
        return fail(ctx, ST_ERR_INVALID_ARG, "st_distill_step: n_steps %d outside 1..%d", n_steps, kMaxSteps);
    {
        const st_status ready = ready_to_run(ctx, "st_distill_step", true);
        if (ready != ST_OK) return ready;
    }
    const bool want_conf = conf_out != nullptr;
    const size_t cc = (size_t)ctx->C * ctx->C;
    ctx->z_current = false;                 // the steps leave z at the forward before the last update
    ctx->z_unkept = false;
    if (want_conf) {
        if (!ctx->conf_buf) {
            cudaError_t e = dev_alloc(ctx, &ctx->conf_buf, (size_t)ctx->S * kMaxSteps * cc);
            if (e != cudaSuccess) return fail(ctx, ST_ERR_OOM, "st_distill_step: %s", cudaGetErrorString(e));
        }
        ST_CUDA(ctx, cudaMemsetAsync(ctx->conf_buf, 0, (size_t)ctx->S * kMaxSteps * cc * sizeof(unsigned long long), ctx->stream));
    }

    st_status st = ST_OK;
    if (ctx->use_graphs) {
        GraphKey key{n_steps, want_conf, false, 0};
        auto it = ctx->graphs.find(key);
        if (it == ctx->graphs.end()) {
            cudaGraph_t graph = nullptr;
            const int64_t before = ctx->launches;
            ST_CUDA(ctx, cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal));
            for (int k = 0; k < n_steps && st == ST_OK; ++k) st = enqueue_step(ctx, k, want_conf, nullptr, k == n_steps - 1);
            if (st == ST_OK && ctx->adam) { launch_step_tick(ctx->step_base, ctx->S, n_steps, nullptr, ctx->stream); ctx->launches += 1; }
            cudaError_t e = cudaStreamEndCapture(ctx->stream, &graph);
            const int64_t n_launches = ctx->launches - before;
            ctx->launches = before;
            if (st != ST_OK) { if (graph) cudaGraphDestroy(graph); return st; }
            if (e != cudaSuccess) return fail(ctx, ST_ERR_CUDA, "st_distill_step: graph capture: %s", cudaGetErrorString(e));
            cudaGraphExec_t exec = nullptr;
            e = cudaGraphInstantiate(&exec, graph, 0);
            cudaGraphDestroy(graph);
            if (e != cudaSuccess) return fail(ctx, ST_ERR_CUDA, "st_distill_step: graph instantiate: %s", cudaGetErrorString(e));
            it = ctx->graphs.emplace(key, st_ctx::StepGraph{exec, n_launches}).first;
        }
        ctx->launches += it->second.n_launches;   // a replay launches the captured kernels again
        ST_CUDA(ctx, cudaGraphLaunch(it->second.exec, ctx->stream));
    } else {
        for (int k = 0; k < n_steps; ++k) {
            st = enqueue_step(ctx, k, want_conf, nullptr, k == n_steps - 1);
            if (st != ST_OK) return st;
        }
        if (ctx->adam) { launch_step_tick(ctx->step_base, ctx->S, n_steps, nullptr, ctx->stream); ctx->launches += 1; }
    }
    if (loss_out)
        ST_CUDA(ctx, cudaMemcpy2DAsync(loss_out, (size_t)n_steps * sizeof(float), ctx->loss_buf, kMaxSteps * sizeof(float),
                                       (size_t)n_steps * sizeof(float), ctx->S, cudaMemcpyDefault, ctx->stream));
    if (conf_out)
        ST_CUDA(ctx, cudaMemcpy2DAsync(conf_out, (size_t)n_steps * cc * 8, ctx->conf_buf, (size_t)kMaxSteps * cc * 8,
                                       (size_t)n_steps * cc * 8, ctx->S, cudaMemcpyDefault, ctx->stream));
    return ST_OK;
}

namespace {
TrainCtl train_ctl(st_ctx* c, int iter, int max_updates, double threshold)
{
    TrainCtl t;
    t.conf = c->conf_buf + (int64_t)iter * c->C * c->C;
    t.conf_stream_stride = (int64_t)kMaxSteps * c->C * c->C;
    t.C = c->C; t.iter = iter; t.max_updates = max_updates; t.threshold = threshold;
    t.done = c->ctl_done; t.best = c->ctl_best; t.metric = c->ctl_metric;
    t.n_updates = c->ctl_n_updates; t.best_iter = c->ctl_best_iter; t.better = c->ctl_better;
    t.theta = c->theta; t.best_theta = c->best_theta; t.n_params = c->n_params; t.S = c->S;
    t.param_begin = c->trained_begin;
    return t;
}

// Train of Algorithm 1 for all streams: one prediction per pass (forward, loss + gradient + confusion), the backward,
// then the update kernel, which first assesses the prediction (metric, best_student, break) and takes the step only
// where the loop goes on.  The backward of the pass in which a loop ends is therefore computed and not used; from the
// next pass on the stream's blocks of the tensor-core GEMMs and of the loss kernel return at once (the fp32
// convolutions still run: their results are simply not used).
st_status enqueue_train(st_ctx* c, int max_updates, double threshold)
{
    st_status st = ST_OK;
    for (int i = 0; i <= max_updates && st == ST_OK; ++i) {
        const int* ended_before = i > 0 ? c->ctl_done + i : nullptr;        // done[s][i]: no prediction i for stream s
        st = enqueue_forward(c, nullptr, ended_before, kCtlPitch, false, true);           // prediction <- Forward(student, frame)
        if (st == ST_OK) st = enqueue_loss(c, c->conf_buf + (int64_t)i * c->C * c->C, nullptr, ended_before, kCtlPitch, i > 0, false);   // loss, gradient, confusion
        // metric, best_student, break: assessed by an extra block of the backward's first tensor-core kernel while that
        // kernel works, or, where there is none (fp32 convolutions; the last prediction, after which every loop ends),
        // by the update itself, which in any case takes the step only where the loop goes on
        const TrainCtl ctl = train_ctl(c, i, max_updates, threshold);
        const bool side = c->bf16_mode && i < max_updates;
        if (st == ST_OK && i < max_updates) st = enqueue_backward(c, nullptr, ended_before, kCtlPitch, side ? &ctl : nullptr);
        if (st == ST_OK) st = enqueue_update(c, i, nullptr, 0, nullptr, &ctl, side ? 2 : 1);
    }
    if (st != ST_OK) return st;
    launch_train_commit(train_ctl(c, 0, max_updates, threshold), c->theta, c->stream);    // student <- best_student
    launch_refresh_shadow(make_update_args(c, 0), c->stream);
    c->launches += 2;
    if (c->adam) { launch_step_tick(c->step_base, c->S, 0, c->ctl_n_updates, c->stream); c->launches += 1; }   // steps taken
    return check_launch(c, "train commit");
}
}  // namespace

st_status st_train_key_frame(st_ctx* ctx, double threshold, int32_t max_updates, int32_t* n_updates_out,
                             double* best_metric_out, double* metric_out, float* loss_out, int64_t* conf_out)
{
    if (!ctx) return ST_ERR_INVALID_ARG;
    if (max_updates < 0 || max_updates > kMaxSteps - 1)
        return fail(ctx, ST_ERR_INVALID_ARG, "st_train_key_frame: max_updates %d outside 0..%d", max_updates, kMaxSteps - 1);
    if (!(threshold == threshold))
        return fail(ctx, ST_ERR_INVALID_ARG, "st_train_key_frame: threshold is not a number");
    {
        const st_status ready = ready_to_run(ctx, "st_train_key_frame", true);
        if (ready != ST_OK) return ready;
    }
    const size_t cc = (size_t)ctx->C * ctx->C;
    ctx->z_current = false;
    ctx->z_unkept = ctx->fused_fwd != 0;    // the loop's logits never leave the loss kernel
    cudaError_t e = cudaSuccess;
    if (!ctx->conf_buf) e = dev_alloc(ctx, &ctx->conf_buf, (size_t)ctx->S * kMaxSteps * cc);
    if (e == cudaSuccess && !ctx->best_theta) {
        e = dev_alloc(ctx, &ctx->best_theta, (size_t)ctx->S * ctx->n_params);
        if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->ctl_done, (size_t)ctx->S * kCtlPitch);
        if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->ctl_best, (size_t)ctx->S * kCtlPitch);
        if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->ctl_metric, (size_t)ctx->S * kCtlPitch);
        if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->ctl_n_updates, (size_t)ctx->S);
        if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->ctl_best_iter, (size_t)ctx->S);
        if (e == cudaSuccess) e = dev_alloc(ctx, &ctx->ctl_better, (size_t)ctx->S * kCtlPitch);
    }
    if (e != cudaSuccess) return fail(ctx, ST_ERR_OOM, "st_train_key_frame: %s", cudaGetErrorString(e));
    ST_CUDA(ctx, cudaMemsetAsync(ctx->conf_buf, 0, (size_t)ctx->S * kMaxSteps * cc * sizeof(unsigned long long), ctx->stream));

    st_status st = ST_OK;
    if (ctx->use_graphs) {
        uint64_t thr_bits;
        memcpy(&thr_bits, &threshold, sizeof thr_bits);
        GraphKey key{max_updates, true, true, thr_bits};
        auto it = ctx->graphs.find(key);
        if (it == ctx->graphs.end()) {
            cudaGraph_t graph = nullptr;
            const int64_t before = ctx->launches;
            ST_CUDA(ctx, cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal));
            st = enqueue_train(ctx, max_updates, threshold);
            e = cudaStreamEndCapture(ctx->stream, &graph);
            const int64_t n_launches = ctx->launches - before;
            ctx->launches = before;
            if (st != ST_OK) { if (graph) cudaGraphDestroy(graph); return st; }
            if (e != cudaSuccess) return fail(ctx, ST_ERR_CUDA, "st_train_key_frame: graph capture: %s", cudaGetErrorString(e));
            cudaGraphExec_t exec = nullptr;
            e = cudaGraphInstantiate(&exec, graph, 0);
            cudaGraphDestroy(graph);
            if (e != cudaSuccess) return fail(ctx, ST_ERR_CUDA, "st_train_key_frame: graph instantiate: %s", cudaGetErrorString(e));
            it = ctx->graphs.emplace(key, st_ctx::StepGraph{exec, n_launches}).first;
        }
        ctx->launches += it->second.n_launches;
        ST_CUDA(ctx, cudaGraphLaunch(it->second.exec, ctx->stream));
    } else {
        st = enqueue_train(ctx, max_updates, threshold);
        if (st != ST_OK) return st;
    }
    const int n_pred = max_updates + 1;
    bool host_out = false;
    if (n_updates_out) {
        ST_CUDA(ctx, cudaMemcpyAsync(n_updates_out, ctx->ctl_n_updates, (size_t)ctx->S * sizeof(int), cudaMemcpyDefault, ctx->stream));
        host_out |= !is_device_ptr(n_updates_out);
    }
    if (best_metric_out) {     // best_metric after the last prediction was assessed
        ST_CUDA(ctx, cudaMemcpy2DAsync(best_metric_out, sizeof(double), ctx->ctl_best + n_pred, kCtlPitch * sizeof(double),
                                       sizeof(double), ctx->S, cudaMemcpyDefault, ctx->stream));
        host_out |= !is_device_ptr(best_metric_out);
    }
    if (metric_out) {
        ST_CUDA(ctx, cudaMemcpy2DAsync(metric_out, (size_t)n_pred * sizeof(double), ctx->ctl_metric, kCtlPitch * sizeof(double),
                                       (size_t)n_pred * sizeof(double), ctx->S, cudaMemcpyDefault, ctx->stream));
        host_out |= !is_device_ptr(metric_out);
    }
    if (loss_out) {
        ST_CUDA(ctx, cudaMemcpy2DAsync(loss_out, (size_t)n_pred * sizeof(float), ctx->loss_buf, kMaxSteps * sizeof(float),
                                       (size_t)n_pred * sizeof(float), ctx->S, cudaMemcpyDefault, ctx->stream));
        host_out |= !is_device_ptr(loss_out);
    }
    if (conf_out) {
        ST_CUDA(ctx, cudaMemcpy2DAsync(conf_out, (size_t)n_pred * cc * 8, ctx->conf_buf, (size_t)kMaxSteps * cc * 8,
                                       (size_t)n_pred * cc * 8, ctx->S, cudaMemcpyDefault, ctx->stream));
        host_out |= !is_device_ptr(conf_out);
    }
    if (host_out) ST_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return ST_OK;
}

st_status st_profile_step(st_ctx* ctx, int32_t n_steps, int32_t* n_stages, float* ms_out, const char** names_out)
{
    if (!ctx) return ST_ERR_INVALID_ARG;
    if (n_steps < 1 || !n_stages || !ms_out || !names_out)
        return fail(ctx, ST_ERR_INVALID_ARG, "st_profile_step: n_steps >= 1 and non-NULL outputs are required");
    {
        const st_status ready = ready_to_run(ctx, "st_profile_step", true);
        if (ready != ST_OK) return ready;
    }
    ctx->z_current = false;
    StageTimer t;
    t.repeat = 8;
    for (int i = 0; i <= StageTimer::kMax; ++i) ST_CUDA(ctx, cudaEventCreate(&t.ev[i]));
    double acc[StageTimer::kMax] = {0};
    st_status st = ST_OK;
    int n = 0;
    for (int k = 0; k < n_steps && st == ST_OK; ++k) {
        t.n = 0;
        cudaEventRecord(t.ev[0], ctx->stream);
        st = enqueue_step(ctx, 0, false, &t);
        if (st != ST_OK) break;
        if (ctx->adam) { launch_step_tick(ctx->step_base, ctx->S, 1, nullptr, ctx->stream); ctx->launches += 1; }
        if (cudaStreamSynchronize(ctx->stream) != cudaSuccess) { st = fail(ctx, ST_ERR_CUDA, "st_profile_step: synchronize failed"); break; }
        n = t.n;
        for (int i = 0; i < n; ++i) {
            float ms = 0.f;
            cudaEventElapsedTime(&ms, t.ev[i], t.ev[i + 1]);
            acc[i] += ms / t.launches[i];
        }
    }
    for (int i = 0; i <= StageTimer::kMax; ++i) cudaEventDestroy(t.ev[i]);
    if (st != ST_OK) return st;
    *n_stages = n;
    for (int i = 0; i < n; ++i) { ms_out[i] = (float)(acc[i] / n_steps); names_out[i] = t.name[i]; }
    return ST_OK;
}

st_status st_pack_updated_params(st_ctx* ctx, int32_t stream, void* dst, size_t dst_capacity, size_t* nbytes)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    const size_t need = (size_t)ctx->n_trained * sizeof(float);      // UpdatedPart: the layers behind the freeze boundary
    if (nbytes) *nbytes = need;
    if (!dst) return fail(ctx, ST_ERR_INVALID_ARG, "st_pack_updated_params: NULL destination");
    if (dst_capacity < need)
        return fail(ctx, ST_ERR_BUFFER_TOO_SMALL, "st_pack_updated_params: capacity %zu < %zu bytes", dst_capacity, need);
    const float* src = ctx->theta + (int64_t)stream * ctx->n_params;
    if (is_device_ptr(dst)) {
        launch_pack(src, (float*)dst, ctx->layout, ctx->trained_begin, ctx->n_trained, 1, ctx->stream);
        ctx->launches += 1;
        return check_launch(ctx, "pack");
    }
    // host destination: pack into the staging buffer, then copy out
    st = ensure_staging(ctx, need);
    if (st != ST_OK) return st;
    launch_pack(src, (float*)ctx->staging, ctx->layout, ctx->trained_begin, ctx->n_trained, 1, ctx->stream);
    ctx->launches += 1;
    st = check_launch(ctx, "pack");
    if (st != ST_OK) return st;
    ST_CUDA(ctx, cudaMemcpyAsync(dst, ctx->staging, need, cudaMemcpyDeviceToHost, ctx->stream));
    ST_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return ST_OK;
}

st_status st_apply_update(st_ctx* ctx, int32_t stream, const void* src, size_t nbytes)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    const size_t need = (size_t)ctx->n_trained * sizeof(float);
    if (!src) return fail(ctx, ST_ERR_INVALID_ARG, "st_apply_update: NULL source");
    if (nbytes != need) return fail(ctx, ST_ERR_INVALID_ARG, "st_apply_update: %zu bytes given, the updated part has %zu", nbytes, need);
    const void* dev = nullptr;
    st = to_device(ctx, src, need, &dev);
    if (st != ST_OK) return st;
    ctx->z_current = false;
    launch_unpack((const float*)dev, ctx->theta + (int64_t)stream * ctx->n_params, ctx->layout, ctx->trained_begin, ctx->n_trained, 1, ctx->stream);
    ctx->launches += 1;
    if (ctx->bf16_mode) { launch_refresh_shadow(make_update_args(ctx, -1), ctx->stream); ctx->launches += 1; }
    return check_launch(ctx, "apply update");
}

namespace {
// forward of all streams with the current parameters, then the mask kernel on `stream`
st_status student_forward(st_ctx* ctx, int32_t stream, const char* who)
{
    (void)stream;                           // the forward runs on all streams
    st_status ready = ready_to_run(ctx, who, false);
    if (ready != ST_OK) return ready;
    if (ctx->z_current) return ST_OK;       // an earlier call already ran it and nothing has changed since
    st_status st = enqueue_forward(ctx);
    ctx->z_current = st == ST_OK;
    if (st == ST_OK) ctx->z_unkept = false;
    return st;
}

StudentMaskArgs mask_args(st_ctx* ctx, int32_t stream, uint8_t* mask)
{
    StudentMaskArgs a{};
    a.z = ctx->z + (int64_t)stream * ctx->C * ctx->p;
    a.C = ctx->C; a.h = ctx->h; a.w = ctx->w;
    a.mask = mask;
    if (ctx->fused_fwd) {               // the mask kernel multiplies the logits itself: no forward before it, `z` is not read
        a.fused = 1; a.kblocks = ctx->Cin / 64; a.stream = stream;
        a.bias = ctx->theta + (int64_t)stream * ctx->n_params + ctx->layout.b_off[ctx->layout.n_layers - 1];
        a.err = ctx->bad + 2;
        a.x_map = &ctx->fx_map; a.w_map = &ctx->fw_map;
    }
    return a;
}
}  // namespace

st_status st_student_mask(st_ctx* ctx, int32_t stream, uint8_t* mask_out)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    if (!mask_out) return fail(ctx, ST_ERR_INVALID_ARG, "st_student_mask: NULL destination");
    st = ctx->fused_fwd ? ready_to_run(ctx, "st_student_mask", false) : student_forward(ctx, stream, "st_student_mask");
    if (st != ST_OK) return st;
    const bool dev = is_device_ptr(mask_out);
    // the kernel writes the mask two pixels (16 bits) at a time: a destination at an odd address gets its
    // mask through the context's own buffer
    const bool direct = dev && ((uintptr_t)mask_out & 1u) == 0;
    uint8_t* dst = direct ? mask_out : ctx->mask_tmp;
    launch_student_mask(mask_args(ctx, stream, dst), ctx->stream);
    ctx->launches += 1;
    st = check_launch(ctx, "student mask");
    if (st != ST_OK) return st;
    if (!direct) ST_CUDA(ctx, cudaMemcpyAsync(mask_out, dst, (size_t)ctx->P, cudaMemcpyDefault, ctx->stream));
    if (!dev) ST_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return ST_OK;
}

st_status st_agreement(st_ctx* ctx, int32_t stream, const uint8_t* pred, const uint8_t* label, int64_t* conf, double* miou)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    const uint8_t* d_label = nullptr;
    const uint8_t* d_pred = nullptr;
    if (label) {
        // the fused kernel reads labels two pixels (16 bits) at a time: a device map at an odd address is copied
        // into the context's buffer like a host map (the plain confusion kernel takes any address)
        if (is_device_ptr(label) && (pred || ((uintptr_t)label & 1u) == 0)) d_label = label;
        else {
            ST_CUDA(ctx, cudaMemcpyAsync(ctx->mask_tmp2, label, (size_t)ctx->P, cudaMemcpyDefault, ctx->stream));
            d_label = ctx->mask_tmp2;
        }
    } else {
        if (!ctx->has_labels[stream]) return fail(ctx, ST_ERR_BAD_STATE, "st_agreement: stream %d has no labels yet", stream);
        d_label = ctx->labels + (int64_t)stream * ctx->P;
    }
    const size_t cc = (size_t)ctx->C * ctx->C, cbytes = cc * sizeof(unsigned long long);
    // Where the kernel delivers the finished matrix and the mean IoU: straight into the caller's device buffers where
    // it gave some (the call is then one kernel and nothing else), else into the context's, to be copied out below.
    const bool conf_direct = conf && is_device_ptr(conf) && ((uintptr_t)conf & 7u) == 0;
    const bool miou_direct = miou && is_device_ptr(miou) && ((uintptr_t)miou & 7u) == 0;
    unsigned long long* conf_res = conf_direct ? reinterpret_cast<unsigned long long*>(conf) : ctx->conf_tmp + cc + 1;
    double* miou_res = miou_direct ? miou : ctx->miou_tmp;
    if (!pred && student_mask_fused_supported(ctx->C)) {
        // the student's own mask: arg-max, confusion and mean IoU in one kernel, the mask itself is not stored
        st = ctx->fused_fwd ? ready_to_run(ctx, "st_agreement", false) : student_forward(ctx, stream, "st_agreement");
        if (st != ST_OK) return st;
        StudentMaskArgs a = mask_args(ctx, stream, nullptr);
        a.labels = d_label; a.conf = ctx->conf_tmp; a.bad = ctx->bad + 1; a.miou = miou_res;
        a.ticket = reinterpret_cast<unsigned int*>(ctx->conf_tmp + cc);
        a.conf_out = conf_res;
        launch_student_mask(a, ctx->stream);
        ctx->launches += 1;
    } else {
        if (pred) {
            if (is_device_ptr(pred)) d_pred = pred;
            else {
                ST_CUDA(ctx, cudaMemcpyAsync(ctx->mask_tmp, pred, (size_t)ctx->P, cudaMemcpyHostToDevice, ctx->stream));
                d_pred = ctx->mask_tmp;
            }
        } else {
            st = st_student_mask(ctx, stream, ctx->mask_tmp);
            if (st != ST_OK) return st;
            d_pred = ctx->mask_tmp;
        }
        // one kernel: its last block turns the counts into the mean IoU, delivers the matrix and clears the counters
        const ConfusionFinish fin = {conf_res, miou_res, reinterpret_cast<unsigned int*>(ctx->conf_tmp + cc)};
        launch_confusion(d_label, d_pred, ctx->P, ctx->C, ctx->conf_tmp, ctx->bad + 1, ctx->stream, &fin);
        ctx->launches += 1;
    }
    st = check_launch(ctx, "confusion");
    if (st != ST_OK) return st;
    if (conf && !conf_direct) ST_CUDA(ctx, cudaMemcpyAsync(conf, conf_res, cbytes, cudaMemcpyDefault, ctx->stream));
    if (miou && is_device_ptr(miou)) {
        // device destination: nothing to wait for; bad labels surface at the next call that does wait
        if (!miou_direct) ST_CUDA(ctx, cudaMemcpyAsync(miou, ctx->miou_tmp, sizeof(double), cudaMemcpyDeviceToDevice, ctx->stream));
        return ST_OK;
    }
    st = fetch_status(ctx);
    if (st != ST_OK) return st;
    if (miou) *miou = ctx->status_host[0];
    return report_status(ctx, true);
}

st_status st_read_tensor(st_ctx* ctx, int32_t stream, st_tensor which, float* dst_host, size_t dst_capacity, size_t* nbytes)
{
    st_status st = check_stream_index(ctx, stream);
    if (st != ST_OK) return st;
    size_t count = 0;
    switch (which) {
        case ST_TENSOR_LOGITS: case ST_TENSOR_LOGIT_GRAD: count = (size_t)ctx->C * ctx->p; break;
        case ST_TENSOR_PARAM_GRAD: case ST_TENSOR_MOMENTUM: count = (size_t)ctx->n_params; break;
        case ST_TENSOR_HIDDEN: case ST_TENSOR_HIDDEN_GRAD:
            if (!ctx->Ch) return fail(ctx, ST_ERR_INVALID_ARG, "st_read_tensor: the head has no hidden layer");
            if (which == ST_TENSOR_HIDDEN_GRAD && ctx->bf16_mode && !ctx->blk[ctx->n_blocks - 1].dout)
                return fail(ctx, ST_ERR_INVALID_ARG, "st_read_tensor: the last block is frozen, no gradient is formed for it");
            count = (size_t)ctx->Ch * ctx->p; break;
        case ST_TENSOR_HIDDEN_FIRST: case ST_TENSOR_HIDDEN_GRAD_FIRST:
            if (ctx->n_blocks < 2) return fail(ctx, ST_ERR_INVALID_ARG, "st_read_tensor: the head has no second block");
            if (which == ST_TENSOR_HIDDEN_GRAD_FIRST && !ctx->blk[0].dout)
                return fail(ctx, ST_ERR_INVALID_ARG, "st_read_tensor: the first block is frozen, no gradient is formed for it");
            count = (size_t)ctx->blk[0].c_out * ctx->p; break;
        case ST_TENSOR_FEATURES: count = (size_t)ctx->Cin * ctx->p; break;
        default: return fail(ctx, ST_ERR_INVALID_ARG, "st_read_tensor: unknown tensor %d", (int)which);
    }
    const size_t need = count * sizeof(float);
    if (nbytes) *nbytes = need;
    if (!dst_host) return fail(ctx, ST_ERR_INVALID_ARG, "st_read_tensor: NULL destination");
    if (dst_capacity < need) return fail(ctx, ST_ERR_BUFFER_TOO_SMALL, "st_read_tensor: capacity %zu < %zu bytes", dst_capacity, need);
    if (ctx->read_tmp_bytes < need) {
        ST_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
        if (ctx->read_tmp) cudaFree(ctx->read_tmp);
        ctx->read_tmp = nullptr; ctx->read_tmp_bytes = 0;
        ST_CUDA(ctx, cudaMalloc((void**)&ctx->read_tmp, need));
        ctx->read_tmp_bytes = need;
    }
    const float* src = nullptr;
    const int64_t s = stream;
    if ((which == ST_TENSOR_LOGITS || which == ST_TENSOR_LOGIT_GRAD) && ctx->z_unkept) {
        st = student_forward(ctx, stream, "st_read_tensor");     // the forward of the student the last call left behind
        if (st != ST_OK) return st;
    }
    switch (which) {
        case ST_TENSOR_LOGITS: src = ctx->z + s * ctx->C * ctx->p; break;
        case ST_TENSOR_LOGIT_GRAD:
            if (ctx->bf16_mode) {     // the step wrote the bf16 copy only: same logits, same labels, same arithmetic once more
                launch_upsample_ce(k3_args(ctx, true, false, nullptr), &ctx->k3_map, ctx->stream);
                ctx->launches += 1;
            }
            src = ctx->dz + s * ctx->C * ctx->p;
            break;
        case ST_TENSOR_PARAM_GRAD: launch_pack(ctx->grad + s * ctx->n_params, ctx->read_tmp, ctx->layout, 0, ctx->n_params, 1, ctx->stream); src = ctx->read_tmp; break;
        case ST_TENSOR_MOMENTUM: launch_pack(ctx->vel + s * ctx->n_params, ctx->read_tmp, ctx->layout, 0, ctx->n_params, 1, ctx->stream); src = ctx->read_tmp; break;
        case ST_TENSOR_HIDDEN:
            if (ctx->bf16_mode) { launch_nhwc_bf16_to_chw(ctx->blk[ctx->n_blocks - 1].out + s * ctx->p * ctx->Ch, ctx->Ch, ctx->p, ctx->read_tmp, ctx->stream); src = ctx->read_tmp; }
            else src = ctx->hid_f32 + s * ctx->Ch * ctx->p;
            break;
        case ST_TENSOR_HIDDEN_GRAD:
            if (ctx->bf16_mode) { launch_nhwc_bf16_to_chw(ctx->blk[ctx->n_blocks - 1].dout + s * ctx->p * ctx->Ch, ctx->Ch, ctx->p, ctx->read_tmp, ctx->stream); src = ctx->read_tmp; }
            else src = ctx->dhid_f32 + s * ctx->Ch * ctx->p;
            break;
        case ST_TENSOR_HIDDEN_FIRST:
            launch_nhwc_bf16_to_chw(ctx->blk[0].out + s * ctx->p * ctx->blk[0].c_out, ctx->blk[0].c_out, ctx->p, ctx->read_tmp, ctx->stream);
            src = ctx->read_tmp;
            break;
        case ST_TENSOR_HIDDEN_GRAD_FIRST:
            launch_nhwc_bf16_to_chw(ctx->blk[0].dout + s * ctx->p * ctx->blk[0].c_out, ctx->blk[0].c_out, ctx->p, ctx->read_tmp, ctx->stream);
            src = ctx->read_tmp;
            break;
        case ST_TENSOR_FEATURES:
            if (ctx->bf16_mode) { launch_nhwc_bf16_to_chw(ctx->x_bf16 + s * ctx->p * ctx->Cin, ctx->Cin, ctx->p, ctx->read_tmp, ctx->stream); src = ctx->read_tmp; }
            else src = ctx->x_f32 + s * ctx->Cin * ctx->p;
            break;
    }
    st = check_launch(ctx, "read tensor");
    if (st != ST_OK) return st;
    ST_CUDA(ctx, cudaMemcpyAsync(dst_host, src, need, cudaMemcpyDeviceToHost, ctx->stream));
    ST_CUDA(ctx, cudaStreamSynchronize(ctx->stream));
    return report_bad_labels(ctx, 0, "an earlier st_distill_step");
}

}  // extern "C"
