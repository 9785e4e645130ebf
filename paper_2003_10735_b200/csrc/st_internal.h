// Internal declarations shared by the kernels' translation units and the C-ABI layer.
// Nothing here is part of the public interface (see include/shadowtutor.h).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <utility>

namespace st {

typedef __nv_bfloat16 bf16;

// ---- programmatic dependent launch -----------------------------------------------------------------
// The kernels of a step form a chain.  Launched with the programmatic-serialization attribute a kernel
// may start while its predecessor is still draining; everything it does before pdl_wait() (barrier
// set-up, tensor-memory allocation, index arithmetic) then overlaps the predecessor's tail.
// pdl_wait() returns once the predecessor grid has completed and its writes are visible; no global
// memory is read or written before it.  pdl_launch_dependents() lets the successor start launching.
#ifdef __CUDACC__
// One 32-byte store (a whole sector) from eight 32-bit registers; the address must be 32-byte aligned.  Where the
// lanes of a warp write to rows that lie far apart (pixel-major activations), a sector written as two 16-byte halves
// reaches L2 as two partial writes; this store writes it once.
__device__ __forceinline__ void store_256(void* dst, const uint32_t* r)
{
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 :: "l"(dst), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

bool pdl_enabled();   // true unless the environment variable ST_PDL is set to 0

// `early`: launch with the programmatic-serialization attribute, i.e. the kernel may start before its predecessor on
// the stream has completed and must call pdl_wait() before it touches anything the predecessor writes.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_early(bool early, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = early ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

// A kernel of the step's chain; `early` is the context's choice (the `chain_early` field of the argument structs).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chain(bool early, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args)
{
    return launch_early(early, kernel, grid, block, smem, s, std::forward<Args>(args)...);
}
#endif

constexpr int kUp = 4;            // bilinear upsample factor of the head (frame = feature map * 4)
constexpr int kMaxSteps = 64;     // upper bound of n_steps in one st_distill_step call
constexpr int kClassPad = 32;     // class rows of bf16 GEMM operands are padded to this (UMMA N)
constexpr int kMaxBlocks = 2;     // student blocks in front of the classifier (Section 5.2: SB5, SB6)
constexpr int kMaxLayers = kMaxBlocks + 1;

// ---- K1: teacher logits -> uint8 labels -------------------------------------------------------
void launch_argmax_u8(const float* logits, int C, int64_t P, uint8_t* labels, cudaStream_t s);

// ---- K6: confusion matrix of two uint8 masks ---------------------------------------------------
// conf: int64 [C][C], accumulated into (caller zeroes it); bad: count of pixels with l or q >= C.
// With `finish` the kernel completes the measurement by itself: its last block writes the matrix to `result` and the
// mean IoU (Section 3.2) to `miou`, then clears `conf` and the ticket, so that the next launch needs no memset
// (`conf` and `*ticket` must be zero before the first launch).
struct ConfusionFinish { unsigned long long* result; double* miou; unsigned int* ticket; };
void launch_confusion(const uint8_t* label, const uint8_t* pred, int64_t P, int C,
                      unsigned long long* conf, unsigned int* bad, cudaStream_t s, const ConfusionFinish* finish = nullptr);

// ---- K8: frozen features fp32 [Cin][p] -> bf16 [p][Cin] ---------------------------------------
void launch_feat_to_bf16_nhwc(const float* feat_chw, int Cin, int64_t p, bf16* out, cudaStream_t s);
// reverse (verification only): bf16 [p][C] -> fp32 [C][p]
void launch_nhwc_bf16_to_chw(const bf16* in, int C, int64_t p, float* out, cudaStream_t s);

// ---- loss weighting near objects: labels [H][W] of one stream -> labels with bit 7 set where the pixel is within
// `radius` of a non-background pixel; tmp is a scratch map of H*W bytes
void launch_object_weight_tags(const uint8_t* labels, int H, int W, int background, int radius, uint8_t* tmp, uint8_t* tagged,
                               cudaStream_t s);

// ---- K3: upsample x4 + softmax cross-entropy + gradient w.r.t. the low-res logits ---------------
struct UpsampleCeArgs {
    const float* z;          // [S][C][h][w]
    const uint8_t* labels;   // [S][H][W]
    float* dz;               // [S][C][h][w]     gradient of the mean loss, or nullptr (only the bf16 copy is wanted)
    bf16* dz_bf16;           // [S][kClassPad][dz_bf16_pitch] or nullptr (rows >= C untouched)
    int64_t dz_bf16_pitch;
    float* loss_part;        // [S][n_blocks]    per-block partial sums of per-pixel losses
    float* db_part;          // [S][n_blocks][C] per-block partial sums of dz over the block's pixels
    unsigned long long* conf;// nullptr, or int64 [C][C] per stream: confusion of label vs argmax of the upsampled logits
    int64_t conf_stream_stride; // elements between the matrices of consecutive streams
    unsigned int* bad;       // count of labels >= C
    unsigned int* err;       // device word: first wait that gave up (0 = none)
    int S, C, h, w;
    int has_map;             // the launch carries a tile map of z (see make_logit_tile_map)
    const int* skip;         // nullptr, or one flag per stream (skip[s * skip_stride]): non-zero = the stream's blocks return at once
    int64_t skip_stride;
    int heavy_w;             // 1, or the integer weight (2..5) of the pixels whose label byte has bit 7 set
                             //   (`labels` is then the tagged map made by launch_object_weight_tags)
    int chain_early;         // launch so that the kernel may start while its predecessor on the stream drains
    // The block multiplies its own logit tile instead of reading `z` (Forward for a 1x1 classifier over bf16 features,
    // row-walking kernel only; the launch then carries tile maps of the features and of the bf16 weights):
    int fused;               // 0, or 1: ignore `z`, compute the tile from the maps
    int x_early;             // the features are not written by the kernel just before this one: fetch them before waiting for it
    int kblocks;             // 64-channel slices of the classifier's input
    const float* theta;      // parameters (for the bias: theta[s * n_params + b_off + c])
    int64_t n_params, b_off;
    float* z_out;            // nullptr, or [S][C][h][w]: the logits are written here as well
    int test_stall;          // test of the give-up path: the first wait of the block's forward runs out (see fused_tile.cuh)
};
// Tile map of the logits for the row-walking kernel: fp32 tensor {w, h, S*C}, one box = the block's tile of all
// classes.  False if the shape does not allow it (w not a multiple of 4, C > 32) or the driver entry point is
// missing; the kernel then fetches its tile with plain loads.
bool make_logit_tile_map(CUtensorMap* m, const float* z, int S, int C, int h, int w);
// general form: any element type and swizzle; dims innermost first, strides (bytes) for dimensions 1..rank-1
bool encode_tensor_map(CUtensorMap* m, CUtensorMapDataType dtype, CUtensorMapSwizzle swizzle, const void* base, int rank,
                       const uint64_t* dims, const uint64_t* strides, const uint32_t* box, char* err, size_t err_len,
                       const char* what);
int upsample_ce_blocks(int h, int w, int C);   // blocks per stream (sizes loss_part / db_part)
cudaError_t prepare_upsample_ce(int C);   // once per device and class count, outside any stream capture
// z_map: host copy, used if a.has_map; x_map, w_map: host copies, needed if a.fused (without them, or for a shape
// fused_forward_supported rejects, the launch falls back to reading `z`)
void launch_upsample_ce(const UpsampleCeArgs& a, const CUtensorMap* z_map, cudaStream_t s, const CUtensorMap* x_map = nullptr,
                        const CUtensorMap* w_map = nullptr);
bool fused_forward_supported(int C, int h, int w, int c_in);
// Tile map of bf16 features [S][h][w][c_in] for the fused forward: {c_in, w, h, S}, one box = 64 channels of the block's tile
bool make_feature_tile_map(CUtensorMap* m, const bf16* x, int S, int c_in, int h, int w);
// register-resident variant for C <= 32 (k_upsample_ce_rows.cu); launch_upsample_ce dispatches to it
bool upsample_ce_rows_supported(int C);
int upsample_ce_rows_blocks(int h, int w);
cudaError_t prepare_upsample_ce_rows(int C);
void launch_upsample_ce_rows(const UpsampleCeArgs& a, const CUtensorMap* z_map, cudaStream_t s, const CUtensorMap* x_map = nullptr,
                             const CUtensorMap* w_map = nullptr);
// student mask: argmax_c of the upsampled logits, uint8 [H][W]; with `labels` also the confusion matrix of
// (label, mask) added into `conf`, and with `miou` the mean IoU written by the last block (k_student_mask.cu)
struct StudentMaskArgs {
    const float* z;            // [C][h][w] logits of one stream
    int C, h, w;
    uint8_t* mask;             // [H][W] or nullptr (confusion only)
    const uint8_t* labels;     // [H][W] or nullptr (mask only)
    unsigned long long* conf;  // [C][C], zero on entry
    unsigned int* bad;         // count of labels >= C
    double* miou;              // nullptr: no mean IoU
    unsigned int* ticket;      // zero between launches (block counter for the mean IoU)
    unsigned long long* conf_out;  // with `miou`: the last block writes the finished matrix here and clears `conf`
    // One-layer head with bf16 features: the kernel multiplies the logits itself (k_student_eval.cu) and `z` is not read
    int fused;                 // 0, or 1: the fields below are set
    int kblocks, stream;       // 64-channel slices of the features; the stream (a coordinate of the tile maps)
    const float* bias;         // the classifier's bias of that stream (fp32 master parameters)
    unsigned int* err;         // device word: first wait that gave up
    const CUtensorMap* x_map;  // host copies of the tile maps of the features (make_feature_tile_map) and of the bf16 weights
    const CUtensorMap* w_map;
};
cudaError_t prepare_student_eval(int C);    // once per device and class count, outside any stream capture
cudaError_t launch_student_eval(const StudentMaskArgs& a, cudaStream_t s);
bool student_mask_fused_supported(int C);   // confusion counters fit shared memory
cudaError_t prepare_student_mask(int C);    // once per device and class count, outside any stream capture
void launch_student_mask(const StudentMaskArgs& a, cudaStream_t s);

// ---- fp32 CUDA-core convolutions (gemm_precision 0), planar [C][h][w] -------------------------
void launch_conv_fwd_f32(const float* in, int Cin, int h, int w, const float* Wt, const float* b,
                         int Cout, int ks, bool relu, float* out, int S, int64_t in_stride,
                         int64_t w_stride, int64_t b_stride, int64_t out_stride, cudaStream_t s);
void launch_conv_wgrad_f32(const float* in, const float* dout, int Cin, int Cout, int h, int w, int ks,
                           float* dW, int S, int64_t in_stride, int64_t dout_stride,
                           int64_t dw_stride, cudaStream_t s);
void launch_conv1x1_dgrad_relu_f32(const float* W2, const float* dz, const float* Hact, int C, int Ch,
                                   int64_t p, float* dH, int S, int64_t w_stride, int64_t dz_stride,
                                   int64_t h_stride, cudaStream_t s);
// db[c] = sum_p d[c][p] (one block per channel, fixed-order reduction)
void launch_bias_grad_f32(const float* d, int C, int64_t p, float* db, int S, int64_t d_stride,
                          int64_t db_stride, cudaStream_t s);

// ---- control of Algorithm 1 (Train): assessed once per prediction, per stream, by the update kernel that follows the
// prediction (metric of the prediction, best_student, the break) ----------------------------------------------
// History arrays are indexed by the number of updates behind a prediction, so that a launch reads only what
// earlier launches wrote: done[s][i] = the loop of stream s had ended before prediction i was made,
// best[s][i] = best_metric before prediction i was assessed.
constexpr int kCtlPitch = kMaxSteps + 2;
struct TrainCtl {
    const unsigned long long* conf;   // confusion matrix of this prediction, stream 0
    int64_t conf_stream_stride;       // elements between the matrices of consecutive streams
    int C;
    int iter;                         // i: number of updates behind this prediction
    int max_updates;                  // MAX_UPDATES
    double threshold;                 // THRESHOLD
    int* done;                        // [S][kCtlPitch]
    double* best;                     // [S][kCtlPitch]
    double* metric;                   // [S][kCtlPitch]  metric of prediction i; -1 where the loop had ended before
    int* better;                      // [S][kCtlPitch]  prediction i was the best so far (best_student <- student)
    int* n_updates;                   // [S] updates taken when the loop ended
    int* best_iter;                   // [S] updates behind best_student
    const float* theta;               // [S][n_params]
    float* best_theta;                // [S][n_params]  best_student
    int64_t n_params;
    int64_t param_begin;              // parameters before this index are frozen: best_student never differs from the student there
    int S;
};

// ---- K5: SGD(+momentum) update, loss finalisation, bf16 shadow refresh -------------------------
struct LayerUpdate {
    int64_t w_off, b_off;      // offsets (floats) of weight / bias in one stream's parameter buffer
    int cout, cin, taps;       // weight in internal order [tap][cout][cin]
    const float* w_partials;   // nullptr: grad buffer already holds dW; else split-K partial sums whose
    int n_split;               //   element index equals the internal weight index
    int64_t w_split_stride;    // floats between splits
    int64_t w_stream_stride;   // floats between streams
    const float* b_partials;   // nullptr: grad buffer already holds db; else [S][n_bpart][cout]
    int n_bpart;
    bf16* shadow;              // nullptr or the bf16 copy of the weight read by the GEMMs (same linear index)
    int64_t shadow_stream_stride;
    bf16* shadow_t;            // nullptr, or a second bf16 copy [9][c_take][cout] with the taps mirrored and the channels
    int64_t shadow_t_stream_stride;   // transposed, for the first c_take input channels: what the gradient passed back
    int c_take;                //   through this 3x3 layer multiplies
    int streamed;              // set by the launcher: the streaming kernel updates this layer's weights, the grouped one skips them
};
struct UpdateArgs {
    float* theta;      // [S][n_params]   internal order
    float* vel;        // [S][n_params]
    float* grad;       // [S][n_params]   holds the applied gradient after the call
    int64_t n_params;
    int S;
    float lr, mu;
    LayerUpdate layer[kMaxLayers];
    int n_layers;
    int64_t param_begin;     // parameters before this index belong to frozen layers and are left alone
    const float* loss_part;  // [S][n_loss_part] per-block sums of per-pixel losses
    int n_loss_part;
    float* loss_buf;         // [S][kMaxSteps]
    int loss_slot;           // slot of loss_buf written by this step
    double inv_P;
    const int* skip;         // nullptr, or one flag per stream (skip[s * skip_stride]): non-zero = leave the stream's
    int64_t skip_stride;     //   parameters and momentum untouched (the loss is still finalised)
    // Adam (optimizer 1): `vel` is the first moment, `vel2` the second; step number t = step_base[s] + loss_slot + 1
    int adam;
    float* vel2;             // [S][n_params]
    double b1, b2, eps, ln_b1, ln_b2;
    const long long* step_base;   // [S] optimisation steps taken before this call
    int chain_early;         // launch so that the kernel may start while its predecessor on the stream drains
    // Train (Algorithm 1): the update also assesses the prediction it follows.  Every block works the metric out from the
    // prediction's confusion matrix (same counts, same arithmetic, same answer), keeps the old value of its parameters
    // as best_student's where the metric is the best so far, and leaves them alone where the loop has ended; block 0
    // writes the history.  `skip` is then not used.
    int has_ctl;             // 0; 1: this kernel assesses the prediction; 2: the backward before it has (see tc_backward), read the outcome
    TrainCtl ctl;
};
// step_base[s] += add (add_per_stream == nullptr) or += add_per_stream[s]
void launch_step_tick(long long* step_base, int S, int add, const int* add_per_stream, cudaStream_t s);
int launch_sgd_update(const UpdateArgs& a, cudaStream_t s);   // returns the number of kernels launched
// refresh the bf16 shadows from the fp32 master parameters (after init)
void launch_refresh_shadow(const UpdateArgs& a, cudaStream_t s);
// mean IoU (Section 3.2) from an int64 confusion matrix, in double, one block
void launch_miou(const unsigned long long* conf, int C, double* out, cudaStream_t s);
// student <- best_student for the trained parameters (the caller refreshes the bf16 copies afterwards)
void launch_train_commit(const TrainCtl& t, float* theta, cudaStream_t s);


// ---- K7: packed parameter buffer <-> internal order ---------------------------------------------
// packed: per layer weight [cout][cin][kh][kw] then bias; internal: weight [tap][cout][cin] then bias.
// `begin`, `count`: the range of one stream's parameters that the packed buffer carries (all of them at initialisation;
// the trained layers, which come last, in UpdatedPart); packed buffers of consecutive streams lie `count` floats apart.
struct PackLayout { int n_layers; int64_t w_off[kMaxLayers], b_off[kMaxLayers]; int cout[kMaxLayers], cin[kMaxLayers], taps[kMaxLayers]; int64_t n_params; };
void launch_pack(const float* internal, float* packed, const PackLayout& L, int64_t begin, int64_t count, int n_bufs, cudaStream_t s);
void launch_unpack(const float* packed, float* internal, const PackLayout& L, int64_t begin, int64_t count, int n_bufs, cudaStream_t s);

// ---- bf16 tensor-core GEMMs (gemm_precision 1) -------------------------------------------------
struct TcPlan;   // tensor maps and launch geometry; built once per context
// One student block of the trainable back part: 3x3 convolution (zero padding 1) over the concatenation of the previous
// block's output (the frozen part's output for the first block) and the block's skip input, then ReLU.
struct TcBlock {
    int c_prev, c_skip, c_out;
    const bf16* in_prev;     // [S][p][c_prev]
    const bf16* in_skip;     // [S][p][c_skip] or nullptr
    const bf16* w;           // [S][9][c_out][c_prev + c_skip]  bf16 copy of the weight, tap-major
    const bf16* w_t;         // [S][9][c_prev][c_out]  taps mirrored, channels transposed (pass_back only)
    int64_t b_off;           // offset of the bias in one stream's parameters
    bf16* out;               // [S][p][c_out]
    uint32_t* relu_bits;     // [S][p][c_out/32]: one bit per output value, set where it is > 0
    bf16* dout;              // [S][p][c_out]     gradient with respect to the output, after the ReLU mask
    float* w_partials;       // [S][n_split1][9][c_out][c_prev + c_skip]
    float* b_partials;       // [S][n_bpart][c_out]: 128-pixel tiles for the last block, 4 x 32 tiles for the others
    int trained;             // the block lies behind the freeze boundary: its gradients are formed
    int pass_back;           // ... and so does the block before it: the gradient is passed on to it
};
struct TcBuffers {
    int S, c_in, C, h, w;
    int n_blocks;
    TcBlock blk[kMaxBlocks];
    const bf16* x;        // [S][p][c_in]     cached features, pixel-major
    const bf16* w2;       // [S][kClassPad][c_last]  bf16 copy of the 1x1 weight, rows >= C zero
    const float* theta;   // [S][n_params]    biases are read from the master parameters
    int64_t n_params, b2_off, w2_off;
    float* z;             // [S][C][p]
    const float* dz;      // [S][C][p]
    const bf16* dz_bf16;  // [S][kClassPad][tc_dz_pitch]
    float* w2_partials;   // [S][n_split2][kClassPad][c_last]
    unsigned int* err;    // device word: first wait that gave up (0 = none)
    int chain_early;      // launch the kernels so that each may start while its predecessor on the stream drains
};
// Geometry is fixed by the shapes alone, so scratch can be sized before the plan exists.
int tc_wgrad_splits(int layer /*1: 3x3, 2: 1x1*/, int c_last, int h, int w);
int tc_b1_partials(int h, int w);   // 128-pixel tiles (bias-gradient partials of the block in front of the classifier)
int tc_tile3_count(int h, int w);   // 4 x 32 pixel tiles of a 3x3 layer per stream (bias-gradient partials of earlier blocks)
int tc_dz_pitch(int h, int w);      // row pitch (elements) of the bf16 logit gradient [S][kClassPad][pitch]
TcPlan* tc_plan_create(const TcBuffers& b, char* err, size_t err_len);
void tc_plan_destroy(TcPlan*);
// Optional per-kernel timing: an event is recorded on the stream after each kernel's launches.  Kernels whose
// result does not depend on how often they run (everything but the parameter update) are launched `repeat` times
// back to back, so that the time between two events is `repeat` kernel durations plus one launch gap.
struct StageTimer {
    static constexpr int kMax = 12;
    cudaEvent_t ev[kMax + 1];
    const char* name[kMax];
    int launches[kMax];
    int repeat = 1;
    int n = 0;
    void mark(const char* what, cudaStream_t s, int n_launches) { if (n < kMax) { name[n] = what; launches[n] = n_launches; cudaEventRecord(ev[n + 1], s); ++n; } }
};
#define ST_REPEAT(t) for (int r_ = 0, R_ = (t) ? (t)->repeat : 1; r_ < R_; ++r_)
inline int st_repeats(const StageTimer* t) { return t ? t->repeat : 1; }
// `skip`: nullptr, or one flag per stream (skip[s * skip_stride]); the blocks of a flagged stream return at once.
// Returns the number of kernels launched.  `after_update`: the kernel launched just before on this stream is the
// parameter update of the previous iteration, which writes weights but no activations; the forward of a one-layer head
// may then fetch its activation tiles while that update is still running.  `first_block`: the blocks before it are
// frozen and their outputs already computed for this key frame (tc_forward_blocks).
int tc_forward(const TcPlan*, cudaStream_t s, StageTimer* t = nullptr, const int* skip = nullptr, int64_t skip_stride = 0,
               bool after_update = false, int first_block = 0);
int tc_forward_blocks(const TcPlan*, int first, int last, cudaStream_t s, StageTimer* t = nullptr, const int* skip = nullptr,
                      int64_t skip_stride = 0);
// `ctl` (Train): one extra block per stream of the first kernel assesses the prediction the backward belongs to, beside the
// kernel's own work; the update that follows reads the outcome.
int tc_backward(const TcPlan*, cudaStream_t s, StageTimer* t = nullptr, const int* skip = nullptr, int64_t skip_stride = 0,
                const TrainCtl* ctl = nullptr);

}  // namespace st
