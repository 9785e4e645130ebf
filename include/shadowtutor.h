/*
 * shadowtutor.h — C ABI of the key-frame partial-distillation step (ShadowTutor, ICPP'20).
 *
 * The library implements the body of the server loop (Algorithm 3) minus the teacher
 * network and the transport: the teacher's per-pixel class logits are reduced to a
 * one-byte label map, the student's trainable back part (its "head") is trained against
 * those labels for K optimisation steps over the cached output of the frozen front part
 * (Algorithm 1's loop body; partial distillation, Section 4.2), the trained subset is
 * packed for the client (UpdatedPart, Algorithm 3) and student/teacher agreement is
 * measured as mean IoU (Section 3.2).
 *
 * Conventions that hold for every entry point
 *   - Plain C types only.  "device" = pointer into CUDA device memory of the current
 *     device; "host" = ordinary (preferably pinned) host memory.  Where a parameter says
 *     "host or device", the library looks the pointer up and copies from/to host memory
 *     on the context's CUDA stream itself.
 *   - The caller owns every buffer it passes.  The library reads or writes it only on the
 *     context's CUDA stream during work enqueued by that call; it keeps no reference
 *     afterwards.  Inputs must stay alive until the stream has passed that work.
 *   - No pointer needs more than the alignment of its element type (one byte for label maps and masks, four
 *     for fp32 tensors); 16-byte aligned, contiguous buffers take the fastest paths.
 *   - Calls enqueue work on `cuda_stream` and return.  Only calls with a host out-value
 *     (`st_pack_updated_params` with a host destination, `st_agreement` unless its `miou` is a
 *     device pointer, `st_read_tensor`) wait for the stream.
 *   - Errors are status codes; nothing aborts, throws or traps.  `st_last_error` gives a
 *     text for the most recent failure on that context (or, with NULL, of the last failed
 *     `st_init_head` on this thread).  All shapes are validated on the host before any
 *     kernel is launched.
 *   - A context is bound to the device that was current in `st_init_head`, and must be
 *     used from one host thread at a time.
 */
#ifndef SHADOWTUTOR_H_
#define SHADOWTUTOR_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define ST_API __attribute__((visibility("default")))
#else
#define ST_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct st_ctx st_ctx; /* opaque, library-owned */

typedef enum st_status {
    ST_OK = 0,
    ST_ERR_INVALID_ARG = 1,      /* NULL where a pointer is required, bad index, bad shape, label >= n_classes */
    ST_ERR_BAD_STATE = 2,        /* call order: features/labels missing for the stream */
    ST_ERR_BUFFER_TOO_SMALL = 3, /* destination capacity below the required size */
    ST_ERR_UNSUPPORTED = 4,      /* a shape the kernels do not cover (see st_init_head) */
    ST_ERR_OOM = 5,              /* device or host allocation failed */
    ST_ERR_CUDA = 6              /* a CUDA call or kernel reported an error */
} st_status;

/* Description of S independent heads of identical shape (one per client video stream). */
typedef struct st_head_desc {
    int32_t n_streams;      /* S >= 1: independent heads, each with its own features/labels/parameters */
    int32_t c_in;           /* channels of the frozen part's output */
    int32_t c_hidden;       /* 0: head = 1x1 conv c_in -> n_classes;
                               >0: 3x3 conv c_in -> c_hidden (zero pad 1) + ReLU, then 1x1 conv -> n_classes */
    int32_t n_classes;      /* 2..255 (labels are one byte, Table 4) */
    int32_t feat_h, feat_w; /* spatial size of the frozen part's output */
    int32_t up;             /* frame = feature map * up, bilinear (half-pixel centres); must be 4 */
    int32_t gemm_precision; /* 0: fp32 FMA convolutions; 1: bf16 operands on tensor cores, fp32 accumulate */
    float lr;               /* learning rate of OptimStep */
    float momentum;         /* heavy-ball momentum; 0 = plain gradient descent (optimizer 0 only) */
    void *cuda_stream;      /* cudaStream_t on which all work is enqueued (NULL = default stream) */
    int32_t optimizer;      /* 0: gradient descent with momentum (Section 4.1.4); 1: Adam (the optimiser of the
                               paper's experiments, Section 5.2) */
    double adam_beta1;      /* Adam's decay rates and epsilon; the paper does not state them.  0 selects the */
    double adam_beta2;      /*   constants of the published algorithm: 0.9, 0.999, 1e-8.                       */
    double adam_eps;        /* epsilon is added to the root of the bias-corrected second moment */
    int32_t object_weight;  /* loss weighting against class imbalance (Section 5.2): the cross-entropy of pixels near
                               and within non-background objects is scaled by this factor (5 in the paper; whole
                               numbers 2..5; 0 or 1 = off, plain mean cross-entropy).  The normaliser stays the
                               number of pixels.  Needs n_classes <= 32. */
    int32_t object_radius;  /* what counts as "near" (the paper gives no distance): within this many rows and
                               columns of a pixel whose label is not the background class; 0..64 */
    int32_t background_class; /* the background class, below n_classes */
    /* The back part as a stack of student blocks (Section 5.2: the blocks SB5 and SB6, each fed by the block before
       it and by a feature map of the frozen front part concatenated to its input), with the freeze boundary of partial
       distillation (Section 4.2) anywhere inside it.  The paper's drawing of a block is not in its text; reading
       taken: block b = 3x3 convolution with zero padding 1 over the concatenation (channels of the previous block's
       output, or of the frozen part's output for block 0, first; then the channels of skip input b), followed by ReLU;
       blocks and skip inputs share the resolution feat_h x feat_w; the classifier is a 1x1 convolution. */
    int32_t n_blocks;         /* 0: the head given by c_hidden.  1..ST_MAX_BLOCKS: this many blocks, then the classifier
                                 (c_hidden must be 0, gemm_precision 1) */
    int32_t block_c_out[2];   /* output channels of each block: multiples of 64, at most 256 */
    int32_t block_c_skip[2];  /* channels of each block's skip input (0: none): multiples of 64 */
    int32_t first_trained;    /* blocks before this index keep their parameters: no gradient is formed for them and none
                                 is passed back into them.  0 trains every block, n_blocks the classifier alone. */
} st_head_desc;
#define ST_MAX_BLOCKS 2

/* Number of fp32 values in one head's packed parameter buffer:
 * per layer in forward order, weight [Cout][Cin][kh][kw] then bias [Cout]. */
ST_API size_t st_param_count(int32_t c_in, int32_t c_hidden, int32_t n_classes);

/* The same for any description: *n_all (may be NULL) = values of all layers of the back part, which st_init_head
 * takes; *n_trained (may be NULL) = values of the layers behind the freeze boundary, which UpdatedPart carries.  For a
 * head without blocks both equal st_param_count.  ST_ERR_INVALID_ARG on a NULL or inconsistent description. */
ST_API st_status st_head_param_counts(const st_head_desc *desc, size_t *n_all, size_t *n_trained);

/*
 * st_init_head — create the server-side copy of the student's trainable part
 * (Algorithm 3 starts from the pre-trained student; Section 4.2 fixes which part is trained).
 *   desc         host; copied.
 *   init_params  host or device; S packed buffers back to back (S * st_param_count floats),
 *                layout as above; copied into fp32 master parameters.  Momentum starts at 0.
 *   out          host; receives the context.
 * Allocates all device state (parameters, momentum, caches, scratch) for S streams.
 * ST_ERR_UNSUPPORTED: up != 4; with gemm_precision 1: c_in or c_hidden not a multiple of
 * 64, c_hidden > 256, or n_classes > 32.
 */
ST_API st_status st_init_head(const st_head_desc *desc, const float *init_params, st_ctx **out);

/*
 * st_set_frozen_features — cache the frozen front part's output for one key frame.
 * The frozen layers' outputs do not change across the K steps (Section 4.2), so they are
 * stored once in the layout the head's GEMMs read (bf16 [h][w][c_in] with
 * gemm_precision 1, fp32 [c_in][h][w] otherwise).
 *   stream    0 <= stream < S.
 *   feat_chw  host or device; fp32 [c_in][feat_h][feat_w], contiguous.
 */
ST_API st_status st_set_frozen_features(st_ctx *ctx, int32_t stream, const float *feat_chw);

/*
 * st_set_skip_features — cache the skip input of one block for one key frame: the feature map of the frozen front
 * part that Section 5.2 concatenates to the block's input (SB2's output for SB5, SB1's for SB6), already at the
 * resolution feat_h x feat_w.  Like the frozen part's output it does not change while the back part is trained.
 *   block     0 <= block < n_blocks, a block with block_c_skip > 0.
 *   feat_chw  host or device; fp32 [block_c_skip][feat_h][feat_w], contiguous.
 */
ST_API st_status st_set_skip_features(st_ctx *ctx, int32_t stream, int32_t block, const float *feat_chw);

/*
 * st_teacher_labels — pseudo-label of the key frame (Algorithm 3: label <- Forward(teacher)):
 * label[y][x] = argmax_c logits[c][y][x], lowest class index on ties; one byte per pixel.
 *   logits_chw  host or device; fp32 [n_classes][H][W], H = feat_h*up, W = feat_w*up.
 *   labels_out  host or device, or NULL; uint8 [H][W].  A copy is always kept in the context
 *               as the training target of `stream`.
 */
ST_API st_status st_teacher_labels(st_ctx *ctx, int32_t stream, const float *logits_chw, uint8_t *labels_out);

/*
 * st_prefetch_key_frame / st_use_prefetched_key_frame — bring the next key frame's inputs to the device while the
 * current key frame is still being trained.  In the server loop (Algorithm 3) a key frame arrives from the client
 * while the previous one may still be in Train; the copy of its inputs from host memory is by far the longest part
 * of handling it (136 MB against 0.35 ms of kernels at 720p), so it runs on a CUDA stream of the library's own, beside
 * the context's stream.
 *   st_prefetch_key_frame   feat_chw, logits_chw: host (pinned memory makes the copy asynchronous) or device, shapes
 *                           as in st_set_frozen_features / st_teacher_labels.  Returns at once; the buffers must stay
 *                           alive and unchanged until st_use_prefetched_key_frame for this stream has returned and the
 *                           context's stream has passed its work.  A second prefetch for the same stream before the
 *                           first is used replaces it.  Device memory for one key frame's inputs is allocated per
 *                           stream on first use (ST_ERR_OOM / ST_ERR_CUDA on failure).
 *   st_use_prefetched_key_frame   makes the prefetched inputs the current key frame of `stream`: the context's stream
 *                           waits for the copy (the host does not), then runs what st_set_frozen_features and
 *                           st_teacher_labels run.  labels_out as in st_teacher_labels.  ST_ERR_BAD_STATE if nothing
 *                           was prefetched for the stream.
 * Everything else about the two inputs is as documented for the two plain calls.
 */
ST_API st_status st_prefetch_key_frame(st_ctx *ctx, int32_t stream, const float *feat_chw, const float *logits_chw);
ST_API st_status st_use_prefetched_key_frame(st_ctx *ctx, int32_t stream, uint8_t *labels_out);

/* Install an existing label map (uint8 [H][W], host or device) as the training target. */
ST_API st_status st_set_labels(st_ctx *ctx, int32_t stream, const uint8_t *labels);

/*
 * st_distill_step — n_steps iterations of Algorithm 1's loop body on all S streams:
 * head forward, bilinear x4 upsample, mean per-pixel softmax cross-entropy against the
 * stored labels (Section 5.2), gradients of the head only (PartialBackward, Section 4.2),
 * OptimStep with the descriptor's optimiser (gradient descent with momentum, or Adam).  With object_weight > 1 the
 * cross-entropy is the weighted one of Section 5.2.
 *   n_steps   1..64.
 *   loss_out  host or device, or NULL; fp32 [S][n_steps]: loss of each step's forward.
 *   conf_out  host or device, or NULL; int64 [S][n_steps][C][C]: conf[label][prediction] of the
 *             forward that produced that step's loss (the prediction before that step's update).
 * ST_ERR_BAD_STATE if a stream has no features or labels yet.
 * Labels >= n_classes are skipped (no loss, no gradient) and make the call that finds them
 * return ST_ERR_INVALID_ARG at its next synchronising point (`st_agreement`, `st_read_tensor`).
 */
ST_API st_status st_distill_step(st_ctx *ctx, int32_t n_steps, float *loss_out, int64_t *conf_out);

/*
 * st_train_key_frame — Train(student, frame, label), the whole of Algorithm 1, on all S streams, each
 * stream with its own control flow, decided on the device:
 *     prediction <- Forward(student, frame); best_metric <- ComputeMetric(prediction, label); best_student <- student
 *     if best_metric < THRESHOLD: for i = 1 .. MAX_UPDATES:
 *         one iteration as in st_distill_step; prediction <- Forward; metric <- ComputeMetric(prediction, label)
 *         if metric > best_metric: best_metric, best_student <- metric, student
 *         if metric > THRESHOLD: break
 * The metric is the mean IoU of Section 3.2 between the student's mask (arg-max of the upsampled logits) and the
 * stored labels; THRESHOLD and MAX_UPDATES are the algorithm's two parameters (Section 4.1.3).
 * On return the context's parameters are best_student (Algorithm 3: student, metric <- Train(...)); the momentum
 * buffer is optimiser state and keeps its latest value.
 *   threshold        THRESHOLD.
 *   max_updates      MAX_UPDATES, 0..63.
 *   n_updates_out    host or device, or NULL; int32 [S]: optimisation steps taken before the loop ended.
 *   best_metric_out  host or device, or NULL; double [S]: best_metric.
 *   metric_out       host or device, or NULL; double [S][max_updates + 1]: metric of the prediction after i updates;
 *                    -1 for predictions the algorithm did not make (i > n_updates).
 *   loss_out         host or device, or NULL; fp32 [S][max_updates + 1]: loss of the prediction after i updates,
 *                    meaningful for i <= n_updates.
 *   conf_out         host or device, or NULL; int64 [S][max_updates + 1][C][C]: confusion matrix of each prediction,
 *                    meaningful for i <= n_updates.
 * The work is enqueued on the context's stream (a replayed CUDA graph per (max_updates, threshold)); the call waits
 * for the stream only if an output pointer is host memory.  The launches of all max_updates iterations are always
 * enqueued; once a stream's loop has ended, the blocks of its later kernels return at once (with gemm_precision 0
 * the fp32 convolutions still run and only the update is suppressed).
 * ST_ERR_BAD_STATE if a stream has no features or labels yet; ST_ERR_INVALID_ARG for max_updates outside 0..63 or a
 * NaN threshold.
 */
ST_API st_status st_train_key_frame(st_ctx *ctx, double threshold, int32_t max_updates, int32_t *n_updates_out,
                                    double *best_metric_out, double *metric_out, float *loss_out, int64_t *conf_out);

/*
 * st_pack_updated_params — UpdatedPart(student) (Algorithm 3; Table 4 sizes are fp32):
 * the current values of every trainable tensor of `stream`, fp32 little-endian, per layer in
 * forward order weight [Cout][Cin][kh][kw] then bias [Cout]; no header, no padding.
 *   dst           host or device.
 *   dst_capacity  bytes available at dst; ST_ERR_BUFFER_TOO_SMALL if below the packed size.
 *   nbytes        host, may be NULL; receives the packed size (also on BUFFER_TOO_SMALL).
 * Momentum is not part of the buffer.  Feeding the buffer back to st_init_head reproduces
 * the parameters bit for bit.
 */
ST_API st_status st_pack_updated_params(st_ctx *ctx, int32_t stream, void *dst, size_t dst_capacity, size_t *nbytes);

/*
 * st_apply_update — ApplyUpdate(student, student_diff) (Algorithm 4): install a buffer produced by
 * st_pack_updated_params as the parameters of `stream`.  The updated part carries values, not differences, so the
 * trainable tensors are simply replaced; the momentum buffer is left as it is.  This is what the client does with
 * the server's reply, and what a server does to move a student between contexts.
 *   src     host or device; the packed buffer (layout of st_pack_updated_params).
 *   nbytes  its size; must equal st_param_count * 4, else ST_ERR_INVALID_ARG.
 * pack -> apply -> pack reproduces the buffer bit for bit.
 */
ST_API st_status st_apply_update(st_ctx *ctx, int32_t stream, const void *src, size_t nbytes);

/*
 * st_student_mask — prediction of the current student at frame resolution:
 * argmax over classes of the upsampled head logits (fresh forward of the current parameters).
 *   mask_out  host or device; uint8 [H][W].
 */
ST_API st_status st_student_mask(st_ctx *ctx, int32_t stream, uint8_t *mask_out);

/*
 * st_agreement — ComputeMetric (Algorithm 1): confusion matrix and mean IoU
 * (Section 3.2: IoU_c = |pred_c ∩ label_c| / |pred_c ∪ label_c|, averaged over the classes
 * present in the label).
 *   pred   host or device uint8 [H][W], or NULL = the current student's mask (fresh forward).
 *   label  host or device uint8 [H][W], or NULL = the stored teacher labels of `stream`.
 *   conf   host or device, or NULL; int64 [C][C], conf[l][q] = #pixels with label l and prediction q.
 *   miou   host or device, or NULL; mean IoU in double.
 * Pixels whose label or prediction is >= n_classes are skipped and the call returns
 * ST_ERR_INVALID_ARG (the counts of the valid pixels are still delivered).
 * Waits for the stream, unless `miou` points to device memory: then the value is written there by
 * work enqueued on the stream, the call returns at once, and skipped pixels are reported by the next
 * call that does wait.
 */
ST_API st_status st_agreement(st_ctx *ctx, int32_t stream, const uint8_t *pred, const uint8_t *label,
                       int64_t *conf, double *miou);

/* Intermediate tensors of the most recent step, for verification. */
typedef enum st_tensor {
    ST_TENSOR_LOGITS = 0,      /* z, fp32 [C][h][w]: head output of the last forward (after st_distill_step: of its last
                                  step, before that step's update; after st_train_key_frame: of the student the call
                                  leaves behind, computed when asked for) */
    ST_TENSOR_LOGIT_GRAD = 1,  /* dz, fp32 [C][h][w]: gradient of the mean loss w.r.t. z */
    ST_TENSOR_PARAM_GRAD = 2,  /* fp32, packed order: gradient applied by the last update */
    ST_TENSOR_MOMENTUM = 3,    /* fp32, packed order */
    ST_TENSOR_HIDDEN = 4,      /* fp32 [c_hidden][h][w]: ReLU output of the 3x3 layer (two-layer head; last block of a stack) */
    ST_TENSOR_HIDDEN_GRAD = 5, /* fp32 [c_hidden][h][w]: gradient w.r.t. the hidden activation (after the ReLU mask) */
    ST_TENSOR_FEATURES = 6,    /* fp32 [c_in][h][w]: the cached features as the GEMMs see them */
    ST_TENSOR_HIDDEN_FIRST = 7,      /* a stack of two blocks: output of block 0, fp32 [block_c_out[0]][h][w] */
    ST_TENSOR_HIDDEN_GRAD_FIRST = 8  /* ... and the gradient with respect to it (after the ReLU mask) */
} st_tensor;

/*
 * st_read_tensor — copy one intermediate tensor of `stream` to host memory as fp32 in the
 * planar layout listed above (converted from the internal layout/precision).
 *   dst_host      host; capacity in bytes; *nbytes (may be NULL) receives the size.
 * Waits for the stream.
 */
ST_API st_status st_read_tensor(st_ctx *ctx, int32_t stream, st_tensor which, float *dst_host,
                         size_t dst_capacity, size_t *nbytes);

/*
 * st_profile_step — time the kernels of the step one by one.  Runs n_steps ordinary steps of
 * Algorithm 1's loop body (they do update the parameters) without graph replay, with a CUDA event
 * recorded on the context's stream after every kernel, and returns the mean time per launch.
 * Every kernel except the parameter update is launched 8 times back to back between two events (its
 * result does not depend on how often it runs), so that the launch gap of a 10-microsecond kernel
 * does not dominate its figure; the update is launched once and its figure includes that gap.
 *   n_stages   host; receives the number of kernels in one step (<= ST_MAX_STAGES).
 *   ms_out     host float[ST_MAX_STAGES]; mean milliseconds per launch of each kernel, in launch order.
 *   names_out  host const char*[ST_MAX_STAGES]; static strings naming the kernels.
 * Waits for the stream after every step.  A measuring aid, not part of the method.
 */
#define ST_MAX_STAGES 12
ST_API st_status st_profile_step(st_ctx *ctx, int32_t n_steps, int32_t *n_stages, float *ms_out,
                                 const char **names_out);

/*
 * st_measure_arithmetic_peaks — what this device sustains in plain fp32 multiply-adds and in exp2 evaluations
 * (special-function unit), measured with two register-only kernels of a few hundred microseconds each.  These
 * are the ceilings of the fused upsample + cross-entropy kernel (ComputeLoss and the start of PartialBackward
 * of Algorithm 1), which is bound by arithmetic, not by memory.  A measuring aid, not part of the method.
 *   cuda_stream  cudaStream_t on which the kernels run (NULL = default stream).
 *   fma_tflops   host, may be NULL; 10^12 fp32 operations per second, a multiply-add counted as two.
 *   ex2_tops     host, may be NULL; 10^12 exp2 evaluations per second.
 * Allocates four bytes of device memory for the duration of the call and waits for the stream.
 */
ST_API st_status st_measure_arithmetic_peaks(void *cuda_stream, double *fma_tflops, double *ex2_tops);

/*
 * st_agreement_noalloc — confusion matrix and mean IoU of two masks without any allocation.
 * (The paper has no counterpart: this entry point exists for the sake of callers, not of the method.)
 *
 * Some callers cannot allocate device memory: a process that gave all of HBM to its own pool at
 * start-up, a latency-critical loop that cannot take the device-wide synchronisation that
 * cudaMalloc/cudaFree imply, or code running while allocation calls are forbidden.  st_agreement
 * needs a context and creating one allocates; this variant takes no context and calls no cudaMalloc,
 * cudaFree or any allocating routine.  Its counters live in a fixed __device__ array inside the
 * library (about 33 KB, held by every GPU that loads the library until the process exits).
 *
 *   pred, label  device; uint8 [n_pixels] each.  Pixels with a value >= n_classes are skipped
 *                (and, unlike st_agreement, not reported: this call never waits for the stream).
 *   n_classes    2..ST_NOALLOC_MAX_CLASSES; larger values return ST_ERR_UNSUPPORTED.
 *   cuda_stream  cudaStream_t on which the work is enqueued (NULL = default stream).
 *   conf_out     device; int64 [n_classes][n_classes], conf[l][q] = #pixels with label l, prediction q.
 *   miou_out     device; one double (Section 3.2's mean IoU over the classes present in the label).
 * Returns after enqueueing; results are valid once the stream has passed the work.
 * The first call on each device looks up the address of the internal array
 * (cudaGetSymbolAddress, with that device current); make that first call before any stream capture.
 * All calls share the internal array, which is cleared at the start of each call: calls whose work
 * overlaps on the GPU (different streams without ordering between them) race and give wrong counts.
 * Errors: ST_ERR_INVALID_ARG (NULL pointer, n_classes < 2, n_pixels < 0), ST_ERR_UNSUPPORTED, ST_ERR_CUDA.
 */
#define ST_NOALLOC_MAX_CLASSES 64
ST_API st_status st_agreement_noalloc(const uint8_t *pred, const uint8_t *label, int64_t n_pixels,
                                      int32_t n_classes, void *cuda_stream, int64_t *conf_out,
                                      double *miou_out);

/* ---- host-side pieces around the step: no device work, callable without a GPU ------------------------ */

/*
 * st_next_stride — NextStride (Algorithm 2): distance to the next key frame from the current stride and the
 * student's metric in [0, 1].  ratio = metric / THRESHOLD below the threshold (the line through (0,0) and
 * (THRESHOLD,1)), (metric - 2 THRESHOLD + 1) / (1 - THRESHOLD) from the threshold on (the line through
 * (THRESHOLD,1) and (1,2)); stride <- ratio * stride, cut to whole frames, clamped to [min_stride, max_stride].
 */
ST_API int32_t st_next_stride(int32_t stride, double metric, double threshold, int32_t min_stride, int32_t max_stride);

/*
 * st_client_schedule — the key frames the client's loop (Algorithm 4) picks among n_frames frames.  The first
 * frame is a key frame.  The reply to a key frame (updated part, metric) is applied min(delay, MIN_STRIDE) frames
 * after it: when it has arrived, or when the client stops to wait for it (Section 4.3).  The stride is recomputed with
 * st_next_stride at that moment and counts from the key frame, so the next key frame is NextStride(stride, metric)
 * frames after the last one, whatever the delay.
 *   metrics       host; metrics[j] = metric returned for the j-th key frame; n_metrics entries.
 *   delay         frames until a reply is complete, >= 1 (it decides when an update is applied, not where the key
 *                 frames fall).
 *   key_frames    host, capacity entries; receives the frame indices.
 *   n_key_frames  host; receives their number (also when capacity is too small: ST_ERR_BUFFER_TOO_SMALL).
 * ST_ERR_INVALID_ARG: bad parameters (threshold must lie strictly between 0 and 1), or fewer metrics than key frames.
 */
ST_API st_status st_client_schedule(int64_t n_frames, const double *metrics, int64_t n_metrics, double threshold,
                                    int32_t min_stride, int32_t max_stride, int32_t delay, int64_t *key_frames,
                                    int64_t capacity, int64_t *n_key_frames);

/* Latencies of Section 4.4 (Table 1), in seconds. */
typedef struct st_latencies {
    double t_si;  /* student inference */
    double t_sd;  /* one student distillation step */
    double t_ti;  /* teacher inference */
    double t_net; /* network latency of one key frame */
} st_latencies;

/*
 * st_throughput_bounds — frames per second the system can reach at least and at most (Section 4.4):
 *   lower = MIN_STRIDE / (MIN_STRIDE t_si + MAX_UPDATES t_sd + t_ti + t_net)
 *   upper = MAX_STRIDE / ((MAX_STRIDE - MIN_STRIDE) t_si + max(MIN_STRIDE t_si, t_net + t_ti))
 * st_traffic_bounds — networked data per second, in the unit of s_net (data per key frame) per second:
 *   lower = s_net / (MAX_STRIDE t_si + MAX_UPDATES t_sd + t_ti + t_net)
 *   upper = s_net / max(MIN_STRIDE t_si, t_net + t_ti)
 * st_choose_max_updates — Section 5.3's rule: the largest MAX_UPDATES whose throughput lower bound is still
 * above fps_floor; -1 if none is (or on bad arguments).
 * Output pointers are host and may be NULL.  ST_ERR_INVALID_ARG on non-positive t_si, negative values or
 * min_stride > max_stride.
 */
ST_API st_status st_throughput_bounds(const st_latencies *lat, int32_t min_stride, int32_t max_stride,
                                      int32_t max_updates, double *fps_lower, double *fps_upper);
ST_API st_status st_traffic_bounds(const st_latencies *lat, double s_net, int32_t min_stride, int32_t max_stride,
                                   int32_t max_updates, double *per_second_lower, double *per_second_upper);
ST_API int32_t st_choose_max_updates(const st_latencies *lat, int32_t min_stride, int32_t max_stride, double fps_floor);

/* Number of kernels this library has launched on the context so far. */
ST_API int64_t st_launch_count(const st_ctx *ctx);

ST_API void st_destroy(st_ctx *ctx);
ST_API const char *st_last_error(const st_ctx *ctx);
ST_API const char *st_status_name(st_status s);

#ifdef __cplusplus
}
#endif
#endif /* SHADOWTUTOR_H_ */
