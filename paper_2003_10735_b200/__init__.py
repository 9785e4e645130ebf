"""Thin Python binding of the key-frame partial-distillation library (libshadowtutor.so).

Argument marshalling only: every function has the name and the meaning of the C entry
point declared in ``include/shadowtutor.h`` and forwards pointers and sizes to it.  Tensors
may be ``torch`` tensors (CUDA or CPU) or ``numpy`` arrays; they must be contiguous and of
the dtype the C interface states.  No arithmetic of the method happens here, and there is
no fallback: if the CUDA library has not been built the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libshadowtutor.so")

ST_OK = 0
ST_ERR_INVALID_ARG = 1
ST_ERR_BAD_STATE = 2
ST_ERR_BUFFER_TOO_SMALL = 3
ST_ERR_UNSUPPORTED = 4
ST_ERR_OOM = 5
ST_ERR_CUDA = 6

ST_TENSOR_LOGITS = 0
ST_TENSOR_LOGIT_GRAD = 1
ST_TENSOR_PARAM_GRAD = 2
ST_TENSOR_MOMENTUM = 3
ST_TENSOR_HIDDEN = 4
ST_TENSOR_HIDDEN_GRAD = 5
ST_TENSOR_FEATURES = 6
ST_TENSOR_HIDDEN_FIRST = 7
ST_TENSOR_HIDDEN_GRAD_FIRST = 8
ST_MAX_BLOCKS = 2

EXPORTED = [
    "st_param_count", "st_init_head", "st_set_frozen_features", "st_teacher_labels", "st_set_labels",
    "st_distill_step", "st_pack_updated_params", "st_student_mask", "st_agreement", "st_read_tensor",
    "st_launch_count", "st_destroy", "st_last_error", "st_status_name", "st_profile_step",
    "st_agreement_noalloc", "st_train_key_frame", "st_next_stride", "st_client_schedule", "st_throughput_bounds",
    "st_traffic_bounds", "st_choose_max_updates", "st_apply_update", "st_measure_arithmetic_peaks",
    "st_prefetch_key_frame", "st_use_prefetched_key_frame", "st_head_param_counts", "st_set_skip_features",
]
ST_NOALLOC_MAX_CLASSES = 64
ST_MAX_STAGES = 12


class st_head_desc(ctypes.Structure):
    _fields_ = [
        ("n_streams", ctypes.c_int32), ("c_in", ctypes.c_int32), ("c_hidden", ctypes.c_int32),
        ("n_classes", ctypes.c_int32), ("feat_h", ctypes.c_int32), ("feat_w", ctypes.c_int32),
        ("up", ctypes.c_int32), ("gemm_precision", ctypes.c_int32),
        ("lr", ctypes.c_float), ("momentum", ctypes.c_float), ("cuda_stream", ctypes.c_void_p),
        ("optimizer", ctypes.c_int32), ("adam_beta1", ctypes.c_double), ("adam_beta2", ctypes.c_double),
        ("adam_eps", ctypes.c_double), ("object_weight", ctypes.c_int32), ("object_radius", ctypes.c_int32),
        ("background_class", ctypes.c_int32),
        ("n_blocks", ctypes.c_int32), ("block_c_out", ctypes.c_int32 * 2), ("block_c_skip", ctypes.c_int32 * 2),
        ("first_trained", ctypes.c_int32),
    ]


class StError(RuntimeError):
    def __init__(self, status: int, name: str, message: str):
        super().__init__(f"{name}: {message}")
        self.status = status
        self.status_name = name


_lib = None


def load_library() -> ctypes.CDLL:
    """Load libshadowtutor.so (built by ``python -m paper_2003_10735_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2003_10735_b200.build` "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    lib.st_param_count.restype = ctypes.c_size_t
    lib.st_param_count.argtypes = [i32, i32, i32]
    lib.st_head_param_counts.restype = ctypes.c_int
    lib.st_head_param_counts.argtypes = [ctypes.POINTER(st_head_desc), ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
    lib.st_set_skip_features.restype = ctypes.c_int
    lib.st_set_skip_features.argtypes = [vp, i32, i32, vp]
    lib.st_init_head.restype = ctypes.c_int
    lib.st_init_head.argtypes = [ctypes.POINTER(st_head_desc), vp, ctypes.POINTER(vp)]
    lib.st_set_frozen_features.restype = ctypes.c_int
    lib.st_set_frozen_features.argtypes = [vp, i32, vp]
    lib.st_teacher_labels.restype = ctypes.c_int
    lib.st_teacher_labels.argtypes = [vp, i32, vp, vp]
    lib.st_prefetch_key_frame.restype = ctypes.c_int
    lib.st_prefetch_key_frame.argtypes = [vp, i32, vp, vp]
    lib.st_use_prefetched_key_frame.restype = ctypes.c_int
    lib.st_use_prefetched_key_frame.argtypes = [vp, i32, vp]
    lib.st_set_labels.restype = ctypes.c_int
    lib.st_set_labels.argtypes = [vp, i32, vp]
    lib.st_distill_step.restype = ctypes.c_int
    lib.st_distill_step.argtypes = [vp, i32, vp, vp]
    lib.st_train_key_frame.restype = ctypes.c_int
    lib.st_train_key_frame.argtypes = [vp, ctypes.c_double, i32, vp, vp, vp, vp, vp]
    dbl = ctypes.c_double
    lib.st_next_stride.restype = i32
    lib.st_next_stride.argtypes = [i32, dbl, dbl, i32, i32]
    lib.st_client_schedule.restype = ctypes.c_int
    lib.st_client_schedule.argtypes = [i64, vp, i64, dbl, i32, i32, i32, vp, i64, ctypes.POINTER(i64)]
    lib.st_throughput_bounds.restype = ctypes.c_int
    lib.st_throughput_bounds.argtypes = [vp, i32, i32, i32, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
    lib.st_traffic_bounds.restype = ctypes.c_int
    lib.st_traffic_bounds.argtypes = [vp, dbl, i32, i32, i32, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
    lib.st_choose_max_updates.restype = i32
    lib.st_choose_max_updates.argtypes = [vp, i32, i32, dbl]
    lib.st_apply_update.restype = ctypes.c_int
    lib.st_apply_update.argtypes = [vp, i32, vp, ctypes.c_size_t]
    lib.st_pack_updated_params.restype = ctypes.c_int
    lib.st_pack_updated_params.argtypes = [vp, i32, vp, ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]
    lib.st_student_mask.restype = ctypes.c_int
    lib.st_student_mask.argtypes = [vp, i32, vp]
    lib.st_agreement.restype = ctypes.c_int
    lib.st_agreement.argtypes = [vp, i32, vp, vp, vp, vp]
    lib.st_read_tensor.restype = ctypes.c_int
    lib.st_read_tensor.argtypes = [vp, i32, ctypes.c_int, vp, ctypes.c_size_t, ctypes.POINTER(ctypes.c_size_t)]
    lib.st_profile_step.restype = ctypes.c_int
    lib.st_profile_step.argtypes = [vp, i32, ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_float),
                                    ctypes.POINTER(ctypes.c_char_p)]
    lib.st_agreement_noalloc.restype = ctypes.c_int
    lib.st_agreement_noalloc.argtypes = [vp, vp, i64, i32, vp, vp, vp]
    lib.st_measure_arithmetic_peaks.restype = ctypes.c_int
    lib.st_measure_arithmetic_peaks.argtypes = [vp, ctypes.POINTER(dbl), ctypes.POINTER(dbl)]
    lib.st_launch_count.restype = i64
    lib.st_launch_count.argtypes = [vp]
    lib.st_destroy.restype = None
    lib.st_destroy.argtypes = [vp]
    lib.st_last_error.restype = ctypes.c_char_p
    lib.st_last_error.argtypes = [vp]
    lib.st_status_name.restype = ctypes.c_char_p
    lib.st_status_name.argtypes = [ctypes.c_int]
    _lib = lib
    return lib


# ---------------------------------------------------------------------------- marshalling
_NP_OF = {"float32": np.float32, "float64": np.float64, "uint8": np.uint8, "int32": np.int32, "int64": np.int64}


def _ptr(buf, dtype: str, min_elems: int, what: str) -> Optional[int]:
    """Address of a contiguous torch tensor / numpy array of the given dtype, or None."""
    if buf is None:
        return None
    if isinstance(buf, np.ndarray):
        if buf.dtype != _NP_OF[dtype] or not buf.flags.c_contiguous:
            raise TypeError(f"{what}: need a C-contiguous {dtype} array, got {buf.dtype}")
        if buf.size < min_elems:
            raise ValueError(f"{what}: {buf.size} elements, need {min_elems}")
        return buf.ctypes.data
    if hasattr(buf, "data_ptr"):
        if str(buf.dtype) != "torch." + dtype or not buf.is_contiguous():
            raise TypeError(f"{what}: need a contiguous {dtype} tensor, got {buf.dtype}")
        if buf.numel() < min_elems:
            raise ValueError(f"{what}: {buf.numel()} elements, need {min_elems}")
        return buf.data_ptr()
    raise TypeError(f"{what}: expected a torch tensor or numpy array")


class _Ctx:
    """Handle of an st_ctx plus the shape facts needed to size buffers."""

    def __init__(self, handle, desc: st_head_desc):
        self.handle = handle
        self.desc = desc
        self.S, self.C = desc.n_streams, desc.n_classes
        self.p = desc.feat_h * desc.feat_w
        self.P = self.p * desc.up * desc.up
        # n_params: the values UpdatedPart carries (the trained layers); n_params_all: every layer of the back part
        self.n_params_all, self.n_params = st_head_param_counts(desc)

    def __del__(self):
        try:
            st_destroy(self)
        except Exception:
            pass


def _check(status: int, ctx: Optional[_Ctx]) -> None:
    if status == ST_OK:
        return
    lib = load_library()
    msg = lib.st_last_error(ctx.handle if ctx is not None else None)
    raise StError(status, lib.st_status_name(status).decode(), (msg or b"").decode())


# ---------------------------------------------------------------------------- entry points
def st_param_count(c_in: int, c_hidden: int, n_classes: int) -> int:
    return int(load_library().st_param_count(c_in, c_hidden, n_classes))


def st_head_param_counts(desc: st_head_desc):
    """(values of all layers of the back part, values of the trained layers) for a description."""
    n_all, n_trained = ctypes.c_size_t(0), ctypes.c_size_t(0)
    _status_only(load_library().st_head_param_counts(ctypes.byref(desc), ctypes.byref(n_all), ctypes.byref(n_trained)),
                 "st_head_param_counts")
    return int(n_all.value), int(n_trained.value)


def st_init_head(*, n_streams: int = 1, c_in: int, c_hidden: int = 0, n_classes: int, feat_h: int,
                 feat_w: int, up: int = 4, gemm_precision: int = 0, lr: float = 0.01, momentum: float = 0.0,
                 cuda_stream: int = 0, init_params, optimizer: int = 0, adam_beta1: float = 0.0,
                 adam_beta2: float = 0.0, adam_eps: float = 0.0, object_weight: int = 0, object_radius: int = 0,
                 background_class: int = 0, blocks=(), first_trained: int = 0) -> _Ctx:
    """`blocks`: (c_out, c_skip) per student block in front of the classifier (at most ST_MAX_BLOCKS); `init_params`
    holds every layer of the back part, frozen ones included."""
    lib = load_library()
    if len(blocks) > ST_MAX_BLOCKS:
        raise ValueError(f"at most {ST_MAX_BLOCKS} blocks")
    c_out = (ctypes.c_int32 * 2)(*([b[0] for b in blocks] + [0] * (2 - len(blocks))))
    c_skip = (ctypes.c_int32 * 2)(*([b[1] for b in blocks] + [0] * (2 - len(blocks))))
    desc = st_head_desc(n_streams, c_in, c_hidden, n_classes, feat_h, feat_w, up, gemm_precision,
                        lr, momentum, cuda_stream or None, optimizer, adam_beta1, adam_beta2, adam_eps,
                        object_weight, object_radius, background_class, len(blocks), c_out, c_skip, first_trained)
    counts_all, _ = ctypes.c_size_t(0), None
    if lib.st_head_param_counts(ctypes.byref(desc), ctypes.byref(counts_all), None) != ST_OK:
        counts_all = ctypes.c_size_t(int(lib.st_param_count(c_in, c_hidden, n_classes)))    # the library reports what is wrong
    n = n_streams * int(counts_all.value)
    out = ctypes.c_void_p()
    status = lib.st_init_head(ctypes.byref(desc), _ptr(init_params, "float32", n, "init_params"), ctypes.byref(out))
    _check(status, None)
    return _Ctx(out.value, desc)


def st_set_frozen_features(ctx: _Ctx, stream: int, feat_chw) -> None:
    n = ctx.desc.c_in * ctx.p
    _check(load_library().st_set_frozen_features(ctx.handle, stream, _ptr(feat_chw, "float32", n, "feat_chw")), ctx)


def st_set_skip_features(ctx: _Ctx, stream: int, block: int, feat_chw) -> None:
    n = ctx.desc.block_c_skip[block] * ctx.p if 0 <= block < ST_MAX_BLOCKS else 0
    _check(load_library().st_set_skip_features(ctx.handle, stream, block, _ptr(feat_chw, "float32", n, "feat_chw")), ctx)


def st_teacher_labels(ctx: _Ctx, stream: int, logits_chw, labels_out=None) -> None:
    _check(load_library().st_teacher_labels(ctx.handle, stream, _ptr(logits_chw, "float32", ctx.C * ctx.P, "logits_chw"),
                                            _ptr(labels_out, "uint8", ctx.P, "labels_out")), ctx)


def st_prefetch_key_frame(ctx: _Ctx, stream: int, feat_chw, logits_chw) -> None:
    """Start copying the next key frame's inputs to the device on the library's own copy stream."""
    _check(load_library().st_prefetch_key_frame(ctx.handle, stream, _ptr(feat_chw, "float32", ctx.desc.c_in * ctx.p, "feat_chw"),
                                                _ptr(logits_chw, "float32", ctx.C * ctx.P, "logits_chw")), ctx)


def st_use_prefetched_key_frame(ctx: _Ctx, stream: int, labels_out=None) -> None:
    """Make the prefetched inputs the current key frame of `stream` (feature cache + labels)."""
    _check(load_library().st_use_prefetched_key_frame(ctx.handle, stream, _ptr(labels_out, "uint8", ctx.P, "labels_out")), ctx)


def st_set_labels(ctx: _Ctx, stream: int, labels) -> None:
    _check(load_library().st_set_labels(ctx.handle, stream, _ptr(labels, "uint8", ctx.P, "labels")), ctx)


def st_distill_step(ctx: _Ctx, n_steps: int, loss_out=None, conf_out=None) -> None:
    _check(load_library().st_distill_step(ctx.handle, n_steps,
                                          _ptr(loss_out, "float32", ctx.S * max(n_steps, 0), "loss_out"),
                                          _ptr(conf_out, "int64", ctx.S * max(n_steps, 0) * ctx.C * ctx.C, "conf_out")), ctx)


def st_train_key_frame(ctx: _Ctx, threshold: float, max_updates: int, n_updates=None, best_metric=None,
                       metrics=None, losses=None, conf=None) -> None:
    """Algorithm 1 (Train) on all streams.  Outputs (each optional; numpy array or tensor):
    n_updates int32 [S], best_metric float64 [S], metrics float64 [S][max_updates+1],
    losses float32 [S][max_updates+1], conf int64 [S][max_updates+1][C][C]."""
    n = max(max_updates, 0) + 1
    _check(load_library().st_train_key_frame(
        ctx.handle, float(threshold), int(max_updates), _ptr(n_updates, "int32", ctx.S, "n_updates"),
        _ptr(best_metric, "float64", ctx.S, "best_metric"), _ptr(metrics, "float64", ctx.S * n, "metrics"),
        _ptr(losses, "float32", ctx.S * n, "losses"), _ptr(conf, "int64", ctx.S * n * ctx.C * ctx.C, "conf")), ctx)


def st_pack_updated_params(ctx: _Ctx, stream: int, dst, dst_capacity: Optional[int] = None) -> int:
    """Returns the packed size in bytes."""
    if dst is None:
        cap, addr = 0, None
    else:
        nelem = dst.size if isinstance(dst, np.ndarray) else dst.numel()
        cap = nelem * 4 if dst_capacity is None else dst_capacity
        addr = _ptr(dst, "float32", 0, "dst")
    nbytes = ctypes.c_size_t(0)
    _check(load_library().st_pack_updated_params(ctx.handle, stream, addr, cap, ctypes.byref(nbytes)), ctx)
    return int(nbytes.value)


def st_apply_update(ctx: _Ctx, stream: int, src) -> None:
    """ApplyUpdate (Algorithm 4): install a packed parameter buffer (float32, numpy or tensor) for `stream`."""
    _check(load_library().st_apply_update(ctx.handle, stream, _ptr(src, "float32", ctx.n_params, "src"),
                                          ctx.n_params * 4), ctx)


def st_student_mask(ctx: _Ctx, stream: int, mask_out) -> None:
    _check(load_library().st_student_mask(ctx.handle, stream, _ptr(mask_out, "uint8", ctx.P, "mask_out")), ctx)


def st_agreement(ctx: _Ctx, stream: int, pred=None, label=None, conf=None, miou_out=None):
    """Returns the mean IoU; `conf` (int64 [C][C]) is filled if given.  With `miou_out` (a CUDA float64
    tensor) the mean IoU is written there by work on the context's stream, the call does not wait and
    returns None."""
    if miou_out is not None:
        if not getattr(miou_out, "is_cuda", False) or str(miou_out.dtype) != "torch.float64" or miou_out.numel() < 1:
            raise TypeError("miou_out: need a CUDA float64 tensor with one element")
        _check(load_library().st_agreement(ctx.handle, stream, _ptr(pred, "uint8", ctx.P, "pred"),
                                           _ptr(label, "uint8", ctx.P, "label"),
                                           _ptr(conf, "int64", ctx.C * ctx.C, "conf"),
                                           ctypes.c_void_p(miou_out.data_ptr())), ctx)
        return None
    miou = ctypes.c_double(0.0)
    _check(load_library().st_agreement(ctx.handle, stream, _ptr(pred, "uint8", ctx.P, "pred"),
                                       _ptr(label, "uint8", ctx.P, "label"),
                                       _ptr(conf, "int64", ctx.C * ctx.C, "conf"),
                                       ctypes.cast(ctypes.byref(miou), ctypes.c_void_p)), ctx)
    return float(miou.value)


def st_read_tensor(ctx: _Ctx, stream: int, which: int) -> np.ndarray:
    """Copy of one intermediate tensor as a flat fp32 numpy array (verification only)."""
    lib = load_library()
    nbytes = ctypes.c_size_t(0)
    status = lib.st_read_tensor(ctx.handle, stream, which, None, 0, ctypes.byref(nbytes))
    if nbytes.value == 0:
        _check(status, ctx)
    out = np.empty(nbytes.value // 4, dtype=np.float32)
    _check(lib.st_read_tensor(ctx.handle, stream, which, out.ctypes.data, out.nbytes, ctypes.byref(nbytes)), ctx)
    return out


def st_profile_step(ctx: _Ctx, n_steps: int):
    """[(kernel name, mean milliseconds), ...] of one step, in launch order."""
    n = ctypes.c_int32(0)
    ms = (ctypes.c_float * ST_MAX_STAGES)()
    names = (ctypes.c_char_p * ST_MAX_STAGES)()
    _check(load_library().st_profile_step(ctx.handle, n_steps, ctypes.byref(n), ms, names), ctx)
    return [(names[i].decode(), float(ms[i])) for i in range(n.value)]


def st_agreement_noalloc(pred, label, n_classes: int, cuda_stream: int, conf_out, miou_out) -> None:
    """Confusion matrix and mean IoU of two device uint8 masks for callers that must not allocate
    device memory (no context, no cudaMalloc; the counters live in a fixed array inside the library).
    `conf_out` (int64 [C][C]) and `miou_out` (float64 [1]) are device tensors filled asynchronously on
    `cuda_stream`.  Calls share the internal array: do not let two of them overlap on the GPU."""
    n = pred.numel()
    if label.numel() != n:
        raise ValueError("pred and label differ in size")
    for t, what in ((pred, "pred"), (label, "label"), (conf_out, "conf_out"), (miou_out, "miou_out")):
        if not getattr(t, "is_cuda", False):
            raise TypeError(f"{what}: a CUDA tensor is required")
    if str(miou_out.dtype) != "torch.float64" or miou_out.numel() < 1:
        raise TypeError("miou_out: need a float64 tensor with one element")
    status = load_library().st_agreement_noalloc(
        _ptr(pred, "uint8", n, "pred"), _ptr(label, "uint8", n, "label"), n, n_classes, cuda_stream or None,
        _ptr(conf_out, "int64", max(n_classes, 0) ** 2, "conf_out"), miou_out.data_ptr())
    if status != ST_OK:
        raise StError(status, load_library().st_status_name(status).decode(), "st_agreement_noalloc")


def st_measure_arithmetic_peaks(cuda_stream: int = 0):
    """(fp32 multiply-add rate in TFLOP/s, exp2 rate in 10^12 per second) measured on the current device."""
    fma, ex2 = ctypes.c_double(0), ctypes.c_double(0)
    _status_only(load_library().st_measure_arithmetic_peaks(cuda_stream or None, ctypes.byref(fma), ctypes.byref(ex2)),
                 "st_measure_arithmetic_peaks")
    return fma.value, ex2.value


class st_latencies(ctypes.Structure):
    _fields_ = [("t_si", ctypes.c_double), ("t_sd", ctypes.c_double), ("t_ti", ctypes.c_double), ("t_net", ctypes.c_double)]


def _status_only(status: int, what: str) -> None:
    if status != ST_OK:
        raise StError(status, load_library().st_status_name(status).decode(), what)


def st_next_stride(stride: int, metric: float, threshold: float, min_stride: int, max_stride: int) -> int:
    """NextStride (Algorithm 2)."""
    return int(load_library().st_next_stride(stride, metric, threshold, min_stride, max_stride))


def st_client_schedule(n_frames: int, metrics, threshold: float, min_stride: int, max_stride: int, delay: int):
    """Key-frame indices picked by the client's loop (Algorithm 4) as a list."""
    m = np.ascontiguousarray(metrics, dtype=np.float64)
    cap = n_frames // max(min_stride, 1) + 2
    out = np.zeros(cap, np.int64)
    n = ctypes.c_int64(0)
    _status_only(load_library().st_client_schedule(n_frames, m.ctypes.data, m.size, threshold, min_stride, max_stride, delay,
                                                   out.ctypes.data, cap, ctypes.byref(n)), "st_client_schedule")
    return out[:n.value].tolist()


def st_throughput_bounds(lat: st_latencies, min_stride: int, max_stride: int, max_updates: int):
    lo, hi = ctypes.c_double(0), ctypes.c_double(0)
    _status_only(load_library().st_throughput_bounds(ctypes.byref(lat), min_stride, max_stride, max_updates,
                                                     ctypes.byref(lo), ctypes.byref(hi)), "st_throughput_bounds")
    return lo.value, hi.value


def st_traffic_bounds(lat: st_latencies, s_net: float, min_stride: int, max_stride: int, max_updates: int):
    lo, hi = ctypes.c_double(0), ctypes.c_double(0)
    _status_only(load_library().st_traffic_bounds(ctypes.byref(lat), s_net, min_stride, max_stride, max_updates,
                                                  ctypes.byref(lo), ctypes.byref(hi)), "st_traffic_bounds")
    return lo.value, hi.value


def st_choose_max_updates(lat: st_latencies, min_stride: int, max_stride: int, fps_floor: float) -> int:
    return int(load_library().st_choose_max_updates(ctypes.byref(lat), min_stride, max_stride, fps_floor))


def st_launch_count(ctx: _Ctx) -> int:
    return int(load_library().st_launch_count(ctx.handle))


def st_destroy(ctx: _Ctx) -> None:
    if ctx is not None and ctx.handle:
        load_library().st_destroy(ctx.handle)
        ctx.handle = None


def st_last_error(ctx: Optional[_Ctx]) -> str:
    return (load_library().st_last_error(ctx.handle if ctx else None) or b"").decode()
