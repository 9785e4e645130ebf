"""CPU oracle of the key-frame partial-distillation step (ShadowTutor).

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  It never imports the CUDA package and the CUDA
package never imports it.

The arithmetic lives in ``st_oracle.c`` (plain C loops, fp32 storage, double
accumulators; a pure-double build exists for finite differences).  This module
compiles it with gcc on first use, wraps it with ctypes, and strings the
functions together in the order of Algorithm 1's loop body:

    prediction = Forward(student, frame)        head_forward + upsample
    loss       = ComputeLoss(prediction, label) softmax_ce
    gradients  = PartialBackward(loss)          upsample_adjoint, conv_wgrad (+ dgrad between head layers)
    student    = OptimStep(student, gradients)  sgd
    metric     = ComputeMetric(prediction,label) confusion + miou      (Section 3.2)

and UpdatedPart(student) (Algorithm 3) = ``pack``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "st_oracle.c")
_LIBS = {}

_c_i64 = ctypes.c_int64
_c_int = ctypes.c_int


def build(force: bool = False) -> None:
    """Compile st_oracle.c twice: fp32 storage and fp64 storage."""
    for tag, ctype in (("f32", "float"), ("f64", "double")):
        out = os.path.join(_HERE, f"libst_oracle_{tag}.so")
        if (not force and os.path.exists(out)
                and os.path.getmtime(out) >= os.path.getmtime(_SRC)):
            continue
        tmp = out + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-fPIC", "-shared", "-std=c99",
               f"-DST_REAL={ctype}", _SRC, "-o", tmp, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, out)


def _lib(dtype) -> ctypes.CDLL:
    tag = "f64" if np.dtype(dtype) == np.float64 else "f32"
    if tag not in _LIBS:
        build()
        lib = ctypes.CDLL(os.path.join(_HERE, f"libst_oracle_{tag}.so"))
        lib.so_miou.restype = ctypes.c_double
        lib.so_softmax_ce.restype = _c_i64
        lib.so_confusion.restype = _c_i64
        assert lib.so_sizeof_real() == (8 if tag == "f64" else 4)
        _LIBS[tag] = lib
    return _LIBS[tag]


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _real(dtype):
    return ctypes.c_double if np.dtype(dtype) == np.float64 else ctypes.c_float


def _c(a, dtype=None) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=dtype)


# ----------------------------------------------------------------------------
# single operations
# ----------------------------------------------------------------------------
def teacher_labels(T: np.ndarray) -> np.ndarray:
    """Pseudo-label map from teacher logits [C][H][W] (Algorithm 3): uint8 [H][W]."""
    T = _c(T)
    C, H, W = T.shape
    out = np.empty((H, W), dtype=np.uint8)
    _lib(T.dtype).so_labels(_p(T), _c_int(C), _c_i64(H * W), _p(out))
    return out


def conv_fwd(x: np.ndarray, W: np.ndarray, b: np.ndarray, relu: bool = False) -> np.ndarray:
    x = _c(x)
    W = _c(W, x.dtype)
    b = _c(b, x.dtype)
    Cin, h, w = x.shape
    Cout, Cin2, ks, ks2 = W.shape
    assert Cin2 == Cin and ks == ks2 and ks in (1, 3)
    out = np.empty((Cout, h, w), dtype=x.dtype)
    _lib(x.dtype).so_conv_fwd(_p(x), _c_int(Cin), _c_int(h), _c_int(w), _p(W), _p(b),
                              _c_int(Cout), _c_int(ks), _c_int(int(relu)), _p(out))
    return out


def upsample(z: np.ndarray, s: int) -> np.ndarray:
    z = _c(z)
    C, h, w = z.shape
    u = np.empty((C, h * s, w * s), dtype=z.dtype)
    _lib(z.dtype).so_upsample(_p(z), _c_int(C), _c_int(h), _c_int(w), _c_int(s), _p(u))
    return u


def upsample_adjoint(g: np.ndarray, s: int) -> np.ndarray:
    g = _c(g)
    C, H, W = g.shape
    h, w = H // s, W // s
    dz = np.empty((C, h, w), dtype=g.dtype)
    _lib(g.dtype).so_upsample_adjoint(_p(g), _c_int(C), _c_int(h), _c_int(w), _c_int(s), _p(dz))
    return dz


def softmax_ce(u: np.ndarray, labels: np.ndarray, want_grad: bool = True, weights: Optional[np.ndarray] = None):
    """(mean loss as float, gradient [C][H][W] or None, number of out-of-range labels).
    `weights` (uint8 [H][W]) scales each pixel's loss and gradient (Section 5.2's loss weighting)."""
    u = _c(u)
    labels = _c(labels, np.uint8)
    C, H, W = u.shape
    g = np.empty_like(u) if want_grad else None
    loss = ctypes.c_double(0.0)
    lib = _lib(u.dtype)
    lib.so_softmax_ce_weighted.restype = _c_i64
    wg = _c(weights, np.uint8) if weights is not None else None
    bad = lib.so_softmax_ce_weighted(_p(u), _p(labels), _p(wg) if wg is not None else None, _c_int(C), _c_i64(H * W),
                                     _p(g) if want_grad else None, ctypes.byref(loss))
    return loss.value, g, int(bad)


def object_weights(labels: np.ndarray, background: int, radius: int, factor: int) -> np.ndarray:
    """uint8 [H][W]: `factor` for pixels within `radius` (square window) of a non-background pixel, else 1."""
    labels = _c(labels, np.uint8)
    H, W = labels.shape
    out = np.empty((H, W), np.uint8)
    _lib(np.float32).so_object_weights(_p(labels), _c_int(H), _c_int(W), _c_int(background), _c_int(radius), _c_int(factor), _p(out))
    return out


def conv_wgrad(x: np.ndarray, dout: np.ndarray, ks: int):
    x = _c(x)
    dout = _c(dout, x.dtype)
    Cin, h, w = x.shape
    Cout = dout.shape[0]
    dW = np.empty((Cout, Cin, ks, ks), dtype=x.dtype)
    db = np.empty((Cout,), dtype=x.dtype)
    _lib(x.dtype).so_conv_wgrad(_p(x), _p(dout), _c_int(Cin), _c_int(Cout), _c_int(h), _c_int(w),
                                _c_int(ks), _p(dW), _p(db))
    return dW, db


def bias_grad(dout: np.ndarray) -> np.ndarray:
    dout = _c(dout)
    Cout = dout.shape[0]
    db = np.empty((Cout,), dtype=dout.dtype)
    _lib(dout.dtype).so_bias_grad(_p(dout), _c_int(Cout), _c_i64(dout.size // Cout), _p(db))
    return db


def conv1x1_dgrad(W2: np.ndarray, dz: np.ndarray) -> np.ndarray:
    dz = _c(dz)
    W2 = _c(W2, dz.dtype)
    C, h, w = dz.shape
    Ch = W2.shape[1]
    dH = np.empty((Ch, h, w), dtype=dz.dtype)
    _lib(dz.dtype).so_conv1x1_dgrad(_p(W2), _p(dz), _c_int(C), _c_int(Ch), _c_i64(h * w), _p(dH))
    return dH


def conv_dgrad(dout: np.ndarray, W: np.ndarray, c_take: Optional[int] = None) -> np.ndarray:
    """Gradient with respect to the first `c_take` input channels of a convolution layer (all of them by default)."""
    dout = _c(dout)
    W = _c(W, dout.dtype)
    Cout, Cin, ks, _ = W.shape
    _, h, w = dout.shape
    take = Cin if c_take is None else int(c_take)
    din = np.empty((take, h, w), dtype=dout.dtype)
    _lib(dout.dtype).so_conv_dgrad(_p(dout), _p(W), _c_int(Cin), _c_int(take), _c_int(Cout), _c_int(h), _c_int(w), _c_int(ks), _p(din))
    return din


def relu_mask_(dH: np.ndarray, Hact: np.ndarray) -> None:
    assert dH.flags.c_contiguous and Hact.flags.c_contiguous and dH.dtype == Hact.dtype
    _lib(dH.dtype).so_relu_mask(_p(dH), _p(Hact), _c_i64(dH.size))


def sgd_(theta: np.ndarray, v: np.ndarray, g: np.ndarray, lr: float, mu: float) -> None:
    assert theta.flags.c_contiguous and v.flags.c_contiguous
    g = _c(g, theta.dtype)
    R = _real(theta.dtype)
    _lib(theta.dtype).so_sgd(_p(theta), _p(v), _p(g), _c_i64(theta.size), R(lr), R(mu))


def adam_(theta: np.ndarray, m: np.ndarray, v: np.ndarray, g: np.ndarray, lr: float, b1: float, b2: float, eps: float,
          t: int) -> None:
    """Step t (1-based) of Adam on theta in place; m, v are the two moment buffers."""
    assert theta.flags.c_contiguous and m.flags.c_contiguous and v.flags.c_contiguous
    g = _c(g, theta.dtype)
    _lib(theta.dtype).so_adam(_p(theta), _p(m), _p(v), _p(g), _c_i64(theta.size), ctypes.c_double(lr), ctypes.c_double(b1),
                              ctypes.c_double(b2), ctypes.c_double(eps), _c_i64(t))


def confusion(labels: np.ndarray, pred: np.ndarray, C: int):
    """(conf int64 [C][C] with conf[label][pred], number of skipped pixels)."""
    labels = _c(labels, np.uint8)
    pred = _c(pred, np.uint8)
    conf = np.zeros((C, C), dtype=np.int64)
    bad = _lib(np.float32).so_confusion(_p(labels), _p(pred), _c_i64(labels.size), _c_int(C), _p(conf))
    return conf, int(bad)


def miou(conf: np.ndarray) -> float:
    conf = _c(conf, np.int64)
    return float(_lib(np.float32).so_miou(_p(conf), _c_int(conf.shape[0])))


def round_bf16(a: np.ndarray) -> np.ndarray:
    out = _c(a).copy()
    _lib(out.dtype).so_round_bf16(_p(out), _c_i64(out.size))
    return out


# ----------------------------------------------------------------------------
# the head and one iteration of Algorithm 1's loop body
# ----------------------------------------------------------------------------
def param_shapes(c_in: int, c_hidden: int, n_classes: int):
    if c_hidden == 0:
        return [((n_classes, c_in, 1, 1), (n_classes,))]
    return [((c_hidden, c_in, 3, 3), (c_hidden,)), ((n_classes, c_hidden, 1, 1), (n_classes,))]


@dataclass
class Head:
    """Trainable back part of the student: conv weights/biases plus momentum buffers."""
    c_in: int
    c_hidden: int
    n_classes: int
    up: int = 4
    lr: float = 0.01
    momentum: float = 0.0
    dtype: type = np.float32
    quantize_bf16: bool = False      # test-only: round GEMM operands to bf16 like the tensor-core path
    theta: np.ndarray = None         # flat parameters in packed order
    vel: np.ndarray = None           # momentum (SGD) / first moment (Adam), same order, starts at zero
    optimizer: str = "sgd"           # "sgd" (heavy-ball momentum) or "adam" (Section 5.2)
    betas: Tuple[float, float] = (0.9, 0.999)   # Adam's decay rates and epsilon: not stated in the paper,
    eps: float = 1e-8                #   the constants of the published algorithm are assumed
    vel2: np.ndarray = None          # Adam's second moment
    t: int = 0                       # optimisation steps taken so far (Adam's bias correction)
    object_weight: int = 1           # Section 5.2's loss weighting: factor for pixels near / within non-background
    object_radius: int = 0           #   objects (5 in the paper), the distance that counts as "near" (not stated
    background: int = 0              #   in the paper) and the background class

    def __post_init__(self):
        n = sum(int(np.prod(ws)) + int(np.prod(bs))
                for ws, bs in param_shapes(self.c_in, self.c_hidden, self.n_classes))
        if self.theta is None:
            self.theta = np.zeros(n, dtype=self.dtype)
        self.theta = np.ascontiguousarray(self.theta, dtype=self.dtype).copy()
        assert self.theta.size == n, (self.theta.size, n)
        self.vel = np.zeros(n, dtype=self.dtype)
        self.vel2 = np.zeros(n, dtype=self.dtype)
        assert self.optimizer in ("sgd", "adam")

    def optim_step(self, grad: np.ndarray) -> None:
        """student <- OptimStep(student, gradients)."""
        self.t += 1
        if self.optimizer == "adam":
            adam_(self.theta, self.vel, self.vel2, grad.astype(self.dtype), self.lr, self.betas[0], self.betas[1], self.eps, self.t)
        else:
            sgd_(self.theta, self.vel, grad.astype(self.dtype), self.lr, self.momentum)

    def layers(self) -> List[Tuple[np.ndarray, np.ndarray]]:
        """Views (weight, bias) into theta, forward order."""
        out, off = [], 0
        for ws, bs in param_shapes(self.c_in, self.c_hidden, self.n_classes):
            nw, nb = int(np.prod(ws)), int(np.prod(bs))
            out.append((self.theta[off:off + nw].reshape(ws), self.theta[off + nw:off + nw + nb]))
            off += nw + nb
        return out

    def _q(self, a):
        return round_bf16(a) if self.quantize_bf16 else a


def head_forward(head: Head, feat: np.ndarray):
    """Forward of the trainable part over the frozen part's output.

    Returns (z [C][h][w], hidden activation [Ch][h][w] or None).
    """
    x = head._q(np.ascontiguousarray(feat, dtype=head.dtype))
    layers = head.layers()
    if head.c_hidden == 0:
        (W, b), = layers
        return conv_fwd(x, head._q(W), b), None
    (W1, b1), (W2, b2) = layers
    Hd = head._q(conv_fwd(x, head._q(W1), b1, relu=True))
    return conv_fwd(Hd, head._q(W2), b2), Hd


def student_mask(head: Head, feat: np.ndarray) -> np.ndarray:
    """Student prediction at frame resolution: argmax of the upsampled head logits."""
    z, _ = head_forward(head, feat)
    return teacher_labels(upsample(z, head.up))


def head_backward(head: Head, x: np.ndarray, Hd: Optional[np.ndarray], dz: np.ndarray) -> np.ndarray:
    """PartialBackward from the logit gradient on (Algorithm 1; Section 4.2): the gradient of every trainable
    tensor, flat, in packed order.  `x` is the frozen part's output as the forward saw it, `Hd` the hidden
    activation of that forward (None for the 1x1 head), `dz` the gradient of the loss with respect to the
    head's logits.  No gradient is formed for `x`.

    With ``quantize_bf16`` the operands of the products are rounded where the tensor-core path rounds them:
    dz where it meets the activations (weight gradient) and the weights (gradient passed back), the 1x1
    weight, and the hidden gradient where it meets `x`.  The bias gradients are sums of the unrounded values.
    """
    layers = head.layers()
    if head.c_hidden == 0:
        dW, db = conv_wgrad(x, head._q(dz), 1)
        if head.quantize_bf16:
            db = bias_grad(dz)
        return np.concatenate([dW.ravel(), db.ravel()])
    (W1, b1), (W2, b2) = layers
    dW2, db2 = conv_wgrad(Hd, head._q(dz), 1)
    dH = conv1x1_dgrad(head._q(W2.reshape(W2.shape[0], W2.shape[1])), head._q(dz))
    relu_mask_(dH, Hd)
    dW1, db1 = conv_wgrad(x, head._q(dH), 3)
    if head.quantize_bf16:
        db2, db1 = bias_grad(dz), bias_grad(dH)
    return np.concatenate([dW1.ravel(), db1.ravel(), dW2.ravel(), db2.ravel()])


def gradients(head: Head, feat: np.ndarray, labels: np.ndarray):
    """Loss and gradient of every trainable tensor (flat, packed order) at the current parameters.

    Also returns the student mask of this forward (the prediction the loss was computed from).
    """
    x = head._q(np.ascontiguousarray(feat, dtype=head.dtype))
    z, Hd = head_forward(head, feat)
    u = upsample(z, head.up)
    wgt = object_weights(labels, head.background, head.object_radius, head.object_weight) if head.object_weight > 1 else None
    loss, g, _ = softmax_ce(u, labels, weights=wgt)
    mask = teacher_labels(u)
    dz = upsample_adjoint(g, head.up)
    return loss, head_backward(head, x, Hd, dz), mask


def distill_step(head: Head, feat: np.ndarray, labels: np.ndarray):
    """One iteration of Algorithm 1's loop: loss and gradients at the current
    parameters, then one optimiser step.  Returns (loss, student mask before the update)."""
    loss, grad, mask = gradients(head, feat, labels)
    head.optim_step(grad)
    return loss, mask


def pack(head: Head) -> bytes:
    """UpdatedPart(student) (Algorithm 3): per trainable layer in forward order the weight
    [Cout][Cin][kh][kw] then the bias [Cout], fp32 little-endian values, no header."""
    return np.ascontiguousarray(head.theta, dtype="<f4").tobytes()


def agreement(labels: np.ndarray, pred: np.ndarray, C: int):
    conf, bad = confusion(labels, pred, C)
    return conf, miou(conf), bad


# ----------------------------------------------------------------------------
# a deeper trainable subset: a stack of student blocks with skip inputs and a freeze boundary inside it
# ----------------------------------------------------------------------------
@dataclass
class StackHead:
    """The back part of the student as a stack of blocks (Section 5.2: blocks SB5 and SB6, each fed by the block before
    it and by a feature map of the frozen front part -- SB2's and SB1's -- concatenated to its input, then the
    classifier), with the freeze boundary of partial distillation (Section 4.2) anywhere inside it.

    The paper's drawing of a student block is not in its text.  Reading taken: block b is a 3x3 convolution with zero
    padding 1 over concat(previous block's output or the frozen part's output, skip input b) followed by ReLU; all
    blocks and their skip inputs share the resolution of the frozen part's output (whatever resampling the skip maps
    need belongs to the frozen part); the classifier is a 1x1 convolution.  Layers before `first_trained` keep their
    parameters: no gradient is formed for them and none is passed back into them ("the gradient computation can stop
    in the middle", Section 4.2).  first_trained = 0 trains every block; = len(blocks) trains the classifier alone.
    """
    c_in: int
    blocks: List[Tuple[int, int]]    # per block (output channels, skip-input channels)
    n_classes: int
    first_trained: int = 0
    up: int = 4
    lr: float = 0.01
    momentum: float = 0.0
    dtype: type = np.float32
    quantize_bf16: bool = False      # test-only: round GEMM operands to bf16 like the tensor-core path
    theta: np.ndarray = None         # flat parameters of ALL layers, forward order: per layer weight then bias
    vel: np.ndarray = None

    def shapes(self):
        out, prev = [], self.c_in
        for c_out, c_skip in self.blocks:
            out.append(((c_out, prev + c_skip, 3, 3), (c_out,)))
            prev = c_out
        out.append(((self.n_classes, prev, 1, 1), (self.n_classes,)))
        return out

    def __post_init__(self):
        n = sum(int(np.prod(ws)) + int(np.prod(bs)) for ws, bs in self.shapes())
        if self.theta is None:
            self.theta = np.zeros(n, dtype=self.dtype)
        self.theta = np.ascontiguousarray(self.theta, dtype=self.dtype).copy()
        assert self.theta.size == n, (self.theta.size, n)
        self.vel = np.zeros(n, dtype=self.dtype)
        assert 0 <= self.first_trained <= len(self.blocks)

    def layers(self):
        out, off = [], 0
        for ws, bs in self.shapes():
            nw, nb = int(np.prod(ws)), int(np.prod(bs))
            out.append((self.theta[off:off + nw].reshape(ws), self.theta[off + nw:off + nw + nb]))
            off += nw + nb
        return out

    def trained_slice(self) -> slice:
        """Where the trained layers sit in theta (they are the last ones): what UpdatedPart carries."""
        off = 0
        for ws, bs in self.shapes()[:self.first_trained]:
            off += int(np.prod(ws)) + int(np.prod(bs))
        return slice(off, self.theta.size)

    def _q(self, a):
        return round_bf16(a) if self.quantize_bf16 else a


def stack_forward(head: StackHead, feat: np.ndarray, skips: List[Optional[np.ndarray]]):
    """(logits [C][h][w], inputs of every block as the convolution saw them, outputs of every block)."""
    layers = head.layers()
    prev = head._q(np.ascontiguousarray(feat, dtype=head.dtype))
    ins, outs = [], []
    for b, (c_out, c_skip) in enumerate(head.blocks):
        x = prev if c_skip == 0 else np.concatenate([prev, head._q(np.ascontiguousarray(skips[b], dtype=head.dtype))], axis=0)
        W, bias = layers[b]
        prev = head._q(conv_fwd(x, head._q(W), bias, relu=True))
        ins.append(x); outs.append(prev)
    Wc, bc = layers[-1]
    return conv_fwd(prev, head._q(Wc), bc), ins, outs


def stack_student_mask(head: StackHead, feat, skips) -> np.ndarray:
    return teacher_labels(upsample(stack_forward(head, feat, skips)[0], head.up))


def stack_gradients(head: StackHead, feat, skips, labels):
    """Loss, gradient of every parameter (zero for the frozen layers) and the student mask of this forward."""
    z, ins, outs = stack_forward(head, feat, skips)
    u = upsample(z, head.up)
    loss, g, _ = softmax_ce(u, labels)
    mask = teacher_labels(u)
    dz = upsample_adjoint(g, head.up)
    layers = head.layers()
    B = len(head.blocks)
    grads = [None] * (B + 1)
    Wc, _ = layers[-1]
    last = outs[-1] if B else head._q(np.ascontiguousarray(feat, dtype=head.dtype))
    dWc, dbc = conv_wgrad(last, head._q(dz), 1)
    if head.quantize_bf16:
        dbc = bias_grad(dz)
    grads[B] = (dWc, dbc)
    if head.first_trained < B:
        dH = conv1x1_dgrad(head._q(Wc.reshape(Wc.shape[0], Wc.shape[1])), head._q(dz))
        relu_mask_(dH, outs[-1])
        for b in range(B - 1, head.first_trained - 1, -1):
            W, _ = layers[b]
            dW, db = conv_wgrad(ins[b], head._q(dH), 3)
            if head.quantize_bf16:
                db = bias_grad(dH)
            grads[b] = (dW, db)
            if b > head.first_trained:             # pass the gradient on to the block before (its own output channels only)
                c_prev = head.blocks[b - 1][0]
                dH = conv_dgrad(head._q(dH), head._q(W), c_prev)
                relu_mask_(dH, outs[b - 1])
    flat = []
    for (ws, bs), gr in zip(head.shapes(), grads):
        if gr is None:
            flat += [np.zeros(int(np.prod(ws)), head.dtype), np.zeros(int(np.prod(bs)), head.dtype)]
        else:
            flat += [gr[0].ravel(), gr[1].ravel()]
    return loss, np.concatenate(flat), mask


def stack_distill_step(head: StackHead, feat, skips, labels):
    """One iteration of Algorithm 1's loop on the trained layers (gradient descent with momentum)."""
    loss, grad, mask = stack_gradients(head, feat, skips, labels)
    sl = head.trained_slice()
    sgd_(head.theta[sl], head.vel[sl], grad[sl].astype(head.dtype), head.lr, head.momentum)
    return loss, mask


def stack_pack(head: StackHead) -> bytes:
    """UpdatedPart(student) (Algorithm 3): the trained layers only, forward order, weight then bias, fp32."""
    return np.ascontiguousarray(head.theta[head.trained_slice()], dtype="<f4").tobytes()


# ----------------------------------------------------------------------------
# Algorithm 1 as a whole: Train(student, frame, label)
# ----------------------------------------------------------------------------
@dataclass
class TrainResult:
    best_metric: float            # the metric returned with best_student
    n_updates: int                # optimisation steps taken before the loop ended
    best_iter: int                # number of updates behind best_student (0 = the incoming student)
    metrics: List[float]          # metric of every prediction: metrics[i] after i updates
    losses: List[float]           # loss of every prediction the loop computed a loss for (one per update)
    masks: List[np.ndarray] = field(default_factory=list)   # the predictions themselves (kept on request)


def train_key_frame(head: Head, feat: np.ndarray, labels: np.ndarray, threshold: float, max_updates: int,
                    keep_masks: bool = False) -> TrainResult:
    """Train(student, frame, label) of Algorithm 1.

    The incoming student is assessed first and is the first best_student; distillation is skipped when it
    already meets the threshold.  Otherwise up to `max_updates` optimisation steps follow, each assessed by
    the metric of the prediction made after it; the best iterate so far is remembered (a later one has to
    be strictly better) and the loop ends at the first metric above the threshold.
    The metric is the mean IoU of Section 3.2 between the student's mask and the pseudo-label.
    On return ``head.theta`` holds best_student (Algorithm 3 continues with the returned student);
    the momentum buffer is optimiser state, not part of the student, and keeps running.
    """
    C = head.n_classes
    prediction = student_mask(head, feat)
    best_metric = agreement(labels, prediction, C)[1]
    best_student = head.theta.copy()
    res = TrainResult(best_metric, 0, 0, [best_metric], [])
    if keep_masks:
        res.masks.append(prediction)
    if best_metric < threshold:
        for i in range(1, max_updates + 1):
            # the loss is a function of the same parameters that produced the prediction assessed last
            loss, _ = distill_step(head, feat, labels)
            res.losses.append(loss)
            res.n_updates = i
            prediction = student_mask(head, feat)
            metric = agreement(labels, prediction, C)[1]
            res.metrics.append(metric)
            if keep_masks:
                res.masks.append(prediction)
            if metric > best_metric:
                best_metric = metric
                best_student = head.theta.copy()
                res.best_iter = i
            if metric > threshold:
                break
    head.theta[:] = best_student
    res.best_metric = best_metric
    return res
