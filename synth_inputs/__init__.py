"""Seeded synthetic inputs shaped like the key-frame distillation workloads.

This module only *draws inputs* (features, teacher logits, initial head
parameters).  It holds none of the method's arithmetic: no argmax, no
convolution, no loss, no metric.  Both the CPU oracle's tests and the CUDA
path's tests/benchmarks feed from it, so the two sides always see identical
arrays.

The shapes follow the paper's workload (ShadowTutor, Section 5.2 and Table 4):
720p HD frames (1280x720), one byte per label pixel, fp32 parameters.  The LVS
videos, the Mask R-CNN teacher and the pre-trained student are not available, so
a Voronoi label map with per-pixel class logits stands in for the teacher output
and ReLU(N(0,1)) noise stands in for the frozen front part's feature map.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Tuple

import numpy as np

__all__ = [
    "WorkloadConfig", "CONFIGS", "get_config", "frozen_features", "voronoi_map",
    "teacher_logits", "head_param_shapes", "head_param_count", "initial_head_params",
    "key_frame_indices", "initial_stack_params", "skip_features",
]


@dataclass(frozen=True)
class WorkloadConfig:
    """One synthetic workload: a head, a frame size and a teacher recipe."""
    name: str
    c_in: int                # feature channels of the frozen part's output
    c_hidden: int            # 0 -> 1x1 head; >0 -> 3x3(c_in->c_hidden, pad 1)+ReLU+1x1
    n_classes: int
    feat_h: int
    feat_w: int
    up: int = 4              # frame = feature map * up
    k_steps: int = 1         # SGD iterations per key frame
    lr: float = 0.01
    momentum: float = 0.0
    n_streams: int = 1
    gemm_precision: int = 0  # 0 fp32 FMA, 1 bf16 tensor core with fp32 accumulate
    n_regions: int = 8       # Voronoi seed points
    teacher: str = "winner"  # "winner" | "onehot_noise" | "blur"
    n_frames: int = 1        # frames in the clip (drift workloads)
    key_stride: int = 0      # key frame every key_stride frames (0: only frame 0)
    drift: int = 0           # per-frame translation step in pixels
    blocks: Tuple[Tuple[int, int], ...] = ()   # a stack of student blocks: (output channels, skip-input channels) each
    first_trained: int = 0   # blocks before this index are frozen

    @property
    def frame_h(self) -> int:
        return self.feat_h * self.up

    @property
    def frame_w(self) -> int:
        return self.feat_w * self.up


CONFIGS = {
    1: WorkloadConfig("tiny_1x1_fp32", 64, 0, 4, 90, 160, k_steps=1, lr=0.01, momentum=0.0,
                      gemm_precision=0, n_regions=8, teacher="winner"),
    2: WorkloadConfig("720p_1x1_bf16", 256, 0, 21, 180, 320, k_steps=8, lr=0.01, momentum=0.9,
                      gemm_precision=1, n_regions=64, teacher="onehot_noise"),
    3: WorkloadConfig("720p_two_layer_drift", 256, 256, 21, 180, 320, k_steps=8, lr=0.005,
                      momentum=0.9, gemm_precision=1, n_regions=64, teacher="onehot_noise",
                      n_frames=16, key_stride=8, drift=2),
    4: WorkloadConfig("1080p_two_layer", 256, 256, 19, 270, 480, k_steps=16, lr=0.005,
                      momentum=0.9, gemm_precision=1, n_regions=128, teacher="blur"),
    5: WorkloadConfig("720p_16_streams", 256, 0, 21, 180, 320, k_steps=8, lr=0.01, momentum=0.9,
                      n_streams=16, gemm_precision=1, n_regions=64, teacher="onehot_noise"),
    # the trained back part in the paper's shape (Section 5.2): two blocks with skip inputs, then the classifier
    6: WorkloadConfig("720p_stack_sb5_sb6", 128, 0, 21, 180, 320, k_steps=8, lr=0.005, momentum=0.9,
                      gemm_precision=1, n_regions=64, teacher="onehot_noise", blocks=((128, 64), (64, 64))),
}


def get_config(idx: int) -> WorkloadConfig:
    return CONFIGS[idx]


def key_frame_indices(cfg: WorkloadConfig) -> List[int]:
    if cfg.key_stride <= 0:
        return [0]
    return list(range(0, cfg.n_frames, cfg.key_stride))


# ----------------------------------------------------------------------------
# frozen features
# ----------------------------------------------------------------------------
def frozen_features(c_in: int, h: int, w: int, seed: int) -> np.ndarray:
    """ReLU(N(0,1)) feature map, fp32 [c_in][h][w]."""
    rng = np.random.default_rng(seed)
    x = rng.standard_normal((c_in, h, w), dtype=np.float32)
    np.maximum(x, 0.0, out=x)
    return x


def label_informed_features(c_in: int, h: int, w: int, class_map: np.ndarray, up: int, seed: int,
                            strength: float = 2.0) -> np.ndarray:
    """ReLU(N(0,1)) features plus `strength` on channel c wherever the frame's class map shows class c at the
    centre of the feature pixel: a stand-in for a frozen front part whose output says something about the
    frame, so that the trainable part can actually improve its agreement with the labels (the plain noise
    features cannot).  `class_map` is uint8 [h*up][w*up] with values below c_in."""
    x = frozen_features(c_in, h, w, seed)
    low = class_map[up // 2::up, up // 2::up][:h, :w].astype(np.int64)
    yy, xx = np.meshgrid(np.arange(h), np.arange(w), indexing="ij")
    x[low, yy, xx] += np.float32(strength)
    return x


# ----------------------------------------------------------------------------
# teacher logits
# ----------------------------------------------------------------------------
def voronoi_map(H: int, W: int, n_regions: int, n_classes: int, seed: int,
                shift: Tuple[int, int] = (0, 0)) -> np.ndarray:
    """Class id per pixel from a Voronoi partition of the frame.

    Seed points are uniform in the frame; region r carries class r mod n_classes;
    a pixel belongs to the nearest point (squared Euclidean, lowest r on ties).
    `shift` = (dx, dy) translates the whole map (pixel (y, x) shows the partition
    at (y - dy, x - dx)), which is how drifting clips are drawn.
    """
    rng = np.random.default_rng(seed)
    py = rng.uniform(0.0, H, size=n_regions)
    px = rng.uniform(0.0, W, size=n_regions)
    dx, dy = shift
    ys = (np.arange(H, dtype=np.float64) - dy)[:, None]
    xs = (np.arange(W, dtype=np.float64) - dx)[None, :]
    best = np.full((H, W), np.inf)
    region = np.zeros((H, W), dtype=np.int32)
    for r in range(n_regions):
        d = (ys - py[r]) ** 2 + (xs - px[r]) ** 2
        closer = d < best            # strict: the lowest r keeps ties
        best = np.where(closer, d, best)
        region = np.where(closer, r, region)
    return (region % n_classes).astype(np.uint8)


def _blur_clamped(plane: np.ndarray, sigma: float, radius: int) -> np.ndarray:
    """Separable Gaussian blur with edge-clamped borders (fp64 in, fp64 out)."""
    t = np.arange(-radius, radius + 1, dtype=np.float64)
    k = np.exp(-0.5 * (t / sigma) ** 2)
    k /= k.sum()
    out = plane
    for axis in (0, 1):
        pad = [(0, 0), (0, 0)]
        pad[axis] = (radius, radius)
        padded = np.pad(out, pad, mode="edge")
        acc = np.zeros_like(out)
        n = out.shape[axis]
        for i, kv in enumerate(k):
            sl = [slice(None), slice(None)]
            sl[axis] = slice(i, i + n)
            acc += kv * padded[tuple(sl)]
        out = acc
    return out


def teacher_logits(cfg: WorkloadConfig, stream: int = 0, frame: int = 0) -> np.ndarray:
    """Per-pixel class logits standing in for the teacher's output, fp32 [C][H][W].

    "winner":       the region's class gets exactly 4.0, every other class N(0, 0.5).
    "onehot_noise": 4.0 * onehot(region class) + N(0, 0.5) on every entry.
    "blur":         Gaussian blur (sigma 3 px, radius 9, clamped edges) of
                    4.0 * onehot, no noise: exact ties occur at symmetric boundaries.
    Drifting clips translate the Voronoi map by a cumulative per-frame step drawn
    from {-drift, 0, +drift}^2 without (0, 0).
    """
    H, W, C = cfg.frame_h, cfg.frame_w, cfg.n_classes
    shift = (0, 0)
    if cfg.drift and frame > 0:
        rng = np.random.default_rng(4000 + stream)
        choices = [(a, b) for a in (-cfg.drift, 0, cfg.drift) for b in (-cfg.drift, 0, cfg.drift)
                   if (a, b) != (0, 0)]
        steps = rng.integers(0, len(choices), size=cfg.n_frames)
        sx = sum(choices[s][0] for s in steps[1:frame + 1])
        sy = sum(choices[s][1] for s in steps[1:frame + 1])
        shift = (sx, sy)
    cls = voronoi_map(H, W, cfg.n_regions, C, 2000 + stream, shift)
    noise_rng = np.random.default_rng(3000 + stream + 100 * frame)
    if cfg.teacher == "winner":
        T = noise_rng.standard_normal((C, H, W), dtype=np.float32) * np.float32(0.5)
        np.put_along_axis(T, cls[None].astype(np.int64), np.float32(4.0), axis=0)
        return T
    if cfg.teacher == "onehot_noise":
        T = noise_rng.standard_normal((C, H, W), dtype=np.float32) * np.float32(0.5)
        hot = np.zeros((C, H, W), dtype=np.float32)
        np.put_along_axis(hot, cls[None].astype(np.int64), np.float32(4.0), axis=0)
        T += hot
        return T
    if cfg.teacher == "blur":
        T = np.empty((C, H, W), dtype=np.float32)
        for c in range(C):
            plane = np.where(cls == c, 4.0, 0.0)
            T[c] = _blur_clamped(plane, 3.0, 9).astype(np.float32)
        return T
    raise ValueError(cfg.teacher)


# ----------------------------------------------------------------------------
# head parameters (packed order: per layer weight [Cout][Cin][kh][kw], then bias [Cout])
# ----------------------------------------------------------------------------
def head_param_shapes(c_in: int, c_hidden: int, n_classes: int):
    """[(weight shape, bias shape), ...] in forward order."""
    if c_hidden == 0:
        return [((n_classes, c_in, 1, 1), (n_classes,))]
    return [((c_hidden, c_in, 3, 3), (c_hidden,)), ((n_classes, c_hidden, 1, 1), (n_classes,))]


def head_param_count(c_in: int, c_hidden: int, n_classes: int) -> int:
    return sum(int(np.prod(ws)) + int(np.prod(bs))
               for ws, bs in head_param_shapes(c_in, c_hidden, n_classes))


def initial_head_params(c_in: int, c_hidden: int, n_classes: int, seed: int) -> np.ndarray:
    """Kaiming-normal weights (std = sqrt(2 / fan_in)), zero biases, one flat fp32 buffer."""
    rng = np.random.default_rng(seed)
    parts = []
    for ws, bs in head_param_shapes(c_in, c_hidden, n_classes):
        fan_in = ws[1] * ws[2] * ws[3]
        std = np.float32(np.sqrt(2.0 / fan_in))
        parts.append((rng.standard_normal(ws, dtype=np.float32) * std).ravel())
        parts.append(np.zeros(bs, dtype=np.float32))
    return np.concatenate(parts)


def initial_stack_params(c_in: int, blocks, n_classes: int, seed: int) -> np.ndarray:
    """The same initialisation for a stack of blocks: per block the 3x3 weight [c_out][c_prev + c_skip][3][3] and its
    bias, then the 1x1 classifier; one flat fp32 buffer in forward order."""
    rng = np.random.default_rng(seed)
    parts, prev = [], c_in
    shapes = [(co, prev_ + cs, 3) for (co, cs), prev_ in zip(blocks, [c_in] + [b[0] for b in blocks[:-1]])]
    shapes.append((n_classes, blocks[-1][0] if blocks else c_in, 1))
    for co, ci, k in shapes:
        std = np.float32(np.sqrt(2.0 / (ci * k * k)))
        parts.append((rng.standard_normal((co, ci, k, k), dtype=np.float32) * std).ravel())
        parts.append(np.zeros(co, dtype=np.float32))
    return np.concatenate(parts)


def skip_features(cfg: WorkloadConfig, block: int, seed: int) -> np.ndarray:
    """Skip input of one block: a feature map of the frozen front part, drawn like its output."""
    return frozen_features(cfg.blocks[block][1], cfg.feat_h, cfg.feat_w, 5000 + 10 * seed + block)


def stream_inputs(cfg: WorkloadConfig, stream: int = 0, frame: int = 0):
    """(features, teacher logits, initial packed params) for one stream / key frame."""
    feat_seed = stream if cfg.n_streams > 1 else frame
    X = frozen_features(cfg.c_in, cfg.feat_h, cfg.feat_w, feat_seed)
    T = teacher_logits(cfg, stream, frame)
    theta = initial_head_params(cfg.c_in, cfg.c_hidden, cfg.n_classes, 1000 + stream)
    return X, T, theta
