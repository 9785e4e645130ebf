"""CPU oracle of the host-side pieces around the distillation step: key-frame striding (Algorithm 2),
the client's key-frame schedule (Algorithm 4) and the analytic bounds of Section 4.4.

TEST INFRASTRUCTURE ONLY, like the rest of this package: plain Python written from the paper's
equations, imported by the tests alone.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Sequence


# ---------------------------------------------------------------------------- Algorithm 2
def next_stride_ratio(metric: float, threshold: float) -> float:
    """Ratio of the next stride to the current one: the line through (0, 0) and (THRESHOLD, 1) below the
    threshold, the line through (THRESHOLD, 1) and (1, 2) from the threshold on."""
    if metric < threshold:
        return metric / threshold
    return (metric - 2.0 * threshold + 1.0) / (1.0 - threshold)


def next_stride(stride: int, metric: float, threshold: float, min_stride: int, max_stride: int) -> int:
    """Algorithm 2.  The stride counts frames, so the product is cut to a whole number (toward zero) before
    it is clamped to [MIN_STRIDE, MAX_STRIDE]."""
    s = math.floor(next_stride_ratio(metric, threshold) * stride)
    return max(min_stride, min(max_stride, s))


# ---------------------------------------------------------------------------- Algorithm 4 (control flow only)
def client_schedule(n_frames: int, metrics: Sequence[float], threshold: float, min_stride: int, max_stride: int,
                    delay: int) -> List[int]:
    """Indices of the key frames Algorithm 4 picks among n_frames frames.

    metrics[j] is the metric the server returns for the j-th key frame; the reply to a key frame is complete
    `delay` frames after it was sent (1 <= delay; the client waits for it at step = MIN_STRIDE at the latest,
    so a larger delay acts like MIN_STRIDE)."""
    keys: List[int] = []
    stride = min_stride
    step = stride                      # first frame as key frame
    updated = True
    metric = None
    for f in range(n_frames):
        if step == stride:             # key frame
            metric = metrics[len(keys)]
            keys.append(f)
            step = 0
            updated = False
        step += 1                      # (student inference on this frame happens here)
        if not updated:
            completed = step >= delay
            if step == min_stride:
                completed = True       # WaitUntilComplete
            if completed:
                stride = next_stride(stride, metric, threshold, min_stride, max_stride)
                updated = True
    return keys


# ---------------------------------------------------------------------------- Section 4.4
@dataclass
class Latencies:
    t_si: float     # student inference
    t_sd: float     # one student distillation step
    t_ti: float     # teacher inference
    t_net: float    # network latency of one key frame


def t_c_bounds(L: Latencies, min_stride: int):
    """(lower, upper) of t_c, the time of the MIN_STRIDE frames after a key frame (Eq. 1)."""
    return max(min_stride * L.t_si, L.t_net + L.t_ti), min_stride * L.t_si + L.t_net + L.t_ti


def t_total(L: Latencies, n: int, k: float, d: float, t_c: float, min_stride: int) -> float:
    """Eq. 2: total time for n frames with k key frames and d distillation steps."""
    return (n - k * min_stride) * L.t_si + d * L.t_sd + k * t_c


def throughput_bounds(L: Latencies, min_stride: int, max_stride: int, max_updates: int):
    """(lower, upper) frames per second: Eq. 11 and Eq. 12."""
    lo = min_stride / (min_stride * L.t_si + max_updates * L.t_sd + L.t_ti + L.t_net)
    hi = max_stride / ((max_stride - min_stride) * L.t_si + max(min_stride * L.t_si, L.t_net + L.t_ti))
    return lo, hi


def traffic_bounds(L: Latencies, s_net: float, min_stride: int, max_stride: int, max_updates: int):
    """(lower, upper) of networked data per second, in the unit of s_net per second: Eq. 7 and Eq. 10."""
    lo = s_net / (max_stride * L.t_si + max_updates * L.t_sd + L.t_ti + L.t_net)
    hi = s_net / max(min_stride * L.t_si, L.t_net + L.t_ti)
    return lo, hi


def choose_max_updates(L: Latencies, min_stride: int, max_stride: int, fps_floor: float, limit: int = 1024) -> int:
    """Section 5.3's rule: the largest MAX_UPDATES whose throughput lower bound is still above fps_floor
    (-1 if even MAX_UPDATES = 0 is not)."""
    best = -1
    for m in range(0, limit + 1):
        if throughput_bounds(L, min_stride, max_stride, m)[0] > fps_floor:
            best = m
        else:
            break
    return best
