#!/usr/bin/env python
"""Benchmark of the key-frame partial-distillation step on B200.

One bench "step" is one pass of the whole hot path over one synthetic 720p key frame:
cache the frozen features, reduce the teacher logits to labels, K = 8 SGD iterations of the
head, pack the updated parameters, and measure student/teacher agreement.  The reported
metric counts SGD iterations per second (8 per bench step), whole job, all GPUs.

    python bench.py --gpus 1 --steps 2000 --warmup 10
    python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...
    python bench.py --impl reference        # the CPU oracle, timed on the host cores

Every rank prints nothing except rank 0, which prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "720p key-frame partial-distill steps/s (K=8)"
N_SETS = 4            # distinct key frames the device-resident run rotates over (4 x 136 MB > 126 MB L2)
# Algorithmic work of the fused upsample + cross-entropy kernel per class and frame pixel: two horizontal and one vertical
# interpolation step, exponent scale and shift, the sum, the normalisation and three adjoint multiply-adds -- 10
# multiply-add equivalents = 20 flop (12 to 16 separate fp32 operations when written without fused multiply-adds) --
# and one exponential.
ALU_FLOP_PER_CLASS_PIXEL = 20.0
EX2_PER_CLASS_PIXEL = 1.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch, ncu capture of (workload, kernel); see profiles/.
# An entry is removed whenever its kernel changes and put back after the next capture.
NCU_DRAM_BYTES = {
    (2, "upsample_ce"): 5.85e6,      # profiles/upsample_ce_rows_720p.md
    # profiles/fwd1x1_upsample_ce_rows_720p.md: a capture starts with cold caches, so the feature map (29.5 MB, L2 resident
    # over the K iterations of the step loop) is read from DRAM once; labels 0.92 MB
    (2, "fwd1x1_upsample_ce"): 30.53e6,
}
# st_init_head reads this when a context is made: "0" keeps the classifier's forward in a kernel of its own
FUSED_SWITCH = "ST_FUSED_FORWARD"


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "sm_max_mhz": float(p.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "sm_max_mhz": 1965.0,
            "source": "fallback"}


# --------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.path = tempfile.NamedTemporaryFile(prefix="st_clocks_", suffix=".csv", delete=False).name
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(gpu_index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None
        self.t0 = self.t1 = None

    def begin(self):
        self.t0 = time.time()

    def end(self):
        self.t1 = time.time()

    def finish(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        import datetime
        with open(self.path) as f:
            for line in f:
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 10:
                    continue
                try:
                    ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                    rows.append((ts, float(parts[2]), float(parts[3]), parts[6:10]))
                except ValueError:
                    continue
        try:
            os.unlink(self.path)
        except OSError:
            pass
        inside = [r for r in rows if self.t0 - 0.05 <= r[0] <= self.t1 + 0.05] or rows[-3:]
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"], "samples": 0}
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in inside for n, v in zip(names, r[3]) if v.lower().startswith("active")})
        return {"sm_mhz": statistics.median(r[1] for r in inside), "sm_max_mhz": inside[0][2],
                "reasons": reasons, "samples": len(inside)}


# --------------------------------------------------------------------------------------------
# the CPU oracle, timed (cpu_baseline leg and --impl reference)
# --------------------------------------------------------------------------------------------
def oracle_key_frame(cfg, feat, T, theta, rows=None):
    """One key frame through the oracle as it stands; returns seconds.  `rows` crops the feature map
    to its first `rows` rows (and the frame to 4*rows) for a bounded sample."""
    import oracle
    if rows is not None:
        feat = np.ascontiguousarray(feat[:, :rows])
        T = np.ascontiguousarray(T[:, :rows * cfg.up])
    t0 = time.perf_counter()
    labels = oracle.teacher_labels(T)
    head = oracle.Head(cfg.c_in, cfg.c_hidden, cfg.n_classes, up=cfg.up, lr=cfg.lr, momentum=cfg.momentum, theta=theta)
    for _ in range(cfg.k_steps):
        oracle.distill_step(head, feat, labels)
    oracle.pack(head)
    oracle.agreement(labels, oracle.student_mask(head, feat), cfg.n_classes)
    return time.perf_counter() - t0


def host_cores():
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    feat, T, theta = si.stream_inputs(cfg)
    # calibrate on a thin band, then size the per-step sample so that the whole run stays within ~3 minutes
    t_band = oracle_key_frame(cfg, feat, T, theta, rows=4)
    per_row = t_band / 4
    budget = 150.0 / max(1, args.steps + args.warmup)
    rows = int(max(4, min(cfg.feat_h, budget / max(per_row, 1e-9))))
    for _ in range(args.warmup):
        oracle_key_frame(cfg, feat, T, theta, rows=rows)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_key_frame(cfg, feat, T, theta, rows=rows)
    dt = time.perf_counter() - t0
    frac = rows / cfg.feat_h
    key_frames_per_s = args.steps / dt * frac          # scaled to the full frame by pixel count
    value = key_frames_per_s * cfg.k_steps
    sample = f"{rows} of {cfg.feat_h} feature rows per step, scaled to the full frame by pixel count"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3 / frac,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": cfg.name, "k_steps": cfg.k_steps, "frame": [cfg.frame_h, cfg.frame_w]},
        "cpu_baseline": {"value": value, "unit": "steps/s", "cores": host_cores(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------
# multi-GPU plumbing: the path shards by client stream, ranks exchange nothing but the timing
# --------------------------------------------------------------------------------------------
def rank_streams(streams_per_rank: int, world: int, rank: int):
    """Global ids of the client streams a rank owns (disjoint, covering 0 .. world*streams_per_rank - 1)."""
    return [rank * streams_per_rank + s for s in range(streams_per_rank)]


def max_over_ranks(value: float, dist, device=None) -> float:
    """Largest value over all ranks (the job is as slow as its slowest rank); identity without a group."""
    if dist is None:
        return float(value)
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Units all ranks processed per second, timed by the slowest rank."""
    return world * units_per_rank / (ms_max / 1e3)


# --------------------------------------------------------------------------------------------
# the CUDA path
# --------------------------------------------------------------------------------------------
def timed_blocks(torch, stream, barrier, n_blocks, steps, body, between=None):
    """ms of each of n_blocks timed regions of `steps` calls of body(i), each bracketed by barrier + synchronize
    and timed with CUDA events on the launching stream; `between` runs outside the timed regions."""
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    out, i = [], 0
    for _ in range(n_blocks):
        if between is not None:
            between()
        barrier()
        ev0.record(stream)
        for _ in range(steps):
            body(i)
            i += 1
        ev1.record(stream)
        barrier()
        out.append(ev0.elapsed_time(ev1))
    return out


def kernel_table(st, ctx, cfg, peaks, arith, n_profile_steps):
    """Per-kernel CUDA-event times of one step (st_profile_step) with the roofline each kernel is held against."""
    S, C, K = cfg.n_streams, cfg.n_classes, cfg.k_steps
    p, P = cfg.feat_h * cfg.feat_w, cfg.frame_h * cfg.frame_w
    blocks = [tuple(b) for b in cfg.blocks] or ([(cfg.c_hidden, 0)] if cfg.c_hidden else [])
    c_last = blocks[-1][0] if blocks else cfg.c_in

    def block_flop(i):                  # one 3x3 layer over its concatenated input
        c_prev = cfg.c_in if i == 0 else blocks[i - 1][0]
        return 2.0 * S * p * blocks[i][0] * 9 * (c_prev + blocks[i][1])
    hbm, tensor_peak = peaks["hbm_gbs"], peaks["bf16_tflops"]
    kernels = {}
    for name, ms in st.st_profile_step(ctx, n_profile_steps):
        k = {"ms": ms, "per_key_frame": K}
        if name in ("upsample_ce", "fwd1x1_upsample_ce"):
            class_pixels = float(C) * P * S
            k.update(bound="alu", achieved=ALU_FLOP_PER_CLASS_PIXEL * class_pixels / ms / 1e9, peak=arith["fma_tflops"],
                     unit="TFLOP/s", hbm_gbs=S * (2 * C * p * 4 + P) / ms / 1e6,
                     xu={"achieved": EX2_PER_CLASS_PIXEL * class_pixels / ms / 1e9, "peak": arith["ex2_tops"],
                         "unit": "1e12 exp2/s", "frac": EX2_PER_CLASS_PIXEL * class_pixels / ms / 1e9 / arith["ex2_tops"]})
            if name == "fwd1x1_upsample_ce":
                # the kernel also multiplies its own logit tiles (Forward of the 1x1 classifier): every block fetches the
                # 9 x 32 nodes around its 7 x 30 from L2, so the launch streams 288/210 of the feature map
                n_tiles = -(-cfg.feat_h // 7) * -(-cfg.feat_w // 30)
                k.update(hbm_gbs=S * (p * c_last * 2 + P) / ms / 1e6,
                         forward={"tensor_tflops": 2.0 * S * n_tiles * 384 * 32 * c_last / ms / 1e9,
                                  "feature_bytes_fetched_by_blocks": S * n_tiles * 288 * c_last * 2,
                                  "note": "replaces tc_fwd1x1 + upsample_ce (see kernels_unfused for those two)"})
        elif name == "tc_fwd1x1":
            k.update(bound="hbm", achieved=S * (p * c_last * 2 + C * p * 4) / ms / 1e6, peak=hbm, unit="GB/s",
                     tflops=2.0 * S * p * C * c_last / ms / 1e9)
        elif name == "tc_wgrad1x1":
            k.update(bound="hbm", achieved=S * (p * c_last * 2 + C * p * 2) / ms / 1e6, peak=hbm, unit="GB/s",
                     tflops=2.0 * S * p * C * c_last / ms / 1e9)
        elif name.startswith("tc_fwd3x3") or name.startswith("tc_wgrad3x3"):
            k.update(bound="tensor", achieved=block_flop(1 if name.endswith("#2") else 0) / ms / 1e9, peak=tensor_peak, unit="TFLOP/s")
        elif name == "tc_dgrad3x3":     # through block 1 into block 0's output channels
            k.update(bound="tensor", achieved=2.0 * S * p * blocks[0][0] * 9 * blocks[1][0] / ms / 1e9, peak=tensor_peak, unit="TFLOP/s")
        elif name == "tc_dgrad":
            k.update(bound="hbm", achieved=S * (2 * p * c_last * 2 + C * p * 4) / ms / 1e6, peak=hbm, unit="GB/s")
        else:
            k.update(bound="latency")
        kernels[name] = k
    for k in kernels.values():
        if "achieved" in k and k.get("peak"):
            k["frac"] = k["achieved"] / k["peak"]
    return kernels


def make_context(st, stream, cfg, theta0, **kw):
    args = dict(n_streams=cfg.n_streams, c_in=cfg.c_in, c_hidden=cfg.c_hidden, n_classes=cfg.n_classes, feat_h=cfg.feat_h,
                feat_w=cfg.feat_w, gemm_precision=cfg.gemm_precision, lr=cfg.lr, momentum=cfg.momentum,
                cuda_stream=stream.cuda_stream, init_params=theta0)
    args.update(kw)
    return st.st_init_head(**args)


def run_other_workload(st, torch, stream, idx, feats_d, logits_d, peaks, arith, local_rank):
    """A few key frames of another workload of the same frame size (the two-layer head, the 16-stream 1x1 head) on the
    input sets already on the device (stream s takes set s mod N_SETS); no CPU baseline."""
    cfg = si.get_config(idx)
    S, C, K = cfg.n_streams, cfg.n_classes, cfg.k_steps
    if cfg.blocks:                      # the stack of blocks has its own channel counts: one input set of its own
        theta0 = si.initial_stack_params(cfg.c_in, cfg.blocks, C, 1000)
        ctx = make_context(st, stream, cfg, theta0, blocks=[tuple(b) for b in cfg.blocks], first_trained=cfg.first_trained)
        own = torch.from_numpy(si.frozen_features(cfg.c_in, cfg.feat_h, cfg.feat_w, 0)).cuda()
        feats_d = [[own]] * N_SETS
        for b in range(len(cfg.blocks)):
            st.st_set_skip_features(ctx, 0, b, torch.from_numpy(si.skip_features(cfg, b, 0)).cuda())
    else:
        theta0 = np.concatenate([si.initial_head_params(cfg.c_in, cfg.c_hidden, C, 1000 + s) for s in range(S)])
        ctx = make_context(st, stream, cfg, theta0)
    packed = torch.empty((S, ctx.n_params), dtype=torch.float32, device="cuda")
    conf = torch.zeros((S, C, C), dtype=torch.int64, device="cuda")
    miou = torch.zeros(S, dtype=torch.float64, device="cuda")
    loss = torch.zeros((S, K), dtype=torch.float32, device="cuda")

    def key_frame(i):
        for s in range(S):
            st.st_set_frozen_features(ctx, s, feats_d[(i + s) % N_SETS][0])
            st.st_teacher_labels(ctx, s, logits_d[(i + s) % N_SETS][0])
        st.st_distill_step(ctx, K, loss)
        for s in range(S):
            st.st_pack_updated_params(ctx, s, packed[s])
            st.st_agreement(ctx, s, None, None, conf[s], miou_out=miou[s:s + 1])

    def sync():
        torch.cuda.synchronize()

    for i in range(3):
        key_frame(i)
    steps = 10 if S == 1 else 4
    clocks = ClockSampler(local_rank)
    clocks.begin()
    ms = timed_blocks(torch, stream, sync, 5, steps, key_frame)
    ms_loop = timed_blocks(torch, stream, sync, 5, steps, lambda i: st.st_distill_step(ctx, K, loss))
    clocks.end()
    kernels = kernel_table(st, ctx, cfg, peaks, arith, 5)
    st.st_destroy(ctx)
    med = statistics.median(ms) / steps
    return {"workload": cfg.name, "steps_per_s": K * S / (med / 1e3), "ms_per_key_frame": med,
            "ms_per_key_frame_min": min(ms) / steps,
            "distill_loop_only": {"steps_per_s": K * S / (statistics.median(ms_loop) / steps / 1e3),
                                  "ms_per_step": statistics.median(ms_loop) / steps / K},
            "streams": S, "c_hidden": cfg.c_hidden, "blocks": [list(b) for b in cfg.blocks], "kernels": kernels, "clocks": clocks.finish(),
            "inputs": f"the {N_SETS} input sets of the main run, stream s on set (key frame + s) mod {N_SETS}"}


def run_confident_student(st, torch, stream, cfg, peaks, arith):
    """The main workload with a student that has learnt its frame: features that carry the class map, trained until the
    mean IoU passes the paper's THRESHOLD of 0.8 (Section 5.3).  Its logits are steep at class boundaries, which is the
    expensive case of the fused upsample + cross-entropy kernel."""
    C, K = cfg.n_classes, cfg.k_steps
    cls = si.voronoi_map(cfg.frame_h, cfg.frame_w, cfg.n_regions, C, 2000)
    feat = si.label_informed_features(cfg.c_in, cfg.feat_h, cfg.feat_w, cls, cfg.up, 0, strength=3.0)
    theta0 = si.initial_head_params(cfg.c_in, cfg.c_hidden, C, 1000)
    ctx = make_context(st, stream, cfg, theta0, lr=0.5)
    st.st_set_frozen_features(ctx, 0, torch.from_numpy(feat).cuda())
    st.st_set_labels(ctx, 0, torch.from_numpy(cls).cuda())
    miou, n_steps = 0.0, 0
    while miou <= 0.8 and n_steps < 200:
        st.st_distill_step(ctx, K)
        n_steps += K
        miou = st.st_agreement(ctx, 0, None, None, None)
    loss = torch.zeros((1, K), dtype=torch.float32, device="cuda")
    ms = timed_blocks(torch, stream, torch.cuda.synchronize, 5, 20, lambda i: st.st_distill_step(ctx, K, loss))
    kernels = kernel_table(st, ctx, cfg, peaks, arith, 10)
    loss_kernel = "fwd1x1_upsample_ce" if "fwd1x1_upsample_ce" in kernels else "upsample_ce"
    out = {"miou_when_timed": miou, "steps_to_get_there": n_steps, "ms_per_step": statistics.median(ms) / 20 / K,
           "upsample_ce_ms": kernels[loss_kernel]["ms"], "upsample_ce_frac": kernels[loss_kernel].get("frac"),
           "loss_kernel": loss_kernel,
           "miou_after": st.st_agreement(ctx, 0, None, None, None)}
    st.st_destroy(ctx)
    return out


def run_ours(args, cfg):
    import torch
    import paper_2003_10735_b200 as st

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    torch.cuda.set_device(local_rank)
    stream = torch.cuda.Stream()
    peaks = read_peaks()
    S, C, K = cfg.n_streams, cfg.n_classes, cfg.k_steps
    H, W, p, P = cfg.frame_h, cfg.frame_w, cfg.feat_h * cfg.feat_w, cfg.frame_h * cfg.frame_w

    with torch.cuda.stream(stream):
        # ---- this device's plain-arithmetic ceilings (fp32 multiply-add, exp2), measured, a few milliseconds
        fma_tflops, ex2_tops = st.st_measure_arithmetic_peaks(stream.cuda_stream)
        arith = {"fma_tflops": fma_tflops, "ex2_tops": ex2_tops}
        # ---- seeded synthetic inputs (each rank its own streams: the path shards by stream, no exchange)
        feats_h, logits_h, thetas = [], [], []
        for i in range(N_SETS):
            per_stream_f, per_stream_t = [], []
            for gs in rank_streams(S, world, rank):
                f = si.frozen_features(cfg.c_in, cfg.feat_h, cfg.feat_w, seed=10 * gs + i)
                t = si.teacher_logits(cfg, stream=gs, frame=i)
                per_stream_f.append(torch.from_numpy(f).pin_memory())
                per_stream_t.append(torch.from_numpy(t).pin_memory())
            feats_h.append(per_stream_f)
            logits_h.append(per_stream_t)
        for s in range(S):
            thetas.append(si.initial_stack_params(cfg.c_in, cfg.blocks, C, 1000 + s) if cfg.blocks
                          else si.initial_head_params(cfg.c_in, cfg.c_hidden, C, 1000 + s))
        theta0 = np.concatenate(thetas)
        theta0_d = torch.from_numpy(theta0).cuda().reshape(S, -1)
        feats_d = [[f.cuda(non_blocking=True) for f in fs] for fs in feats_h]
        logits_d = [[t.cuda(non_blocking=True) for t in ts] for ts in logits_h]
        stack_kw = dict(blocks=[tuple(b) for b in cfg.blocks], first_trained=cfg.first_trained) if cfg.blocks else {}
        ctx = make_context(st, stream, cfg, theta0, **stack_kw)
        for s in range(S if cfg.blocks else 0):      # a stack of blocks: the skip inputs are cached like the features
            for b in range(len(cfg.blocks)):
                st.st_set_skip_features(ctx, s, b, torch.from_numpy(si.skip_features(cfg, b, s)).cuda())
        n_params = ctx.n_params
        packed_d = torch.empty((S, n_params), dtype=torch.float32, device="cuda")
        packed_h = torch.empty((S, n_params), dtype=torch.float32).pin_memory()
        conf_d = torch.zeros((S, C, C), dtype=torch.int64, device="cuda")
        loss_d = torch.zeros((S, K), dtype=torch.float32, device="cuda")
        mious = [0.0] * S
        miou_d = torch.zeros(S, dtype=torch.float64, device="cuda")

        def key_frame(i, feats, logits, packed, results_on_device=True):
            fs, ts = feats[i % N_SETS], logits[i % N_SETS]
            for s in range(S):
                st.st_set_frozen_features(ctx, s, fs[s])
                st.st_teacher_labels(ctx, s, ts[s])
            st.st_distill_step(ctx, K, loss_d)
            for s in range(S):
                st.st_pack_updated_params(ctx, s, packed[s])
                if results_on_device:       # the mean IoU stays on the device like the packed parameters: no wait
                    st.st_agreement(ctx, s, None, None, conf_d[s], miou_out=miou_d[s:s + 1])
                else:                       # end to end: the mean IoU comes back to the host every key frame
                    mious[s] = st.st_agreement(ctx, s, None, None, conf_d[s])

        def barrier():
            if dist is not None:
                dist.barrier()
            torch.cuda.synchronize()

        def reset_parameters():             # outside every timed region: each block starts from the initial student
            for s in range(S):
                st.st_apply_update(ctx, s, theta0_d[s])

        # A timed block is exactly --steps key frames.  Short blocks are repeated so that about two thousand key frames
        # are timed in all; the reported value is the median block (the minimum is given beside it).
        n_blocks = args.blocks if args.blocks > 0 else max(1, min(101, -(-2000 // args.steps)))
        if n_blocks > 1 and n_blocks % 2 == 0:
            n_blocks += 1

        # ---- device-resident run
        for i in range(args.warmup):
            key_frame(i, feats_d, logits_d, packed_d)
        clocks = ClockSampler(local_rank) if rank == 0 else None
        barrier()
        launches0 = st.st_launch_count(ctx)
        if clocks:
            clocks.begin()
        block_ms = timed_blocks(torch, stream, barrier, n_blocks, args.steps,
                                lambda i: key_frame(i, feats_d, logits_d, packed_d), between=reset_parameters)
        if clocks:
            clocks.end()
        launches = (st.st_launch_count(ctx) - launches0 - n_blocks * S * (2 if cfg.gemm_precision == 1 else 1)) // n_blocks
        last_miou_dev = float(miou_d[0].item())
        block_ms = [max_over_ranks(m, dist, "cuda") for m in block_ms]
        ms_total = statistics.median(block_ms)
        clock_info = clocks.finish() if clocks else None

        # ---- the K-step loop alone (inputs already cached), for the per-step view
        n_loop = max(10, min(args.steps, 200))
        ms_loop = statistics.median(timed_blocks(torch, stream, barrier, 5, n_loop, lambda i: st.st_distill_step(ctx, K, loss_d),
                                                 between=reset_parameters)) / n_loop

        # ---- end to end through the C ABI with host buffers (pinned): H2D of the inputs, D2H of the results.
        # Every key frame's inputs cross PCIe inside the timed region; the copy of key frame i+1 is started (on the
        # library's copy stream) as soon as key frame i has been handed to the kernels, so that it runs beside them.
        e2e_steps = max(3, min(args.steps, 100))

        def key_frame_e2e(i):
            for s in range(S):
                st.st_use_prefetched_key_frame(ctx, s)
            for s in range(S):
                st.st_prefetch_key_frame(ctx, s, feats_h[(i + 1) % N_SETS][s], logits_h[(i + 1) % N_SETS][s])
            st.st_distill_step(ctx, K, loss_d)
            for s in range(S):
                st.st_pack_updated_params(ctx, s, packed_h[s])
                mious[s] = st.st_agreement(ctx, s, None, None, conf_d[s])

        e2e_plain_ms = timed_blocks(torch, stream, barrier, 1, e2e_steps,
                                    lambda i: key_frame(i, feats_h, logits_h, packed_h, results_on_device=False), between=reset_parameters)

        def prime():                        # block b starts at key frame b * e2e_steps: its inputs are on their way
            reset_parameters()
            for s in range(S):
                st.st_prefetch_key_frame(ctx, s, feats_h[prime.next % N_SETS][s], logits_h[prime.next % N_SETS][s])
            prime.next += e2e_steps
        prime.next = 0
        e2e_ms = timed_blocks(torch, stream, barrier, 3, e2e_steps, key_frame_e2e, between=prime)
        ms_e2e = statistics.median([max_over_ranks(m, dist, "cuda") for m in e2e_ms])
        h2d = S * (cfg.c_in * p * 4 + C * P * 4)
        d2h = S * (n_params * 4 + 8)

        # ---- per-kernel times with CUDA events on the launching stream
        kernels, train, others, confident, unfused = {}, {}, {}, None, None
        if rank == 0:
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

            def timed(fn, reps=20):
                ev0.record(stream)
                for r in range(reps):
                    fn(r)
                ev1.record(stream)
                torch.cuda.synchronize()
                return ev0.elapsed_time(ev1) / reps
            t_arg = timed(lambda r: st.st_teacher_labels(ctx, 0, logits_d[r % N_SETS][0]))
            t_feat = timed(lambda r: st.st_set_frozen_features(ctx, 0, feats_d[r % N_SETS][0]))
            hbm = peaks["hbm_gbs"]
            kernels["argmax_u8"] = {"ms": t_arg, "bound": "hbm", "achieved": (C * P * 4 + P) / t_arg / 1e6,
                                    "peak": hbm, "unit": "GB/s", "per_key_frame": S}
            if cfg.gemm_precision == 1:
                kernels["feat_to_bf16_nhwc"] = {"ms": t_feat, "bound": "hbm", "achieved": cfg.c_in * p * 6 / t_feat / 1e6,
                                                "peak": hbm, "unit": "GB/s", "per_key_frame": S}
            # agreement of two given masks: the kernel alone (results delivered into device buffers: one launch, no copy,
            # no wait; launched back to back) and the whole call with the mean IoU read back by the host
            rng = np.random.default_rng(0)
            lab_map = si.voronoi_map(H, W, cfg.n_regions, C, 2000)
            # a prediction like a trained student's: the same regions with their borders a few pixels off, plus 1 % of stray pixels
            moved = np.roll(lab_map, (3, 5), axis=(0, 1))
            noisy = np.where(rng.random((H, W)) < 0.99, moved, rng.integers(0, C, (H, W))).astype(np.uint8)
            m_coh = [torch.from_numpy(lab_map).cuda(), torch.from_numpy(noisy).cuda()]
            m_rnd = [torch.randint(0, C, (H, W), dtype=torch.uint8, device="cuda") for _ in range(2)]
            agree = {}
            for name, (a, b) in (("coherent_masks", m_coh), ("random_masks", m_rnd)):
                t_k = timed(lambda r: st.st_agreement(ctx, 0, a, b, conf_d[0], miou_out=miou_d[0:1]), reps=50)
                t_c = timed(lambda r: st.st_agreement(ctx, 0, a, b, conf_d[0]), reps=20)
                agree[name] = {"kernel_us": t_k * 1e3, "call_us": t_c * 1e3, "kernel_gbs": 2 * P / t_k / 1e6,
                               "kernel_frac_of_hbm": 2 * P / t_k / 1e6 / hbm}
            # the same counting kernel on sixteen frames' worth of pixels in one launch (the no-context entry point takes
            # any length): what the kernel reaches when it has more than one wave of work
            big = [m.repeat(16, 1) for m in m_coh]
            t_big = timed(lambda r: st.st_agreement_noalloc(big[1], big[0], C, stream.cuda_stream, conf_d[0], miou_d[0:1]), reps=20)
            agree["coherent_masks_16_frames"] = {"kernel_us": t_big * 1e3, "kernel_gbs": 32 * P / t_big / 1e6,
                                                 "kernel_frac_of_hbm": 32 * P / t_big / 1e6 / hbm,
                                                 "note": "memset + counting kernel + mean-IoU kernel of st_agreement_noalloc"}
            del big
            t_own = timed(lambda r: st.st_agreement(ctx, 0, None, None, conf_d[0], miou_out=miou_d[0:1]), reps=50)
            agree["student_mask_fused"] = {"kernel_us": t_own * 1e3, "note": "arg-max of the upsampled logits + confusion + mean IoU, forward reused"}
            kernels["agreement"] = {"ms": agree["coherent_masks"]["kernel_us"] / 1e3, "bound": "latency", "per_key_frame": S, **agree}
            kernels.update(kernel_table(st, ctx, cfg, peaks, arith, 20))
            if "fwd1x1_upsample_ce" in kernels:
                # the same step with the classifier's forward in its own kernel, for the two kernels' own rooflines
                os.environ[FUSED_SWITCH] = "0"
                ctx_u = make_context(st, stream, cfg, theta0)
                os.environ.pop(FUSED_SWITCH)
                st.st_set_frozen_features(ctx_u, 0, feats_d[0][0])
                st.st_teacher_labels(ctx_u, 0, logits_d[0][0])
                for _ in range(3):
                    st.st_distill_step(ctx_u, K, loss_d[0:1])
                ms_u = statistics.median(timed_blocks(torch, stream, barrier, 5, 50, lambda i: st.st_distill_step(ctx_u, K, loss_d[0:1]))) / 50
                unfused = kernel_table(st, ctx_u, si.get_config(args.workload), peaks, arith, 20)
                unfused["distill_loop_only_ms_per_step"] = ms_u / K
                st.st_destroy(ctx_u)
            # Train of Algorithm 1 (forward, metric, break test and best-student snapshot per update, all on the device):
            # the full loop (a threshold no mean IoU reaches) and a loop that ends on the first metric
            for name, thr in (("full_loop", 2.0), ("ends_at_once", 0.0)):
                for _ in range(3):
                    st.st_train_key_frame(ctx, thr, K)
                train[name + "_ms"] = timed(lambda r: st.st_train_key_frame(ctx, thr, K), reps=20)
            train["max_updates"] = K

        result = None
        if rank == 0:
            ms_step = ms_total / args.steps
            value = whole_job_rate(K * S * args.steps, world, ms_total)      # SGD iterations of all streams of all ranks
            dominant = max(kernels, key=lambda n: kernels[n]["ms"] * kernels[n]["per_key_frame"])
            dk = kernels[dominant]
            # DRAM bytes per launch from the ncu capture summarised in profiles/ (same kernel, same workload)
            traffic = NCU_DRAM_BYTES.get((args.workload, dominant))
            roofline = {"kernel": dominant, "bound": dk.get("bound"), "achieved": dk.get("achieved"), "peak": dk.get("peak"),
                        "unit": dk.get("unit"), "frac": dk.get("frac"), "traffic": traffic,
                        "peak_source": f"of {peaks['source']}" if dk.get("bound") in ("hbm", "tensor") else
                                       "fp32 multiply-add rate measured on this device by st_measure_arithmetic_peaks",
                        "ms_per_launch": dk["ms"]}
            if dk.get("bound") == "alu":
                roofline.update(algorithmic_flop_per_class_pixel=ALU_FLOP_PER_CLASS_PIXEL, xu=dk.get("xu"),
                                derived_fma_peak_tflops=148 * 128 * 2 * peaks["sm_max_mhz"] * 1e6 / 1e12)
            result = {
                "metric": METRIC, "value": value, "unit": "steps/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16" if cfg.gemm_precision == 1 else "f32", "data": "synthetic",
                "config": {"workload": cfg.name, "k_steps": K, "frame": [H, W], "features": [cfg.c_in, cfg.feat_h, cfg.feat_w],
                           "classes": C, "streams_per_gpu": S, "c_hidden": cfg.c_hidden,
                           "step": "features cache + labels + K SGD iterations + pack + agreement per key frame",
                           "l2": f"inputs rotate over {N_SETS} key frames ({N_SETS * S * (cfg.c_in * p + C * P) * 4 / 1e6:.0f} MB) > 126 MB L2",
                           "parallelism": f"replicas x{world}, no collective",
                           "timed_blocks": f"{n_blocks} blocks of {args.steps} key frames, parameters reset before each; value = median block"},
                "timed_blocks": {"n": n_blocks, "ms_median": ms_total, "ms_min": min(block_ms), "ms_max": max(block_ms),
                                 "value_of_fastest_block": whole_job_rate(K * S * args.steps, world, min(block_ms))},
                "clocks": clock_info,
                "e2e": {"value": world * K * S * e2e_steps / (ms_e2e / 1e3), "unit": "steps/s", "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / e2e_steps,
                        "calls": "st_use_prefetched_key_frame, st_prefetch_key_frame (next key frame), st_distill_step, "
                                 "st_pack_updated_params (host), st_agreement (host)",
                        "ms_per_step_without_prefetch": e2e_plain_ms[0] / e2e_steps},
                "gpu_launches": int(launches),
                "roofline": roofline,
                "arithmetic_peaks": arith,
                "key_frames_per_s": world * args.steps / (ms_total / 1e3),
                "distill_loop_only": {"steps_per_s": K * S / (ms_loop / 1e3), "ms_per_k_steps": ms_loop},
                "kernels": kernels, "kernels_unfused": unfused, "train_key_frame": train,
                "last_loss": float(loss_d[0, -1].item()), "last_miou": mious[0], "last_miou_device_run": last_miou_dev,
            }
        st.st_destroy(ctx)

        # ---- beside the headline: the same workload with a trained student, and the other workloads of this frame size
        if rank == 0 and world == 1 and not args.headline_only and args.workload == 2:
            result["confident_student"] = run_confident_student(st, torch, stream, cfg, peaks, arith)
            result["other_workloads"] = {str(idx): run_other_workload(st, torch, stream, idx, feats_d, logits_d, peaks, arith, local_rank)
                                         for idx in (3, 5, 6)}

    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            oracle.build()
            feat, T, theta = si.stream_inputs(cfg)
            rows = cfg.feat_h if cfg.c_hidden == 0 else max(4, cfg.feat_h // 16)
            t_first = oracle_key_frame(cfg, feat, T, theta, rows=rows)       # also warms the oracle's library up
            n_rep = int(max(1, min(40, round(12.0 / max(t_first, 1e-3)))))    # about 12 s of CPU work in all
            t = sum(oracle_key_frame(cfg, feat, T, theta, rows=rows) for _ in range(n_rep)) / n_rep
            frac = rows / cfg.feat_h
            result["cpu_baseline"] = {
                "value": cfg.k_steps / t * frac, "unit": "steps/s", "cores": host_cores(), "kind": "oracle",
                "sample": (f"{n_rep} key frames (labels, {cfg.k_steps} steps, pack, agreement) of one stream on {rows} of "
                           f"{cfg.feat_h} feature rows, {t:.2f} s each, scaled by pixel count"),
            }
        print(json.dumps(result), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=2, help="index into the synthetic workload table (2 = 720p, 1x1 head, K=8)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--blocks", type=int, default=0, help="timed blocks of --steps key frames (0: enough for about 2000 key frames)")
    ap.add_argument("--headline-only", action="store_true", help="skip the trained-student and other-workload runs")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = si.get_config(args.workload)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
