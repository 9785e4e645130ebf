"""Full-size workloads in the launch configuration the benchmark uses, checked against the oracle
where it finishes in seconds (a stream or a few steps computed in full) and through properties that
hold at any size for the rest."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
import paper_2003_10735_b200 as st

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(autouse=True)
def side_stream():
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        yield s
    s.synchronize()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def ctx_for(cfg, theta, S=1):
    return st.st_init_head(n_streams=S, c_in=cfg.c_in, c_hidden=cfg.c_hidden, n_classes=cfg.n_classes,
                           feat_h=cfg.feat_h, feat_w=cfg.feat_w, gemm_precision=cfg.gemm_precision, lr=cfg.lr,
                           momentum=cfg.momentum, cuda_stream=torch.cuda.current_stream().cuda_stream, init_params=theta)


def packed(ctx, s=0):
    out = np.empty(ctx.n_params, np.float32)
    st.st_pack_updated_params(ctx, s, out)
    return out


def rel_l2(a, b):
    return float(np.linalg.norm(a.astype(np.float64) - b) / max(np.linalg.norm(b), 1e-30))


def check_step_properties(conf, lab, C):
    for k in range(conf.shape[0]):
        assert conf[k].sum() == lab.size                                           # every pixel counted once
        np.testing.assert_array_equal(conf[k].sum(1), np.bincount(lab.ravel(), minlength=C))


def two_layer_prefix_vs_oracle(cfg, feat, T, theta, n_ref_steps):
    """GPU K = n_ref_steps from the initial parameters against the oracle, element by element."""
    ctx = ctx_for(cfg, theta)
    st.st_set_frozen_features(ctx, 0, dev(feat))
    st.st_teacher_labels(ctx, 0, dev(T))
    loss = np.zeros(n_ref_steps, np.float32)
    st.st_distill_step(ctx, n_ref_steps, loss)
    got = packed(ctx)
    st.st_destroy(ctx)
    lab = oracle.teacher_labels(T)
    head = oracle.Head(cfg.c_in, cfg.c_hidden, cfg.n_classes, lr=cfg.lr, momentum=cfg.momentum, theta=theta)
    ref_loss = [oracle.distill_step(head, feat, lab)[0] for _ in range(n_ref_steps)]
    np.testing.assert_allclose(loss, ref_loss, rtol=1e-4)                            # stated: 1e-4 relative
    off = 0
    for ws, bs in oracle.param_shapes(cfg.c_in, cfg.c_hidden, cfg.n_classes):
        for n in (int(np.prod(ws)), int(np.prod(bs))):
            g, r = got[off:off + n], head.theta[off:off + n]
            assert np.abs(g - r).max() / max(np.abs(r).max(), 1e-6) <= 2e-2            # stated: 2e-2 max relative
            off += n
    assert np.abs(got - head.theta).mean() <= 1e-3                                   # stated: 1e-3 mean absolute
    assert rel_l2(got - theta, head.theta.astype(np.float64) - theta) <= 2e-2        # update vector
    return lab


def test_config3_two_layer_720p_two_key_frames():
    cfg = si.get_config(3)
    theta = si.initial_head_params(cfg.c_in, cfg.c_hidden, cfg.n_classes, 1000)
    frames = si.key_frame_indices(cfg)
    assert frames == [0, 8]
    feat0, T0 = si.frozen_features(cfg.c_in, cfg.feat_h, cfg.feat_w, 0), si.teacher_logits(cfg, 0, 0)
    two_layer_prefix_vs_oracle(cfg, feat0, T0, theta, 1)
    # the whole clip on the GPU: parameters and momentum persist across key frames
    ctx = ctx_for(cfg, theta)
    K, C = cfg.k_steps, cfg.n_classes
    losses = []
    for f in frames:
        feat, T = si.frozen_features(cfg.c_in, cfg.feat_h, cfg.feat_w, f), si.teacher_logits(cfg, 0, f)
        labels = torch.empty((cfg.frame_h, cfg.frame_w), dtype=torch.uint8, device="cuda")
        st.st_set_frozen_features(ctx, 0, dev(feat))
        st.st_teacher_labels(ctx, 0, dev(T), labels)
        lab = oracle.teacher_labels(T)
        np.testing.assert_array_equal(labels.cpu().numpy(), lab)
        loss = torch.zeros(K, dtype=torch.float32, device="cuda")
        conf = torch.zeros((K, C, C), dtype=torch.int64, device="cuda")
        st.st_distill_step(ctx, K, loss, conf)
        check_step_properties(conf.cpu().numpy(), lab, C)
        losses.append(loss.cpu().numpy())
        mask = torch.empty_like(labels)
        st.st_student_mask(ctx, 0, mask)
        gconf = np.zeros((C, C), np.int64)
        m = st.st_agreement(ctx, 0, None, None, gconf)
        oconf, om, _ = oracle.agreement(lab, mask.cpu().numpy(), C)
        np.testing.assert_array_equal(gconf, oconf)
        assert m == om
    assert np.isfinite(np.concatenate(losses)).all()
    assert losses[0][-1] < losses[0][0]                         # training makes progress on a key frame
    raw = packed(ctx)
    assert raw.nbytes == 2381908
    assert np.isfinite(raw).all()
    st.st_destroy(ctx)


GAP = 4e-2      # top-2 logit gap below which a pixel counts as a near-tie of the bf16 student: twice the largest
                # logit error that bf16 operands cause in these heads (about 3e-3 typical, 1.5e-2 at most)


@pytest.mark.parametrize("idx,rows", [(3, 10), (4, 10)])
def test_two_layer_full_channels_full_width_band_k8_two_key_frames(idx, rows):
    """The two-layer workloads at their full channel counts (256 -> 256 -> 21 / 19) and full width, on a band of
    feature rows the oracle finishes in seconds: K = 8 steps with momentum on each of two key frames (parameters and
    momentum carried over), every step's loss, the final parameters of each key frame and every step's fused
    confusion matrix against the plain oracle."""
    full = si.get_config(idx)
    cfg = si.WorkloadConfig("band", full.c_in, full.c_hidden, full.n_classes, rows, full.feat_w, k_steps=8, lr=full.lr,
                            momentum=full.momentum, gemm_precision=1, n_regions=24, teacher=full.teacher)
    C, K = cfg.n_classes, cfg.k_steps
    theta = si.initial_head_params(cfg.c_in, cfg.c_hidden, C, 1000)
    ctx = ctx_for(cfg, theta)
    head = oracle.Head(cfg.c_in, cfg.c_hidden, C, lr=cfg.lr, momentum=cfg.momentum, theta=theta)
    # the oracle with its operands rounded where the tensor-core path rounds them: what is left is summation order
    # and the rare hidden value that rounds the other way
    head_q = oracle.Head(cfg.c_in, cfg.c_hidden, C, lr=cfg.lr, momentum=cfg.momentum, theta=theta, quantize_bf16=True)
    # The stated 1e-4 on the loss is for whole frames; the rounding noise of bf16 operands averages down with the
    # square root of the pixel count, and this band has a sixteenth to a twenty-seventh of a frame's pixels.
    loss_tol = 1e-4 * np.sqrt(full.feat_h / rows)
    start = theta
    for frame in (0, 1):
        feat = si.frozen_features(cfg.c_in, cfg.feat_h, cfg.feat_w, 7 + frame)
        T = si.teacher_logits(cfg, stream=frame, frame=0)
        st.st_set_frozen_features(ctx, 0, dev(feat))
        st.st_teacher_labels(ctx, 0, dev(T))
        loss = np.zeros(K, np.float32)
        conf = np.zeros((K, C, C), np.int64)
        st.st_distill_step(ctx, K, loss, conf)
        got = packed(ctx)
        lab = oracle.teacher_labels(T)
        ref_loss, masks, near_ties = [], [], []
        for _ in range(K):
            z_ref, _ = oracle.head_forward(head, feat)
            top2 = np.sort(oracle.upsample(z_ref, cfg.up), axis=0)[-2:]
            near_ties.append(int((top2[1] - top2[0] < GAP).sum()))                       # pixels whose class a logit error can flip
            l, m = oracle.distill_step(head, feat, lab)
            ref_loss.append(l); masks.append(m)
        # the logits of the last step's forward: bf16 operands against the plain oracle, well inside the gap that
        # defines a near-tie (two logits moving toward each other by this much close a gap of twice as much)
        z = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGITS)
        assert np.abs(z - z_ref.ravel()).max() <= GAP / 2
        np.testing.assert_allclose(loss, ref_loss, rtol=loss_tol)
        q_loss = [oracle.distill_step(head_q, feat, lab)[0] for _ in range(K)]
        np.testing.assert_allclose(loss, q_loss, rtol=3e-5)
        q_upd = rel_l2(got - start, head_q.theta.astype(np.float64) - start)
        assert q_upd <= 5e-3, q_upd
        off = 0
        for ws, bs in oracle.param_shapes(cfg.c_in, cfg.c_hidden, C):
            for n in (int(np.prod(ws)), int(np.prod(bs))):
                g, r = got[off:off + n], head.theta[off:off + n]
                assert np.abs(g - r).max() / max(np.abs(r).max(), 1e-6) <= 2e-2            # stated: 2e-2 max relative
                off += n
        assert np.abs(got - head.theta).mean() <= 1e-3                                   # stated: 1e-3 mean absolute
        upd = rel_l2(got - start, head.theta.astype(np.float64) - start)
        print(f"workload {idx} band, key frame {frame}: loss err {np.abs(loss / np.array(ref_loss) - 1).max():.1e} "
              f"(rounded-operand oracle {np.abs(loss / np.array(q_loss) - 1).max():.1e}), update rel-L2 {upd:.1e} ({q_upd:.1e})")
        assert upd <= 2e-2                                                                # update of this key frame
        check_step_properties(conf, lab, C)
        for k in range(K):
            # the student's class may differ from the oracle's only at near-ties; each such pixel moves two cells by one
            ref_c, _, _ = oracle.agreement(lab, masks[k], C)
            moved = int(np.abs(conf[k] - ref_c).sum())
            assert moved <= 2 * near_ties[k], k
            assert near_ties[k] <= lab.size // 5, k                                       # near-ties stay the exception
            # what Algorithm 1 decides on: the metric of the step's prediction
            assert abs(oracle.miou(conf[k]) - oracle.miou(ref_c)) <= 5e-3, k
            if k in (0, K - 1):
                print(f"  step {k}: {moved // 2} of {lab.size} pixels differ, {near_ties[k]} near-ties, "
                      f"mIoU {oracle.miou(conf[k]):.4f} vs {oracle.miou(ref_c):.4f}")
        start = head.theta.copy()
    st.st_destroy(ctx)


def test_config4_two_layer_1080p_k16_agreement_every_step():
    cfg = si.get_config(4)
    feat, T, theta = si.stream_inputs(cfg)
    lab = two_layer_prefix_vs_oracle(cfg, feat, T, theta, 1)
    ctx = ctx_for(cfg, theta)
    K, C = cfg.k_steps, cfg.n_classes
    st.st_set_frozen_features(ctx, 0, dev(feat))
    labels = torch.empty((cfg.frame_h, cfg.frame_w), dtype=torch.uint8, device="cuda")
    st.st_teacher_labels(ctx, 0, dev(T), labels)
    np.testing.assert_array_equal(labels.cpu().numpy(), lab)    # blurred boundaries: exact ties, lowest class wins
    loss = torch.zeros(K, dtype=torch.float32, device="cuda")
    conf = torch.zeros((K, C, C), dtype=torch.int64, device="cuda")
    st.st_distill_step(ctx, K, loss, conf)
    c = conf.cpu().numpy()
    check_step_properties(c, lab, C)
    l = loss.cpu().numpy()
    assert np.isfinite(l).all() and l[-1] < l[0]
    # mIoU of every step from the fused counts, through the oracle's definition
    mious = [oracle.miou(c[k]) for k in range(K)]
    assert all(0.0 <= m <= 1.0 for m in mious)
    assert packed(ctx).nbytes == 2379852
    st.st_destroy(ctx)


def test_config5_sixteen_streams_grouped():
    cfg = si.get_config(5)
    S, K, C = cfg.n_streams, cfg.k_steps, cfg.n_classes
    thetas = [si.initial_head_params(cfg.c_in, 0, C, 1000 + s) for s in range(S)]
    ctx = ctx_for(cfg, np.concatenate(thetas), S=S)
    keep = {}
    for s in range(S):
        feat = si.frozen_features(cfg.c_in, cfg.feat_h, cfg.feat_w, s)
        T = si.teacher_logits(cfg, s, 0)
        st.st_set_frozen_features(ctx, s, dev(feat))
        st.st_teacher_labels(ctx, s, dev(T))
        if s in (0, 11):
            keep[s] = (feat, T)
    loss = torch.zeros((S, K), dtype=torch.float32, device="cuda")
    conf = torch.zeros((S, K, C, C), dtype=torch.int64, device="cuda")
    st.st_distill_step(ctx, K, loss, conf)
    l = loss.cpu().numpy()
    c = conf.cpu().numpy()
    assert np.isfinite(l).all()
    for s in range(S):
        assert c[s].sum() == K * cfg.frame_h * cfg.frame_w
        assert packed(ctx, s).nbytes == 21588
    for s, (feat, T) in keep.items():                           # two streams in full against the oracle
        lab = oracle.teacher_labels(T)
        head = oracle.Head(cfg.c_in, 0, C, lr=cfg.lr, momentum=cfg.momentum, theta=thetas[s])
        ref = [oracle.distill_step(head, feat, lab)[0] for _ in range(K)]
        np.testing.assert_allclose(l[s], ref, rtol=1e-4)
        got = packed(ctx, s)
        assert np.abs(got - head.theta).max() / np.abs(head.theta).max() <= 2e-2
        assert np.abs(got - head.theta).mean() <= 1e-3
        assert rel_l2(got - thetas[s], head.theta.astype(np.float64) - thetas[s]) <= 2e-2
        check_step_properties(c[s], lab, C)
        gconf = np.zeros((C, C), np.int64)
        mask = torch.empty((cfg.frame_h, cfg.frame_w), dtype=torch.uint8, device="cuda")
        st.st_student_mask(ctx, s, mask)
        m = st.st_agreement(ctx, s, None, None, gconf)
        oconf, om, _ = oracle.agreement(lab, mask.cpu().numpy(), C)
        np.testing.assert_array_equal(gconf, oconf)
        assert m == om
    st.st_destroy(ctx)


def test_train_key_frame_720p_early_exit_is_cheaper_than_the_full_loop():
    """Algorithm 1 at frame size (720p, 1x1 head, bf16 GEMMs) on label-informed features: the loop ends as soon as
    the mean IoU passes THRESHOLD, the result is the plain loop's iterate, and the ended loop costs little."""
    cfg = si.get_config(2)
    C, K = cfg.n_classes, 8
    cls = si.voronoi_map(cfg.frame_h, cfg.frame_w, cfg.n_regions, C, 2000)
    feat = si.label_informed_features(cfg.c_in, cfg.feat_h, cfg.feat_w, cls, 4, 0, strength=3.0)
    theta = si.initial_head_params(cfg.c_in, 0, C, 1000)
    stream = torch.cuda.current_stream()

    def fresh():
        ctx = st.st_init_head(n_streams=1, c_in=cfg.c_in, c_hidden=0, n_classes=C, feat_h=cfg.feat_h, feat_w=cfg.feat_w,
                              gemm_precision=1, lr=0.5, momentum=0.9, cuda_stream=stream.cuda_stream, init_params=theta)
        st.st_set_frozen_features(ctx, 0, torch.from_numpy(feat).cuda())
        st.st_set_labels(ctx, 0, torch.from_numpy(cls).cuda())
        return ctx

    def timed(ctx, thr):
        n_upd = np.zeros(1, np.int32); best = np.zeros(1, np.float64); met = np.zeros((1, K + 1), np.float64)
        st.st_train_key_frame(ctx, thr, K, n_upd, best, met)            # first call: captures the graph
        out = (int(n_upd[0]), float(best[0]), met[0].copy())
        ts = []
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d_n = torch.zeros(1, dtype=torch.int32, device="cuda")
        for _ in range(3):
            e0.record(stream); st.st_train_key_frame(ctx, thr, K, d_n); e1.record(stream); stream.synchronize()
            ts.append(e0.elapsed_time(e1))
        return out, min(ts)

    ctx = fresh()
    (n_full, best_full, met_full), _ = timed(ctx, 2.0)
    assert n_full == K and met_full[-1] > met_full[0] + 0.3, met_full      # the student learns the frame
    st.st_destroy(ctx)
    thr = 0.5 * (met_full[1] + met_full[2])                                  # passed after the second update
    ctx = fresh()
    (n, best, met), _ = timed(ctx, thr)
    assert n == 2 and best == met[2] > thr and (met[3:] == -1).all()
    ref = fresh()
    st.st_distill_step(ref, 2, None, torch.zeros((1, 2, C, C), dtype=torch.int64, device="cuda"))   # same loss-kernel instantiation as Train
    a, b = np.empty(ctx.n_params, np.float32), np.empty(ctx.n_params, np.float32)
    st.st_pack_updated_params(ctx, 0, a); st.st_pack_updated_params(ref, 0, b)
    # (the timed replays above ran Train again from the returned student: with the threshold already met they take
    # no step, so the parameters are still those of the first call)
    assert a.tobytes() == b.tobytes()
    # cost of a call whose loop ends at once (threshold met by the incoming student) vs the full loop
    _, t_done = timed(ctx, thr)
    full = fresh()
    _, t_full = timed(full, 2.0)
    print(f"Train 720p K=8: full loop {t_full * 1e3:.0f} us, loop ended at once {t_done * 1e3:.0f} us")
    assert t_done < 0.5 * t_full
    for c in (ctx, ref, full):
        st.st_destroy(c)
