"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by element,
on the same seeded inputs.  Integer/byte results must be bit-exact; floating point within the
tolerances written next to each assertion."""
import numpy as np
import pytest

import oracle
import synth_inputs as si
import paper_2003_10735_b200 as st

pytestmark = pytest.mark.gpu
torch = pytest.importorskip("torch")


@pytest.fixture(autouse=True)
def side_stream():
    """Run every test on a non-default stream (step loops are then replayed as CUDA graphs)."""
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        yield s
    s.synchronize()


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def make_ctx(c_in, c_hidden, C, h, w, theta, S=1, prec=0, lr=0.01, mu=0.0):
    return st.st_init_head(n_streams=S, c_in=c_in, c_hidden=c_hidden, n_classes=C, feat_h=h, feat_w=w,
                           gemm_precision=prec, lr=lr, momentum=mu,
                           cuda_stream=torch.cuda.current_stream().cuda_stream, init_params=theta)


def packed(ctx, stream=0):
    out = np.empty(ctx.n_params, np.float32)
    assert st.st_pack_updated_params(ctx, stream, out) == out.nbytes
    return out


def rand_problem(seed, c_in, C, h, w, blobs=True):
    rng = np.random.default_rng(seed)
    feat = np.maximum(rng.standard_normal((c_in, h, w)), 0).astype(np.float32)
    if blobs:
        cfg = si.WorkloadConfig("t", c_in, 0, C, h, w, n_regions=max(4, C), teacher="onehot_noise")
        T = si.teacher_logits(cfg, stream=seed)
    else:
        T = rng.standard_normal((C, 4 * h, 4 * w)).astype(np.float32)
    return feat, T


# ---------------------------------------------------------------------------- K1 labels
@pytest.mark.parametrize("C,h,w", [(4, 90, 160), (21, 13, 17), (2, 1, 1), (255, 3, 5)])
def test_teacher_labels_bit_exact(C, h, w):
    rng = np.random.default_rng(C)
    T = rng.integers(-3, 4, size=(C, 4 * h, 4 * w)).astype(np.float32)       # plenty of exact ties
    T += (rng.random(T.shape) < 0.5) * rng.standard_normal(T.shape).astype(np.float32)
    ctx = make_ctx(8, 0, C, h, w, np.zeros(st.st_param_count(8, 0, C), np.float32))
    out = torch.empty((4 * h, 4 * w), dtype=torch.uint8, device="cuda")
    st.st_teacher_labels(ctx, 0, dev(T), out)
    ref = oracle.teacher_labels(T)
    np.testing.assert_array_equal(out.cpu().numpy(), ref)
    # host input and host output go through the same kernel
    out_h = np.empty((4 * h, 4 * w), np.uint8)
    st.st_teacher_labels(ctx, 0, T, out_h)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(out_h, ref)
    st.st_destroy(ctx)


def test_teacher_labels_blurred_boundaries_full_1080p():
    cfg = si.get_config(4)
    T = si.teacher_logits(cfg)
    ctx = make_ctx(8, 0, cfg.n_classes, cfg.feat_h, cfg.feat_w, np.zeros(st.st_param_count(8, 0, cfg.n_classes), np.float32))
    out = torch.empty((cfg.frame_h, cfg.frame_w), dtype=torch.uint8, device="cuda")
    st.st_teacher_labels(ctx, 0, dev(T), out)
    np.testing.assert_array_equal(out.cpu().numpy(), oracle.teacher_labels(T))
    st.st_destroy(ctx)


# ---------------------------------------------------------------------------- K6 agreement
@pytest.mark.parametrize("C,h,w", [(4, 90, 160), (21, 45, 80), (3, 1, 1), (200, 5, 7)])
def test_confusion_and_miou_bit_exact(C, h, w):
    rng = np.random.default_rng(C + 1)
    P = 16 * h * w
    lab = np.repeat(rng.integers(0, C, P // 8 + 1), 8)[:P].astype(np.uint8).reshape(4 * h, 4 * w)   # coherent runs
    pred = np.where(rng.random((4 * h, 4 * w)) < 0.7, lab, rng.integers(0, C, (4 * h, 4 * w))).astype(np.uint8)
    ctx = make_ctx(8, 0, C, h, w, np.zeros(st.st_param_count(8, 0, C), np.float32))
    conf = torch.zeros((C, C), dtype=torch.int64, device="cuda")
    m = st.st_agreement(ctx, 0, dev(pred), dev(lab), conf)
    ref_conf, ref_m, _ = oracle.agreement(lab, pred, C)
    np.testing.assert_array_equal(conf.cpu().numpy(), ref_conf)
    assert m == ref_m                                              # same integer counts, same double arithmetic order
    conf_h = np.zeros((C, C), np.int64)
    m2 = st.st_agreement(ctx, 0, pred, lab, conf_h)                # host masks
    np.testing.assert_array_equal(conf_h, ref_conf)
    assert m2 == ref_m
    m_dev = torch.zeros(1, dtype=torch.float64, device="cuda")     # device destination: written on the stream, no wait
    assert st.st_agreement(ctx, 0, dev(pred), dev(lab), conf, miou_out=m_dev) is None
    torch.cuda.current_stream().synchronize()
    assert float(m_dev.item()) == ref_m
    st.st_destroy(ctx)


def test_prefetched_key_frames_equal_plain_ones():
    """Inputs brought in by st_prefetch_key_frame (the library's copy stream, while the previous key frame trains) give
    exactly the labels, losses and parameters of the plain calls."""
    C, c_in, h, w, K = 6, 8, 11, 19, 3
    theta = si.initial_head_params(c_in, 0, C, 3)
    frames = [rand_problem(20 + f, c_in, C, h, w) for f in range(3)]
    pinned = [(torch.from_numpy(f).pin_memory(), torch.from_numpy(T).pin_memory()) for f, T in frames]
    plain, pre = make_ctx(c_in, 0, C, h, w, theta, lr=0.05, mu=0.9), make_ctx(c_in, 0, C, h, w, theta, lr=0.05, mu=0.9)
    with pytest.raises(st.StError) as ei:
        st.st_use_prefetched_key_frame(pre, 0)
    assert ei.value.status == st.ST_ERR_BAD_STATE
    st.st_prefetch_key_frame(pre, 0, *pinned[0])
    for f in range(3):
        lab_a = torch.empty((4 * h, 4 * w), dtype=torch.uint8, device="cuda")
        lab_b = torch.empty_like(lab_a)
        st.st_set_frozen_features(plain, 0, pinned[f][0]); st.st_teacher_labels(plain, 0, pinned[f][1], lab_a)
        st.st_use_prefetched_key_frame(pre, 0, lab_b)
        if f + 1 < 3:
            st.st_prefetch_key_frame(pre, 0, *pinned[f + 1])          # copied while the steps below run
        la, lb = np.zeros(K, np.float32), np.zeros(K, np.float32)
        st.st_distill_step(plain, K, la); st.st_distill_step(pre, K, lb)
        torch.cuda.synchronize()
        assert torch.equal(lab_a, lab_b)
        np.testing.assert_array_equal(lab_a.cpu().numpy(), oracle.teacher_labels(frames[f][1]))
        assert la.tobytes() == lb.tobytes()
        assert packed(plain).tobytes() == packed(pre).tobytes()
    with pytest.raises(st.StError):
        st.st_use_prefetched_key_frame(pre, 0)                         # nothing pending any more
    st.st_destroy(plain); st.st_destroy(pre)


def test_masks_at_odd_addresses_give_the_same_results():
    """Label maps and masks are byte arrays: a view that starts at an odd address (a tensor sliced by one byte) must
    give the same mask, confusion matrix and mean IoU as an aligned buffer."""
    C, c_in, h, w = 5, 8, 9, 14
    P = 16 * h * w
    feat, T = rand_problem(3, c_in, C, h, w)
    ctx = make_ctx(c_in, 0, C, h, w, si.initial_head_params(c_in, 0, C, 4))
    st.st_set_frozen_features(ctx, 0, dev(feat))
    st.st_teacher_labels(ctx, 0, dev(T))
    lab = oracle.teacher_labels(T)
    mask = torch.empty((4 * h, 4 * w), dtype=torch.uint8, device="cuda")
    st.st_student_mask(ctx, 0, mask)
    conf = torch.zeros((C, C), dtype=torch.int64, device="cuda")
    m = st.st_agreement(ctx, 0, None, dev(lab), conf)
    for shift in (1, 3):
        raw = torch.zeros(P + 16, dtype=torch.uint8, device="cuda")
        mask_odd = raw[shift:shift + P]
        assert mask_odd.data_ptr() % 2 == 1
        st.st_student_mask(ctx, 0, mask_odd)
        assert torch.equal(mask_odd.view(4 * h, 4 * w), mask) and int(raw[:shift].sum()) == 0 and int(raw[shift + P:].sum()) == 0
        lab_raw = torch.zeros(P + 16, dtype=torch.uint8, device="cuda")
        lab_odd = lab_raw[shift:shift + P]
        lab_odd.copy_(dev(lab).view(-1))
        conf2 = torch.zeros_like(conf)
        assert st.st_agreement(ctx, 0, None, lab_odd, conf2) == m               # the student's own mask, fused kernel
        assert torch.equal(conf2, conf)
        conf3 = torch.zeros_like(conf)
        assert st.st_agreement(ctx, 0, mask_odd, lab_odd, conf3) == m           # two masks, both at odd addresses
        assert torch.equal(conf3, conf)
    ref_conf, ref_m, _ = oracle.agreement(lab, mask.cpu().numpy(), C)
    np.testing.assert_array_equal(conf.cpu().numpy(), ref_conf)
    assert m == ref_m
    st.st_destroy(ctx)


def test_agreement_reports_out_of_range_labels():
    C, h, w = 3, 2, 2
    lab = np.zeros((8, 8), np.uint8)
    pred = np.zeros((8, 8), np.uint8)
    lab[3, 3] = 9
    ctx = make_ctx(8, 0, C, h, w, np.zeros(st.st_param_count(8, 0, C), np.float32))
    conf = np.zeros((C, C), np.int64)
    with pytest.raises(st.StError) as ei:
        st.st_agreement(ctx, 0, pred, lab, conf)
    assert ei.value.status == st.ST_ERR_INVALID_ARG
    assert conf[0, 0] == 63                                        # the valid pixels are still counted
    assert st.st_agreement(ctx, 0, pred, pred, conf) == 1.0        # the error does not stick
    st.st_destroy(ctx)


# ---------------------------------------------------------------------------- call order, pack
def test_call_order_and_pack_errors():
    C, cin, h, w = 3, 8, 4, 4
    theta = si.initial_head_params(cin, 0, C, 1)
    ctx = make_ctx(cin, 0, C, h, w, theta)
    with pytest.raises(st.StError) as ei:
        st.st_distill_step(ctx, 1)
    assert ei.value.status == st.ST_ERR_BAD_STATE
    with pytest.raises(st.StError) as ei:
        st.st_set_frozen_features(ctx, 1, np.zeros((cin, h, w), np.float32))
    assert ei.value.status == st.ST_ERR_INVALID_ARG
    small = np.zeros(3, np.float32)
    with pytest.raises(st.StError) as ei:
        st.st_pack_updated_params(ctx, 0, small)
    assert ei.value.status == st.ST_ERR_BUFFER_TOO_SMALL
    with pytest.raises(st.StError) as ei:
        st.st_distill_step(ctx, 0)
    assert ei.value.status == st.ST_ERR_INVALID_ARG
    # K = 0 steps taken: pack returns the initial values bit for bit (host and device destination)
    np.testing.assert_array_equal(packed(ctx), theta)
    d = torch.empty(ctx.n_params, dtype=torch.float32, device="cuda")
    st.st_pack_updated_params(ctx, 0, d)
    np.testing.assert_array_equal(d.cpu().numpy(), theta)
    st.st_destroy(ctx)


@pytest.mark.parametrize("prec", [0, 1])
def test_pack_roundtrip_two_layer(prec):
    cin, ch, C, h, w = 64, 64, 5, 4, 4
    n = st.st_param_count(cin, ch, C)
    theta = np.arange(n, dtype=np.float32)
    ctx = make_ctx(cin, ch, C, h, w, theta, prec=prec)
    raw = packed(ctx)
    assert raw.tobytes() == np.arange(n, dtype="<f4").tobytes()
    ctx2 = make_ctx(cin, ch, C, h, w, raw, prec=prec)
    np.testing.assert_array_equal(packed(ctx2), raw)
    st.st_destroy(ctx); st.st_destroy(ctx2)


# ---------------------------------------------------------------------------- fp32 steps
def run_both(cfg_like, feat, T, theta, n_steps, prec, want_conf=False, quantize=False):
    c_in, ch, C, h, w, lr, mu = cfg_like
    ctx = make_ctx(c_in, ch, C, h, w, theta, prec=prec, lr=lr, mu=mu)
    st.st_set_frozen_features(ctx, 0, dev(feat))
    labels = torch.empty((4 * h, 4 * w), dtype=torch.uint8, device="cuda")
    st.st_teacher_labels(ctx, 0, dev(T), labels)
    loss = torch.zeros(n_steps, dtype=torch.float32, device="cuda")
    conf = torch.zeros((n_steps, C, C), dtype=torch.int64, device="cuda") if want_conf else None
    st.st_distill_step(ctx, n_steps, loss, conf)
    head = oracle.Head(c_in, ch, C, lr=lr, momentum=mu, theta=theta, quantize_bf16=quantize)
    lab_ref = oracle.teacher_labels(T)
    np.testing.assert_array_equal(labels.cpu().numpy(), lab_ref)
    ref_loss, ref_masks = [], []
    for _ in range(n_steps):
        l, m = oracle.distill_step(head, feat, lab_ref)
        ref_loss.append(l); ref_masks.append(m)
    return ctx, head, loss.cpu().numpy(), np.array(ref_loss), (conf.cpu().numpy() if want_conf else None), ref_masks, lab_ref


def check_weights(ctx, head, theta0, max_rel, mean_abs, upd_rel):
    got = packed(ctx)
    ref = head.theta
    off = 0
    for ws, bs in oracle.param_shapes(head.c_in, head.c_hidden, head.n_classes):
        for n in (int(np.prod(ws)), int(np.prod(bs))):
            g, r = got[off:off + n], ref[off:off + n]
            scale = max(np.abs(r).max(), 1e-6)
            assert np.abs(g - r).max() / scale <= max_rel, (off, np.abs(g - r).max() / scale)
            off += n
    assert np.abs(got - ref).mean() <= mean_abs
    du, dr = got - theta0, ref - theta0
    rel = np.linalg.norm(du - dr) / max(np.linalg.norm(dr), 1e-30)
    assert rel <= upd_rel, rel        # a wrong gradient cannot pass this one
    return rel


def test_config1_tiny_fp32_step():
    cfg = si.get_config(1)
    feat, T, theta = si.stream_inputs(cfg)
    like = (cfg.c_in, 0, cfg.n_classes, cfg.feat_h, cfg.feat_w, cfg.lr, cfg.momentum)
    ctx, head, loss, ref_loss, conf, ref_masks, lab = run_both(like, feat, T, theta, 1, 0, want_conf=True)
    assert abs(loss[0] - ref_loss[0]) <= 1e-4 * abs(ref_loss[0])             # stated tolerance: 1e-4 relative
    check_weights(ctx, head, theta, max_rel=1e-5, mean_abs=1e-5, upd_rel=1e-4)  # fp32 GEMMs: 1e-5
    # logits and their gradient, element by element
    z = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGITS)
    # (z was produced by the forward of step 1, i.e. with the initial weights)
    head0 = oracle.Head(cfg.c_in, 0, cfg.n_classes, theta=theta)
    z_ref, _ = oracle.head_forward(head0, feat)
    np.testing.assert_allclose(z, z_ref.ravel(), rtol=1e-5, atol=1e-5)
    u = oracle.upsample(z_ref, 4)
    _, g, _ = oracle.softmax_ce(u, lab)
    dz_ref = oracle.upsample_adjoint(g, 4)
    dz = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGIT_GRAD)
    np.testing.assert_allclose(dz, dz_ref.ravel(), rtol=1e-4, atol=1e-9)
    # fused confusion of the pre-update forward vs. oracle mask: differing pixels only at near-ties
    ref_conf, _, _ = oracle.agreement(lab, ref_masks[0], cfg.n_classes)
    assert conf[0].sum() == lab.size
    assert np.abs(conf[0] - ref_conf).sum() <= 2 * max(2, lab.size // 1000)
    # agreement after the step: the GPU's own mask, counted by the oracle, must match bit for bit
    mask = torch.empty(lab.shape, dtype=torch.uint8, device="cuda")
    st.st_student_mask(ctx, 0, mask)
    gconf = np.zeros((cfg.n_classes, cfg.n_classes), np.int64)
    m = st.st_agreement(ctx, 0, None, None, gconf)
    oconf, om, _ = oracle.agreement(lab, mask.cpu().numpy(), cfg.n_classes)
    np.testing.assert_array_equal(gconf, oconf)
    assert m == om
    # and the mask itself agrees with the oracle's except at near-ties of the top-2 logits
    omask = oracle.student_mask(head, feat)
    diff = mask.cpu().numpy() != omask
    assert diff.mean() <= 1e-3
    if diff.any():
        zz, _ = oracle.head_forward(head, feat)
        uu = np.sort(oracle.upsample(zz, 4), axis=0)
        gap = (uu[-1] - uu[-2])[diff]
        assert gap.max() <= 1e-5 * max(1.0, np.abs(uu).max())
    st.st_destroy(ctx)


@pytest.mark.parametrize("c_in,ch,C,h,w,K,mu", [
    (5, 0, 3, 7, 9, 3, 0.9),        # odd sizes: ragged tiles in every kernel
    (8, 0, 21, 17, 33, 2, 0.0),
    (6, 7, 4, 9, 11, 3, 0.9),       # two-layer head, fp32
    (4, 0, 40, 3, 5, 2, 0.5),       # more classes than one register tile
    (3, 0, 2, 1, 1, 2, 0.0),        # single feature pixel: every frame pixel is border
])
def test_small_fp32_steps(c_in, ch, C, h, w, K, mu):
    feat, T = rand_problem(7, c_in, C, h, w)
    theta = si.initial_head_params(c_in, ch, C, 3)
    if ch:
        theta[ch * c_in * 9: ch * c_in * 9 + ch] = 0.05
    like = (c_in, ch, C, h, w, 0.05, mu)
    ctx, head, loss, ref_loss, conf, _, lab = run_both(like, feat, T, theta, K, 0)
    np.testing.assert_allclose(loss, ref_loss, rtol=1e-4)
    check_weights(ctx, head, theta, max_rel=1e-5, mean_abs=1e-5, upd_rel=2e-4)
    # the applied gradient of the last step and the momentum buffer
    v = st.st_read_tensor(ctx, 0, st.ST_TENSOR_MOMENTUM)
    np.testing.assert_allclose(v, head.vel, rtol=2e-3, atol=1e-7)
    st.st_destroy(ctx)


def test_wildly_varying_logits_take_the_exact_maximum_path():
    # neighbouring nodes carry logits +-300 in different classes: halfway between them every class is
    # 150 below the largest node logit, so a softmax normalised by a neighbourhood bound would underflow
    c_in, C, h, w = 2, 3, 6, 40
    rng = np.random.default_rng(3)
    f = (rng.random((h, w)) < 0.5).astype(np.float32)
    feat = np.stack([f, 1.0 - f])
    theta = np.array([300.0, 0.0, 0.0, 300.0, 10.0, 10.0, 0.0, 0.0, 0.0], np.float32)   # W [3][2], b [3]
    lab = rng.integers(0, C, (4 * h, 4 * w)).astype(np.uint8)
    ctx = make_ctx(c_in, 0, C, h, w, theta, lr=1e-4)
    st.st_set_frozen_features(ctx, 0, feat)
    st.st_set_labels(ctx, 0, lab)
    loss = np.zeros(1, np.float32)
    st.st_distill_step(ctx, 1, loss)
    head = oracle.Head(c_in, 0, C, lr=1e-4, theta=theta)
    ref, _ = oracle.distill_step(head, feat, lab)
    assert np.isfinite(loss[0]) and abs(loss[0] - ref) <= 1e-4 * abs(ref)
    dz = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGIT_GRAD)
    assert np.isfinite(dz).all()
    np.testing.assert_allclose(packed(ctx), head.theta, rtol=1e-4, atol=1e-5)
    st.st_destroy(ctx)


def test_two_streams_are_independent_fp32():
    c_in, C, h, w = 6, 3, 5, 7
    probs = [rand_problem(20 + s, c_in, C, h, w) for s in range(2)]
    thetas = [si.initial_head_params(c_in, 0, C, 30 + s) for s in range(2)]
    ctx = make_ctx(c_in, 0, C, h, w, np.concatenate(thetas), S=2, lr=0.05, mu=0.9)
    for s in range(2):
        st.st_set_frozen_features(ctx, s, dev(probs[s][0]))
        st.st_teacher_labels(ctx, s, dev(probs[s][1]))
    loss = torch.zeros((2, 3), dtype=torch.float32, device="cuda")
    st.st_distill_step(ctx, 3, loss)
    for s in range(2):
        head = oracle.Head(c_in, 0, C, lr=0.05, momentum=0.9, theta=thetas[s])
        lab = oracle.teacher_labels(probs[s][1])
        ref = [oracle.distill_step(head, probs[s][0], lab)[0] for _ in range(3)]
        np.testing.assert_allclose(loss[s].cpu().numpy(), ref, rtol=1e-4)
        np.testing.assert_allclose(packed(ctx, s), head.theta, rtol=1e-4, atol=1e-6)
    st.st_destroy(ctx)


def test_out_of_range_training_labels_are_skipped_and_reported():
    c_in, C, h, w = 4, 3, 2, 3
    feat, T = rand_problem(5, c_in, C, h, w)
    lab = oracle.teacher_labels(T).copy()
    lab[2, 5] = 200
    theta = si.initial_head_params(c_in, 0, C, 1)
    ctx = make_ctx(c_in, 0, C, h, w, theta, lr=0.05)
    st.st_set_frozen_features(ctx, 0, feat)
    st.st_set_labels(ctx, 0, lab)
    loss = np.zeros(1, np.float32)
    st.st_distill_step(ctx, 1, loss)
    with pytest.raises(st.StError) as ei:
        st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGITS)
    assert ei.value.status == st.ST_ERR_INVALID_ARG
    head = oracle.Head(c_in, 0, C, lr=0.05, theta=theta)
    ref, _ = oracle.distill_step(head, feat, lab)
    assert abs(loss[0] - ref) <= 1e-4 * abs(ref)
    np.testing.assert_allclose(packed(ctx), head.theta, rtol=1e-4, atol=1e-6)
    st.st_destroy(ctx)


def test_default_stream_runs_without_graph_capture():
    c_in, C, h, w = 8, 5, 9, 13
    feat, T = rand_problem(9, c_in, C, h, w)
    theta = si.initial_head_params(c_in, 0, C, 2)
    outs = []
    for stream in (torch.cuda.default_stream(), torch.cuda.current_stream()):
        with torch.cuda.stream(stream):
            ctx = make_ctx(c_in, 0, C, h, w, theta, lr=0.05, mu=0.9)
            st.st_set_frozen_features(ctx, 0, feat); st.st_teacher_labels(ctx, 0, T)
            st.st_distill_step(ctx, 2)
            st.st_distill_step(ctx, 2)
            outs.append(packed(ctx))
            st.st_destroy(ctx)
    assert outs[0].tobytes() == outs[1].tobytes()


def test_steps_are_bit_reproducible():
    c_in, C, h, w = 8, 5, 9, 13
    feat, T = rand_problem(9, c_in, C, h, w)
    theta = si.initial_head_params(c_in, 0, C, 2)
    outs = []
    for _ in range(2):
        ctx = make_ctx(c_in, 0, C, h, w, theta, lr=0.05, mu=0.9)
        st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_teacher_labels(ctx, 0, dev(T))
        st.st_distill_step(ctx, 4)
        outs.append(packed(ctx))
        st.st_destroy(ctx)
    assert outs[0].tobytes() == outs[1].tobytes()


def test_profile_step_times_every_kernel_and_takes_real_steps():
    c_in, C, h, w = 8, 5, 9, 13
    feat, T = rand_problem(9, c_in, C, h, w)
    theta = si.initial_head_params(c_in, 0, C, 2)
    ctx = make_ctx(c_in, 0, C, h, w, theta, lr=0.05)
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_teacher_labels(ctx, 0, dev(T))
    stages = st.st_profile_step(ctx, 2)
    names = [n for n, _ in stages]
    assert names == ["conv1x1_fwd_f32", "upsample_ce", "conv1x1_wgrad_f32", "sgd_update"]
    assert all(ms > 0 for _, ms in stages)
    head = oracle.Head(c_in, 0, C, lr=0.05, theta=theta)
    lab = oracle.teacher_labels(T)
    for _ in range(2):
        oracle.distill_step(head, feat, lab)
    np.testing.assert_allclose(packed(ctx), head.theta, rtol=1e-4, atol=1e-6)     # the profiled steps are ordinary steps
    assert st.st_launch_count(ctx) >= 8
    st.st_destroy(ctx)


# ---------------------------------------------------------------------------- ApplyUpdate (Algorithm 4)
@pytest.mark.parametrize("c_hidden,prec", [(0, 0), (64, 1)])
def test_apply_update_moves_a_student_between_contexts(c_hidden, prec):
    c_in, C, h, w = 64, 5, 9, 12
    feat, T = rand_problem(3, c_in, C, h, w)
    lab = oracle.teacher_labels(T)
    theta = si.initial_head_params(c_in, c_hidden, C, 7)
    server = make_ctx(c_in, c_hidden, C, h, w, theta, prec=prec, lr=0.05, mu=0.9)
    st.st_set_frozen_features(server, 0, dev(feat)); st.st_set_labels(server, 0, dev(lab))
    st.st_distill_step(server, 3)
    update = packed(server)                                        # UpdatedPart(student)
    client = make_ctx(c_in, c_hidden, C, h, w, theta, prec=prec)   # still holds the old student
    st.st_set_frozen_features(client, 0, dev(feat))
    m_old = torch.empty((4 * h, 4 * w), dtype=torch.uint8, device="cuda")
    st.st_student_mask(client, 0, m_old)
    st.st_apply_update(client, 0, update)                          # host buffer
    assert packed(client).tobytes() == update.tobytes()
    m_new, m_srv = torch.empty_like(m_old), torch.empty_like(m_old)
    st.st_student_mask(client, 0, m_new); st.st_student_mask(server, 0, m_srv)
    assert torch.equal(m_new, m_srv)                               # the client now predicts what the server's student predicts
    # the oracle's student after the same three steps predicts the same mask up to near-ties
    head = oracle.Head(c_in, c_hidden, C, lr=0.05, momentum=0.9, theta=theta, quantize_bf16=bool(prec))
    for _ in range(3):
        oracle.distill_step(head, feat, lab)
    assert (m_new.cpu().numpy() != oracle.student_mask(head, feat)).mean() <= (1e-3 if prec == 0 else 2e-2)
    st.st_apply_update(client, 0, dev(theta))                      # device buffer: back to the old student
    assert packed(client).tobytes() == np.asarray(theta, np.float32).tobytes()
    back = torch.empty_like(m_old)
    st.st_student_mask(client, 0, back)
    assert torch.equal(back, m_old)
    with pytest.raises(st.StError) as ei:
        st.load_library().st_apply_update  # symbol exists
        st._check(st.load_library().st_apply_update(client.handle, 0, update.ctypes.data, update.nbytes - 4), client)
    assert ei.value.status == st.ST_ERR_INVALID_ARG
    st.st_destroy(server); st.st_destroy(client)


def test_agreement_of_several_streams_reuses_one_forward_and_notices_changes():
    c_in, C, h, w, S = 8, 4, 9, 12, 3
    probs = [rand_problem(10 + s, c_in, C, h, w) for s in range(S)]
    thetas = [si.initial_head_params(c_in, 0, C, 20 + s) for s in range(S)]
    ctx = make_ctx(c_in, 0, C, h, w, np.concatenate(thetas), S=S, lr=0.1)
    labs = []
    for s, (feat, T) in enumerate(probs):
        st.st_set_frozen_features(ctx, s, dev(feat)); st.st_teacher_labels(ctx, s, dev(T))
        labs.append(oracle.teacher_labels(T))

    def check(thetas_now):
        before = st.st_launch_count(ctx)
        for s, (feat, _) in enumerate(probs):
            conf = np.zeros((C, C), np.int64)
            m = st.st_agreement(ctx, s, None, None, conf)
            mask = torch.empty((4 * h, 4 * w), dtype=torch.uint8, device="cuda")
            st.st_student_mask(ctx, s, mask)
            oconf, om, _ = oracle.agreement(labs[s], mask.cpu().numpy(), C)
            np.testing.assert_array_equal(conf, oconf)
            assert m == om
            ref = oracle.student_mask(oracle.Head(c_in, 0, C, theta=thetas_now[s]), feat)
            assert (mask.cpu().numpy() != ref).mean() < 1e-3
        return st.st_launch_count(ctx) - before

    n1 = check(thetas)
    n2 = check(thetas)                       # nothing changed: no forward at all this time
    assert n2 == n1 - 1
    st.st_apply_update(ctx, 1, thetas[0])   # stream 1 gets stream 0's student: the cached forward is stale
    check([thetas[0], thetas[0], thetas[2]])
    st.st_distill_step(ctx, 2)              # so it is after training steps
    heads = [oracle.Head(c_in, 0, C, lr=0.1, theta=t) for t in (thetas[0], thetas[0], thetas[2])]
    for s, (feat, _) in enumerate(probs):
        for _ in range(2):
            oracle.distill_step(heads[s], feat, labs[s])
    check([hd.theta for hd in heads])
    st.st_destroy(ctx)


@pytest.mark.parametrize("scale", [3.5, 4.2])
def test_steep_logits_inside_the_fast_range_keep_fp32_accuracy(scale):
    """Logits that change by 20 to 28 nats between neighbouring nodes: most cells still take the geometric-progression
    path of the fused loss kernel (its limit is 40 log2-units = 27.7 nats per cell), a few the row-by-row one; the
    gradient must agree with the oracle as on gentle logits."""
    c_in, C, h, w = 32, 21, 45, 80
    cls = si.voronoi_map(4 * h, 4 * w, 24, C, 2005)
    feat = si.label_informed_features(c_in, h, w, cls, 4, 7, strength=3.0)
    theta = (si.initial_head_params(c_in, 0, C, 5) * scale).astype(np.float32)
    ctx = make_ctx(c_in, 0, C, h, w, theta, lr=0.0)
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_set_labels(ctx, 0, dev(cls))
    loss = np.zeros(1, np.float32)
    st.st_distill_step(ctx, 1, loss)
    head = oracle.Head(c_in, 0, C, theta=theta)
    z, _ = oracle.head_forward(head, feat)
    steps = max(np.abs(np.diff(z, axis=1)).max(), np.abs(np.diff(z, axis=2)).max())
    assert 18.0 < steps < 40.0, steps                               # the case is what it is meant to be
    ref_loss, g, _ = oracle.softmax_ce(oracle.upsample(z, 4), cls)
    ref = oracle.upsample_adjoint(g, 4).ravel()
    dz = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGIT_GRAD)
    assert np.linalg.norm(dz - ref) / np.linalg.norm(ref) < 2e-6
    assert abs(loss[0] - ref_loss) <= 1e-5 * abs(ref_loss)
    st.st_destroy(ctx)
