"""GPU parity of the bf16 tensor-core path (gemm_precision 1) against the CPU oracle.

Two comparisons are made.  Against the plain fp32 oracle with the stated tolerances (loss 1e-4
relative; weights 2e-2 max relative / 1e-3 mean absolute; update vector 2e-2 relative L2), and
against the oracle with its GEMM operands rounded to bf16 at the same places, where the
remaining difference is accumulation order only and the tolerance is much tighter."""
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


def make_ctx(c_in, ch, C, h, w, theta, S=1, lr=0.01, mu=0.0, prec=1):
    return st.st_init_head(n_streams=S, c_in=c_in, c_hidden=ch, n_classes=C, feat_h=h, feat_w=w,
                           gemm_precision=prec, lr=lr, momentum=mu,
                           cuda_stream=torch.cuda.current_stream().cuda_stream, init_params=theta)


def packed(ctx, stream=0):
    out = np.empty(ctx.n_params, np.float32)
    st.st_pack_updated_params(ctx, stream, out)
    return out


def problem(seed, c_in, C, h, w):
    rng = np.random.default_rng(seed)
    feat = np.maximum(rng.standard_normal((c_in, h, w)), 0).astype(np.float32)
    cfg = si.WorkloadConfig("t", c_in, 0, C, h, w, n_regions=max(4, C), teacher="onehot_noise")
    return feat, si.teacher_logits(cfg, stream=seed)


def rel_l2(a, b):
    return float(np.linalg.norm(a.astype(np.float64) - b) / max(np.linalg.norm(b), 1e-30))


def check_weights(got, ref, theta0, c_in, ch, C, max_rel=2e-2, mean_abs=1e-3, upd_rel=2e-2):
    off = 0
    for ws, bs in oracle.param_shapes(c_in, ch, C):
        for n in (int(np.prod(ws)), int(np.prod(bs))):
            g, r = got[off:off + n], ref[off:off + n]
            assert np.abs(g - r).max() / max(np.abs(r).max(), 1e-6) <= max_rel
            off += n
    assert np.abs(got - ref).mean() <= mean_abs
    r = rel_l2(got - theta0, ref.astype(np.float64) - theta0)
    assert r <= upd_rel, r
    return r


@pytest.mark.parametrize("c_in,h,w", [(64, 5, 7), (256, 12, 20)])
def test_feature_cache_rounds_to_nearest_even(c_in, h, w):
    feat, _ = problem(1, c_in, 3, h, w)
    feat[0, 0, :4] = [1.00390625, 1.01171875, -1.00390625, 3.0e-39]     # ties and a denormal
    ctx = make_ctx(c_in, 0, 3, h, w, np.zeros(st.st_param_count(c_in, 0, 3), np.float32))
    st.st_set_frozen_features(ctx, 0, dev(feat))
    got = st.st_read_tensor(ctx, 0, st.ST_TENSOR_FEATURES)
    np.testing.assert_array_equal(got, oracle.round_bf16(feat).ravel())
    st.st_destroy(ctx)


@pytest.mark.parametrize("c_in,C,h,w", [
    (64, 5, 9, 13),      # fewer pixels than one 128-pixel tile, ragged chunk
    (128, 21, 24, 40),   # several tiles and a half one
    (256, 32, 17, 31),   # all 32 class rows in use, two channel accumulators
    (192, 2, 8, 8),      # channel count that is not a multiple of 128
    (768, 21, 10, 30),   # more channels than the one-tile forward can hold in shared memory: the persistent form serves
    (1024, 4, 6, 9),     # the largest channel count the path accepts
])
def test_1x1_head_single_step_intermediates(c_in, C, h, w):
    feat, T = problem(3, c_in, C, h, w)
    theta = si.initial_head_params(c_in, 0, C, 5)
    theta[-C:] = np.linspace(-0.5, 0.5, C)                        # non-zero biases
    ctx = make_ctx(c_in, 0, C, h, w, theta, lr=0.05)
    st.st_set_frozen_features(ctx, 0, dev(feat))
    st.st_teacher_labels(ctx, 0, dev(T))
    loss = np.zeros(1, np.float32)
    st.st_distill_step(ctx, 1, loss)
    lab = oracle.teacher_labels(T)
    hq = oracle.Head(c_in, 0, C, lr=0.05, theta=theta, quantize_bf16=True)
    z_ref, _ = oracle.head_forward(hq, feat)
    z = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGITS)
    np.testing.assert_allclose(z, z_ref.ravel(), rtol=2e-5, atol=2e-5)        # same bf16 operands, fp32 accumulation
    l_ref, g_ref, _ = oracle.gradients(hq, feat, lab)
    assert abs(loss[0] - l_ref) <= 2e-5 * abs(l_ref)
    g = st.st_read_tensor(ctx, 0, st.ST_TENSOR_PARAM_GRAD)
    assert rel_l2(g, g_ref) <= 2e-3
    assert np.abs(g - g_ref).max() <= 2e-3 * np.abs(g_ref).max()
    # against the plain fp32 oracle: stated tolerances
    hp = oracle.Head(c_in, 0, C, lr=0.05, theta=theta)
    l_plain, _ = oracle.distill_step(hp, feat, lab)
    # few pixels: the bf16 rounding of X and W does not average out as it does at frame size, where
    # the stated 1e-4 holds (full-size test below); here the bound is the rounding itself
    assert abs(loss[0] - l_plain) <= 2e-3 * abs(l_plain)
    check_weights(packed(ctx), hp.theta, theta, c_in, 0, C)
    st.st_destroy(ctx)


@pytest.mark.parametrize("c_in,ch,C,h,w", [
    (64, 64, 5, 10, 37),      # ragged tile in x and y, one accumulator
    (128, 128, 21, 9, 33),
    (256, 256, 19, 6, 70),    # the full channel counts of the two-layer workloads, all of TMEM
    (64, 192, 3, 4, 4),
])
def test_two_layer_head_single_step_intermediates(c_in, ch, C, h, w):
    feat, T = problem(4, c_in, C, h, w)
    theta = si.initial_head_params(c_in, ch, C, 6)
    nb1 = ch * c_in * 9
    theta[nb1:nb1 + ch] = np.linspace(-0.2, 0.3, ch)
    ctx = make_ctx(c_in, ch, C, h, w, theta, lr=0.02)
    st.st_set_frozen_features(ctx, 0, dev(feat))
    st.st_teacher_labels(ctx, 0, dev(T))
    loss = np.zeros(1, np.float32)
    st.st_distill_step(ctx, 1, loss)
    lab = oracle.teacher_labels(T)
    hq = oracle.Head(c_in, ch, C, lr=0.02, theta=theta, quantize_bf16=True)
    z_ref, hd_ref = oracle.head_forward(hq, feat)
    hd = st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN)
    # bf16 outputs of fp32 sums in different orders: at most one bf16 ulp apart, and rarely
    d = np.abs(hd - hd_ref.ravel())
    assert (d <= 2.0 ** -7 * np.maximum(np.abs(hd_ref.ravel()), 1e-3)).all()
    assert (d > 0).mean() < 0.02
    z = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGITS)
    # a hidden value one bf16 ulp apart moves a logit by about ulp * |W2|; a few of them can add up
    np.testing.assert_allclose(z, z_ref.ravel(), rtol=1e-3, atol=5e-3)
    l_ref, g_ref, _ = oracle.gradients(hq, feat, lab)
    assert abs(loss[0] - l_ref) <= 1e-4 * abs(l_ref)
    g = st.st_read_tensor(ctx, 0, st.ST_TENSOR_PARAM_GRAD)
    off = 0
    for ws, bs in oracle.param_shapes(c_in, ch, C):
        for n in (int(np.prod(ws)), int(np.prod(bs))):
            assert rel_l2(g[off:off + n], g_ref[off:off + n]) <= 1e-2, (off, n)
            off += n
    hp = oracle.Head(c_in, ch, C, lr=0.02, theta=theta)
    l_plain, _ = oracle.distill_step(hp, feat, lab)
    assert abs(loss[0] - l_plain) <= 2e-3 * abs(l_plain)      # few pixels, see the 1x1 test
    # same for the update vector: with a few hundred pixels the rounding noise of bf16 operands is not
    # averaged down to the 2e-2 that holds at frame size; the tight check is the one against the
    # rounded-operand oracle above
    check_weights(packed(ctx), hp.theta, theta, c_in, ch, C, upd_rel=6e-2)
    st.st_destroy(ctx)


def test_hidden_gradient_and_relu_mask():
    c_in, ch, C, h, w = 64, 64, 4, 7, 9
    feat, T = problem(8, c_in, C, h, w)
    theta = si.initial_head_params(c_in, ch, C, 2)
    ctx = make_ctx(c_in, ch, C, h, w, theta)
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_teacher_labels(ctx, 0, dev(T))
    st.st_distill_step(ctx, 1)
    hd = st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN).reshape(ch, h, w)
    dz = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGIT_GRAD).reshape(C, h, w)
    dh = st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN_GRAD).reshape(ch, h, w)
    W2 = theta[ch * c_in * 9 + ch: ch * c_in * 9 + ch + C * ch].reshape(C, ch)
    ref = oracle.conv1x1_dgrad(oracle.round_bf16(W2), oracle.round_bf16(dz))     # both GEMM operands are bf16
    oracle.relu_mask_(ref, np.ascontiguousarray(hd))
    assert (dh[hd <= 0] == 0).all()
    np.testing.assert_allclose(dh, oracle.round_bf16(ref), rtol=2.0 ** -7, atol=1e-12)
    st.st_destroy(ctx)


def test_config2_720p_full_size_k8():
    cfg = si.get_config(2)
    feat, T, theta = si.stream_inputs(cfg)
    ctx = make_ctx(cfg.c_in, 0, cfg.n_classes, cfg.feat_h, cfg.feat_w, theta, lr=cfg.lr, mu=cfg.momentum)
    st.st_set_frozen_features(ctx, 0, dev(feat))
    labels = torch.empty((cfg.frame_h, cfg.frame_w), dtype=torch.uint8, device="cuda")
    st.st_teacher_labels(ctx, 0, dev(T), labels)
    K = cfg.k_steps
    loss = torch.zeros(K, dtype=torch.float32, device="cuda")
    conf = torch.zeros((K, cfg.n_classes, cfg.n_classes), dtype=torch.int64, device="cuda")
    st.st_distill_step(ctx, K, loss, conf)
    lab = oracle.teacher_labels(T)
    np.testing.assert_array_equal(labels.cpu().numpy(), lab)                   # bit-exact labels
    head = oracle.Head(cfg.c_in, 0, cfg.n_classes, lr=cfg.lr, momentum=cfg.momentum, theta=theta)
    ref_loss, masks = [], []
    for _ in range(K):
        l, m = oracle.distill_step(head, feat, lab)
        ref_loss.append(l); masks.append(m)
    np.testing.assert_allclose(loss.cpu().numpy(), ref_loss, rtol=1e-4)         # loss: 1e-4 relative
    raw = packed(ctx)
    assert raw.nbytes == 21588                                                  # 256*21 weights + 21 biases
    check_weights(raw, head.theta, theta, cfg.c_in, 0, cfg.n_classes)
    # per-step fused confusion: totals exact, cells within the near-tie budget of the student mask
    c = conf.cpu().numpy()
    for k in range(K):
        assert c[k].sum() == lab.size
        np.testing.assert_array_equal(c[k].sum(1), np.bincount(lab.ravel(), minlength=cfg.n_classes))
        ref_c, _, _ = oracle.agreement(lab, masks[k], cfg.n_classes)
        assert np.abs(c[k] - ref_c).sum() <= 2 * lab.size // 500
    # agreement from the GPU's own mask is bit-exact with the oracle's count of that mask
    mask = torch.empty_like(labels)
    st.st_student_mask(ctx, 0, mask)
    gconf = np.zeros((cfg.n_classes,) * 2, np.int64)
    m = st.st_agreement(ctx, 0, None, None, gconf)
    oconf, om, _ = oracle.agreement(lab, mask.cpu().numpy(), cfg.n_classes)
    np.testing.assert_array_equal(gconf, oconf)
    assert m == om
    st.st_destroy(ctx)


def test_three_streams_grouped_launch():
    c_in, C, h, w = 64, 6, 11, 19
    S = 3
    probs = [problem(40 + s, c_in, C, h, w) for s in range(S)]
    thetas = [si.initial_head_params(c_in, 0, C, 50 + s) for s in range(S)]
    ctx = make_ctx(c_in, 0, C, h, w, np.concatenate(thetas), S=S, lr=0.05, mu=0.9)
    for s in range(S):
        st.st_set_frozen_features(ctx, s, dev(probs[s][0]))
        st.st_teacher_labels(ctx, s, dev(probs[s][1]))
    loss = torch.zeros((S, 4), dtype=torch.float32, device="cuda")
    st.st_distill_step(ctx, 4, loss)
    for s in range(S):
        head = oracle.Head(c_in, 0, C, lr=0.05, momentum=0.9, theta=thetas[s])
        lab = oracle.teacher_labels(probs[s][1])
        ref = [oracle.distill_step(head, probs[s][0], lab)[0] for _ in range(4)]
        np.testing.assert_allclose(loss[s].cpu().numpy(), ref, rtol=2e-3)     # few pixels
        check_weights(packed(ctx, s), head.theta, thetas[s], c_in, 0, C)
    st.st_destroy(ctx)


def test_bf16_steps_are_bit_reproducible():
    c_in, ch, C, h, w = 64, 64, 5, 9, 35
    feat, T = problem(9, c_in, C, h, w)
    theta = si.initial_head_params(c_in, ch, C, 2)
    outs = []
    for _ in range(2):
        ctx = make_ctx(c_in, ch, C, h, w, theta, lr=0.02, mu=0.9)
        st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_teacher_labels(ctx, 0, dev(T))
        st.st_distill_step(ctx, 3)
        outs.append(packed(ctx))
        st.st_destroy(ctx)
    assert outs[0].tobytes() == outs[1].tobytes()


@pytest.mark.parametrize("c_in,ch,h,w", [
    (64, 128, 72, 352),     # 198 tiles of 128 pixels: on 148 SMs the last 50 are cut into two channel ranges each
    (64, 256, 56, 352),     # 154 tiles: the last 6 are cut into four channel ranges each
])
def test_two_layer_forward_with_a_partly_filled_last_round(c_in, ch, h, w):
    C = 5
    rng = np.random.default_rng(9)
    feat = np.maximum(rng.standard_normal((c_in, h, w)), 0).astype(np.float32)
    theta = si.initial_head_params(c_in, ch, C, 8)
    nb1 = ch * c_in * 9
    theta[nb1:nb1 + ch] = np.linspace(-0.2, 0.3, ch)
    ctx = make_ctx(c_in, ch, C, h, w, theta)
    st.st_set_frozen_features(ctx, 0, dev(feat))
    mask = torch.empty((4 * h, 4 * w), dtype=torch.uint8, device="cuda")
    st.st_student_mask(ctx, 0, mask)                              # runs the forward
    hq = oracle.Head(c_in, ch, C, theta=theta, quantize_bf16=True)
    z_ref, hd_ref = oracle.head_forward(hq, feat)
    hd = st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN)
    d = np.abs(hd - hd_ref.ravel())
    assert (d <= 2.0 ** -7 * np.maximum(np.abs(hd_ref.ravel()), 1e-3)).all()
    assert (d > 0).mean() < 0.02
    z = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGITS)
    np.testing.assert_allclose(z, z_ref.ravel(), rtol=1e-3, atol=5e-3)
    # the ReLU bits written by the same epilogue drive the backward pass: one step's hidden gradient is zero exactly
    # where the hidden activation is zero
    lab = rng.integers(0, C, (4 * h, 4 * w)).astype(np.uint8)
    st.st_set_labels(ctx, 0, dev(lab))
    st.st_distill_step(ctx, 1)
    hd1 = st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN)
    dh = st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN_GRAD)
    assert (dh[hd1 == 0] == 0).all() and (dh[hd1 > 0] != 0).mean() > 0.9
    st.st_destroy(ctx)


def test_a_wait_that_runs_out_is_reported_and_nothing_else_breaks(monkeypatch):
    """Every wait inside the tensor-core kernels is bounded.  A test-only switch makes the forward's first barrier
    expect 16 bytes more than its copies deliver and shortens the limit: the wait runs out, the kernel records where,
    writes nothing, frees its tensor memory and returns; the host reports ST_ERR_CUDA at the next call that waits.
    Nothing faults or hangs, the device stays usable, and a context made without the switch works as ever."""
    c_in, C, h, w = 64, 5, 9, 13
    feat, T = problem(12, c_in, C, h, w)
    theta = si.initial_head_params(c_in, 0, C, 5)
    monkeypatch.setenv("ST_TEST_STALL_FWD1X1", "1")
    ctx = make_ctx(c_in, 0, C, h, w, theta, lr=0.05)
    monkeypatch.delenv("ST_TEST_STALL_FWD1X1")
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_teacher_labels(ctx, 0, dev(T))
    st.st_distill_step(ctx, 1)
    with pytest.raises(st.StError) as ei:
        st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGITS)
    assert ei.value.status == st.ST_ERR_CUDA
    assert "gave up waiting (code 1, block 0)" in str(ei.value)         # code 1: a wait for data to arrive
    assert (st.st_read_tensor(ctx, 0, st.ST_TENSOR_FEATURES) == oracle.round_bf16(feat).ravel()).all()   # reported once; the context answers
    st.st_destroy(ctx)
    good = make_ctx(c_in, 0, C, h, w, theta, lr=0.05)
    st.st_set_frozen_features(good, 0, dev(feat)); st.st_teacher_labels(good, 0, dev(T))
    loss = np.zeros(1, np.float32)
    st.st_distill_step(good, 1, loss)
    hq = oracle.Head(c_in, 0, C, lr=0.05, theta=theta, quantize_bf16=True)
    l_ref, _, _ = oracle.gradients(hq, feat, oracle.teacher_labels(T))
    assert abs(loss[0] - l_ref) <= 2e-5 * abs(l_ref)
    st.st_destroy(good)


def test_a_wait_that_runs_out_inside_the_loss_kernels_own_forward(monkeypatch):
    """The same for the forward that a one-layer head's loss kernel runs inside its blocks: with the test-only switch
    the first feature slice's barrier expects 16 bytes more than the copy delivers and the limit is short.  Every block
    gives up, writes nothing, frees its tensor memory and returns; the error is reported once and the device stays
    usable."""
    c_in, C, h, w = 128, 5, 20, 64
    feat, T = problem(13, c_in, C, h, w)
    theta = si.initial_head_params(c_in, 0, C, 5)
    monkeypatch.setenv("ST_TEST_STALL_FUSED", "1")
    ctx = make_ctx(c_in, 0, C, h, w, theta, lr=0.05)
    monkeypatch.delenv("ST_TEST_STALL_FUSED")
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_teacher_labels(ctx, 0, dev(T))
    st.st_distill_step(ctx, 2)
    with pytest.raises(st.StError) as ei:
        st.st_read_tensor(ctx, 0, st.ST_TENSOR_FEATURES)
    assert ei.value.status == st.ST_ERR_CUDA
    assert "gave up waiting (code 1," in str(ei.value)                    # code 1: a wait for data to arrive
    assert (st.st_read_tensor(ctx, 0, st.ST_TENSOR_FEATURES) == oracle.round_bf16(feat).ravel()).all()   # reported once
    st.st_destroy(ctx)
    good = make_ctx(c_in, 0, C, h, w, theta, lr=0.05)
    st.st_set_frozen_features(good, 0, dev(feat)); st.st_teacher_labels(good, 0, dev(T))
    loss = np.zeros(1, np.float32)
    st.st_distill_step(good, 1, loss)
    hq = oracle.Head(c_in, 0, C, lr=0.05, theta=theta, quantize_bf16=True)
    l_ref, _, _ = oracle.gradients(hq, feat, oracle.teacher_labels(T))
    assert abs(loss[0] - l_ref) <= 2e-5 * abs(l_ref)
    st.st_destroy(good)


@pytest.mark.parametrize("c_in,C,h,w,S", [
    (64, 5, 9, 32, 1),       # the smallest map the block-level forward takes: one tile, one 64-channel slice
    (128, 21, 24, 40, 2),    # two streams, ragged tiles in both directions
    (192, 32, 23, 95, 1),    # three slices, all 32 class rows, a last tile column of five nodes
    (256, 19, 30, 61, 1),    # four slices (the ring of two is refilled), a last tile column of one node
])
def test_forward_inside_the_loss_kernel_equals_the_separate_forward(c_in, C, h, w, S, monkeypatch):
    """A one-layer head multiplies its logits inside the loss kernel and inside the student-mask kernel.  With
    ST_FUSED_FORWARD=0 at context creation the same steps run with the forward as a kernel of its own.  Both forms
    multiply the same bf16 operands in the same order, so the logits agree bit by bit as long as the parameters do.
    The loss kernel shifts its exponentials by the largest logit of the block's tile, and the two forms' tiles differ
    (36 columns from a multiple of four against 32 from the block's first node), so sums of exponentials can round
    differently in the last place: everything downstream is compared to a few units in the last place, integer
    counts to a handful of pixels."""
    K = 3
    probs = [problem(10 + s, c_in, C, h, w) for s in range(S)]
    theta = np.concatenate([si.initial_head_params(c_in, 0, C, 20 + s) for s in range(S)])

    def run(fused):
        if not fused:
            monkeypatch.setenv("ST_FUSED_FORWARD", "0")
        ctx = make_ctx(c_in, 0, C, h, w, theta, S=S, lr=0.05, mu=0.9)
        monkeypatch.delenv("ST_FUSED_FORWARD", raising=False)
        for s in range(S):
            st.st_set_frozen_features(ctx, s, dev(probs[s][0]))
            st.st_teacher_labels(ctx, s, dev(probs[s][1]))
        loss = np.zeros((S, K), np.float32)
        conf = np.zeros((S, K, C, C), np.int64)
        st.st_distill_step(ctx, K, loss, conf)
        out = {"loss": loss, "conf": conf, "launches": st.st_launch_count(ctx)}
        out["z"] = [st.st_read_tensor(ctx, s, st.ST_TENSOR_LOGITS) for s in range(S)]
        out["dz"] = [st.st_read_tensor(ctx, s, st.ST_TENSOR_LOGIT_GRAD) for s in range(S)]
        out["theta"] = [packed(ctx, s) for s in range(S)]
        masks, agree = [], []
        for s in range(S):
            m = torch.empty((4 * h, 4 * w), dtype=torch.uint8, device="cuda")
            st.st_student_mask(ctx, s, m)
            masks.append(m.cpu().numpy())
            c = np.zeros((C, C), np.int64)
            agree.append((st.st_agreement(ctx, s, None, None, c), c))
        out["mask"], out["agree"] = masks, agree
        n_upd = np.zeros(S, np.int32); best = np.zeros(S, np.float64); met = np.zeros((S, K + 1), np.float64)
        st.st_train_key_frame(ctx, 2.0, K, n_upd, best, met)
        out["train"] = (n_upd, best, met, [packed(ctx, s) for s in range(S)])
        st.st_destroy(ctx)
        return out

    a, b = run(True), run(False)
    assert a["launches"] < b["launches"]                      # the forward really was part of another kernel
    P = 16 * h * w
    np.testing.assert_allclose(a["loss"], b["loss"], rtol=2e-6)
    assert np.abs(a["conf"] - b["conf"]).sum(axis=(2, 3)).max() <= 2 * max(4, P // 1000)
    for s in range(S):
        np.testing.assert_allclose(a["z"][s], b["z"][s], rtol=1e-5, atol=1e-5)
        np.testing.assert_allclose(a["dz"][s], b["dz"][s], rtol=1e-4, atol=1e-10)
        np.testing.assert_allclose(a["theta"][s], b["theta"][s], rtol=1e-5, atol=1e-7)
        assert (a["mask"][s] != b["mask"][s]).sum() <= max(4, P // 1000)
        assert abs(a["agree"][s][0] - b["agree"][s][0]) <= 1e-3
        assert np.abs(a["agree"][s][1] - b["agree"][s][1]).sum() <= 2 * max(4, P // 1000)
        assert int(a["agree"][s][1].sum()) == P and int(b["agree"][s][1].sum()) == P
        np.testing.assert_allclose(a["train"][3][s], b["train"][3][s], rtol=1e-4, atol=1e-6)
    assert (a["train"][0] == b["train"][0]).all()             # updates taken
    np.testing.assert_allclose(a["train"][1], b["train"][1], atol=1e-3)
    np.testing.assert_allclose(a["train"][2], b["train"][2], atol=1e-3)
