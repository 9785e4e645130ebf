"""GPU parity of the deeper trainable subset: a stack of student blocks with skip inputs and a freeze boundary inside
it (Section 5.2's SB5 / SB6; Section 4.2), bf16 tensor-core path, against the CPU oracle (oracle.StackHead)."""
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


def rel_l2(a, b):
    return float(np.linalg.norm(a.astype(np.float64) - b) / max(np.linalg.norm(b), 1e-30))


def stack_problem(seed, c_in, blocks, C, h, w):
    rng = np.random.default_rng(seed)
    feat = np.maximum(rng.standard_normal((c_in, h, w)), 0).astype(np.float32)
    skips = [np.maximum(rng.standard_normal((cs, h, w)), 0).astype(np.float32) if cs else None for _, cs in blocks]
    cfg = si.WorkloadConfig("t", c_in, 0, C, h, w, n_regions=max(4, C), teacher="onehot_noise")
    T = si.teacher_logits(cfg, stream=seed)
    theta, prev = [], c_in
    for co, cs in blocks:                                    # Kaiming-normal weights, small non-zero biases
        fan = (prev + cs) * 9
        theta += [rng.standard_normal(co * fan).astype(np.float32) * np.float32(np.sqrt(2.0 / fan)),
                  np.linspace(-0.2, 0.3, co).astype(np.float32)]
        prev = co
    theta += [rng.standard_normal(C * prev).astype(np.float32) * np.float32(np.sqrt(2.0 / prev)), np.linspace(-0.1, 0.1, C).astype(np.float32)]
    return feat, skips, T, np.concatenate(theta)


def make_ctx(c_in, blocks, C, h, w, theta, first_trained, S=1, lr=0.02, mu=0.9):
    return st.st_init_head(n_streams=S, c_in=c_in, n_classes=C, feat_h=h, feat_w=w, gemm_precision=1, lr=lr, momentum=mu,
                           cuda_stream=torch.cuda.current_stream().cuda_stream, init_params=theta, blocks=blocks,
                           first_trained=first_trained)


def feed(ctx, s, feat, skips, T):
    st.st_set_frozen_features(ctx, s, dev(feat))
    for b, sk in enumerate(skips):
        if sk is not None:
            st.st_set_skip_features(ctx, s, b, dev(sk))
    st.st_teacher_labels(ctx, s, dev(T))


def ulp_close(got, ref, frac=0.02):
    """bf16 values of fp32 sums taken in different orders: at most one bf16 step apart, and rarely."""
    d = np.abs(got - ref)
    assert (d <= 2.0 ** -7 * np.maximum(np.abs(ref), 1e-3)).all()
    assert (d > 0).mean() < frac


@pytest.mark.parametrize("c_in,blocks,C,h,w", [
    (64, [(64, 64), (128, 64)], 5, 10, 37),       # ragged tiles, both blocks with a skip input
    (128, [(128, 0), (64, 128)], 21, 9, 33),      # first block without a skip input
    (64, [(256, 64), (256, 0)], 19, 6, 70),       # widest blocks: all of tensor memory in the weight gradient
])
def test_stack_single_step_intermediates(c_in, blocks, C, h, w):
    feat, skips, T, theta = stack_problem(5, c_in, blocks, C, h, w)
    ctx = make_ctx(c_in, blocks, C, h, w, theta, 0)
    assert ctx.n_params == ctx.n_params_all == theta.size
    feed(ctx, 0, feat, skips, T)
    loss = np.zeros(1, np.float32)
    st.st_distill_step(ctx, 1, loss)
    lab = oracle.teacher_labels(T)
    hq = oracle.StackHead(c_in, blocks, C, lr=0.02, momentum=0.9, theta=theta, quantize_bf16=True)
    z_ref, ins, outs = oracle.stack_forward(hq, feat, skips)
    ulp_close(st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN_FIRST), outs[0].ravel())
    # the second block reads the first one's output, where a value here and there sits one bf16 step away from the
    # oracle's: its own sums move by about that step times a weight, which a value next to zero feels in full
    h1 = st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN)
    np.testing.assert_allclose(h1, outs[1].ravel(), rtol=2.0 ** -7, atol=2e-3)
    assert (h1 != outs[1].ravel()).mean() < 0.1
    np.testing.assert_allclose(st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGITS), z_ref.ravel(), rtol=2e-3, atol=1e-2)
    l_ref, g_ref, _ = oracle.stack_gradients(hq, feat, skips, lab)
    assert abs(loss[0] - l_ref) <= 2e-4 * abs(l_ref)
    g = st.st_read_tensor(ctx, 0, st.ST_TENSOR_PARAM_GRAD)
    off = 0
    for ws, bs in hq.shapes():
        for n in (int(np.prod(ws)), int(np.prod(bs))):
            assert rel_l2(g[off:off + n], g_ref[off:off + n]) <= 2e-2, (off, n)
            off += n
    # the gradient that reaches the first block: zero exactly where that block's output is zero
    h0 = st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN_FIRST)
    dh0 = st.st_read_tensor(ctx, 0, st.ST_TENSOR_HIDDEN_GRAD_FIRST)
    assert (dh0[h0 <= 0] == 0).all() and np.abs(dh0).max() > 0
    st.st_destroy(ctx)


@pytest.mark.parametrize("first_trained", [0, 1, 2])
def test_stack_trains_behind_the_freeze_boundary(first_trained):
    c_in, blocks, C, h, w, K = 64, [(64, 64), (128, 64)], 6, 11, 35, 3
    feat, skips, T, theta = stack_problem(7 + first_trained, c_in, blocks, C, h, w)
    ctx = make_ctx(c_in, blocks, C, h, w, theta, first_trained)
    feed(ctx, 0, feat, skips, T)
    loss = np.zeros(K, np.float32)
    conf = np.zeros((K, C, C), np.int64)
    st.st_distill_step(ctx, K, loss, conf)
    lab = oracle.teacher_labels(T)
    plain = oracle.StackHead(c_in, blocks, C, first_trained=first_trained, lr=0.02, momentum=0.9, theta=theta)
    quant = oracle.StackHead(c_in, blocks, C, first_trained=first_trained, lr=0.02, momentum=0.9, theta=theta, quantize_bf16=True)
    ref_loss = [oracle.stack_distill_step(plain, feat, skips, lab)[0] for _ in range(K)]
    q_loss = [oracle.stack_distill_step(quant, feat, skips, lab)[0] for _ in range(K)]
    np.testing.assert_allclose(loss, q_loss, rtol=2e-4)
    np.testing.assert_allclose(loss, ref_loss, rtol=3e-3)              # few pixels: bf16 rounding is not averaged away
    sl = plain.trained_slice()
    got = np.empty(ctx.n_params, np.float32)
    assert st.st_pack_updated_params(ctx, 0, got) == len(oracle.stack_pack(plain)) == (theta.size - sl.start) * 4
    assert rel_l2(got - theta[sl], quant.theta[sl].astype(np.float64) - theta[sl]) <= 1e-2      # update, same roundings
    assert rel_l2(got - theta[sl], plain.theta[sl].astype(np.float64) - theta[sl]) <= 8e-2      # update, plain oracle
    assert np.abs(got - plain.theta[sl]).max() <= 2e-2 * np.abs(plain.theta[sl]).max()
    g = st.st_read_tensor(ctx, 0, st.ST_TENSOR_PARAM_GRAD)
    assert not g[:sl.start].any() and g[sl].any()                       # no gradient for the frozen layers
    v = st.st_read_tensor(ctx, 0, st.ST_TENSOR_MOMENTUM)
    assert not v[:sl.start].any()
    for k in range(K):
        assert conf[k].sum() == lab.size
        np.testing.assert_array_equal(conf[k].sum(1), np.bincount(lab.ravel(), minlength=C))
    # the student's mask with the final parameters, counted by the oracle
    mask = torch.empty((4 * h, 4 * w), dtype=torch.uint8, device="cuda")
    st.st_student_mask(ctx, 0, mask)
    gconf = np.zeros((C, C), np.int64)
    m = st.st_agreement(ctx, 0, None, None, gconf)
    oconf, om, _ = oracle.agreement(lab, mask.cpu().numpy(), C)
    np.testing.assert_array_equal(gconf, oconf)
    assert m == om
    # UpdatedPart installed in a fresh context reproduces the student (ApplyUpdate); frozen layers never left theirs
    other = make_ctx(c_in, blocks, C, h, w, theta, first_trained)
    feed(other, 0, feat, skips, T)
    st.st_apply_update(other, 0, got)
    mask2 = torch.empty_like(mask)
    st.st_student_mask(other, 0, mask2)
    assert torch.equal(mask, mask2)
    again = np.empty(ctx.n_params, np.float32)
    st.st_pack_updated_params(other, 0, again)
    assert again.tobytes() == got.tobytes()
    st.st_destroy(ctx); st.st_destroy(other)


def test_stack_two_streams_and_a_second_key_frame():
    c_in, blocks, C, h, w, K = 64, [(64, 0), (64, 64)], 4, 8, 34, 2
    probs = [stack_problem(20 + s, c_in, blocks, C, h, w) for s in range(2)]
    theta = np.concatenate([p[3] for p in probs])
    ctx = make_ctx(c_in, blocks, C, h, w, theta, 1, S=2)
    heads = [oracle.StackHead(c_in, blocks, C, first_trained=1, lr=0.02, momentum=0.9, theta=p[3], quantize_bf16=True) for p in probs]
    with pytest.raises(st.StError) as ei:
        st.st_set_frozen_features(ctx, 0, dev(probs[0][0])); st.st_teacher_labels(ctx, 0, dev(probs[0][2]))
        st.st_set_frozen_features(ctx, 1, dev(probs[1][0])); st.st_teacher_labels(ctx, 1, dev(probs[1][2]))
        st.st_distill_step(ctx, 1)                                   # block 1's skip input is missing
    assert ei.value.status == st.ST_ERR_BAD_STATE
    for frame in range(2):                                           # the second key frame swaps the two streams' inputs
        for s in range(2):
            feat, skips, T, _ = probs[(s + frame) % 2]
            feed(ctx, s, feat, skips, T)
        loss = np.zeros((2, K), np.float32)
        st.st_distill_step(ctx, K, loss)
        for s in range(2):
            feat, skips, T, _ = probs[(s + frame) % 2]
            lab = oracle.teacher_labels(T)
            ref = [oracle.stack_distill_step(heads[s], feat, skips, lab)[0] for _ in range(K)]
            np.testing.assert_allclose(loss[s], ref, rtol=3e-4)
    for s in range(2):
        got = np.empty(ctx.n_params, np.float32)
        st.st_pack_updated_params(ctx, s, got)
        sl = heads[s].trained_slice()
        assert rel_l2(got - probs[s][3][sl], heads[s].theta[sl].astype(np.float64) - probs[s][3][sl]) <= 2e-2
    st.st_destroy(ctx)


def test_stack_workload_full_width_band_and_full_frame():
    """The stack workload (two blocks with skip inputs, 128 -> 128 -> 64 -> 21) at full width: a band of rows against
    the oracle over K = 4 steps with momentum, then the whole 720p frame through its invariants."""
    full = si.get_config(6)
    blocks, C = [tuple(b) for b in full.blocks], full.n_classes
    theta = si.initial_stack_params(full.c_in, blocks, C, 1000)
    # ---- a band the oracle finishes in seconds
    rows, K = 10, 4
    cfg = si.WorkloadConfig("band", full.c_in, 0, C, rows, full.feat_w, n_regions=24, teacher="onehot_noise", blocks=full.blocks)
    feat = si.frozen_features(cfg.c_in, rows, cfg.feat_w, 3)
    skips = [si.skip_features(cfg, b, 3) for b in range(2)]
    T = si.teacher_logits(cfg, stream=1)
    ctx = make_ctx(cfg.c_in, blocks, C, rows, cfg.feat_w, theta, 0, lr=full.lr, mu=full.momentum)
    feed(ctx, 0, feat, skips, T)
    loss = np.zeros(K, np.float32)
    st.st_distill_step(ctx, K, loss)
    lab = oracle.teacher_labels(T)
    plain = oracle.StackHead(cfg.c_in, blocks, C, lr=full.lr, momentum=full.momentum, theta=theta)
    quant = oracle.StackHead(cfg.c_in, blocks, C, lr=full.lr, momentum=full.momentum, theta=theta, quantize_bf16=True)
    ref = [oracle.stack_distill_step(plain, feat, skips, lab)[0] for _ in range(K)]
    q = [oracle.stack_distill_step(quant, feat, skips, lab)[0] for _ in range(K)]
    np.testing.assert_allclose(loss, q, rtol=3e-5)
    np.testing.assert_allclose(loss, ref, rtol=1e-4 * np.sqrt(full.feat_h / rows))
    got = np.empty(ctx.n_params, np.float32)
    st.st_pack_updated_params(ctx, 0, got)
    assert rel_l2(got - theta, quant.theta.astype(np.float64) - theta) <= 5e-3
    assert rel_l2(got - theta, plain.theta.astype(np.float64) - theta) <= 2e-2
    st.st_destroy(ctx)
    # ---- the whole frame
    K = full.k_steps
    ctx = make_ctx(full.c_in, blocks, C, full.feat_h, full.feat_w, theta, 0, lr=full.lr, mu=full.momentum)
    T = si.teacher_logits(full)
    feed(ctx, 0, si.frozen_features(full.c_in, full.feat_h, full.feat_w, 0), [si.skip_features(full, b, 0) for b in range(2)], T)
    loss = np.zeros(K, np.float32)
    conf = np.zeros((K, C, C), np.int64)
    st.st_distill_step(ctx, K, loss, conf)
    lab = oracle.teacher_labels(T)
    assert np.isfinite(loss).all() and loss[-1] < loss[0]
    for k in range(K):
        assert conf[k].sum() == lab.size
        np.testing.assert_array_equal(conf[k].sum(1), np.bincount(lab.ravel(), minlength=C))
    assert st.st_pack_updated_params(ctx, 0, np.empty(ctx.n_params, np.float32)) == theta.size * 4
    st.st_destroy(ctx)
