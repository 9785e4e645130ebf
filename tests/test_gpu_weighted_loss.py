"""GPU parity of Section 5.2's loss weighting (cross-entropy of pixels near and within non-background objects
scaled by an integer factor) against the oracle: which pixels are weighted (through the zero-weights closed form,
where the loss is ln C times the mean weight), loss, logit gradient and parameter gradient on smooth and on steep
logits (both code paths of the fused kernel), for both heads, fp32 and bf16 GEMMs."""
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


def object_labels(h, w, C, seed, bg=0):
    """Mostly background with a few objects, one touching the frame corner and one the right edge."""
    rng = np.random.default_rng(seed)
    lab = np.full((4 * h, 4 * w), bg, np.uint8)
    lab[:3, :5] = (bg + 1) % C
    lab[4 * h // 2: 4 * h // 2 + 6, 4 * w - 2:] = (bg + 2) % C
    for _ in range(4):
        y, x = rng.integers(0, 4 * h - 4), rng.integers(0, 4 * w - 6)
        lab[y:y + rng.integers(1, 5), x:x + rng.integers(1, 7)] = rng.integers(0, C)
    return lab


def ctx_for(c_in, c_hidden, C, h, w, theta, prec, weight, radius, bg=0, lr=0.05, mu=0.0):
    return st.st_init_head(n_streams=1, c_in=c_in, c_hidden=c_hidden, n_classes=C, feat_h=h, feat_w=w, gemm_precision=prec,
                           lr=lr, momentum=mu, cuda_stream=torch.cuda.current_stream().cuda_stream, init_params=theta,
                           object_weight=weight, object_radius=radius, background_class=bg)


@pytest.mark.parametrize("h,w,C,radius,weight,bg", [(10, 37, 4, 0, 5, 0), (45, 64, 21, 3, 5, 0), (9, 12, 3, 9, 2, 1), (23, 40, 5, 64, 3, 0)])
def test_zero_weights_give_ln_c_times_the_mean_weight(h, w, C, radius, weight, bg):
    lab = object_labels(h, w, C, h + radius, bg)
    wgt = oracle.object_weights(lab, bg, radius, weight)
    theta = np.zeros(st.st_param_count(8, 0, C), np.float32)
    ctx = ctx_for(8, 0, C, h, w, theta, 0, weight, radius, bg)
    st.st_set_frozen_features(ctx, 0, dev(si.frozen_features(8, h, w, 1))); st.st_set_labels(ctx, 0, dev(lab))
    loss = torch.zeros(1, dtype=torch.float32, device="cuda")
    st.st_distill_step(ctx, 1, loss)
    # uniform softmax: every pixel's loss is ln C, so the weighted mean is ln C * mean(weight): this pins the set of
    # weighted pixels (the two sides agree on the sum of the weights to a small fraction of one weight step)
    assert abs(float(loss.item()) / np.log(C) * lab.size - wgt.astype(np.int64).sum()) < 1e-5 * wgt.astype(np.int64).sum() + 0.5
    # and db_c = sum_p w_p (1/C - [label_p = c]) / P
    g = st.st_read_tensor(ctx, 0, st.ST_TENSOR_PARAM_GRAD)[-C:]
    ref = np.array([(wgt.astype(np.float64) * (1.0 / C - (lab == c))).sum() / lab.size for c in range(C)])
    np.testing.assert_allclose(g, ref, rtol=0, atol=2e-6)
    st.st_destroy(ctx)


@pytest.mark.parametrize("c_in,c_hidden,C,h,w,prec,scale", [
    (8, 0, 4, 19, 45, 0, 1.0), (8, 0, 4, 19, 45, 0, 60.0), (8, 8, 5, 12, 20, 0, 1.0), (64, 0, 21, 24, 40, 1, 1.0), (64, 64, 5, 24, 40, 1, 1.0)])
def test_weighted_steps_match_the_oracle(c_in, c_hidden, C, h, w, prec, scale):
    lab = object_labels(h, w, C, 5)
    feat = si.frozen_features(c_in, h, w, 2)
    theta = (si.initial_head_params(c_in, c_hidden, C, 3) * scale).astype(np.float32)   # scale 60: steep logits, the row-by-row path
    ctx = ctx_for(c_in, c_hidden, C, h, w, theta, prec, 5, 2)
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_set_labels(ctx, 0, dev(lab))
    head = oracle.Head(c_in, c_hidden, C, lr=0.05, theta=theta, object_weight=5, object_radius=2, quantize_bf16=bool(prec))
    ref_loss, ref_grad, _ = oracle.gradients(head, feat, lab)
    plain_loss = oracle.gradients(oracle.Head(c_in, c_hidden, C, theta=theta, quantize_bf16=bool(prec)), feat, lab)[0]
    assert abs(ref_loss - plain_loss) > 0.02 * plain_loss                  # the weighting matters in this case
    loss = torch.zeros(2, dtype=torch.float32, device="cuda")
    st.st_distill_step(ctx, 1, loss[:1])
    assert float(loss[0]) == pytest.approx(ref_loss, rel=1e-4 if prec == 0 else 2e-3)
    g = st.st_read_tensor(ctx, 0, st.ST_TENSOR_PARAM_GRAD)
    assert rel_l2(g, ref_grad) < (2e-5 if prec == 0 else 1e-2)
    # the logit gradient itself (fp32 copy, produced on demand with bf16 GEMMs)
    z, _ = oracle.head_forward(head, feat)
    wgt = oracle.object_weights(lab, 0, 2, 5)
    _, gfull, _ = oracle.softmax_ce(oracle.upsample(z, 4), lab, weights=wgt)
    dz = st.st_read_tensor(ctx, 0, st.ST_TENSOR_LOGIT_GRAD)
    assert rel_l2(dz, oracle.upsample_adjoint(gfull, 4).ravel()) < (2e-5 if prec == 0 else 2e-3)
    # a second step continues from the first
    oracle.distill_step(head, feat, lab)
    ref2 = oracle.gradients(head, feat, lab)[0]
    st.st_distill_step(ctx, 1, loss[1:])
    assert float(loss[1]) == pytest.approx(ref2, rel=1e-4 if prec == 0 else 3e-3)
    st.st_destroy(ctx)


def test_weighting_off_and_bad_arguments():
    c_in, C, h, w = 8, 4, 6, 8
    lab = object_labels(h, w, C, 1)
    feat = si.frozen_features(c_in, h, w, 2)
    theta = si.initial_head_params(c_in, 0, C, 3)
    out = []
    for weight in (0, 1):                                                   # both mean "off": the plain loss
        ctx = ctx_for(c_in, 0, C, h, w, theta, 0, weight, 3)
        st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_set_labels(ctx, 0, dev(lab))
        loss = torch.zeros(1, dtype=torch.float32, device="cuda")
        st.st_distill_step(ctx, 1, loss)
        out.append(float(loss.item()))
        st.st_destroy(ctx)
    ref = oracle.gradients(oracle.Head(c_in, 0, C, theta=theta), feat, lab)[0]
    assert out[0] == out[1] == pytest.approx(ref, rel=1e-5)
    for kw, status in ((dict(weight=6, radius=1), st.ST_ERR_UNSUPPORTED), (dict(weight=5, radius=65), st.ST_ERR_UNSUPPORTED),
                       (dict(weight=5, radius=-1), st.ST_ERR_INVALID_ARG), (dict(weight=5, radius=1, bg=4), st.ST_ERR_INVALID_ARG)):
        with pytest.raises(st.StError) as ei:
            ctx_for(c_in, 0, C, h, w, theta, 0, **kw)
        assert ei.value.status == status
    with pytest.raises(st.StError) as ei:                                   # more than 32 classes: the other loss kernel has no weighting
        ctx_for(c_in, 0, 40, h, w, np.zeros(st.st_param_count(c_in, 0, 40), np.float32), 0, 5, 1)
    assert ei.value.status == st.ST_ERR_UNSUPPORTED
