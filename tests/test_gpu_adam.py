"""GPU parity of the Adam optimiser (Section 5.2) against the oracle: parameters, both moment buffers and the
loss trajectory over several steps, across two calls (the step count of the bias correction carries over), for both
heads in fp32 and with bf16 GEMMs, and inside Train (Algorithm 1)."""
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


def packed(ctx, s=0):
    out = np.empty(ctx.n_params, np.float32)
    st.st_pack_updated_params(ctx, s, out)
    return out


def rel_l2(a, b):
    return float(np.linalg.norm(a.astype(np.float64) - b) / max(np.linalg.norm(b), 1e-30))


@pytest.mark.parametrize("c_in,c_hidden,C,h,w,prec", [
    (8, 0, 4, 11, 13, 0), (8, 16, 4, 11, 13, 0), (64, 0, 5, 24, 40, 1), (64, 64, 5, 24, 40, 1)])
def test_adam_steps_match_the_oracle(c_in, c_hidden, C, h, w, prec):
    cls = si.voronoi_map(4 * h, 4 * w, 6, C, 2001)
    feat = si.label_informed_features(c_in, h, w, cls, 4, 3)
    theta = si.initial_head_params(c_in, c_hidden, C, 1003)
    betas, eps, lr = (0.8, 0.99), 1e-6, 0.01
    ctx = st.st_init_head(n_streams=1, c_in=c_in, c_hidden=c_hidden, n_classes=C, feat_h=h, feat_w=w, gemm_precision=prec,
                          lr=lr, cuda_stream=torch.cuda.current_stream().cuda_stream, init_params=theta,
                          optimizer=1, adam_beta1=betas[0], adam_beta2=betas[1], adam_eps=eps)
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_set_labels(ctx, 0, dev(cls))
    head = oracle.Head(c_in, c_hidden, C, lr=lr, optimizer="adam", betas=betas, eps=eps, theta=theta, quantize_bf16=bool(prec))
    losses = []
    for n in (3, 2):                                            # two calls: step numbers 1..3, then 4..5
        out = torch.zeros(n, dtype=torch.float32, device="cuda")
        st.st_distill_step(ctx, n, out)
        losses += out.cpu().tolist()
    ref = [oracle.distill_step(head, feat, cls)[0] for _ in range(5)]
    tol = 1e-5 if prec == 0 else 2e-3
    np.testing.assert_allclose(losses, ref, rtol=1e-4 if prec == 0 else 2e-3)
    got = packed(ctx)
    assert rel_l2(got - theta, head.theta - theta) < (2e-4 if prec == 0 else 3e-2)       # the update itself
    np.testing.assert_allclose(got, head.theta, rtol=0, atol=tol * max(1.0, np.abs(head.theta).max()))
    # an Adam step is about lr long in every coordinate (at most lr (1 - b1) / sqrt(1 - b2) = 2 lr here)
    assert 2 * lr < np.abs(got - theta).max() <= 5 * 2 * lr
    m = st.st_read_tensor(ctx, 0, st.ST_TENSOR_MOMENTUM) if hasattr(st, "ST_TENSOR_MOMENTUM") else st.st_read_tensor(ctx, 0, 3)
    assert rel_l2(m, head.vel) < (1e-4 if prec == 0 else 3e-2)
    st.st_destroy(ctx)


def test_default_constants_and_bad_arguments():
    c_in, C, h, w = 8, 3, 5, 7
    cls = si.voronoi_map(4 * h, 4 * w, 4, C, 2002)
    feat = si.label_informed_features(c_in, h, w, cls, 4, 1)
    theta = si.initial_head_params(c_in, 0, C, 1)
    kw = dict(n_streams=1, c_in=c_in, n_classes=C, feat_h=h, feat_w=w, lr=0.01,
              cuda_stream=torch.cuda.current_stream().cuda_stream, init_params=theta)
    ctx = st.st_init_head(optimizer=1, **kw)                   # zeros select 0.9, 0.999, 1e-8
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_set_labels(ctx, 0, dev(cls))
    st.st_distill_step(ctx, 2)
    head = oracle.Head(c_in, 0, C, lr=0.01, optimizer="adam", theta=theta)
    for _ in range(2):
        oracle.distill_step(head, feat, cls)
    np.testing.assert_allclose(packed(ctx), head.theta, rtol=0, atol=2e-6)
    st.st_destroy(ctx)
    for bad in (dict(optimizer=2), dict(optimizer=1, adam_beta1=1.0), dict(optimizer=1, adam_beta2=-0.5), dict(optimizer=1, adam_eps=-1.0)):
        with pytest.raises(st.StError) as ei:
            st.st_init_head(**bad, **kw)
        assert ei.value.status == st.ST_ERR_INVALID_ARG


def test_train_key_frame_with_adam_counts_only_the_steps_it_took():
    c_in, C, h, w, K = 8, 4, 12, 20, 6
    cls = si.voronoi_map(4 * h, 4 * w, 6, C, 2001)
    feat = si.label_informed_features(c_in, h, w, cls, 4, 1)
    theta = si.initial_head_params(c_in, 0, C, 1001)
    mk = lambda: oracle.Head(c_in, 0, C, lr=0.05, optimizer="adam", theta=theta)
    full = oracle.train_key_frame(mk(), feat, cls, 2.0, K).metrics
    thr = 0.5 * (full[1] + full[2])
    assert full[2] > thr > full[1] and all(abs(x - thr) > 1e-2 for x in full[:3])
    ctx = st.st_init_head(n_streams=1, c_in=c_in, n_classes=C, feat_h=h, feat_w=w, lr=0.05, optimizer=1,
                          cuda_stream=torch.cuda.current_stream().cuda_stream, init_params=theta)
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_set_labels(ctx, 0, dev(cls))
    n_upd = np.zeros(1, np.int32)
    st.st_train_key_frame(ctx, thr, K, n_upd)                  # ends after two updates
    head = mk()
    r = oracle.train_key_frame(head, feat, cls, thr, K)
    assert n_upd[0] == r.n_updates == 2
    np.testing.assert_allclose(packed(ctx), head.theta, rtol=0, atol=2e-6)
    # the next plain step is step number 3 of Adam on both sides (not number K + 1)
    st.st_distill_step(ctx, 1)
    oracle.distill_step(head, feat, cls)
    assert head.t == 3
    np.testing.assert_allclose(packed(ctx), head.theta, rtol=0, atol=3e-6)
    st.st_destroy(ctx)
