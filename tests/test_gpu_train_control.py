"""GPU parity of st_train_key_frame (Algorithm 1, Train) against the oracle's train_key_frame.

The loop's decisions compare mean IoUs with THRESHOLD and with each other; the GPU's masks may differ from the
oracle's in a few near-tie pixels, so (i) the decisions are checked exactly by replaying Algorithm 1's rules on the
GPU's own confusion matrices with the oracle's metric, (ii) the metrics are compared with the oracle's within a small
tolerance, and where the oracle's decisions are robust to that tolerance the control flow must be identical,
(iii) the returned parameters must be bit-identical to the GPU's own plain loop of best_iter steps when that loop also
asks for the per-step confusion matrices (the same instantiation of the loss kernel), and equal to rounding otherwise."""
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


def problem(seed, c_in, c_hidden, C, h, w, strength=2.0):
    cls = si.voronoi_map(4 * h, 4 * w, max(6, C), C, 2000 + seed)
    feat = si.label_informed_features(c_in, h, w, cls, 4, seed, strength)
    theta = si.initial_head_params(c_in, c_hidden, C, 1000 + seed)
    return feat, cls, theta


def make_ctx(c_in, c_hidden, C, h, w, thetas, S, prec, lr, mu):
    return st.st_init_head(n_streams=S, c_in=c_in, c_hidden=c_hidden, n_classes=C, feat_h=h, feat_w=w,
                           gemm_precision=prec, lr=lr, momentum=mu,
                           cuda_stream=torch.cuda.current_stream().cuda_stream, init_params=np.concatenate(thetas))


def packed(ctx, s=0):
    out = np.empty(ctx.n_params, np.float32)
    st.st_pack_updated_params(ctx, s, out)
    return out


def rules(metrics, threshold, max_updates):
    """Algorithm 1's rules on a list of metrics: (n_updates, best_iter, best_metric)."""
    best, best_i, n = metrics[0], 0, 0
    if metrics[0] < threshold:
        for i in range(1, max_updates + 1):
            n = i
            if metrics[i] > best:
                best, best_i = metrics[i], i
            if metrics[i] > threshold:
                break
    return n, best_i, best


def run_train(ctx, S, C, thr, K):
    n_upd = np.zeros(S, np.int32); best = np.zeros(S, np.float64)
    met = np.zeros((S, K + 1), np.float64); los = np.zeros((S, K + 1), np.float32)
    conf = np.zeros((S, K + 1, C, C), np.int64)
    st.st_train_key_frame(ctx, thr, K, n_upd, best, met, los, conf)
    return n_upd, best, met, los, conf


CASES = [  # c_in, c_hidden, C, h, w, prec, lr, mu
    (8, 0, 4, 12, 20, 0, 0.5, 0.9),
    (8, 8, 4, 12, 20, 0, 0.5, 0.9),
    (64, 0, 5, 24, 40, 1, 0.5, 0.9),
    (64, 64, 5, 24, 40, 1, 0.2, 0.9),
]


@pytest.mark.parametrize("c_in,c_hidden,C,h,w,prec,lr,mu", CASES)
def test_train_key_frame_matches_algorithm_1(c_in, c_hidden, C, h, w, prec, lr, mu):
    K = 8
    feat, labels, theta = problem(1, c_in, c_hidden, C, h, w)
    P = labels.size
    # the oracle's metric after 0..K plain steps
    # bf16 GEMMs: the reference rounds its GEMM operands at the same places (the lr of this test amplifies rounding
    # noise over the steps, and the point here is the control flow)
    ref = oracle.train_key_frame(oracle.Head(c_in, c_hidden, C, lr=lr, momentum=mu, theta=theta, quantize_bf16=bool(prec)),
                                 feat, labels, 2.0, K)
    m_ref = ref.metrics
    assert max(m_ref) > m_ref[0] + 0.05, m_ref
    tol = 5e-3 if prec == 0 else 3e-2          # mean IoU moves by about (flipped pixels / P) * few; bf16 logits flip more
    thresholds = [0.0, 2.0] + sorted(set(0.5 * (a + b) for a, b in zip(sorted(m_ref)[:-1], sorted(m_ref)[1:])))[::2]
    exits = set()
    for thr in thresholds:
        ctx = make_ctx(c_in, c_hidden, C, h, w, [theta], 1, prec, lr, mu)
        st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_set_labels(ctx, 0, dev(labels))
        n_upd, best, met, los, conf = run_train(ctx, 1, C, thr, K)
        n = int(n_upd[0])
        # (i) the device's decisions follow Algorithm 1 exactly, given its own confusion matrices
        m_gpu = [oracle.miou(conf[0, i]) for i in range(n + 1)]
        assert [int(conf[0, i].sum()) for i in range(n + 1)] == [P] * (n + 1)
        # predictions the loop never made are marked; the others carry the metric of their confusion matrix
        np.testing.assert_array_equal(met[0, :n + 1], m_gpu)
        assert (met[0, n + 1:] == -1.0).all()
        # ... and the rules applied to them by hand give the same exit and the same best
        full = m_gpu + [0.0] * (K - n)
        n_r, bi_r, best_r = rules(full, thr, K)
        assert (n, float(best[0])) == (n_r, best_r), (thr, m_gpu)
        # (ii) metrics and losses agree with the oracle's
        np.testing.assert_allclose(m_gpu, m_ref[:n + 1], atol=tol)
        np.testing.assert_allclose(los[0, :n], ref.losses[:n], rtol=2e-3 if prec else 1e-4)
        # where no oracle metric is within tol of the threshold or of the running best, the control flow is the oracle's
        n_o, bi_o, _ = rules(m_ref, thr, K)
        robust = all(abs(x - thr) > 2 * tol for x in m_ref[:n_o + 1])
        if robust:
            assert n == n_o, (thr, m_ref, m_gpu)
        # (iii) the returned student is the GPU's own iterate after best_iter plain steps: bit for bit against the loop
        # that also computes the per-step confusion (the loss kernel is instantiated with and without it, and the two
        # instantiations round a few gradient values differently in the last place), to rounding against the other
        ctx2 = make_ctx(c_in, c_hidden, C, h, w, [theta], 1, prec, lr, mu)
        st.st_set_frozen_features(ctx2, 0, dev(feat)); st.st_set_labels(ctx2, 0, dev(labels))
        ctx3 = make_ctx(c_in, c_hidden, C, h, w, [theta], 1, prec, lr, mu)
        st.st_set_frozen_features(ctx3, 0, dev(feat)); st.st_set_labels(ctx3, 0, dev(labels))
        if bi_r > 0:
            st.st_distill_step(ctx2, bi_r, None, torch.zeros((1, bi_r, C, C), dtype=torch.int64, device="cuda"))
            st.st_distill_step(ctx3, bi_r)
        assert packed(ctx).tobytes() == packed(ctx2).tobytes(), (thr, bi_r)
        np.testing.assert_allclose(packed(ctx), packed(ctx3), rtol=0, atol=(1e-5 if prec == 0 else 1e-3) * np.abs(packed(ctx3)).max())
        st.st_destroy(ctx3)
        # the stored student is usable at once: its mask reproduces best_metric
        cf = np.zeros((C, C), np.int64)
        assert st.st_agreement(ctx, 0, None, None, cf) == float(best[0])
        exits.add(n)
        st.st_destroy(ctx); st.st_destroy(ctx2)
    assert 0 in exits and K in exits and len(exits) >= 3, exits


def test_streams_end_their_loops_independently():
    c_in, C, h, w, K, lr, mu = 8, 4, 12, 20, 8, 0.5, 0.9
    probs = [problem(s, c_in, 0, C, h, w, strength=[2.0, 0.0, 3.0][s]) for s in range(3)]   # stream 1 cannot learn
    refs = [oracle.train_key_frame(oracle.Head(c_in, 0, C, lr=lr, momentum=mu, theta=p[2]), p[0], p[1], 2.0, K).metrics for p in probs]
    thr = 0.5 * (refs[0][0] + max(refs[0]))
    ctx = make_ctx(c_in, 0, C, h, w, [p[2] for p in probs], 3, 0, lr, mu)
    for s, (feat, labels, _) in enumerate(probs):
        st.st_set_frozen_features(ctx, s, dev(feat)); st.st_set_labels(ctx, s, dev(labels))
    n_upd, best, met, los, conf = run_train(ctx, 3, C, thr, K)
    for s, (feat, labels, theta) in enumerate(probs):
        r = oracle.train_key_frame(oracle.Head(c_in, 0, C, lr=lr, momentum=mu, theta=theta), feat, labels, thr, K)
        m_gpu = [oracle.miou(conf[s, i]) for i in range(int(n_upd[s]) + 1)]
        assert rules(m_gpu + [0.0] * K, thr, K)[0] == n_upd[s]
        if all(abs(x - thr) > 1e-2 for x in r.metrics):
            assert n_upd[s] == r.n_updates
        head = oracle.Head(c_in, 0, C, lr=lr, momentum=mu, theta=theta)
        for _ in range(rules(m_gpu + [0.0] * K, thr, K)[1]):
            oracle.distill_step(head, feat, labels)
        np.testing.assert_allclose(packed(ctx, s), head.theta, rtol=1e-4, atol=1e-6)
    assert len(set(int(x) for x in n_upd)) >= 2, n_upd            # the streams really took different exits
    st.st_destroy(ctx)


def test_train_key_frame_argument_errors_and_replay():
    c_in, C, h, w = 8, 3, 4, 4
    feat, labels, theta = problem(0, c_in, 0, C, h, w)
    ctx = make_ctx(c_in, 0, C, h, w, [theta], 1, 0, 0.1, 0.0)
    with pytest.raises(st.StError) as ei:
        st.st_train_key_frame(ctx, 0.5, 3)
    assert ei.value.status == st.ST_ERR_BAD_STATE
    st.st_set_frozen_features(ctx, 0, dev(feat)); st.st_set_labels(ctx, 0, dev(labels))
    for bad in (-1, 64):
        with pytest.raises(st.StError) as ei:
            st.st_train_key_frame(ctx, 0.5, bad)
        assert ei.value.status == st.ST_ERR_INVALID_ARG
    with pytest.raises(st.StError):
        st.st_train_key_frame(ctx, float("nan"), 3)
    # MAX_UPDATES = 0: one prediction, no update
    n_upd, best, met, los, conf = run_train(ctx, 1, C, 2.0, 0)
    assert n_upd[0] == 0 and packed(ctx).tobytes() == np.asarray(theta, np.float32).tobytes()
    # two calls in a row (the second one replays the captured graph) continue from the returned student
    a = run_train(ctx, 1, C, 2.0, 3)
    b = run_train(ctx, 1, C, 2.0, 3)
    assert a[0][0] == 3 and b[0][0] == 3 and b[2][0, 0] == a[1][0]      # the second call starts from the first one's best
    st.st_destroy(ctx)


@pytest.mark.parametrize("c_hidden", [0, 64])
def test_streams_end_independently_with_tensor_core_kernels(c_hidden):
    """Three streams with bf16 GEMMs: once a stream's loop has ended, the blocks of its GEMMs and of its loss kernel
    return at once (the persistent 3x3 forward leaves its tiles out) while the other streams keep training."""
    c_in, C, h, w, K, lr, mu = 64, 5, 24, 40, 6, 0.3, 0.9
    strengths = [3.0, 0.0, 2.0]                                       # stream 1 cannot learn: its loop runs to the end
    probs = [problem(s, c_in, c_hidden, C, h, w, strength=strengths[s]) for s in range(3)]
    mk = lambda s: oracle.Head(c_in, c_hidden, C, lr=lr, momentum=mu, theta=probs[s][2], quantize_bf16=True)
    full = [oracle.train_key_frame(mk(s), probs[s][0], probs[s][1], 2.0, K).metrics for s in range(3)]
    thr = 0.5 * (full[0][1] + full[0][2]) if full[0][2] > full[0][1] else 0.5 * (full[0][0] + max(full[0]))
    ctx = make_ctx(c_in, c_hidden, C, h, w, [p[2] for p in probs], 3, 1, lr, mu)
    for s, (feat, labels, _) in enumerate(probs):
        st.st_set_frozen_features(ctx, s, dev(feat)); st.st_set_labels(ctx, s, dev(labels))
    n_upd, best, met, los, conf = run_train(ctx, 3, C, thr, K)
    exits = []
    for s, (feat, labels, theta) in enumerate(probs):
        n = int(n_upd[s])
        m_gpu = [oracle.miou(conf[s, i]) for i in range(n + 1)]
        n_r, bi_r, best_r = rules(m_gpu + [0.0] * K, thr, K)
        assert (n, float(best[s])) == (n_r, best_r), (s, m_gpu)      # the device followed Algorithm 1 on its own metrics
        assert (met[s, n + 1:] == -1.0).all()
        # the stream's returned student: its own plain loop of best_iter steps (same kernels, no other stream involved)
        solo = make_ctx(c_in, c_hidden, C, h, w, [theta], 1, 1, lr, mu)
        st.st_set_frozen_features(solo, 0, dev(feat)); st.st_set_labels(solo, 0, dev(labels))
        if bi_r > 0:
            st.st_distill_step(solo, bi_r, None, torch.zeros((1, bi_r, C, C), dtype=torch.int64, device="cuda"))
        assert packed(ctx, s).tobytes() == packed(solo).tobytes(), s
        st.st_destroy(solo)
        np.testing.assert_allclose(m_gpu, full[s][:n + 1], atol=3e-2)
        exits.append(n)
    assert len(set(exits)) >= 2, exits                               # some loops went on after others had ended
    # a second call starts from the returned students: those already past the threshold take no step
    n2 = np.zeros(3, np.int32)
    st.st_train_key_frame(ctx, thr, K, n2)
    for s in range(3):
        if best[s] >= thr:
            assert n2[s] == 0, (s, n2)
    st.st_destroy(ctx)
