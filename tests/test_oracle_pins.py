"""Pins for the CPU oracle: each function is checked against something other than
itself (closed forms, invariants, brute force, library routines, the paper's
printed sizes), so that a dropped term, a wrong sign/index or a transposed
operand fails at least one test.  CPU only.
"""
import itertools
import os

import numpy as np
import pytest

import oracle
import synth_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, *v = line.split()
            out[k] = [float(t) for t in v]
    return out


# ---------------------------------------------------------------------------- labels
def test_labels_brute_force_and_ties():
    rng = np.random.default_rng(1)
    T = rng.integers(-2, 3, size=(5, 7, 9)).astype(np.float32)   # many exact ties
    got = oracle.teacher_labels(T)
    for y in range(7):
        for x in range(9):
            col = T[:, y, x]
            best = max(col)
            first = [c for c in range(5) if col[c] == best][0]   # lowest index wins
            assert got[y, x] == first
    assert got.dtype == np.uint8
    # property: chosen value >= all others, strictly greater than every lower index
    chosen = np.take_along_axis(T, got[None].astype(np.int64), 0)[0]
    assert (chosen[None] >= T).all()
    for c in range(5):
        lower = (np.arange(5)[:, None, None] < got[None]) & (T == chosen[None])
        assert not lower.any()


def test_labels_recover_voronoi_map():
    cfg = si.get_config(1)
    T = si.teacher_logits(cfg)
    cls = si.voronoi_map(cfg.frame_h, cfg.frame_w, cfg.n_regions, cfg.n_classes, 2000)
    # the winner is exactly 4.0 and the noise N(0, 0.5) never reaches 4.0 (8 sigma)
    assert (oracle.teacher_labels(T) == cls).all()


def test_label_map_is_one_byte_per_pixel_table4():
    g = _golden("table4_sizes.txt")
    lab = oracle.teacher_labels(np.zeros((2, 720, 1280), np.float32))
    assert lab.nbytes == 1280 * 720
    assert round(lab.nbytes / 2**20, 3) == g["label_map_to_client_mb"][0]
    assert round(1280 * 720 * 3 / 2**20, 3) == g["frame_to_server_mb"][0]


# ---------------------------------------------------------------------------- conv forward
def test_conv1x1_is_a_matrix_product():
    rng = np.random.default_rng(2)
    x = rng.standard_normal((6, 5, 7)).astype(np.float32)
    W = rng.standard_normal((4, 6, 1, 1)).astype(np.float32)
    b = rng.standard_normal(4).astype(np.float32)
    got = oracle.conv_fwd(x, W, b)
    ref = (W.reshape(4, 6).astype(np.float64) @ x.reshape(6, -1).astype(np.float64)
           + b[:, None]).reshape(4, 5, 7)
    np.testing.assert_allclose(got, ref, rtol=1e-6, atol=1e-6)
    # W[co][ci] is not W[ci][co]: a transposed operand would fail on a non-square case above


def test_conv3x3_centre_tap_reduces_to_1x1_and_border_counts():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((3, 6, 8)).astype(np.float32)
    W1 = rng.standard_normal((5, 3, 1, 1)).astype(np.float32)
    b = rng.standard_normal(5).astype(np.float32)
    W3 = np.zeros((5, 3, 3, 3), np.float32)
    W3[:, :, 1, 1] = W1[:, :, 0, 0]
    np.testing.assert_array_equal(oracle.conv_fwd(x, W3, b), oracle.conv_fwd(x, W1, b))
    ones = np.ones((1, 4, 5), np.float32)
    cnt = oracle.conv_fwd(ones, np.ones((1, 1, 3, 3), np.float32), np.zeros(1, np.float32))[0]
    assert cnt[0, 0] == 4 and cnt[0, 2] == 6 and cnt[2, 0] == 6 and cnt[1, 1] == 9 and cnt[3, 4] == 4


def test_conv3x3_single_tap_shifts_the_right_way():
    # weight at (ky,kx)=(0,2) reads in[y-1][x+1]
    x = np.zeros((1, 5, 5), np.float32)
    x[0, 1, 3] = 7.0
    W = np.zeros((1, 1, 3, 3), np.float32)
    W[0, 0, 0, 2] = 1.0
    out = oracle.conv_fwd(x, W, np.zeros(1, np.float32))[0]
    assert out[2, 2] == 7.0 and out.sum() == 7.0


def test_conv_and_relu_vs_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(4)
    x = rng.standard_normal((4, 7, 9)).astype(np.float32)
    W = rng.standard_normal((6, 4, 3, 3)).astype(np.float32)
    b = rng.standard_normal(6).astype(np.float32)
    ref = torch.relu(torch.nn.functional.conv2d(torch.from_numpy(x)[None].double(),
                                                torch.from_numpy(W).double(),
                                                torch.from_numpy(b).double(), padding=1))[0].numpy()
    np.testing.assert_allclose(oracle.conv_fwd(x, W, b, relu=True), ref, rtol=1e-5, atol=1e-5)


# ---------------------------------------------------------------------------- upsample
def test_upsample_invariants():
    const = np.full((2, 3, 5), 1.7, np.float32)
    assert (oracle.upsample(const, 4) == np.float32(1.7)).all()
    rng = np.random.default_rng(5)
    z = rng.standard_normal((2, 4, 6)).astype(np.float32)
    np.testing.assert_array_equal(oracle.upsample(z, 1), z)
    # affine ramp reproduced exactly in the interior (away from the clamped border)
    yy, xx = np.meshgrid(np.arange(6.0), np.arange(7.0), indexing="ij")
    ramp = (2.0 * yy - 3.0 * xx + 1.0)[None].astype(np.float64)
    u = oracle.upsample(ramp, 4)[0]
    Y, X = np.meshgrid(np.arange(24.0), np.arange(28.0), indexing="ij")
    ref = 2.0 * ((Y + 0.5) / 4 - 0.5) - 3.0 * ((X + 0.5) / 4 - 0.5) + 1.0
    np.testing.assert_allclose(u[2:-2, 2:-2], ref[2:-2, 2:-2], rtol=0, atol=1e-12)
    # borders clamp to the edge value
    assert u[0, 0] == ramp[0, 0, 0] and u[-1, -1] == ramp[0, -1, -1]


def test_upsample_row_weights_are_eighths():
    # for s = 4 and Y = 4q + r the two source rows carry weights (3/8,5/8), (1/8,7/8), (7/8,1/8), (5/8,3/8)
    z = np.zeros((1, 3, 1), np.float64)
    z[0, 1, 0] = 1.0
    u = oracle.upsample(z, 4)[0, :, 0]
    np.testing.assert_array_equal(u, [0, 0, 1 / 8, 3 / 8, 5 / 8, 7 / 8, 7 / 8, 5 / 8, 3 / 8, 1 / 8, 0, 0])


def test_upsample_vs_torch_interpolate():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(6)
    z = rng.standard_normal((3, 5, 7)).astype(np.float32)
    ref = torch.nn.functional.interpolate(torch.from_numpy(z)[None].double(), scale_factor=4,
                                          mode="bilinear", align_corners=False)[0].numpy()
    np.testing.assert_allclose(oracle.upsample(z, 4), ref, rtol=1e-6, atol=1e-6)
    ref2 = torch.nn.functional.interpolate(torch.from_numpy(z)[None].double(), scale_factor=2,
                                           mode="bilinear", align_corners=False)[0].numpy()
    np.testing.assert_allclose(oracle.upsample(z, 2), ref2, rtol=1e-6, atol=1e-6)


def test_adjoint_dot_product_identity():
    rng = np.random.default_rng(7)
    a = rng.standard_normal((2, 4, 5))
    g = rng.standard_normal((2, 16, 20))
    lhs = float((oracle.upsample(a, 4) * g).sum())
    rhs = float((a * oracle.upsample_adjoint(g, 4)).sum())
    assert abs(lhs - rhs) <= 1e-11 * max(1.0, abs(lhs))


# ---------------------------------------------------------------------------- loss and its gradient
def test_ce_gradient_closed_form():
    rng = np.random.default_rng(8)
    u = rng.standard_normal((5, 6, 7)) * 3
    lab = rng.integers(0, 5, size=(6, 7)).astype(np.uint8)
    loss, g, bad = oracle.softmax_ce(u, lab)
    assert bad == 0
    P = 42
    e = np.exp(u - u.max(0))
    p = e / e.sum(0)
    onehot = (np.arange(5)[:, None, None] == lab[None])
    np.testing.assert_allclose(g, (p - onehot) / P, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(g.sum(0), 0, atol=1e-15)            # rows of p - onehot sum to 0
    ref_loss = float(np.mean(np.log(np.exp(u).sum(0)) - np.take_along_axis(u, lab[None].astype(np.int64), 0)[0]))
    assert abs(loss - ref_loss) < 1e-12
    # shift invariance and a large offset (the max subtraction must be there)
    loss2, _, _ = oracle.softmax_ce(u + 900.0, lab)
    assert abs(loss2 - loss) < 1e-9


def test_ce_vs_torch():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(9)
    u = rng.standard_normal((4, 5, 6)).astype(np.float32)
    lab = rng.integers(0, 4, size=(5, 6)).astype(np.uint8)
    loss, _, _ = oracle.softmax_ce(u, lab)
    ref = torch.nn.functional.cross_entropy(torch.from_numpy(u)[None].double(),
                                            torch.from_numpy(lab.astype(np.int64))[None]).item()
    assert abs(loss - ref) < 1e-7


def test_zero_weights_closed_form():
    # W = 0, b = 0 -> logits 0 -> loss = ln C, db[c] = 1/C - n_c/P, dW rows sum to 0 over classes
    cfgC, cin, h, w = 5, 3, 4, 6
    rng = np.random.default_rng(10)
    feat = rng.standard_normal((cin, h, w))
    lab = rng.integers(0, cfgC, size=(4 * h, 4 * w)).astype(np.uint8)
    head = oracle.Head(cin, 0, cfgC, dtype=np.float64)
    loss, grad, _ = oracle.gradients(head, feat, lab)
    assert abs(loss - np.log(cfgC)) < 1e-12
    dW = grad[:cfgC * cin].reshape(cfgC, cin)
    db = grad[cfgC * cin:]
    counts = np.bincount(lab.ravel(), minlength=cfgC)
    np.testing.assert_allclose(db, 1.0 / cfgC - counts / lab.size, atol=1e-13)
    np.testing.assert_allclose(dW.sum(0), 0, atol=1e-12)


def test_ce_out_of_range_labels_are_skipped_and_counted():
    u = np.zeros((3, 2, 2))
    lab = np.array([[0, 1], [7, 2]], np.uint8)
    loss, g, bad = oracle.softmax_ce(u, lab)
    assert bad == 1 and (g[:, 1, 0] == 0).all()
    assert abs(loss - 3 * np.log(3) / 4) < 1e-12


# ---------------------------------------------------------------------------- whole gradient
def _fd_check(c_hidden):
    rng = np.random.default_rng(11 + c_hidden)
    cin, C, h, w = 3, 3, 3, 5
    feat = np.abs(rng.standard_normal((cin, h, w))) + 0.1
    lab = rng.integers(0, C, size=(4 * h, 4 * w)).astype(np.uint8)
    n = si.head_param_count(cin, c_hidden, C)
    theta = rng.standard_normal(n) * 0.5
    if c_hidden:
        # keep hidden pre-activations away from the ReLU kink: positive weights + positive bias on layer 1
        nw1 = c_hidden * cin * 9
        theta[:nw1] = np.abs(theta[:nw1]) * 0.3
        theta[nw1:nw1 + c_hidden] = 0.5
        theta[nw1] *= -1.0        # one negative weight keeps it generic but far from 0 pre-activation
    head = oracle.Head(cin, c_hidden, C, dtype=np.float64, theta=theta)
    loss, grad, _ = oracle.gradients(head, feat, lab)

    def f(th):
        hd = oracle.Head(cin, c_hidden, C, dtype=np.float64, theta=th)
        z, _ = oracle.head_forward(hd, feat)
        return oracle.softmax_ce(oracle.upsample(z, 4), lab, want_grad=False)[0]

    eps = 1e-6
    fd = np.empty(n)
    for i in range(n):
        tp, tm = theta.copy(), theta.copy()
        tp[i] += eps
        tm[i] -= eps
        fd[i] = (f(tp) - f(tm)) / (2 * eps)
    err = np.abs(fd - grad).max() / max(np.abs(fd).max(), 1e-12)
    assert err < 1e-6, err


def test_finite_differences_1x1_head():
    _fd_check(0)


def test_finite_differences_two_layer_head():
    _fd_check(2)


def test_step_vs_torch_autograd():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(13)
    cin, ch, C, h, w = 4, 5, 3, 4, 6
    feat = np.maximum(rng.standard_normal((cin, h, w)), 0)
    lab = rng.integers(0, C, size=(4 * h, 4 * w)).astype(np.uint8)
    theta = si.initial_head_params(cin, ch, C, 5).astype(np.float64)
    theta[ch * cin * 9: ch * cin * 9 + ch] = 0.05
    head = oracle.Head(cin, ch, C, dtype=np.float64, theta=theta, lr=0.1, momentum=0.9)
    tt = [torch.tensor(a.copy(), requires_grad=True) for wb in head.layers() for a in wb]
    opt = torch.optim.SGD(tt, lr=0.1, momentum=0.9)
    x = torch.from_numpy(feat)[None]
    y = torch.from_numpy(lab.astype(np.int64))[None]
    for _ in range(3):
        loss_o, _ = oracle.distill_step(head, feat, lab)
        opt.zero_grad()
        hdn = torch.relu(torch.nn.functional.conv2d(x, tt[0], tt[1], padding=1))
        z = torch.nn.functional.conv2d(hdn, tt[2], tt[3])
        u = torch.nn.functional.interpolate(z, scale_factor=4, mode="bilinear", align_corners=False)
        loss_t = torch.nn.functional.cross_entropy(u, y)
        loss_t.backward()
        opt.step()
        assert abs(loss_o - loss_t.item()) < 1e-10
    ref = np.concatenate([t.detach().numpy().ravel() for t in tt])
    np.testing.assert_allclose(head.theta, ref, rtol=1e-9, atol=1e-11)


def test_partial_backward_leaves_features_untouched_and_loss_decreases():
    cfg = si.WorkloadConfig("t", 8, 0, 3, 6, 8)
    rng = np.random.default_rng(14)
    feat = np.maximum(rng.standard_normal((8, 6, 8)), 0).astype(np.float32)
    lab = rng.integers(0, 3, size=(24, 32)).astype(np.uint8)
    feat0 = feat.copy()
    head = oracle.Head(8, 0, 3, theta=si.initial_head_params(8, 0, 3, 1), lr=0.05)
    losses = [oracle.distill_step(head, feat, lab)[0] for _ in range(6)]
    np.testing.assert_array_equal(feat, feat0)
    assert all(b < a for a, b in zip(losses, losses[1:]))


# ---------------------------------------------------------------------------- optimiser
def test_sgd_momentum_closed_form():
    g = np.array([0.5, -2.0, 0.0], np.float64)
    theta = np.array([1.0, 2.0, 3.0], np.float64)
    th0 = theta.copy()
    v = np.zeros(3)
    mu, lr = 0.9, 0.01
    total_v = np.zeros(3)
    for t in range(1, 6):
        oracle.sgd_(theta, v, g, lr, mu)
        np.testing.assert_allclose(v, g * (1 - mu**t) / (1 - mu), rtol=1e-13)
        total_v += v
    np.testing.assert_allclose(theta, th0 - lr * total_v, rtol=1e-13)
    # mu = 0 is plain gradient descent
    th = np.array([1.0]); vv = np.zeros(1)
    oracle.sgd_(th, vv, np.array([2.0]), 0.25, 0.0)
    assert th[0] == 0.5 and vv[0] == 2.0


# ---------------------------------------------------------------------------- pack
def test_pack_layout_and_sizes():
    cin, ch, C = 3, 2, 4
    n = si.head_param_count(cin, ch, C)
    head = oracle.Head(cin, ch, C, theta=np.arange(n, dtype=np.float32))
    raw = oracle.pack(head)
    assert raw == np.arange(n, dtype="<f4").tobytes()         # values, fp32, no header
    (W1, b1), (W2, b2) = head.layers()
    assert W1.shape == (ch, cin, 3, 3) and W1[1, 2, 0, 1] == 1 * 27 + 2 * 9 + 1
    assert b1[0] == ch * cin * 9 and W2[0, 0, 0, 0] == ch * cin * 9 + ch
    assert b2[-1] == n - 1
    # sizes of the workloads' packed buffers
    assert si.head_param_count(256, 0, 21) * 4 == 21588
    assert si.head_param_count(64, 0, 4) * 4 == 1040
    assert si.head_param_count(256, 256, 21) * 4 == 2381908
    assert si.head_param_count(256, 256, 19) * 4 == 2379852
    # K = 0 leaves parameters bit-identical; pack -> init -> pack round-trips
    head2 = oracle.Head(cin, ch, C, theta=np.frombuffer(raw, "<f4"))
    assert oracle.pack(head2) == raw


def test_table4_parameter_bytes_are_fp32():
    g = _golden("table4_sizes.txt")
    full = g["student_params_million"][0] * 1e6 * 4 / 2**20
    assert abs(full - g["full_student_mb"][0]) / g["full_student_mb"][0] < 0.02
    part = full * g["trained_fraction"][0]
    assert abs(part - g["updated_part_mb"][0]) / g["updated_part_mb"][0] < 0.02


# ---------------------------------------------------------------------------- metric
def test_confusion_and_miou():
    g = _golden("miou_hand_example.txt")
    lab = np.array(g["label"], np.uint8)
    pred = np.array(g["pred"], np.uint8)
    conf, m, bad = oracle.agreement(lab, pred, 2)
    assert conf.ravel().tolist() == g["conf"] and bad == 0
    assert abs(m - g["miou"][0]) < 1e-15
    _, m3, _ = oracle.agreement(np.array(g["label3"], np.uint8), np.array(g["pred3"], np.uint8), 3)
    assert abs(m3 - g["miou3"][0]) < 1e-15
    rng = np.random.default_rng(15)
    lab = rng.integers(0, 6, 500).astype(np.uint8)
    pred = rng.integers(0, 6, 500).astype(np.uint8)
    conf, m, bad = oracle.agreement(lab, pred, 6)
    brute = np.zeros((6, 6), np.int64)
    for l, q in zip(lab, pred):
        brute[l, q] += 1
    np.testing.assert_array_equal(conf, brute)                  # conf[label][pred], not transposed
    assert conf.sum() == 500
    np.testing.assert_array_equal(conf.sum(1), np.bincount(lab, minlength=6))
    ious = []
    for c in range(6):
        inter = np.sum((lab == c) & (pred == c))
        union = np.sum((lab == c) | (pred == c))
        ious.append(inter / union)
    assert abs(m - np.mean(ious)) < 1e-15
    assert oracle.agreement(lab, lab, 6)[1] == 1.0
    assert oracle.agreement(lab, (lab + 1) % 6, 6)[1] == 0.0
    _, _, bad = oracle.agreement(np.array([0, 9], np.uint8), np.array([0, 0], np.uint8), 6)
    assert bad == 1


def test_round_bf16_ties_to_even():
    a = np.array([1.0, 1.00390625, 1.01171875, -1.00390625, 0.0], np.float32)
    # 1 + 2^-8 is halfway between 1 and 1 + 2^-7 -> even (1.0); 1 + 3*2^-8 -> 1 + 2^-6 (even mantissa)
    np.testing.assert_array_equal(oracle.round_bf16(a),
                                  np.array([1.0, 1.0, 1.015625, -1.0, 0.0], np.float32))
    x = np.random.default_rng(0).standard_normal(1000).astype(np.float32)
    torch = pytest.importorskip("torch")
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(oracle.round_bf16(x), ref)


# ---------------------------------------------------------------------------- Adam (Section 5.2)
def test_adam_first_step_moves_every_weight_by_lr_against_its_gradient_sign():
    # step 1: m_hat = g, v_hat = g^2, so theta moves by lr * g / (|g| + eps): the sign of g, whatever its size
    rng = np.random.default_rng(0)
    for dtype in (np.float32, np.float64):
        theta = rng.standard_normal(50).astype(dtype); g = (rng.standard_normal(50) * 10 ** rng.uniform(-3, 3, 50)).astype(dtype)
        th, m, v = theta.copy(), np.zeros(50, dtype), np.zeros(50, dtype)
        oracle.adam_(th, m, v, g, 0.01, 0.9, 0.999, 1e-8, 1)
        np.testing.assert_allclose(th, theta - 0.01 * g / (np.abs(g) + 1e-8), rtol=0, atol=2e-6 if dtype == np.float32 else 1e-12)
        big = np.abs(g) > 1e-2                                   # there eps / |g| < 1e-6: a plain sign step
        np.testing.assert_allclose(th[big], (theta - 0.01 * np.sign(g))[big], rtol=0, atol=2e-6 if dtype == np.float32 else 2e-8)
        np.testing.assert_allclose(m, 0.1 * g, rtol=1e-6); np.testing.assert_allclose(v, 0.001 * g * g, rtol=1e-6)


def test_adam_constant_gradient_keeps_unit_steps_and_zero_gradient_does_not_move():
    # constant g: m_hat = g and v_hat = g^2 at every step, so every step has length lr
    th, m, v = np.zeros(3), np.zeros(3), np.zeros(3)
    g = np.array([2.0, -0.5, 1e-3])
    for t in range(1, 8):
        oracle.adam_(th, m, v, g, 0.01, 0.9, 0.999, 1e-12, t)
        np.testing.assert_allclose(th, -0.01 * t * np.sign(g), rtol=1e-6)
    th0 = np.ones(4); m, v = np.zeros(4), np.zeros(4)
    oracle.adam_(th0, m, v, np.zeros(4), 0.01, 0.9, 0.999, 1e-8, 1)
    assert (th0 == 1.0).all()


def test_adam_matches_torch_adam_over_several_steps():
    torch = pytest.importorskip("torch")
    rng = np.random.default_rng(1)
    theta0 = rng.standard_normal(40)
    grads = [rng.standard_normal(40) * (1 + k) for k in range(6)]
    th, m, v = theta0.copy(), np.zeros(40), np.zeros(40)
    p = torch.tensor(theta0, dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([p], lr=0.01, betas=(0.8, 0.99), eps=1e-6)
    for t, g in enumerate(grads, 1):
        oracle.adam_(th, m, v, g, 0.01, 0.8, 0.99, 1e-6, t)
        p.grad = torch.tensor(g, dtype=torch.float64)
        opt.step()
        np.testing.assert_allclose(th, p.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_head_with_adam_takes_textbook_steps_on_the_real_gradient():
    rng = np.random.default_rng(2)
    feat = np.maximum(rng.standard_normal((6, 4, 5)), 0).astype(np.float32)
    labels = rng.integers(0, 3, (16, 20)).astype(np.uint8)
    theta = si.initial_head_params(6, 0, 3, 5)
    head = oracle.Head(6, 0, 3, lr=0.01, optimizer="adam", theta=theta)
    th, m, v = np.asarray(theta, np.float64).copy(), np.zeros(theta.size), np.zeros(theta.size)
    for t in range(1, 4):
        _, g, _ = oracle.gradients(head, feat, labels)                 # gradient at the current parameters
        oracle.distill_step(head, feat, labels)
        m = 0.9 * m + 0.1 * g; v = 0.999 * v + 0.001 * g * g            # the update written out once more in numpy
        th = th - 0.01 * (m / (1 - 0.9 ** t)) / (np.sqrt(v / (1 - 0.999 ** t)) + 1e-8)
        np.testing.assert_allclose(head.theta, th, rtol=2e-5, atol=2e-7)
        th = head.theta.astype(np.float64)                               # follow the fp32 trajectory
        m, v = head.vel.astype(np.float64), head.vel2.astype(np.float64)


# ---------------------------------------------------------------------------- loss weighting near objects (Section 5.2)
def test_object_weights_are_a_square_dilation_of_the_non_background_mask():
    ndimage = pytest.importorskip("scipy.ndimage")
    rng = np.random.default_rng(21)
    for H, W, r, bg in [(9, 13, 1, 0), (20, 17, 3, 2), (6, 6, 0, 0), (5, 30, 8, 1)]:
        lab = np.full((H, W), bg, np.uint8)
        for _ in range(3):
            y, x = rng.integers(0, H), rng.integers(0, W)
            lab[y:y + rng.integers(1, 3), x:x + rng.integers(1, 4)] = (bg + 1 + rng.integers(0, 3)) % 5 if bg != 4 else 0
        got = oracle.object_weights(lab, bg, r, 5)
        near = ndimage.maximum_filter((lab != bg).astype(np.uint8), size=2 * r + 1, mode="constant", cval=0).astype(bool)
        np.testing.assert_array_equal(got, np.where(near, 5, 1))
        assert ((got == 5) | (got == 1)).all() and (got[lab != bg] == 5).all()      # "within" objects is always weighted
    # hand case: one object pixel in the middle of a 5x7 background, radius 1 -> a 3x3 block of fives
    lab = np.zeros((5, 7), np.uint8); lab[2, 3] = 4
    exp = np.ones((5, 7), np.uint8); exp[1:4, 2:5] = 5
    np.testing.assert_array_equal(oracle.object_weights(lab, 0, 1, 5), exp)
    # at the frame corner the window is cut, not wrapped
    lab = np.zeros((4, 4), np.uint8); lab[0, 0] = 1
    exp = np.ones((4, 4), np.uint8); exp[:3, :3] = 5
    np.testing.assert_array_equal(oracle.object_weights(lab, 0, 2, 5), exp)


def test_weighted_loss_is_the_plain_loss_plus_four_times_the_near_object_part():
    rng = np.random.default_rng(22)
    C, H, W = 4, 12, 16
    u = rng.standard_normal((C, H, W)) * 2
    lab = rng.integers(0, C, (H, W)).astype(np.uint8)
    wgt = np.where(rng.random((H, W)) < 0.3, 5, 1).astype(np.uint8)
    loss_w, g_w, _ = oracle.softmax_ce(u, lab, weights=wgt)
    loss_1, g_1, _ = oracle.softmax_ce(u, lab)                               # the unweighted function, pinned above
    heavy = wgt == 5
    n = int(heavy.sum())
    loss_h, _, _ = oracle.softmax_ce(u[:, heavy].reshape(C, 1, n), lab[heavy].reshape(1, n))   # mean over the heavy pixels alone
    assert loss_w == pytest.approx(loss_1 + 4.0 * loss_h * n / (H * W), rel=1e-12)
    np.testing.assert_allclose(g_w, g_1 * wgt[None], rtol=1e-12, atol=1e-18)
    # factor 1 everywhere is the plain loss, bit for bit
    l1, g1, _ = oracle.softmax_ce(u, lab, weights=np.ones((H, W), np.uint8))
    assert l1 == pytest.approx(loss_1, rel=1e-14) and g1.tobytes() == g_1.tobytes()


def test_weighted_head_gradient_by_finite_differences_and_background_only_frames():
    rng = np.random.default_rng(23)
    cin, C, h, w = 3, 3, 3, 5
    feat = np.abs(rng.standard_normal((cin, h, w))) + 0.1
    lab = np.zeros((4 * h, 4 * w), np.uint8); lab[3:6, 4:9] = 1; lab[8, 15] = 2
    n = si.head_param_count(cin, 0, C)
    theta = rng.standard_normal(n) * 0.5
    kw = dict(dtype=np.float64, object_weight=5, object_radius=2, background=0)
    loss, grad, _ = oracle.gradients(oracle.Head(cin, 0, C, theta=theta, **kw), feat, lab)
    wgt = oracle.object_weights(lab, 0, 2, 5)
    assert 0 < (wgt == 5).mean() < 1

    def f(th):
        z, _ = oracle.head_forward(oracle.Head(cin, 0, C, dtype=np.float64, theta=th), feat)
        return oracle.softmax_ce(oracle.upsample(z, 4), lab, want_grad=False, weights=wgt)[0]

    fd = np.array([(f(theta + 1e-6 * e) - f(theta - 1e-6 * e)) / 2e-6 for e in np.eye(n)])
    assert np.abs(fd - grad).max() / np.abs(fd).max() < 1e-6
    assert loss == pytest.approx(f(theta), rel=1e-12)
    # a frame with no object: the weighted head computes exactly what the plain head computes
    bgl = np.zeros_like(lab)
    a = oracle.gradients(oracle.Head(cin, 0, C, theta=theta, **kw), feat, bgl)
    b = oracle.gradients(oracle.Head(cin, 0, C, theta=theta, dtype=np.float64), feat, bgl)
    assert a[0] == pytest.approx(b[0], rel=1e-14) and a[1].tobytes() == b[1].tobytes()   # (the loss is an OpenMP reduction)
