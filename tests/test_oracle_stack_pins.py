"""Pins for the oracle of the deeper trainable subset (a stack of student blocks with skip inputs and a freeze
boundary inside it; Section 5.2's SB5 / SB6 and Section 4.2's partial distillation): the gradient passed back through a
3x3 layer against its defining identity and torch, the whole gradient against finite differences and torch autograd
with the frozen layers' parameters excluded, the special cases that reduce to the two heads pinned elsewhere, and the
rounded-operand switch against a restatement with library routines.  CPU only."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle


def n_params(c_in, blocks, C):
    return oracle.StackHead(c_in, blocks, C).theta.size


def tiny_problem(seed, c_in=3, blocks=((4, 2), (5, 1)), C=3, h=3, w=5, dtype=np.float64):
    rng = np.random.default_rng(seed)
    feat = rng.standard_normal((c_in, h, w)).astype(dtype)
    skips = [rng.standard_normal((cs, h, w)).astype(dtype) if cs else None for _, cs in blocks]
    theta = (0.4 * rng.standard_normal(n_params(c_in, list(blocks), C))).astype(dtype)
    labels = rng.integers(0, C, size=(4 * h, 4 * w)).astype(np.uint8)
    return feat, skips, theta, labels


# ---------------------------------------------------------------------------- the gradient through a 3x3 layer
def test_conv_dgrad_is_the_transpose_of_the_convolution():
    rng = np.random.default_rng(1)
    for ks in (1, 3):
        x = rng.standard_normal((5, 6, 7))
        W = rng.standard_normal((4, 5, ks, ks))
        g = rng.standard_normal((4, 6, 7))
        lhs = float((oracle.conv_fwd(x, W, np.zeros(4)) * g).sum())
        rhs = float((x * oracle.conv_dgrad(g, W)).sum())
        assert lhs == pytest.approx(rhs, rel=1e-12)
        ref = F.conv_transpose2d(torch.from_numpy(g)[None], torch.from_numpy(W), padding=ks // 2)[0].numpy()
        np.testing.assert_allclose(oracle.conv_dgrad(g, W), ref, rtol=1e-12, atol=1e-12)
        np.testing.assert_array_equal(oracle.conv_dgrad(g, W, 2), oracle.conv_dgrad(g, W)[:2])     # the first channels only
    # a single tap moves the gradient the opposite way to the forward shift
    W = np.zeros((1, 1, 3, 3)); W[0, 0, 0, 2] = 1.0              # forward: out(y, x) = in(y - 1, x + 1)
    g = np.zeros((1, 4, 4)); g[0, 2, 1] = 1.0
    d = oracle.conv_dgrad(g, W)
    assert d[0, 1, 2] == 1.0 and d.sum() == 1.0


# ---------------------------------------------------------------------------- special cases pinned elsewhere
def test_one_block_without_skip_is_the_two_layer_head():
    rng = np.random.default_rng(2)
    c_in, ch, C, h, w = 4, 6, 3, 4, 5
    feat = rng.standard_normal((c_in, h, w)).astype(np.float32)
    labels = rng.integers(0, C, size=(4 * h, 4 * w)).astype(np.uint8)
    theta = (0.3 * rng.standard_normal(n_params(c_in, [(ch, 0)], C))).astype(np.float32)
    for quant in (False, True):
        a = oracle.Head(c_in, ch, C, lr=0.05, momentum=0.9, theta=theta, quantize_bf16=quant)
        b = oracle.StackHead(c_in, [(ch, 0)], C, lr=0.05, momentum=0.9, theta=theta, quantize_bf16=quant)
        for _ in range(3):
            la, _ = oracle.distill_step(a, feat, labels)
            lb, _ = oracle.stack_distill_step(b, feat, [None], labels)
            assert la == pytest.approx(lb, rel=1e-13)     # the loss is an OpenMP sum: its last bits depend on the thread split
        assert a.theta.tobytes() == b.theta.tobytes()
        assert oracle.pack(a) == oracle.stack_pack(b)


def test_classifier_alone_is_the_1x1_head_on_the_last_block_output():
    feat, skips, theta, labels = tiny_problem(3, dtype=np.float32)
    blocks = [(4, 2), (5, 1)]
    st = oracle.StackHead(3, blocks, 3, first_trained=2, lr=0.1, theta=theta)
    _, _, outs = oracle.stack_forward(st, feat, skips)
    n_cls = 3 * 5 + 3
    one = oracle.Head(5, 0, 3, lr=0.1, theta=theta[-n_cls:])
    l1, g1, _ = oracle.gradients(one, outs[-1], labels)
    l2, g2, _ = oracle.stack_gradients(st, feat, skips, labels)
    assert l1 == pytest.approx(l2, rel=1e-13) and g1.tobytes() == g2[-n_cls:].tobytes() and not g2[:-n_cls].any()
    assert len(oracle.stack_pack(st)) == n_cls * 4                   # UpdatedPart = the trained layers only


# ---------------------------------------------------------------------------- the whole gradient
@pytest.mark.parametrize("first_trained", [0, 1])
def test_stack_gradient_by_finite_differences(first_trained):
    feat, skips, theta, labels = tiny_problem(4)
    blocks = [(4, 2), (5, 1)]

    def loss_at(t):
        hd = oracle.StackHead(3, blocks, 3, first_trained=first_trained, theta=t, dtype=np.float64)
        z, _, outs = oracle.stack_forward(hd, feat, skips)
        return oracle.softmax_ce(oracle.upsample(z, 4), labels, want_grad=False)[0], outs

    hd = oracle.StackHead(3, blocks, 3, first_trained=first_trained, theta=theta, dtype=np.float64)
    _, grad, _ = oracle.stack_gradients(hd, feat, skips, labels)
    sl = hd.trained_slice()
    assert not grad[:sl.start].any()                                 # no gradient for the frozen layers
    # keep away from ReLU kinks: every pre-activation this far from zero keeps its sign under the probes below
    _, outs = loss_at(theta)
    rng = np.random.default_rng(0)
    eps = 1e-6
    for i in rng.choice(np.arange(sl.start, theta.size), size=60, replace=False):
        tp, tm = theta.copy(), theta.copy()
        tp[i] += eps; tm[i] -= eps
        (lp, op), (lm, om) = loss_at(tp), loss_at(tm)
        if any(((a > 0) != (b > 0)).any() for a, b in zip(op, om)):
            continue                                                 # a unit crossed its kink: not differentiable there
        fd = (lp - lm) / (2 * eps)
        assert fd == pytest.approx(grad[i], rel=2e-6, abs=1e-9), i


def torch_stack(c_in, blocks, C, theta, feat, skips, labels, first_trained, steps, lr, mu):
    """The same stack with torch modules in double; frozen layers have requires_grad False."""
    t = torch.from_numpy(np.asarray(theta, np.float64))
    params, off, prev = [], 0, c_in
    shapes = [(co, prev_ + cs) for (co, cs), prev_ in zip(blocks, [c_in] + [b[0] for b in blocks[:-1]])]
    for co, ci in shapes:
        W = t[off:off + co * ci * 9].reshape(co, ci, 3, 3).clone(); off += co * ci * 9
        b = t[off:off + co].clone(); off += co
        params += [W, b]
    Wc = t[off:off + C * blocks[-1][0]].reshape(C, blocks[-1][0], 1, 1).clone(); off += C * blocks[-1][0]
    bc = t[off:off + C].clone()
    params += [Wc, bc]
    for i, p in enumerate(params):
        p.requires_grad_(i // 2 >= first_trained)
    trained = [p for p in params if p.requires_grad]
    opt = torch.optim.SGD(trained, lr=lr, momentum=mu)
    x0 = torch.from_numpy(feat)[None]
    sk = [torch.from_numpy(s)[None] if s is not None else None for s in skips]
    lab = torch.from_numpy(labels.astype(np.int64))[None]
    losses = []
    for _ in range(steps):
        x = x0
        for b in range(len(blocks)):
            xin = x if sk[b] is None else torch.cat([x, sk[b]], dim=1)
            x = F.relu(F.conv2d(xin, params[2 * b], params[2 * b + 1], padding=1))
        z = F.conv2d(x, params[-2], params[-1])
        loss = F.cross_entropy(F.interpolate(z, scale_factor=4, mode="bilinear", align_corners=False), lab)
        opt.zero_grad(); loss.backward(); opt.step()
        losses.append(float(loss.detach()))
    return losses, torch.cat([p.detach().reshape(-1) for p in params]).numpy()


@pytest.mark.parametrize("first_trained", [0, 1, 2])
def test_stack_steps_against_torch_autograd(first_trained):
    feat, skips, theta, labels = tiny_problem(5, h=4, w=6)
    blocks = [(4, 2), (5, 1)]
    hd = oracle.StackHead(3, blocks, 3, first_trained=first_trained, lr=0.2, momentum=0.9, theta=theta, dtype=np.float64)
    losses = [oracle.stack_distill_step(hd, feat, skips, labels)[0] for _ in range(3)]
    ref_losses, ref_theta = torch_stack(3, blocks, 3, theta, feat, skips, labels, first_trained, 3, 0.2, 0.9)
    np.testing.assert_allclose(losses, ref_losses, rtol=1e-10)
    np.testing.assert_allclose(hd.theta, ref_theta, rtol=1e-9, atol=1e-11)
    sl = hd.trained_slice()
    assert hd.theta[:sl.start].tobytes() == theta[:sl.start].tobytes()          # frozen layers are bit-identical
    assert np.abs(hd.theta[sl] - theta[sl]).max() > 1e-4                        # trained ones moved


def test_gradients_of_later_layers_do_not_depend_on_the_freeze_boundary():
    feat, skips, theta, labels = tiny_problem(6, dtype=np.float32)
    blocks = [(4, 2), (5, 1)]
    g = [oracle.stack_gradients(oracle.StackHead(3, blocks, 3, first_trained=ft, theta=theta), feat, skips, labels)[1]
         for ft in (0, 1, 2)]
    s1 = oracle.StackHead(3, blocks, 3, first_trained=1, theta=theta).trained_slice()
    s2 = oracle.StackHead(3, blocks, 3, first_trained=2, theta=theta).trained_slice()
    assert g[0][s1].tobytes() == g[1][s1].tobytes() and g[1][s2].tobytes() == g[2][s2].tobytes()
    assert g[0][:s1.start].any() and not g[1][:s1.start].any()


def test_skip_inputs_enter_the_block_after_the_previous_output():
    """Channel order of a block's input: previous output first, skip input after it.  Zeroing the weights that read the
    skip channels must give the output of the block without its skip input."""
    feat, skips, theta, labels = tiny_problem(7, dtype=np.float32)
    hd = oracle.StackHead(3, [(4, 2)], 3, theta=theta[:n_params(3, [(4, 2)], 3)])
    W, _ = hd.layers()[0]
    W[:, 3:] = 0.0                                                   # channels 3, 4 are the skip input
    z_a = oracle.stack_forward(hd, feat, [skips[0]])[0]
    z_b = oracle.stack_forward(hd, feat, [np.zeros_like(skips[0])])[0]
    assert z_a.tobytes() == z_b.tobytes()
    W[:, :3] = 0.0; W[:, 3:] = 1.0
    assert not np.array_equal(oracle.stack_forward(hd, feat, [skips[0]])[0], z_b)


# ---------------------------------------------------------------------------- the rounded-operand switch
def _bf(t):
    return t.float().bfloat16().double()


def test_rounding_places_of_the_stack_against_a_library_restatement():
    feat, skips, theta, labels = tiny_problem(8, h=4, w=6)
    blocks, C, c_in = [(4, 2), (5, 1)], 3, 3
    hd = oracle.StackHead(c_in, blocks, C, first_trained=0, theta=theta, dtype=np.float64, quantize_bf16=True)
    loss, grad, _ = oracle.stack_gradients(hd, feat, skips, labels)
    t = torch.from_numpy(theta)
    (W1, b1), (W2, b2), (Wc, bc) = [(torch.from_numpy(W.copy()), torch.from_numpy(b.copy())) for W, b in hd.layers()]
    x = _bf(torch.from_numpy(feat))[None]
    s1, s2 = _bf(torch.from_numpy(skips[0]))[None], _bf(torch.from_numpy(skips[1]))[None]
    in1 = torch.cat([x, s1], 1)
    h1 = _bf(F.relu(F.conv2d(in1, _bf(W1), b1, padding=1)))
    in2 = torch.cat([h1, s2], 1)
    h2 = _bf(F.relu(F.conv2d(in2, _bf(W2), b2, padding=1)))
    z = F.conv2d(h2, _bf(Wc), bc).detach().requires_grad_(True)
    l = F.cross_entropy(F.interpolate(z, scale_factor=4, mode="bilinear", align_corners=False),
                        torch.from_numpy(labels.astype(np.int64))[None])
    l.backward()
    dz = z.grad
    dzq = _bf(dz)
    dWc = torch.einsum("ncyx,nkyx->ck", dzq, h2)
    dh2 = torch.einsum("ck,ncyx->nkyx", _bf(Wc).reshape(C, 5), dzq) * (h2 > 0)
    dW2 = torch.nn.grad.conv2d_weight(in2, W2.shape, _bf(dh2), padding=1)
    dh1 = F.conv_transpose2d(_bf(dh2), _bf(W2), padding=1)[:, :4] * (h1 > 0)
    dW1 = torch.nn.grad.conv2d_weight(in1, W1.shape, _bf(dh1), padding=1)
    ref = torch.cat([dW1.reshape(-1), dh1.sum((0, 2, 3)), dW2.reshape(-1), dh2.sum((0, 2, 3)), dWc.reshape(-1),
                     dz.sum((0, 2, 3))]).numpy()
    assert loss == pytest.approx(float(l.detach()), rel=1e-12)
    np.testing.assert_allclose(grad, ref, rtol=0, atol=1e-9 * np.abs(ref).max())
    plain = oracle.stack_gradients(oracle.StackHead(c_in, blocks, C, theta=theta, dtype=np.float64), feat, skips, labels)[1]
    assert np.abs(plain - ref).max() > 1e-5 * np.abs(ref).max()     # what the tolerance is worth
