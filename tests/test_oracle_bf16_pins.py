"""Pins for the oracle's rounded-operand switch (``Head(quantize_bf16=True)``) and for ``bias_grad``.

The tensor-core path multiplies bf16 operands; the oracle's test-only switch rounds the same tensors so
that a GPU test can tell "wrong" from "rounded".  Every tight bf16 comparison on the GPU stands on that
switch, so it is pinned here, on the CPU, against things other than itself:
  - on inputs that are exact bf16 values already, rounding is the identity and the switched path must
    equal the plain path bit for bit (forward, weight gradients, the gradient passed back);
  - ``bias_grad`` is the bias half of ``conv_wgrad``;
  - on generic inputs each gradient stays within the bound that one 2^-9 relative error per rounded
    operand allows, measured from the plain path;
  - a restatement with library routines (torch's bf16 cast, conv2d, conv2d_weight, autograd) that rounds at
    exactly the places the tensor-core path rounds must agree to 1e-9 in double: removing or adding one
    rounding anywhere moves a gradient by about 1e-3 and fails it.
CPU only.
"""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle

EPS = 2.0 ** -9          # largest relative error of rounding to bf16 (8 significant bits, ties to even)


def _head(c_in, ch, C, theta, quant, dtype=np.float32, **kw):
    return oracle.Head(c_in, ch, C, theta=np.asarray(theta, dtype=dtype), dtype=dtype, quantize_bf16=quant, **kw)


def _small_exact_case(ch, seed):
    """Features, parameters, hidden activations and a logit gradient whose values and whose products' sums all
    fit in eight significant bits: rounding to bf16 cannot change any of them."""
    rng = np.random.default_rng(seed)
    c_in, C, h, w = 3, 3, 4, 5
    x = rng.integers(0, 3, size=(c_in, h, w)).astype(np.float32)                       # 0, 1, 2
    n = sum(int(np.prod(ws)) + int(np.prod(bs)) for ws, bs in oracle.param_shapes(c_in, ch, C))
    theta = (rng.integers(-2, 3, size=n) * 0.5).astype(np.float32)                      # -1 .. 1 in halves
    dz = (rng.integers(-7, 8, size=(C, h, w)) / 64.0).astype(np.float32)                # three bits
    return c_in, C, h, w, x, theta, dz


@pytest.mark.parametrize("ch", [0, 4])
def test_rounded_path_is_the_plain_path_on_exact_bf16_values(ch):
    c_in, C, h, w, x, theta, dz = _small_exact_case(ch, 5 + ch)
    plain, quant = _head(c_in, ch, C, theta, False), _head(c_in, ch, C, theta, True)
    zp, hp = oracle.head_forward(plain, x)
    zq, hq = oracle.head_forward(quant, x)
    assert zp.tobytes() == zq.tobytes()
    if ch:
        assert hp.tobytes() == hq.tobytes() and (oracle.round_bf16(hp) == hp).all() and (hp > 0).any()
        dH = oracle.conv1x1_dgrad(plain.layers()[1][0].reshape(C, ch), dz)
        assert (oracle.round_bf16(dH) == dH).all()                                      # the case really is exact
    gp = oracle.head_backward(plain, x, hp, dz)
    gq = oracle.head_backward(quant, x, hq, dz)
    assert gp.tobytes() == gq.tobytes() and np.abs(gp).max() > 0


def test_bias_grad_is_the_bias_half_of_the_weight_gradient():
    rng = np.random.default_rng(11)
    for dtype in (np.float32, np.float64):
        x = rng.standard_normal((5, 6, 7)).astype(dtype)
        d = rng.standard_normal((4, 6, 7)).astype(dtype)
        for ks in (1, 3):
            assert oracle.bias_grad(d).tobytes() == oracle.conv_wgrad(x, d, ks)[1].tobytes()
        np.testing.assert_allclose(oracle.bias_grad(d), d.reshape(4, -1).astype(np.float64).sum(1), rtol=1e-6)
    # the channel axis is the first one: a transposed reading fails on a non-square case
    d = np.zeros((2, 3, 5), np.float32); d[1] = 1.0
    assert oracle.bias_grad(d).tolist() == [0.0, 15.0]


def _abs_wgrad(x, d, ks):
    return oracle.conv_wgrad(np.abs(x), np.abs(d), ks)[0].astype(np.float64)


@pytest.mark.parametrize("ch", [0, 6])
def test_rounded_gradients_stay_within_the_rounding_bound_of_the_plain_ones(ch):
    rng = np.random.default_rng(21 + ch)
    c_in, C, h, w = 5, 4, 6, 7
    x = np.maximum(rng.standard_normal((c_in, h, w)), 0).astype(np.float64)
    n = sum(int(np.prod(ws)) + int(np.prod(bs)) for ws, bs in oracle.param_shapes(c_in, ch, C))
    theta = (0.3 * rng.standard_normal(n))
    dz = (1e-3 * rng.standard_normal((C, h, w)))
    plain = _head(c_in, ch, C, theta, False, np.float64)
    quant = _head(c_in, ch, C, theta, True, np.float64)
    slack = 1.001
    if ch == 0:
        gp = oracle.head_backward(plain, x, None, dz)
        gq = oracle.head_backward(quant, oracle.round_bf16(x), None, dz)
        nW = C * c_in
        # dW = sum x dz with both operands rounded once: |error| <= (2 eps + eps^2) sum |x| |dz|
        bound = (2 * EPS + EPS * EPS) * _abs_wgrad(x, dz, 1).ravel()
        assert (np.abs(gq[:nW] - gp[:nW]) <= slack * bound + 1e-300).all()
        assert np.abs(gq[:nW] - gp[:nW]).max() > 0.02 * bound.max()                 # and rounding did happen
        assert gq[nW:].tobytes() == gp[nW:].tobytes()                                # bias gradient: unrounded sums
        return
    # two-layer head, the same hidden activation on both sides so that only the backward's roundings differ
    _, Hd = oracle.head_forward(quant, x)
    xq = oracle.round_bf16(x)
    gp = oracle.head_backward(plain, xq, Hd, dz)
    gq = oracle.head_backward(quant, xq, Hd, dz)
    n1 = ch * c_in * 9
    W2 = plain.layers()[1][0].reshape(C, ch)
    dW1p, db1p, dW2p, db2p = gp[:n1], gp[n1:n1 + ch], gp[n1 + ch:n1 + ch + C * ch], gp[n1 + ch + C * ch:]
    dW1q, db1q, dW2q, db2q = gq[:n1], gq[n1:n1 + ch], gq[n1 + ch:n1 + ch + C * ch], gq[n1 + ch + C * ch:]
    assert db2q.tobytes() == db2p.tobytes()
    # dW2 = sum Hd dz, dz rounded: eps sum |Hd| |dz|
    b2 = EPS * _abs_wgrad(Hd, dz, 1).ravel()
    assert (np.abs(dW2q - dW2p) <= slack * b2 + 1e-300).all() and np.abs(dW2q - dW2p).max() > 0.02 * b2.max()
    # dH = sum_c W2 dz, both rounded, then the ReLU mask
    A = np.einsum("ck,cyx->kyx", np.abs(W2), np.abs(dz)) * (Hd > 0)
    dHp = oracle.conv1x1_dgrad(W2, dz); oracle.relu_mask_(dHp, Hd)
    e_dH = (2 * EPS + EPS * EPS) * A
    # db1 = sum of the unrounded dH of that side
    assert (np.abs(db1q - db1p) <= slack * e_dH.reshape(ch, -1).sum(1) + 1e-300).all()
    # dW1 = sum x round(dH): |round(dHq) - dHp| <= e_dH + eps (|dHp| + e_dH)
    e_op = e_dH + EPS * (np.abs(dHp) + e_dH)
    b1 = oracle.conv_wgrad(np.abs(xq), e_op, 3)[0].ravel()
    assert (np.abs(dW1q - dW1p) <= slack * b1 + 1e-300).all() and np.abs(dW1q - dW1p).max() > 0.02 * b1.max()


def _bf(t):
    """Round a double tensor to bf16 the way the oracle's switch does (through fp32), keeping doubles."""
    return t.float().bfloat16().double()


def _torch_rounded_gradients(c_in, ch, C, theta, x, labels):
    """The step's gradient with bf16 operands, restated with torch in double: X, the weight copies and the hidden
    activation are rounded in the forward; in the backward dz is rounded where it meets the activations and the
    weights, the hidden gradient where it meets X; bias gradients are sums of the unrounded values."""
    t = torch.from_numpy(np.asarray(theta, np.float64))
    xq = _bf(torch.from_numpy(x))[None]
    lab = torch.from_numpy(labels.astype(np.int64))[None]
    if ch == 0:
        W, b = t[:C * c_in].reshape(C, c_in, 1, 1), t[C * c_in:]
        z = F.conv2d(xq, _bf(W), b).detach().requires_grad_(True)
        Hd = None
    else:
        n1 = ch * c_in * 9
        W1, b1 = t[:n1].reshape(ch, c_in, 3, 3), t[n1:n1 + ch]
        W2, b2 = t[n1 + ch:n1 + ch + C * ch].reshape(C, ch, 1, 1), t[n1 + ch + C * ch:]
        Hd = _bf(F.relu(F.conv2d(xq, _bf(W1), b1, padding=1)))
        z = F.conv2d(Hd, _bf(W2), b2).detach().requires_grad_(True)
    u = F.interpolate(z, scale_factor=4, mode="bilinear", align_corners=False)
    loss = F.cross_entropy(u, lab)
    loss.backward()
    dz = z.grad
    dzq = _bf(dz)
    if ch == 0:
        dW = torch.einsum("ncyx,nkyx->ck", dzq, xq)
        return float(loss.detach()), torch.cat([dW.reshape(-1), dz.sum((0, 2, 3))]).numpy()
    dW2 = torch.einsum("ncyx,nkyx->ck", dzq, Hd)
    dH = torch.einsum("ck,ncyx->nkyx", _bf(W2).reshape(C, ch), dzq) * (Hd > 0)
    dW1 = torch.nn.grad.conv2d_weight(xq, (ch, c_in, 3, 3), _bf(dH), padding=1)
    return float(loss.detach()), torch.cat([dW1.reshape(-1), dH.sum((0, 2, 3)), dW2.reshape(-1), dz.sum((0, 2, 3))]).numpy()


@pytest.mark.parametrize("ch", [0, 6])
def test_rounding_places_against_a_library_restatement(ch):
    rng = np.random.default_rng(31 + ch)
    c_in, C, h, w = 5, 4, 6, 7
    x = np.maximum(rng.standard_normal((c_in, h, w)), 0)
    n = sum(int(np.prod(ws)) + int(np.prod(bs)) for ws, bs in oracle.param_shapes(c_in, ch, C))
    theta = 0.3 * rng.standard_normal(n)
    labels = rng.integers(0, C, size=(4 * h, 4 * w)).astype(np.uint8)
    head = _head(c_in, ch, C, theta, True, np.float64)
    loss, grad, _ = oracle.gradients(head, x, labels)
    ref_loss, ref = _torch_rounded_gradients(c_in, ch, C, theta, x, labels)
    assert loss == pytest.approx(ref_loss, rel=1e-12)
    np.testing.assert_allclose(grad, ref, rtol=0, atol=1e-9 * np.abs(ref).max())
    # what the tolerance is worth: the plain path (no rounding at all) is about 1e-3 away, and so is a
    # restatement with one rounding left out (here: dz is not rounded before it meets the activations)
    plain = _head(c_in, ch, C, theta, False, np.float64)
    g_plain = oracle.gradients(plain, x, labels)[1]
    assert np.abs(g_plain - ref).max() > 1e-5 * np.abs(ref).max()
    global _bf
    keep = _bf
    calls = {"n": 0}

    def skip_one(t):                       # the rounding of dz (first call of the backward) is left out
        calls["n"] += 1
        return t if calls["n"] == (3 if ch == 0 else 5) else keep(t)
    try:
        _bf = skip_one
        _, mutated = _torch_rounded_gradients(c_in, ch, C, theta, x, labels)
    finally:
        _bf = keep
    assert np.abs(mutated - ref).max() > 1e-6 * np.abs(ref).max()
    assert not np.allclose(grad, mutated, rtol=0, atol=1e-9 * np.abs(ref).max())


def test_fp32_storage_follows_the_double_build():
    """The fp32-storage oracle (the one the GPU tests call) and the double build take the same roundings:
    they differ by fp32 storage noise only, far below one bf16 rounding."""
    rng = np.random.default_rng(41)
    c_in, ch, C, h, w = 5, 6, 4, 6, 7
    x = np.maximum(rng.standard_normal((c_in, h, w)), 0).astype(np.float32)
    n = sum(int(np.prod(ws)) + int(np.prod(bs)) for ws, bs in oracle.param_shapes(c_in, ch, C))
    theta = (0.3 * rng.standard_normal(n)).astype(np.float32)
    labels = rng.integers(0, C, size=(4 * h, 4 * w)).astype(np.uint8)
    g32 = oracle.gradients(_head(c_in, ch, C, theta, True, np.float32), x, labels)[1]
    g64 = oracle.gradients(_head(c_in, ch, C, theta, True, np.float64), x, labels)[1]
    rel = np.linalg.norm(g32 - g64) / np.linalg.norm(g64)
    assert rel < 2e-4        # a handful of hidden values sit close enough to a rounding boundary to flip in fp32
