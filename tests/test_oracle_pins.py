"""Pins for the fp64 CPU checker: every function in oracle/ is compared with
something that is not itself - closed forms, hand-worked values stored under
tests/golden/, adjoint identities, finite differences, and torch's own fp64
CPU routines (conv2d, max_pool2d, linear, cross_entropy, autograd)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from conftest import read_golden_blocks

rng = np.random.default_rng(1234)


def nhwc_to_torch(x):
    return torch.from_numpy(np.ascontiguousarray(x)).permute(0, 3, 1, 2).contiguous()


def torch_to_nhwc(t):
    return t.permute(0, 2, 3, 1).contiguous().numpy()


# ---------------------------------------------------------------- convolution

def test_delta_kernel_is_identity():
    N, H, W, C = 2, 5, 7, 4
    x = rng.standard_normal((N, H, W, C))
    Wt = np.zeros((C, 3, 3, C))
    for k in range(C):
        Wt[k, 1, 1, k] = 1.0
    z = oracle.conv3x3_fwd(x, Wt, np.zeros(C))
    assert np.array_equal(z, x)
    assert np.array_equal(oracle.relu_fwd(z), np.maximum(x, 0.0))
    # a delta one step off-centre shifts the image and pulls in a zero border
    Ws = np.zeros((C, 3, 3, C))
    for k in range(C):
        Ws[k, 0, 2, k] = 1.0  # reads x[h-1, w+1]
    zs = oracle.conv3x3_fwd(x, Ws, None)
    expect = np.zeros_like(x)
    expect[:, 1:, :-1, :] = x[:, :-1, 1:, :]
    assert np.array_equal(zs, expect)


@pytest.mark.parametrize("C", [1, 3])
def test_constant_input_closed_form(C):
    a, bias = 2.0, 0.5
    x = np.full((1, 4, 4, C), a)
    Wt = np.ones((2, 3, 3, C))
    z = oracle.conv3x3_fwd(x, Wt, np.array([0.0, bias]))
    counts = np.array([[4, 6, 6, 4], [6, 9, 9, 6], [6, 9, 9, 6], [4, 6, 6, 4]], dtype=float)
    assert np.array_equal(z[0, :, :, 0], counts * a * C)
    assert np.array_equal(z[0, :, :, 1], counts * a * C + bias)
    if C == 1:
        assert z[0, 0, :, 0].tolist() == [8.0, 12.0, 12.0, 8.0]
        assert z[0, 1, :, 0].tolist() == [12.0, 18.0, 18.0, 12.0]


def test_hand_worked_3x3_tells_correlation_from_flip():
    g = read_golden_blocks("hand_conv3x3.txt")
    m = np.arange(1.0, 10.0).reshape(3, 3)
    x = m.reshape(1, 3, 3, 1)
    Wt = m.reshape(1, 3, 3, 1)
    z = oracle.conv3x3_fwd(x, Wt, None)[0, :, :, 0]
    assert np.array_equal(z, g["correlation"])
    assert not np.array_equal(z, g["flipped"])
    ones = np.ones((1, 3, 3, 1))
    assert np.array_equal(oracle.conv3x3_dgrad(ones, Wt)[0, :, :, 0], g["grad_ones"])
    dW, db = oracle.conv3x3_wgrad(x, ones)
    assert np.array_equal(dW[0, :, :, 0], g["grad_ones"])
    assert db[0] == 9.0
    # <conv(x), 1> three ways
    assert z.sum() == 1365.0 == (x * oracle.conv3x3_dgrad(ones, Wt)).sum() == (Wt * dW).sum()


@pytest.mark.parametrize("shape", [(2, 6, 5, 3, 4), (1, 2, 2, 5, 2), (3, 4, 8, 1, 1)])
def test_adjoint_identities(shape):
    N, H, W, Cin, Cout = shape
    x = rng.standard_normal((N, H, W, Cin))
    Wt = rng.standard_normal((Cout, 3, 3, Cin))
    b = rng.standard_normal(Cout)
    dz = rng.standard_normal((N, H, W, Cout))
    z = oracle.conv3x3_fwd(x, Wt, b)
    lhs = ((z - b) * dz).sum()
    dx = oracle.conv3x3_dgrad(dz, Wt)
    dW, db = oracle.conv3x3_wgrad(x, dz)
    assert abs(lhs - (x * dx).sum()) <= 1e-12 * abs(lhs) + 1e-12
    assert abs(lhs - (Wt * dW).sum()) <= 1e-12 * abs(lhs) + 1e-12
    np.testing.assert_allclose(db, dz.sum(axis=(0, 1, 2)), rtol=1e-13, atol=1e-13)


@pytest.mark.parametrize("shape", [(2, 6, 5, 3, 4), (1, 9, 4, 8, 6)])
def test_conv_against_torch_fp64(shape):
    N, H, W, Cin, Cout = shape
    x = rng.standard_normal((N, H, W, Cin))
    Wt = rng.standard_normal((Cout, 3, 3, Cin))
    b = rng.standard_normal(Cout)
    dz = rng.standard_normal((N, H, W, Cout))
    tx = nhwc_to_torch(x).requires_grad_(True)
    tw = torch.from_numpy(Wt).permute(0, 3, 1, 2).contiguous().requires_grad_(True)  # [k,c,r,s]
    tb = torch.from_numpy(b).requires_grad_(True)
    tz = F.conv2d(tx, tw, tb, stride=1, padding=1)
    tz.backward(nhwc_to_torch(dz))
    np.testing.assert_allclose(oracle.conv3x3_fwd(x, Wt, b), torch_to_nhwc(tz.detach()), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(oracle.conv3x3_dgrad(dz, Wt), torch_to_nhwc(tx.grad), rtol=1e-12, atol=1e-12)
    dW, db = oracle.conv3x3_wgrad(x, dz)
    np.testing.assert_allclose(dW, tw.grad.permute(0, 2, 3, 1).numpy(), rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(db, tb.grad.numpy(), rtol=1e-12, atol=1e-12)


def test_wgrad_accumulates():
    x = rng.standard_normal((2, 4, 4, 2))
    dz = rng.standard_normal((2, 4, 4, 3))
    dW, db = oracle.conv3x3_wgrad(x, dz)
    dW2, db2 = oracle.conv3x3_wgrad(x[:1], dz[:1])
    oracle.conv3x3_wgrad(x[1:], dz[1:], dW2, db2)
    np.testing.assert_allclose(dW2, dW, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(db2, db, rtol=1e-13, atol=1e-13)


# ----------------------------------------------------------- ReLU and pooling

def test_relu():
    z = np.array([-2.0, -0.0, 0.0, 1e-300, 3.0])
    assert oracle.relu_fwd(z).tolist() == [0.0, 0.0, 0.0, 1e-300, 3.0]
    dy = np.array([5.0, 6.0, 7.0, 8.0, 9.0])
    assert oracle.relu_bwd(z, dy).tolist() == [0.0, 0.0, 0.0, 8.0, 9.0]  # derivative at 0 is 0


def test_pool_on_a_ramp():
    H, Wd = 6, 8
    ramp = (np.arange(H)[:, None] * Wd + np.arange(Wd)[None, :]).astype(float)
    y = np.stack([ramp, -ramp], axis=-1)[None]  # channel 1 decreasing: max is the first corner
    p = oracle.maxpool2x2_fwd(y)
    i, j = np.meshgrid(np.arange(H // 2), np.arange(Wd // 2), indexing="ij")
    assert np.array_equal(p[0, :, :, 0], (2 * i + 1) * Wd + 2 * j + 1)
    assert np.array_equal(p[0, :, :, 1], -((2 * i) * Wd + 2 * j))
    dp = rng.standard_normal(p.shape)
    dy = oracle.maxpool2x2_bwd(y, dp)
    assert np.array_equal(dy[0, 1::2, 1::2, 0], dp[0, :, :, 0])
    assert np.array_equal(dy[0, 0::2, 0::2, 1], dp[0, :, :, 1])
    assert np.count_nonzero(dy) == dp.size
    assert abs(dy.sum() - dp.sum()) < 1e-12


def test_pool_ties_go_to_first_in_scan_order():
    y = np.zeros((1, 2, 2, 3))
    y[0, :, :, 1] = 4.0                      # four-way tie
    y[0, 0, 1, 2] = y[0, 1, 0, 2] = 7.0      # tie between (0,1) and (1,0)
    dy = oracle.maxpool2x2_bwd(y, np.array([1.0, 2.0, 3.0]).reshape(1, 1, 1, 3))
    assert dy[0, 0, 0, 0] == 1.0 and dy[0, 0, 0, 1] == 2.0 and dy[0, 0, 1, 2] == 3.0
    assert np.count_nonzero(dy) == 3


def test_pool_against_torch():
    y = rng.standard_normal((2, 6, 4, 5))
    dp = rng.standard_normal((2, 3, 2, 5))
    ty = nhwc_to_torch(y).requires_grad_(True)
    tp = F.max_pool2d(ty, 2, 2)
    tp.backward(nhwc_to_torch(dp))
    assert np.array_equal(oracle.maxpool2x2_fwd(y), torch_to_nhwc(tp.detach()))
    assert np.array_equal(oracle.maxpool2x2_bwd(y, dp), torch_to_nhwc(ty.grad))


# ------------------------------------------------------ dense, softmax, loss

def test_dense_10x10_example():
    # section 7.1: dense(W, x, b) = (W * x) .+ b on 10x10 operands
    W = np.arange(100.0).reshape(10, 10)
    x = np.ones((1, 10))
    b = np.full(10, 0.25)
    y = oracle.dense_fwd(x, W, b)
    # row o of W sums to 10*(10 o) + 45
    assert np.array_equal(y[0], 100.0 * np.arange(10) + 45.0 + 0.25)
    x2 = np.eye(10)  # ten columns at once: W * I + b
    assert np.array_equal(oracle.dense_fwd(x2, W, b), W.T + 0.25)
    Wr, xr = rng.standard_normal((10, 10)), rng.standard_normal((10, 10))
    np.testing.assert_allclose(oracle.dense_fwd(xr, Wr, b), xr @ Wr.T + b, rtol=1e-13, atol=1e-13)


def test_dense_backward_adjoint_and_torch():
    N, In, Out = 3, 7, 5
    x, W, dy = rng.standard_normal((N, In)), rng.standard_normal((Out, In)), rng.standard_normal((N, Out))
    dx, dW, db = oracle.dense_bwd(x, W, dy)
    np.testing.assert_allclose(dx, dy @ W, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(dW, dy.T @ x, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(db, dy.sum(0), rtol=1e-13, atol=1e-13)
    tx, tw = torch.from_numpy(x).requires_grad_(True), torch.from_numpy(W).requires_grad_(True)
    F.linear(tx, tw).backward(torch.from_numpy(dy))
    np.testing.assert_allclose(dx, tx.grad.numpy(), rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(dW, tw.grad.numpy(), rtol=1e-13, atol=1e-13)


def test_softmax_and_cross_entropy_closed_forms():
    l = np.full((3, 1000), 1.7)
    p = oracle.softmax(l)
    np.testing.assert_allclose(p, 1e-3, rtol=1e-14)
    labels = np.array([0, 500, 999], dtype=np.int32)
    assert abs(oracle.cross_entropy(l, labels) - 6.907755278982137) < 1e-13  # ln 1000
    # two classes: softmax is the logistic function
    l2 = np.array([[0.0, np.log(3.0)]])
    np.testing.assert_allclose(oracle.softmax(l2), [[0.25, 0.75]], rtol=1e-15)
    assert abs(oracle.cross_entropy(l2, np.array([0], dtype=np.int32)) - np.log(4.0)) < 1e-15
    # large logits must not overflow
    big = np.array([[1000.0, 1000.0 + np.log(3.0)]])
    np.testing.assert_allclose(oracle.softmax(big), [[0.25, 0.75]], rtol=1e-12)
    lr = rng.standard_normal((4, 9)) * 3
    pr = oracle.softmax(lr)
    np.testing.assert_allclose(pr.sum(1), 1.0, rtol=1e-14)
    lab = np.array([1, 8, 0, 3], dtype=np.int32)
    dl = oracle.softmax_ce_bwd(pr, lab)
    np.testing.assert_allclose(dl.sum(1), 0.0, atol=1e-15)
    tl = torch.from_numpy(lr).requires_grad_(True)
    loss = F.cross_entropy(tl, torch.from_numpy(lab).long())
    loss.backward()
    assert abs(oracle.cross_entropy(lr, lab) - loss.item()) < 1e-13
    np.testing.assert_allclose(dl, tl.grad.numpy(), rtol=1e-12, atol=1e-15)
    # chunked batches: n_total divides, chunks add up
    part = oracle.cross_entropy(lr[:2], lab[:2], 4) + oracle.cross_entropy(lr[2:], lab[2:], 4)
    assert abs(part - loss.item()) < 1e-13


def test_softmax_jacobian_of_sum_vanishes():
    # section 7.3 uses sum(m(x)) as the loss; softmax rows sum to one, so the
    # gradient of that loss with respect to the logits is zero
    lr = rng.standard_normal((4, 9)) * 3
    pr = oracle.softmax(lr)
    np.testing.assert_allclose(oracle.softmax_bwd(pr, np.ones_like(pr)), 0.0, atol=1e-15)
    g = rng.standard_normal(pr.shape)
    tl = torch.from_numpy(lr).requires_grad_(True)
    (torch.softmax(tl, 1) * torch.from_numpy(g)).sum().backward()
    np.testing.assert_allclose(oracle.softmax_bwd(pr, g), tl.grad.numpy(), rtol=1e-12, atol=1e-15)


def test_round_bf16_against_torch_and_on_ties():
    v = np.concatenate([rng.standard_normal(20000) * 10.0 ** rng.integers(-30, 30, 20000),
                        np.array([0.0, -0.0, 1.0, -1.0, 2.0 ** -126, 2.0 ** -133, 3.0 * 2.0 ** -134])])
    v = v.astype(np.float32)  # torch rounds from fp32; these are exact doubles too
    ref = torch.from_numpy(v).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(oracle.round_bf16(v.astype(np.float64)), ref)
    # ties go to the even 8-bit significand: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert oracle.round_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert oracle.round_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    assert oracle.round_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1.0 + 2.0 ** -7
    # a value that fp32 double rounding would get wrong is rounded once, from fp64
    x = 1.0 + 2.0 ** -8 + 2.0 ** -30  # fp32 would first drop 2^-30, then tie to even -> 1.0
    assert oracle.round_bf16(np.array([x]))[0] == 1.0 + 2.0 ** -7
    r = oracle.round_bf16(rng.standard_normal(1000))
    assert np.array_equal(oracle.round_bf16(r), r)


def test_bf16_storage_model_only_rounds_what_is_stored():
    params, x, labels = tiny_inputs()
    params, x = oracle.round_bf16(params), oracle.round_bf16(x)
    l64 = oracle.forward(TINY, params, x)
    l16, saved = oracle.forward(TINY, params, x, keep=True, storage="bf16")
    assert 0 < np.abs(l16 - l64).max() < 0.05 * np.abs(l64).max()
    for sv in saved:
        if sv[0] == "conv":
            assert np.array_equal(oracle.round_bf16(sv[2]), sv[2])
    _, g64, _ = oracle.backward(TINY, params, x, labels)
    _, g16, _ = oracle.backward(TINY, params, x, labels, storage="bf16")
    rel = np.linalg.norm(g16 - g64) / np.linalg.norm(g64)
    assert 0 < rel < 0.1


def test_backward_at_a_given_forward_state_reproduces_backward():
    params, x, labels = tiny_inputs()
    loss, grads, logits = oracle.backward(TINY, params, x, labels)
    _, saved = oracle.forward(TINY, params, x, keep=True)
    outputs = []
    for st, sv in zip(TINY, saved):
        outputs.append(sv[2] if st[0] in ("conv", "fc") else None)
    # pool outputs are the next step's input
    for i, st in enumerate(TINY):
        if st[0] == "pool":
            nxt = saved[i + 1]
            outputs[i] = nxt[1] if nxt[0] == "conv" else nxt[1].reshape(nxt[3])
    lg2, state = oracle.state_from_outputs(TINY, x, outputs)
    assert np.array_equal(lg2, logits)
    loss2, grads2, _ = oracle.backward(TINY, params, x, labels, state=(lg2, state))
    assert loss2 == loss and np.array_equal(grads2, grads)


# ------------------------------------------------------------- whole networks

TINY = [("conv", 3), ("conv", 4), ("pool",), ("conv", 2), ("pool",), ("fc", 6, True), ("fc", 5, True), ("fc", 3, False)]


def tiny_inputs(N=2, H=8, W=8, C=2, seed=7, bias=True):
    r = np.random.default_rng(seed)
    shapes = oracle.param_shapes(TINY, H, W, C)
    parts = []
    for ws, bs in shapes:
        fan_in = int(np.prod(ws[1:]))
        parts.append(r.standard_normal(ws).ravel() * np.sqrt(2.0 / fan_in))
        parts.append(r.standard_normal(bs) * 0.1 if bias else np.zeros(bs))
    return np.concatenate(parts), r.standard_normal((N, H, W, C)), r.integers(0, 3, N).astype(np.int32)


def test_finite_differences_on_a_tiny_net():
    params, x, labels = tiny_inputs()
    loss, grads, _ = oracle.backward(TINY, params, x, labels)
    h = 1e-5
    worst = 0.0
    for i in range(params.size):
        pp, pm = params.copy(), params.copy()
        pp[i] += h
        pm[i] -= h
        lp = oracle.cross_entropy(oracle.forward(TINY, pp, x), labels)
        lm = oracle.cross_entropy(oracle.forward(TINY, pm, x), labels)
        fd = (lp - lm) / (2 * h)
        err = abs(fd - grads[i]) / max(abs(fd), abs(grads[i]), 1e-4)
        worst = max(worst, err)
    assert worst <= 1e-6, worst
    assert np.count_nonzero(grads) > 0.5 * grads.size


def test_sgd_step_closed_form_and_descent():
    # quadratic L = a w^2 / 2: gradient a w, so a step gives w (1 - lr a), k steps w (1 - lr a)^k
    w, a, lr = np.array([3.0, -1.5]), 2.0, 0.1
    assert np.allclose(oracle.sgd_step(w, a * w, lr), [2.4, -1.2], rtol=0, atol=1e-15)
    for _ in range(5):
        w = oracle.sgd_step(w, a * w, lr)
    assert np.allclose(w, np.array([3.0, -1.5]) * 0.8 ** 5, rtol=1e-14)
    # on the tiny net a small step along the negative gradient lowers the loss by about lr |g|^2
    params, x, labels = tiny_inputs()
    loss, grads, _ = oracle.backward(TINY, params, x, labels)
    lr = 1e-4
    after = oracle.cross_entropy(oracle.forward(TINY, oracle.sgd_step(params, grads, lr), x), labels)
    assert after < loss
    assert abs((loss - after) - lr * float(grads @ grads)) <= 1e-2 * lr * float(grads @ grads)


def torch_net(steps, params, x, labels):
    shapes = oracle.param_shapes(steps, x.shape[1], x.shape[2], x.shape[3])
    t = torch.from_numpy(params.copy()).requires_grad_(True)
    a = nhwc_to_torch(x)
    off = 0
    pi = 0
    for st in steps:
        if st[0] == "pool":
            a = F.max_pool2d(a, 2, 2)
            continue
        ws, bs = shapes[pi]; pi += 1
        nw, nb = int(np.prod(ws)), int(np.prod(bs))
        w, b = t[off:off + nw].reshape(ws), t[off + nw:off + nw + nb]
        off += nw + nb
        if st[0] == "conv":
            a = F.relu(F.conv2d(a, w.permute(0, 3, 1, 2), b, padding=1))
        else:
            if a.dim() == 4:
                a = a.permute(0, 2, 3, 1).reshape(a.shape[0], -1)  # (h, w, c), c fastest
            a = F.linear(a, w, b)
            if st[2]:
                a = F.relu(a)
    loss = F.cross_entropy(a, torch.from_numpy(labels).long())
    loss.backward()
    return a.detach().numpy(), loss.item(), t.grad.numpy()


def test_whole_network_against_torch_autograd():
    params, x, labels = tiny_inputs(N=3, H=8, W=12, C=3, seed=11)
    loss, grads, logits = oracle.backward(TINY, params, x, labels)
    tl, tloss, tg = torch_net(TINY, params, x, labels)
    np.testing.assert_allclose(logits, tl, rtol=1e-11, atol=1e-12)
    assert abs(loss - tloss) < 1e-12
    np.testing.assert_allclose(grads, tg, rtol=1e-9, atol=1e-13)
    # chunking the batch gives the same sums
    g2 = np.zeros_like(grads)
    l2 = 0.0
    for s in range(3):
        l, _, _ = oracle.backward(TINY, params, x[s:s + 1], labels[s:s + 1], n_total=3, grads=g2)
        l2 += l
    np.testing.assert_allclose(g2, grads, rtol=1e-11, atol=1e-14)
    assert abs(l2 - loss) < 1e-12


def test_vgg19_topology_against_torch_at_32x32():
    # the real 19-layer topology at the small input size, fp64, against torch
    steps = oracle.vgg19_steps()
    r = np.random.default_rng(3)
    shapes = oracle.param_shapes(steps, 32, 32, 3)
    parts = []
    for ws, bs in shapes:
        parts.append(r.standard_normal(ws).ravel() * np.sqrt(2.0 / int(np.prod(ws[1:]))))
        parts.append(r.standard_normal(bs) * 0.05)
    params = np.concatenate(parts)
    assert params.size == 43003944
    x = (r.random((2, 32, 32, 3)) - 0.5) / 0.25
    labels = np.array([3, 977], dtype=np.int32)
    loss, grads, logits = oracle.vgg19_backward(params, x, labels, chunk=1)
    tl, tloss, tg = torch_net(steps, params, x, labels)
    np.testing.assert_allclose(logits, tl, rtol=1e-10, atol=1e-11)
    assert abs(loss - tloss) < 1e-11
    den = np.linalg.norm(tg)
    assert np.linalg.norm(grads - tg) <= 1e-10 * den


def test_forward_is_positively_homogeneous_without_bias():
    params, x, _ = tiny_inputs(bias=False)
    l1 = oracle.forward(TINY, params, x)
    l2 = oracle.forward(TINY, params, 3.5 * x)
    np.testing.assert_allclose(l2, 3.5 * l1, rtol=1e-12, atol=1e-13)


def test_gradient_of_the_papers_sum_loss_is_zero():
    params, x, _ = tiny_inputs()
    loss, grads, _ = oracle.backward(TINY, params, x, loss_kind="sum")
    assert abs(loss - x.shape[0]) < 1e-12
    assert np.abs(grads).max() < 1e-14


def test_structure_matches_the_papers_instruction_counts():
    counts = {}
    with open(__file__.replace("test_oracle_pins.py", "golden/hlo_instruction_counts.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, *v = line.split()
                counts[k] = [int(t) for t in v]
    steps = oracle.vgg19_steps()
    n_conv = sum(1 for s in steps if s[0] == "conv")
    n_pool = sum(1 for s in steps if s[0] == "pool")
    n_fc = sum(1 for s in steps if s[0] == "fc")
    n_relu = n_conv + sum(1 for s in steps if s[0] == "fc" and s[2])
    assert n_conv == counts["convolution"][0] == 16
    assert n_fc == counts["dot"][0] == 3
    assert n_pool == counts["reduce-window"][0] == counts["select-and-scatter"][1] == 5
    assert n_relu + n_pool == counts["maximum"][0] == 23
    # backward: forward convs + one filter gradient each + one input gradient
    # for all but the first layer; dense layers: forward + dX + dW
    assert n_conv + n_conv + (n_conv - 1) == counts["convolution"][1] == 47
    assert 3 * n_conv == counts["convolution"][2]
    assert 3 * n_fc == counts["dot"][1]
    assert n_conv == counts["reverse"][1]
    assert 1 + n_conv + n_fc == counts["reduce"][2]
    shapes = oracle.param_shapes(steps, 224, 224, 3)
    assert sum(int(np.prod(w)) + int(np.prod(b)) for w, b in shapes) == 143667240
