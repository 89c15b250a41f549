"""GPU parity: the CUDA library (through its C ABI) against the fp64 CPU
checker on the same seeded inputs.

Tolerances.  fp32 configuration: relative L2 error of the logits <= 1e-4 (the
stated bar); gradients <= 2e-4 (fp32 FMA sums of up to ~25k terms, two passes
through the network).  bf16 configurations (fp32 accumulation): relative L2
<= 2e-2 on the logits and on every stored activation against the checker's
own forward pass, and <= 2e-2 on each of the 38 gradient tensors against the
checker's backward pass taken at the forward state the device stored (its
activations read back from the workspace).  The ReLU masks and pool
arg-maxima are integer decisions made on those stored values; an
implementation whose forward arithmetic differs by one part in 10^7 flips
enough near-zero pre-activations to move every gradient tensor by 5-25%, so
gradients are compared where they are unique: given the decisions
(tests/test_oracle_bf16_sensitivity.py reproduces that measurement with the
checker alone).  What that comparison cannot see is asserted separately: the
fraction of decisions on which the device's stored state and the checker's own
forward pass differ is small and every differing one is a near-tie, and the
free-running gradient (each side at its own forward state) keeps the direction
of every tensor (cosine >= 0.90).
"""
import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def pkg():
    import paper_1810_09868_b200 as p
    return p


def rel_l2(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def make_inputs(H, W, B, bf16, bias_std=0.0):
    params = si.vgg19_params(H, W, seed=0, bias_std=bias_std, bf16_exact=bf16)
    images = si.images(B, H, W, seed=1, bf16_exact=bf16)
    labels = si.labels(B, seed=2)
    return params, images, labels


def run_backward(net, images, labels):
    x = torch.from_numpy(images).to(DEV).to(net.act_dtype)
    y = torch.from_numpy(labels).to(DEV)
    logits = torch.empty(images.shape[0], 1000, dtype=torch.float32, device=DEV)
    grads, loss = net.backward(x, y, logits=logits)
    net.sync_status()
    return logits.cpu().numpy(), grads.cpu().numpy(), float(loss.item())


def device_state(net, B, images, logits):
    """(logits, saved) of the checker, built from the activations the device stored."""
    p = pkg()
    outs, ci, pi, fi = [], 0, 0, 0
    steps = oracle.vgg19_steps()
    for st in steps:
        if st[0] == "conv":
            idx = ci; ci += 1
        elif st[0] == "pool":
            idx = 16 + pi; pi += 1
        else:
            idx = 21 + fi; fi += 1
        if idx <= 22:
            t = net.saved_tensor(B, p.VGG19_MODE_BACKWARD, idx).float().cpu().numpy().astype(np.float64)
            outs.append(t.reshape(B, 4096) if idx >= 21 else t)
        else:
            outs.append(np.asarray(logits, dtype=np.float64))
    return oracle.state_from_outputs(steps, images, outs)


def pool_argmax(x):
    """Arg-max (0..3, scan order (0,0),(0,1),(1,0),(1,1), first maximum wins) and the four candidates
    of every 2x2 window of an NHWC tensor."""
    N, Hh, Ww, C = x.shape
    w = x.reshape(N, Hh // 2, 2, Ww // 2, 2, C).transpose(0, 1, 3, 5, 2, 4).reshape(N, Hh // 2, Ww // 2, C, 4)
    return np.argmax(w, axis=-1), w


def decision_agreement(d_saved, o_saved):
    """How far the integer decisions of the backward pass (ReLU masks, pool arg-maxima) taken on the
    device's stored forward state are from those the checker takes on its own bf16-storage forward
    pass.  Per step: (kind, fraction of decisions that differ, worst near-tie measure), where the
    near-tie measure of a differing decision is the size of the value that decided it relative to the
    layer's rms: the activation itself for a mask, the checker's margin between the two candidate
    positions for a pooling window.  A correct forward pass differs only on near-ties."""
    out = []
    for sd, so in zip(d_saved, o_saved):
        if sd[0] in ("conv", "fc"):
            if sd[0] == "fc" and not sd[4]:
                continue
            yd, yo = sd[2], so[2]
            rms = float(np.sqrt(np.mean(yo ** 2))) + 1e-300
            differ = (yd > 0) != (yo > 0)
            frac = float(differ.mean())
            worst = float(np.maximum(yd, yo)[differ].max() / rms) if differ.any() else 0.0
            out.append((sd[0] + "-relu", frac, worst))
        else:
            ad, _ = pool_argmax(sd[1])
            ao, wo = pool_argmax(so[1])
            live = wo.max(axis=-1) > 0  # a window of zeros passes no gradient through the ReLU below
            differ = (ad != ao) & live
            frac = float(differ.sum() / max(int(live.sum()), 1))
            rms = float(np.sqrt(np.mean(so[1] ** 2))) + 1e-300
            margin = wo.max(axis=-1) - np.take_along_axis(wo, ad[..., None], axis=-1)[..., 0]
            worst = float(margin[differ].max() / rms) if differ.any() else 0.0
            out.append(("pool", frac, worst))
    return out


# Bounds on the decisions that may differ between the device's forward state and the checker's own.
# Measured at 224x224 on twelve images of the batch-100 pass: at most 0.27 % of a layer's ReLU masks and
# 2.7 % of its live pooling windows (bf16 keeps 8 significant bits, so neighbouring positive activations
# tie or sit one ulp apart often), every one of them a near-tie: the deciding value at most 6 % of the
# layer's rms, while the activations agree to 2e-2 in L2.
MASK_DIFFER_MAX, POOL_DIFFER_MAX, NEAR_TIE_MAX = 0.02, 0.06, 0.25
# Free-running comparison (each side differentiates at its own forward state): direction only.  The
# checker against itself under a 1e-7 weight perturbation keeps 0.978 (32x32); the device against the
# checker measured 0.945 on the least aligned tensor (the first layer's filter, 224x224, 8 images).
FREE_COSINE_MIN = 0.90


def check_decisions(d_saved, o_saved):
    rows = decision_agreement(d_saved, o_saved)
    for kind, frac, worst in rows:
        assert frac <= (POOL_DIFFER_MAX if kind == "pool" else MASK_DIFFER_MAX), rows
        assert worst <= NEAR_TIE_MAX, rows
    return rows


def free_running_cosines(net, grads, o_grads):
    cos = []
    for off, dims in net.param_slices():
        n = int(np.prod(dims))
        a, b = np.asarray(grads[off:off + n], dtype=np.float64), o_grads[off:off + n]
        cos.append(float(a @ b / max(np.linalg.norm(a) * np.linalg.norm(b), 1e-300)))
    return cos


def check_bf16_backward(net, params, images, labels, logits, grads, loss, tol=2e-2):
    """Forward parity on logits and stored activations; the decisions taken on the stored state against
    the checker's own; backward parity at the stored state; direction of the free-running gradient."""
    B = images.shape[0]
    steps = oracle.vgg19_steps()
    p64 = params.astype(np.float64)
    o_logits, o_saved = oracle.forward(steps, p64, images, keep=True, storage="bf16")
    e_logits = rel_l2(logits, o_logits)
    assert e_logits <= tol
    assert rel_l2(logits, oracle.forward(steps, p64, images)) <= tol
    d_logits, d_saved = device_state(net, B, images, logits)
    worst_act = 0.0
    for sd, so in zip(d_saved, o_saved):
        if sd[0] in ("conv", "fc") and sd[2].shape == so[2].shape:
            worst_act = max(worst_act, rel_l2(sd[2], so[2]))
    assert worst_act <= tol
    decisions = check_decisions(d_saved, o_saved)
    o_loss, o_grads, _ = oracle.backward(steps, p64, images, labels, storage="bf16", state=(d_logits, d_saved))
    assert abs(loss - o_loss) <= 1e-3 * abs(o_loss)
    worst = check_grads(net, grads, o_grads, tol)
    _, free_grads, _ = oracle.backward(steps, p64, images, labels, storage="bf16", state=(o_logits, o_saved))
    cos = free_running_cosines(net, grads, free_grads)
    assert min(cos) >= FREE_COSINE_MIN, cos
    print(f"bf16 {images.shape[1]}x{images.shape[2]} B={B}: logits {e_logits:.2e}, worst activation {worst_act:.2e}, "
          f"decisions differing: masks <= {max(f for k, f, _ in decisions if k != 'pool'):.2e}, pools <= "
          f"{max(f for k, f, _ in decisions if k == 'pool'):.2e}, worst near-tie {max(w for _, _, w in decisions):.2e} of rms; "
          f"worst gradient tensor at the stored state {worst:.2e}; free-running: whole-gradient difference "
          f"{rel_l2(grads, free_grads):.2e}, smallest per-tensor cosine {min(cos):.4f}")
    return worst


def check_grads(net, grads, o_grads, tol):
    worst = []
    for i, (off, dims) in enumerate(net.param_slices()):
        n = int(np.prod(dims))
        e = rel_l2(grads[off:off + n], o_grads[off:off + n])
        worst.append((e, i, dims))
    bad = [w for w in worst if not w[0] <= tol]
    assert not bad, f"gradient tensors above {tol}: {bad}"
    return max(w[0] for w in worst)


def test_config1_fp32_forward_32x32_batch1():
    p = pkg()
    params, images, _ = make_inputs(32, 32, 1, False)
    net = p.Net(32, 32, 1, p.VGG19_FP32, params=params, mode=p.VGG19_MODE_FORWARD)
    x = torch.from_numpy(images).to(DEV)
    probs = torch.empty(1, 1000, dtype=torch.float32, device=DEV)
    logits = net.forward(x, probs=probs)
    net.sync_status()
    o = oracle.vgg19_forward(params.astype(np.float64), images)
    assert rel_l2(logits.cpu().numpy(), o) <= 1e-4
    assert rel_l2(probs.cpu().numpy(), oracle.softmax(o)) <= 1e-4
    assert int(logits.argmax()) == int(o.argmax())
    net.close()


@pytest.mark.parametrize("flags", [0, 1])
def test_fp32_backward_32x32(flags):
    p = pkg()
    B = 3
    params, images, labels = make_inputs(32, 32, B, False, bias_std=0.05)
    net = p.Net(32, 32, B, p.VGG19_FP32, params=params, flags=flags)
    logits, grads, loss = run_backward(net, images, labels)
    o_loss, o_grads, o_logits = oracle.vgg19_backward(params.astype(np.float64), images, labels, chunk=B)
    assert rel_l2(logits, o_logits) <= 1e-4
    assert abs(loss - o_loss) <= 1e-4 * abs(o_loss)
    worst = check_grads(net, grads, o_grads, 2e-4)
    print(f"fp32 32x32 B={B}: logits {rel_l2(logits, o_logits):.2e}, worst gradient tensor {worst:.2e}")
    net.close()


@pytest.mark.parametrize("flags", [0, 2])
def test_bf16_backward_32x32(flags):
    p = pkg()
    B = 5
    params, images, labels = make_inputs(32, 32, B, True, bias_std=0.05)
    net = p.Net(32, 32, B, p.VGG19_BF16, params=params, flags=flags)
    logits, grads, loss = run_backward(net, images, labels)
    check_bf16_backward(net, params, images, labels, logits, grads, loss)
    net.close()


def test_smaller_batch_than_batch_max_and_ragged_sizes():
    p = pkg()
    params, images, labels = make_inputs(64, 32, 3, True)
    net = p.Net(64, 32, 7, p.VGG19_BF16, params=params)
    logits, grads, loss = run_backward(net, images, labels)
    check_bf16_backward(net, params, images, labels, logits, grads, loss)
    net.close()


def test_mid_size_image_takes_every_convolution_kernel():
    # 96x64: layer 2 runs on the halo kernel, 48x32 and below on the general kernel in patch
    # (48x32) and im2col (24x16, ...) mode
    p = pkg()
    params, images, labels = make_inputs(96, 64, 3, True, bias_std=0.05)
    net = p.Net(96, 64, 3, p.VGG19_BF16, params=params)
    logits, grads, loss = run_backward(net, images, labels)
    check_bf16_backward(net, params, images, labels, logits, grads, loss)
    net.close()


def test_wide_image_takes_the_large_image_kernels_with_unequal_sides():
    # 96 rows x 224 columns: the row-shift kernel at 96x224 and the halo kernel at 48x112 (height and width enter
    # their tile arithmetic separately), the pair kernels at 24x56, 12x28 and 6x14 with ragged last tiles, and a
    # first dense layer of 3 x 7 x 512 inputs; forward + backward against the checker
    p = pkg()
    params, images, labels = make_inputs(96, 224, 2, True, bias_std=0.05)
    net = p.Net(96, 224, 2, p.VGG19_BF16, params=params)
    logits, grads, loss = run_backward(net, images, labels)
    check_bf16_backward(net, params, images, labels, logits, grads, loss)
    # and the forward-only pass (pools in the epilogues, no pre-pool activation stored) gives the same logits
    x = torch.from_numpy(images).to(DEV).to(torch.bfloat16)
    fwd = net.forward(x).clone()
    net.sync_status()
    assert rel_l2(fwd.cpu().numpy(), logits) <= 1e-3
    net.close()


@pytest.mark.parametrize("B", [1, 3])
def test_full_resolution_odd_batches(B):
    # 224x224 at batch 1 and 3: odd tile counts in the pair kernels (a last pair with one idle CTA), tail rounds
    # of other sizes than at batch 100, a dense M tile of 1 or 3 rows
    p = pkg()
    params, images, labels = make_inputs(224, 224, B, True, bias_std=0.05)
    net = p.Net(224, 224, B, p.VGG19_BF16, params=params)
    logits, grads, loss = run_backward(net, images, labels)
    check_bf16_backward(net, params, images, labels, logits, grads, loss)
    net.close()


@pytest.mark.parametrize("H,W", [(256, 256), (448, 448)])
def test_other_resolutions_forward(H, W):
    # 256x256: a width that is no multiple of 14, so conv1_2 leaves the row-shift kernel for the halo kernel;
    # 448x448: four times the benchmark's pixels (first dense layer 14 x 14 x 512 = 100352 inputs).  Forward-only
    # pass (pools in the epilogues) and training-mode forward give logits within the bf16 bar of the checker.
    p = pkg()
    params, images, labels = make_inputs(H, W, 1, True, bias_std=0.05)
    net = p.Net(H, W, 1, p.VGG19_BF16, params=params)
    x = torch.from_numpy(images).to(DEV).to(torch.bfloat16)
    fwd = net.forward(x).clone()
    net.sync_status()
    ref = oracle.forward(oracle.vgg19_steps(), params.astype(np.float64), images)
    assert np.isfinite(fwd.cpu().numpy()).all()
    assert rel_l2(fwd.cpu().numpy(), ref) <= 2e-2
    logits, grads, loss = run_backward(net, images, labels)
    assert rel_l2(logits, ref) <= 2e-2 and np.isfinite(grads).all()
    net.close()


def test_graph_replay_is_bit_identical_and_matches_direct_launch():
    p = pkg()
    params, images, _ = make_inputs(32, 32, 2, True)
    x = torch.from_numpy(images).to(DEV).to(torch.bfloat16)
    outs = []
    for flags in (0, p.VGG19_FLAG_NO_GRAPH):
        net = p.Net(32, 32, 2, p.VGG19_BF16, params=params, flags=flags, mode=p.VGG19_MODE_FORWARD)
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            a = net.forward(x, stream=s).clone()
            b = net.forward(x, stream=s).clone()
            c = net.forward(x, stream=s).clone()
        net.sync_status(s)
        assert torch.equal(a, b) and torch.equal(b, c)
        outs.append(a.cpu())
        assert p.vgg19_launch_count(net.handle, p.VGG19_MODE_FORWARD) >= 16 + 5 + 3
        net.close()
    assert torch.equal(outs[0], outs[1])


def test_seeded_create_matches_the_generator_and_get_set_params():
    p = pkg()
    h = p.vgg19_create(32, 32, 1, p.VGG19_FP32, 0)
    n_t, n_e = p.vgg19_param_count(h)
    assert n_t == 38 and n_e == 43003944
    host = np.empty(n_e, dtype=np.float32)
    p.vgg19_get_params(h, host)
    assert np.array_equal(host, si.vgg19_params(32, 32, seed=0))
    other = si.vgg19_params(32, 32, seed=5)
    p.vgg19_set_params(h, other)
    p.vgg19_get_params(h, host)
    assert np.array_equal(host, other)
    off, dims = p.vgg19_param_info(h, 0)
    assert off == 0 and dims == (64, 3, 3, 3)
    off, dims = p.vgg19_param_info(h, 32)
    assert dims == (4096, 512)
    text = p.vgg19_describe(h)
    assert text.count("conv") >= 16 and "convolution=16 reduce-window=5 dot=3" in text
    p.vgg19_destroy(h)


def test_error_codes_on_a_device():
    p = pkg()
    h = p.vgg19_create(32, 32, 2, p.VGG19_BF16, 0)
    x = torch.zeros(2, 32, 32, 3, dtype=torch.bfloat16, device=DEV)
    out = torch.zeros(2, 1000, device=DEV)
    with pytest.raises(p.binding.Vgg19Error) as e:
        p.vgg19_forward(h, x, 2, out)
    assert e.value.code == p.VGG19_ERR_WORKSPACE
    need = p.vgg19_workspace_bytes(h, 2, p.VGG19_MODE_FORWARD)
    assert need > 0 and p.vgg19_workspace_bytes(h, 3, p.VGG19_MODE_FORWARD) == 0
    ws = torch.empty(need - 256, dtype=torch.uint8, device=DEV)
    p.vgg19_bind_workspace(h, ws, need - 256)
    with pytest.raises(p.binding.Vgg19Error) as e:
        p.vgg19_forward(h, x, 2, out)
    assert e.value.code == p.VGG19_ERR_WORKSPACE
    with pytest.raises(p.binding.Vgg19Error) as e:
        p.vgg19_forward(h, x, 3, out)
    assert e.value.code == p.VGG19_ERR_ARG
    with pytest.raises(p.binding.Vgg19Error) as e:
        p.vgg19_forward(h, None, 2, out)
    assert e.value.code == p.VGG19_ERR_ARG
    p.vgg19_destroy(h)


def test_host_buffer_entry_points():
    p = pkg()
    B = 2
    params, images, labels = make_inputs(32, 32, B, True)
    net = p.Net(32, 32, B, p.VGG19_BF16, params=params, host_io=True)
    x_host = torch.from_numpy(images).to(torch.bfloat16).pin_memory()
    logits_host = torch.empty(B, 1000, dtype=torch.float32).pin_memory()
    probs_host = torch.empty(B, 1000, dtype=torch.float32).pin_memory()
    s = torch.cuda.Stream()
    p.vgg19_forward_host(net.handle, x_host, B, logits_host, probs_host, s)
    dev_logits = net.forward(x_host.to(DEV))
    torch.cuda.synchronize()
    assert torch.equal(dev_logits.cpu(), logits_host)
    np.testing.assert_allclose(probs_host.sum(1).numpy(), 1.0, rtol=1e-5)
    grads_host = torch.empty(net.n_params, dtype=torch.float32).pin_memory()
    loss_host = torch.empty(1, dtype=torch.float32).pin_memory()
    p.vgg19_backward_host(net.handle, x_host, torch.from_numpy(labels), B, grads_host, loss_host, s)
    grads, loss = net.backward(x_host.to(DEV), torch.from_numpy(labels).to(DEV))
    torch.cuda.synchronize()
    assert torch.equal(grads.cpu(), grads_host) and float(loss) == float(loss_host)
    net.close()


@pytest.mark.parametrize("bf16", [False, True])
def test_sgd_step_updates_every_copy_of_the_parameters(bf16):
    """One gradient-descent step on the device against the checker's w - lr * g, then a second
    forward + backward pass with the updated parameters against the checker: every copy of the
    filters the kernels read (storage type, rotated, tap-major, padded) must have followed."""
    p = pkg()
    B, lr = 2, 0.05
    params, images, labels = make_inputs(32, 32, B, bf16, bias_std=0.1)
    net = p.Net(32, 32, B, p.VGG19_BF16 if bf16 else p.VGG19_FP32, params=params)
    logits0, grads, _ = run_backward(net, images, labels)
    net.sgd_step(torch.from_numpy(grads).to(DEV), lr)
    net.sync_status()
    new = np.empty_like(params)
    p.vgg19_get_params(net.handle, new)
    want = oracle.sgd_step(params, grads, lr)
    assert rel_l2(new, want) <= 1e-6
    assert rel_l2(new, params) > 1e-4  # the step moved the parameters
    logits1, grads1, loss1 = run_backward(net, images, labels)
    assert rel_l2(logits1, logits0) > 1e-3
    if bf16:
        # the device computes with the bf16 rounding of its fp32 master copy
        used = oracle.round_bf16(new.astype(np.float64)).astype(np.float32)
        check_bf16_backward(net, used, images, labels, logits1, grads1, loss1)
    else:
        o_loss, o_grads, o_logits = oracle.backward(oracle.vgg19_steps(), new.astype(np.float64), images, labels)
        assert rel_l2(logits1, o_logits) <= 1e-4
        assert abs(loss1 - o_loss) <= 1e-4 * abs(o_loss)
        check_grads(net, grads1, o_grads, 2e-4)
    net.close()


def test_async_host_entry_point_matches_the_blocking_one():
    """Five batches in flight through vgg19_forward_host_async (two staging slots, uploads on the
    library's own stream) give bit for bit the logits of vgg19_forward_host on the same images."""
    p = pkg()
    B = 3
    params, _, _ = make_inputs(32, 32, B, True)
    net = p.Net(32, 32, B, p.VGG19_BF16, params=params, mode=p.VGG19_MODE_FORWARD, host_io=True)
    stream = torch.cuda.Stream()
    batches = [torch.from_numpy(si.images(B, 32, 32, seed=10 + i, bf16_exact=True)).to(torch.bfloat16).pin_memory()
               for i in range(5)]
    want = []
    for x in batches:
        out = torch.empty(B, 1000, dtype=torch.float32).pin_memory()
        p.vgg19_forward_host(net.handle, x, B, out, None, stream)
        want.append(out.clone())
    got = [torch.full((B, 1000), float("nan"), dtype=torch.float32).pin_memory() for _ in batches]
    for x, out in zip(batches, got):
        p.vgg19_forward_host_async(net.handle, x, B, out, None, stream)
    net.sync_status(stream)
    for g, w in zip(got, want):
        assert torch.equal(g, w)
    assert not torch.equal(want[0], want[1])
    net.close()


def test_async_host_entry_point_with_changing_batch_sizes():
    """The staging slots of vgg19_forward_host_async sit behind the work area of a pass at the call's own
    batch, so a smaller batch right after a larger one (the ragged last batch of a serving loop) would
    upload into memory the larger pass is still using unless the library orders the two.  Alternating
    batch 4 and batch 1 must give the blocking call's logits bit for bit."""
    p = pkg()
    params, _, _ = make_inputs(64, 64, 4, True)
    net = p.Net(64, 64, 4, p.VGG19_BF16, params=params, mode=p.VGG19_MODE_FORWARD, host_io=True)
    stream = torch.cuda.Stream()
    sizes = [4, 1, 4, 1, 1, 4, 2, 4]
    batches = [torch.from_numpy(si.images(b, 64, 64, seed=30 + i, bf16_exact=True)).to(torch.bfloat16).pin_memory()
               for i, b in enumerate(sizes)]
    want = []
    for x, b in zip(batches, sizes):
        out = torch.empty(b, 1000, dtype=torch.float32).pin_memory()
        p.vgg19_forward_host(net.handle, x, b, out, None, stream)
        want.append(out.clone())
    for _ in range(3):
        got = [torch.full((b, 1000), float("nan"), dtype=torch.float32).pin_memory() for b in sizes]
        for x, b, out in zip(batches, sizes, got):
            p.vgg19_forward_host_async(net.handle, x, b, out, None, stream)
        net.sync_status(stream)
        for g, w in zip(got, want):
            assert torch.equal(g, w)
    net.close()


def test_a_bounded_wait_that_runs_out_is_reported_and_the_handle_stays_usable():
    """Every wait inside the tensor-core kernels is bounded; one that runs out records a code and the
    kernel returns.  The library's self-test kernel waits (about a millisecond) on a barrier nothing
    arrives on: vgg19_sync_status must report VGG19_ERR_DEVICE_TIMEOUT once, clear the record, and the
    next pass on the same handle must give the result it gave before."""
    p = pkg()
    params, images, _ = make_inputs(32, 32, 2, True)
    net = p.Net(32, 32, 2, p.VGG19_BF16, params=params, mode=p.VGG19_MODE_FORWARD)
    x = torch.from_numpy(images).to(DEV).to(torch.bfloat16)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        before = net.forward(x, stream=s).clone()
    net.sync_status(s)
    p.vgg19_selftest_wait_timeout(net.handle, s)
    with pytest.raises(p.binding.Vgg19Error) as e:
        net.sync_status(s)
    assert e.value.code == p.VGG19_ERR_DEVICE_TIMEOUT
    net.sync_status(s)  # the record was cleared
    with torch.cuda.stream(s):
        after = net.forward(x, stream=s).clone()
    net.sync_status(s)
    assert torch.equal(before, after)
    net.close()


def test_a_label_out_of_range_is_reported_not_dereferenced():
    p = pkg()
    B = 3
    params, images, labels = make_inputs(32, 32, B, True)
    net = p.Net(32, 32, B, p.VGG19_BF16, params=params)
    x = torch.from_numpy(images).to(DEV).to(torch.bfloat16)
    for bad in (1000, -7, 2 ** 31 - 1):
        y = torch.from_numpy(labels).to(DEV).clone()
        y[1] = bad
        grads, loss = net.backward(x, y)
        with pytest.raises(p.binding.Vgg19Error) as e:
            net.sync_status()
        assert e.value.code == p.VGG19_ERR_ARG
        assert torch.isnan(loss).all()
    grads, loss = net.backward(x, torch.from_numpy(labels).to(DEV))
    net.sync_status()
    assert torch.isfinite(loss).all() and torch.isfinite(grads).all()
    net.close()


@pytest.mark.parametrize("bf16", [False, True])
def test_train_steps_as_one_graph_match_backward_then_sgd_step(bf16):
    """vgg19_train_steps (k training steps recorded as one CUDA graph: forward, loss, backward, parameter
    update and filter-copy rebuild per step, the gradient staying in the workspace) against the same k
    steps made of separate vgg19_backward + vgg19_sgd_step calls (bit for bit: same kernels, same order),
    and the first step against the checker: loss and updated parameters w - lr * dL/dw at the stored
    forward state."""
    p = pkg()
    B, K, lr = 2, 3, 0.02
    dtype = p.VGG19_BF16 if bf16 else p.VGG19_FP32
    params, _, _ = make_inputs(32, 32, B, bf16, bias_std=0.1)
    images = si.images(K * B, 32, 32, seed=1, bf16_exact=bf16)
    labels = si.labels(K * B, seed=2)
    net = p.Net(32, 32, B, dtype, params=params, mode=p.VGG19_MODE_TRAIN)
    x = torch.from_numpy(images).to(DEV).to(net.act_dtype)
    y = torch.from_numpy(labels).to(DEV)
    s = torch.cuda.Stream()
    # reference sequence on the same handle: separate calls
    ref_losses, first_grads, first_logits = [], None, None
    for k in range(K):
        logits = torch.empty(B, 1000, dtype=torch.float32, device=DEV)
        with torch.cuda.stream(s):
            grads, loss = net.backward(x[k * B:(k + 1) * B], y[k * B:(k + 1) * B], logits=logits, stream=s)
            if k == 0:
                net.sync_status(s)
                first_grads, first_logits = grads.cpu().numpy(), logits.cpu().numpy()
                first_state = device_state(net, B, images[:B], first_logits) if bf16 else None
            net.sgd_step(grads, lr, stream=s)
        net.sync_status(s)
        ref_losses.append(float(loss))
    want = np.empty_like(params)
    p.vgg19_get_params(net.handle, want)
    # the same three steps as one graph, from the same starting point, twice (the second run replays the graph)
    for run in range(2):
        p.vgg19_set_params(net.handle, params)
        losses = torch.full((K,), float("nan"), dtype=torch.float32, device=DEV)
        p.vgg19_train_steps(net.handle, x, y, B, K, lr, losses, s)
        net.sync_status(s)
        got = np.empty_like(params)
        p.vgg19_get_params(net.handle, got)
        assert np.array_equal(got, want), run
        assert losses.cpu().tolist() == ref_losses, run
    assert p.vgg19_launch_count(net.handle, p.VGG19_MODE_TRAIN) >= K * (16 + 3 + 1)
    # one step against the checker
    p.vgg19_set_params(net.handle, params)
    loss1 = torch.empty(1, dtype=torch.float32, device=DEV)
    p.vgg19_train_step(net.handle, x[:B], y[:B], B, lr, loss1, s)
    net.sync_status(s)
    after = np.empty_like(params)
    p.vgg19_get_params(net.handle, after)
    steps = oracle.vgg19_steps()
    p64 = params.astype(np.float64)
    if bf16:
        o_loss, o_grads, _ = oracle.backward(steps, p64, images[:B], labels[:B], storage="bf16", state=first_state)
    else:
        o_loss, o_grads, _ = oracle.backward(steps, p64, images[:B], labels[:B])
    assert abs(float(loss1) - o_loss) <= 1e-3 * abs(o_loss)
    o_after = oracle.sgd_step(p64, o_grads, lr)
    # compare the step taken, not the parameters (which barely move): w_after - w_before
    assert rel_l2(after.astype(np.float64) - p64, o_after - p64) <= (2e-2 if bf16 else 2e-4)
    net.close()


def test_dense_gradient_event_fires_inside_the_pass_and_changes_nothing():
    """With vgg19_set_dense_grads_event the backward pass (as a recorded graph and enqueued directly) signals
    the caller's event once the three dense layers' gradients are final: a side stream that waits for the
    event and copies that part of the gradient buffer must get the final values, must be done before the
    pass ends, and the gradients must equal those of a pass without the event."""
    p = pkg()
    B = 4
    params, images, labels = make_inputs(64, 64, B, True)
    x = torch.from_numpy(images).to(DEV).to(torch.bfloat16)
    y = torch.from_numpy(labels).to(DEV)
    for flags in (0, p.VGG19_FLAG_NO_GRAPH):
        net = p.Net(64, 64, B, p.VGG19_BF16, params=params, flags=flags)
        dense_off, _ = p.vgg19_param_info(net.handle, 32)
        s, side = torch.cuda.Stream(), torch.cuda.Stream()
        with torch.cuda.stream(s):
            plain, _ = net.backward(x, y, stream=s)
            plain = plain.clone()
        net.sync_status(s)
        ev = torch.cuda.Event(enable_timing=False)
        ev.record(s)  # creates the underlying event
        p.vgg19_set_dense_grads_event(net.handle, ev)
        grads = torch.zeros(net.n_params, dtype=torch.float32, device=DEV)
        early = torch.zeros(net.n_params - dense_off, dtype=torch.float32, device=DEV)
        done_side, done_pass = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start = torch.cuda.Event(enable_timing=True)
        for rep in range(3):  # first call records the graph, later ones replay it
            grads.zero_()
            torch.cuda.synchronize()
            with torch.cuda.stream(s):
                start.record(s)
                net.backward(x, y, grads=grads, stream=s)
                done_pass.record(s)
            with torch.cuda.stream(side):
                side.wait_event(ev)
                early.copy_(grads[dense_off:])
                done_side.record(side)
            torch.cuda.synchronize()
            net.sync_status(s)
            assert torch.equal(grads, plain)
            assert torch.equal(early, plain[dense_off:]), "the dense gradients were not final when the event fired"
            assert start.elapsed_time(done_side) < start.elapsed_time(done_pass), "the event did not fire before the pass ended"
        p.vgg19_set_dense_grads_event(net.handle, None)
        net.close()
