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
gradients are compared where they are unique: given the decisions.  The
unsynchronised difference is printed for information.
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


def check_bf16_backward(net, params, images, labels, logits, grads, loss, tol=2e-2):
    """Forward parity on logits and stored activations; backward parity at the stored state."""
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
    o_loss, o_grads, _ = oracle.backward(steps, p64, images, labels, storage="bf16", state=(d_logits, d_saved))
    assert abs(loss - o_loss) <= 1e-3 * abs(o_loss)
    worst = check_grads(net, grads, o_grads, tol)
    _, free_grads, _ = oracle.backward(steps, p64, images, labels, storage="bf16")
    print(f"bf16 {images.shape[1]}x{images.shape[2]} B={B}: logits {e_logits:.2e}, worst activation {worst_act:.2e}, "
          f"worst gradient tensor at the stored state {worst:.2e}, whole-gradient difference to the checker's own "
          f"forward state {rel_l2(grads, free_grads):.2e}")
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
