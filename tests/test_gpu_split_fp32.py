"""The fp32 configuration's tensor-core path (VGG19_FLAG_SPLIT_F16): every fp32 value travels as two fp16 terms
and every product is three fp16 products in an fp32 accumulator.  Checked against the fp64 CPU checker on
fp32 inputs (nothing is rounded to 16 bits beforehand).

Tolerance.  hi + lo keeps 22 bits of a 24-bit mantissa: relative error at most 2^-23 per operand, and the
dropped lo*lo term is 2^-22 of a product.  The sums are another matter: the tensor core's fp32 accumulation
truncates, which measured 2.2e-6, 4.3e-6, 8.1e-6 and 1.6e-5 in relative L2 after 216, 432, 864 and 1728 chained
MMAs (layers 2, 5, 9 and 13) and 1.1e-4 to 1.7e-4 on the logits - so the kernels hand their accumulator over
every 32 MMAs and add the chunks with round-to-nearest fp32 additions, which measures 6.6e-7 on every layer
and 1.0e-5 on the logits.  Bars: 2e-6 per layer; through 19 layers the fp32 configuration's own, 1e-4 on
logits and probabilities (section 7.2's configuration), and 3e-5 so that a return of the long chains fails.
"""
import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def rel_l2(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def pkg():
    import paper_1810_09868_b200 as p
    return p


def layer_params(p, net, params, layer):
    (woff, wdims), (boff, bdims) = p.vgg19_param_info(net.handle, 2 * (layer - 1)), p.vgg19_param_info(net.handle, 2 * layer - 1)
    Wt = params[woff:woff + int(np.prod(wdims))].reshape(wdims).astype(np.float64)
    b = params[boff:boff + int(np.prod(bdims))].astype(np.float64)
    return Wt, b


# (layer, H=W at a 224x224 input, Cin, Cout)
SHAPES = [(2, 224, 64, 64), (3, 112, 64, 128), (5, 56, 128, 256), (9, 28, 256, 512), (13, 14, 512, 512)]


@pytest.fixture(scope="module")
def net224():
    p = pkg()
    params = si.vgg19_params(224, 224, seed=0, bias_std=0.1)
    net = p.Net(224, 224, 3, p.VGG19_FP32, params=params, flags=p.VGG19_FLAG_SPLIT_F16, mode=p.VGG19_MODE_FORWARD)
    yield p, net, params
    net.close()


@pytest.mark.parametrize("layer,S,Cin,Cout", SHAPES)
def test_split_conv_layer_forward(net224, layer, S, Cin, Cout):
    p, net, params = net224
    B = 3 if S <= 28 else 1  # 14x14x3 = 588 pixels: a ragged last tile
    x = si.normal(B * S * S * Cin, seed=100 + layer, take_abs=True).reshape(B, S, S, Cin).astype(np.float32)
    Wt, b = layer_params(p, net, params, layer)
    xd = torch.from_numpy(x).to(DEV)
    y = torch.full((B, S, S, Cout), float("nan"), dtype=torch.float32, device=DEV)
    pooled = torch.full((B, S // 2, S // 2, Cout), float("nan"), dtype=torch.float32, device=DEV)
    p.vgg19_conv_layer_forward(net.handle, layer, xd, B, y, pooled, torch.cuda.current_stream())
    net.sync_status()
    ref = oracle.relu_fwd(oracle.conv3x3_fwd(x.astype(np.float64), Wt, b))
    got = y.cpu().numpy()
    assert np.isfinite(got).all()
    err = rel_l2(got, ref)
    print(f"layer {layer}: split-fp16 convolution against the fp64 checker {err:.2e}")
    assert err <= 2e-6
    assert np.array_equal(pooled.cpu().numpy(), oracle.maxpool2x2_fwd(got.astype(np.float64)).astype(np.float32))


@pytest.mark.parametrize("H,B,extra", [(32, 1, 0), (64, 3, 0), (32, 2, 1)])
def test_split_forward_small(H, B, extra):
    """Section 7.2's fp32 configuration (32x32, batch 1) and a larger one, whole pass, bar 1e-4; also without a
    recorded graph (extra = VGG19_FLAG_NO_GRAPH)."""
    p = pkg()
    params = si.vgg19_params(H, H, seed=0, bias_std=0.05)
    images = si.images(B, H, H, seed=1)
    net = p.Net(H, H, B, p.VGG19_FP32, params=params, flags=p.VGG19_FLAG_SPLIT_F16 | extra, mode=p.VGG19_MODE_FORWARD)
    x = torch.from_numpy(images).to(DEV)
    probs = torch.empty(B, 1000, dtype=torch.float32, device=DEV)
    logits = net.forward(x, probs=probs).clone()
    net.sync_status()
    o = oracle.vgg19_forward(params.astype(np.float64), images)
    e_l, e_p = rel_l2(logits.cpu().numpy(), o), rel_l2(probs.cpu().numpy(), oracle.softmax(o))
    print(f"{H}x{H} batch {B}: split-fp16 forward, logits {e_l:.2e}, probabilities {e_p:.2e}")
    assert e_l <= 3e-5 and e_p <= 3e-5
    assert [int(i) for i in logits.argmax(1)] == [int(i) for i in o.argmax(1)]
    # a second pass (the recorded graph) returns the same bits
    again = net.forward(x)
    net.sync_status()
    assert torch.equal(again, logits)
    net.close()


def test_split_forward_224():
    """Full-size images: four of them, each against the checker."""
    p = pkg()
    B = 4
    params = si.vgg19_params(224, 224, seed=0)
    images = si.images(B, 224, 224, seed=1)
    net = p.Net(224, 224, B, p.VGG19_FP32, params=params, flags=p.VGG19_FLAG_SPLIT_F16, mode=p.VGG19_MODE_FORWARD)
    x = torch.from_numpy(images).to(DEV)
    logits = net.forward(x).clone()
    net.sync_status()
    o = oracle.vgg19_forward(params.astype(np.float64), images)
    errs = [rel_l2(logits[i].cpu().numpy(), o[i]) for i in range(B)]
    print(f"224x224 batch {B}: split-fp16 forward, logits per image {['%.2e' % e for e in errs]}")
    assert max(errs) <= 3e-5
    net.close()


def test_split_reports_an_activation_beyond_fp16_range():
    """A value beyond 65504 cannot be carried as fp16 terms: the pass reports it instead of returning infinities
    silently, and the next pass on ordinary inputs is clean."""
    p = pkg()
    params = si.vgg19_params(32, 32, seed=0)
    net = p.Net(32, 32, 1, p.VGG19_FP32, params=params, flags=p.VGG19_FLAG_SPLIT_F16, mode=p.VGG19_MODE_FORWARD)
    big = torch.full((1, 32, 32, 3), 3.0e6, dtype=torch.float32, device=DEV)  # conv1_1's outputs pass 65504
    net.forward(big)
    with pytest.raises(p.Vgg19Error) as ei:
        net.sync_status()
    assert ei.value.code == p.VGG19_ERR_RANGE
    x = torch.from_numpy(si.images(1, 32, 32, seed=1)).to(DEV)
    logits = net.forward(x)
    net.sync_status()
    assert torch.isfinite(logits).all()
    net.close()


def test_split_network_through_the_host_entry_point_and_beside_a_backward_pass():
    """The host-buffer call runs the same split pass (same bits as the device call); a backward pass of the same
    network keeps the CUDA-core fp32 kernels (the flag covers forward-only passes) and still matches the checker."""
    p = pkg()
    B = 2
    params = si.vgg19_params(32, 32, seed=0, bias_std=0.05)
    images, labels = si.images(B, 32, 32, seed=1), si.labels(B, seed=2)
    net = p.Net(32, 32, B, p.VGG19_FP32, params=params, flags=p.VGG19_FLAG_SPLIT_F16, host_io=True)
    assert "split-fp16" in p.vgg19_describe(net.handle)
    x = torch.from_numpy(images)
    logits_host = torch.empty(B, 1000, dtype=torch.float32).pin_memory()
    s = torch.cuda.Stream()
    p.vgg19_forward_host(net.handle, x.pin_memory(), B, logits_host, None, s)
    dev_logits = net.forward(x.to(DEV)).clone()
    net.sync_status()
    assert torch.equal(dev_logits.cpu(), logits_host)
    bl = torch.empty(B, 1000, dtype=torch.float32, device=DEV)
    grads, loss = net.backward(x.to(DEV), torch.from_numpy(labels).to(DEV), logits=bl)
    net.sync_status()
    o_loss, o_grads, o_logits = oracle.vgg19_backward(params.astype(np.float64), images, labels, chunk=B)
    assert rel_l2(bl.cpu().numpy(), o_logits) <= 1e-4 and rel_l2(dev_logits.cpu().numpy(), o_logits) <= 3e-5
    assert rel_l2(grads.cpu().numpy(), o_grads) <= 2e-4
    assert abs(float(loss) - o_loss) <= 1e-4 * abs(o_loss)
    net.close()


def test_split_flag_needs_fp32():
    p = pkg()
    with pytest.raises(Exception):
        p.Net(32, 32, 1, p.VGG19_BF16, seed=0, flags=p.VGG19_FLAG_SPLIT_F16, mode=p.VGG19_MODE_FORWARD)
