"""Per-layer parity of the dense kernels (forward; input, filter and bias gradient) at the three layer shapes of
the 224x224 network, against the fp64 CPU checker fed the same bf16-exact tensors.  Batch 100 (the benchmark's)
for every layer, and 37 rows, a ragged M tile, for layer 1.

Tolerance: as for the convolution layers - fp32 accumulation, bf16 storage of activations and input gradients
(compared with the checker's result rounded to bf16: rare one-ulp flips, bar 1e-3), fp32 filter and bias
gradients unrounded (bar 1e-3)."""
import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# (layer, In, Out, relu, batch)
SHAPES = [(1, 25088, 4096, True, 37), (1, 25088, 4096, True, 100), (2, 4096, 4096, True, 100), (3, 4096, 1000, False, 100)]


def rel_l2(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


@pytest.fixture(scope="module")
def net224():
    import paper_1810_09868_b200 as p
    params = si.vgg19_params(224, 224, seed=0, bias_std=0.1, bf16_exact=True)
    net = p.Net(224, 224, 100, p.VGG19_BF16, params=params)
    yield p, net, params
    net.close()


def layer_params(p, net, params, layer):
    i = 32 + 2 * (layer - 1)  # tensors 0..31 are the convolution layers' weights and biases
    (woff, wdims), (boff, bdims) = p.vgg19_param_info(net.handle, i), p.vgg19_param_info(net.handle, i + 1)
    Wt = params[woff:woff + int(np.prod(wdims))].reshape(wdims).astype(np.float64)
    b = params[boff:boff + int(np.prod(bdims))].astype(np.float64)
    return Wt, b


@pytest.mark.parametrize("layer,In,Out,relu,B", SHAPES)
def test_dense_layer_forward(net224, layer, In, Out, relu, B):
    p, net, params = net224
    x = si.normal(B * In, seed=400 + layer, take_abs=True, bf16_exact=True).reshape(B, In)
    Wt, b = layer_params(p, net, params, layer)
    assert Wt.shape == (Out, In)
    xd = torch.from_numpy(x).to(DEV).to(torch.bfloat16)
    y = torch.full((B, Out), float("nan"), dtype=torch.bfloat16, device=DEV)
    yf = torch.full((B, Out), float("nan"), dtype=torch.float32, device=DEV)
    p.vgg19_dense_layer_forward(net.handle, layer, xd, B, y, yf, torch.cuda.current_stream())
    net.sync_status()
    ref = oracle.dense_fwd(x, Wt, b)
    if relu:
        ref = oracle.relu_fwd(ref)
    assert np.isfinite(yf.cpu().numpy()).all()
    assert rel_l2(yf.cpu().numpy(), ref) <= 1e-3
    assert rel_l2(y.float().cpu().numpy(), oracle.round_bf16(ref)) <= 1e-3
    assert torch.equal(y, yf.to(torch.bfloat16))  # the two outputs are the same values


@pytest.mark.parametrize("layer,In,Out,relu,B", SHAPES)
def test_dense_layer_backward(net224, layer, In, Out, relu, B):
    p, net, params = net224
    x = si.normal(B * In, seed=400 + layer, take_abs=True, bf16_exact=True).reshape(B, In)
    x = x * (si.uniform(x.size, seed=500 + layer).reshape(x.shape) < 0.5)  # a ReLU output: about half zeros
    dy = si.normal(B * Out, seed=600 + layer, stddev=1e-3, bf16_exact=True).reshape(B, Out)
    Wt, _ = layer_params(p, net, params, layer)
    xd = torch.from_numpy(x).to(DEV).to(torch.bfloat16)
    dyd = torch.from_numpy(dy).to(DEV).to(torch.bfloat16)
    dw = torch.full((Out, In), float("nan"), dtype=torch.float32, device=DEV)
    db = torch.full((Out,), float("nan"), dtype=torch.float32, device=DEV)
    dx = torch.full((B, In), float("nan"), dtype=torch.bfloat16, device=DEV)
    # the input of layers 2 and 3 is a ReLU output, whose mask the input gradient applies; layer 1's is a pool output
    mask = xd if layer > 1 else None
    p.vgg19_dense_layer_backward(net.handle, layer, xd, dyd, B, dw, db, dx, mask, torch.cuda.current_stream())
    net.sync_status()
    o_dx, o_dw, o_db = oracle.dense_bwd(x, Wt, dy)
    if layer > 1:
        o_dx = o_dx * (x > 0)
    assert rel_l2(dw.cpu().numpy(), o_dw) <= 1e-3
    assert rel_l2(db.cpu().numpy(), o_db) <= 1e-3
    assert rel_l2(dx.float().cpu().numpy(), oracle.round_bf16(o_dx)) <= 1e-3


def test_dense_layers_fp32_configuration():
    """The fp32 configuration's dense kernels (CUDA cores) through the same entry points, 32x32 network:
    512 -> 4096 -> 4096 -> 1000, bar 1e-5."""
    import paper_1810_09868_b200 as p
    B = 3
    params = si.vgg19_params(32, 32, seed=0, bias_std=0.1)
    net = p.Net(32, 32, B, p.VGG19_FP32, params=params)
    for layer, In, Out, relu in [(1, 512, 4096, True), (2, 4096, 4096, True), (3, 4096, 1000, False)]:
        x = si.normal(B * In, seed=700 + layer, take_abs=True).reshape(B, In).astype(np.float32)
        dy = si.normal(B * Out, seed=800 + layer, stddev=1e-3).reshape(B, Out).astype(np.float32)
        Wt, b = layer_params(p, net, params, layer)
        xd, dyd = torch.from_numpy(x).to(DEV), torch.from_numpy(dy).to(DEV)
        y = torch.full((B, Out), float("nan"), dtype=torch.float32, device=DEV)
        p.vgg19_dense_layer_forward(net.handle, layer, xd, B, y, None, torch.cuda.current_stream())
        dw = torch.full((Out, In), float("nan"), dtype=torch.float32, device=DEV)
        db = torch.full((Out,), float("nan"), dtype=torch.float32, device=DEV)
        dx = torch.full((B, In), float("nan"), dtype=torch.float32, device=DEV)
        p.vgg19_dense_layer_backward(net.handle, layer, xd, dyd, B, dw, db, dx, None, torch.cuda.current_stream())
        net.sync_status()
        ref = oracle.dense_fwd(x.astype(np.float64), Wt, b)
        if relu:
            ref = oracle.relu_fwd(ref)
        o_dx, o_dw, o_db = oracle.dense_bwd(x.astype(np.float64), Wt, dy.astype(np.float64))
        assert rel_l2(y.cpu().numpy(), ref) <= 1e-5
        assert rel_l2(dw.cpu().numpy(), o_dw) <= 1e-5 and rel_l2(db.cpu().numpy(), o_db) <= 1e-5
        assert rel_l2(dx.cpu().numpy(), o_dx) <= 1e-5
    net.close()


def test_dense_layer_arguments():
    import paper_1810_09868_b200 as p
    net = p.Net(32, 32, 2, p.VGG19_BF16, seed=0)
    x = torch.zeros(2, 512, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(p.Vgg19Error) as e:
        p.vgg19_dense_layer_forward(net.handle, 4, x, 2, x, None, torch.cuda.current_stream())
    assert e.value.code == p.VGG19_ERR_ARG
    with pytest.raises(p.Vgg19Error) as e:
        p.vgg19_dense_layer_forward(net.handle, 1, x, 2, None, None, torch.cuda.current_stream())
    assert e.value.code == p.VGG19_ERR_ARG
    net.close()
