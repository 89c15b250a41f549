"""Per-layer parity of the convolution kernels (forward, input gradient, filter
and bias gradient) at the layer shapes of the 224x224 network, on a small
batch, against the fp64 CPU checker fed the same bf16-exact tensors.

Tolerance: the device accumulates in fp32 and stores bf16.  Against the
checker's result rounded to bf16 the only differences are rare one-ulp
rounding flips (relative L2 ~1e-4): bar 1e-3.  fp32 gradient outputs are not
rounded: bar 1e-3 as well (sums of up to ~10^5 bf16 products in fp32).
"""
import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

# (layer, H=W at a 224x224 input, Cin, Cout): the nine distinct shapes
SHAPES = [(1, 224, 3, 64), (2, 224, 64, 64), (3, 112, 64, 128), (4, 112, 128, 128), (5, 56, 128, 256),
          (6, 56, 256, 256), (9, 28, 256, 512), (10, 28, 512, 512), (13, 14, 512, 512)]


def rel_l2(a, b):
    a, b = np.asarray(a, dtype=np.float64), np.asarray(b, dtype=np.float64)
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


@pytest.fixture(scope="module")
def net224():
    import paper_1810_09868_b200 as p
    params = si.vgg19_params(224, 224, seed=0, bias_std=0.1, bf16_exact=True)
    net = p.Net(224, 224, 3, p.VGG19_BF16, params=params)
    yield p, net, params
    net.close()


def layer_params(p, net, params, layer):
    (woff, wdims), (boff, bdims) = p.vgg19_param_info(net.handle, 2 * (layer - 1)), p.vgg19_param_info(net.handle, 2 * layer - 1)
    Wt = params[woff:woff + int(np.prod(wdims))].reshape(wdims).astype(np.float64)
    b = params[boff:boff + int(np.prod(bdims))].astype(np.float64)
    return Wt, b


def layer_input(layer, B, S, Cin):
    if Cin == 3:
        return si.images(B, S, S, seed=1, bf16_exact=True)
    return si.normal(B * S * S * Cin, seed=100 + layer, take_abs=True, bf16_exact=True).reshape(B, S, S, Cin)


@pytest.mark.parametrize("layer,S,Cin,Cout", SHAPES)
def test_conv_layer_forward(net224, layer, S, Cin, Cout):
    p, net, params = net224
    B = 3 if S <= 28 else 1  # 14x14x3 = 588 pixels: a ragged last tile
    x = layer_input(layer, B, S, Cin)
    Wt, b = layer_params(p, net, params, layer)
    xd = torch.from_numpy(x).to(DEV).to(torch.bfloat16)
    y = torch.full((B, S, S, Cout), float("nan"), dtype=torch.bfloat16, device=DEV)
    pooled = torch.full((B, S // 2, S // 2, Cout), float("nan"), dtype=torch.bfloat16, device=DEV)
    p.vgg19_conv_layer_forward(net.handle, layer, xd, B, y, pooled, torch.cuda.current_stream())
    net.sync_status()
    ref = oracle.round_bf16(oracle.relu_fwd(oracle.conv3x3_fwd(x, Wt, b)))
    got = y.float().cpu().numpy()
    assert np.isfinite(got).all()
    assert rel_l2(got, ref) <= 1e-3
    assert np.array_equal(pooled.float().cpu().numpy(), oracle.maxpool2x2_fwd(got))


@pytest.mark.parametrize("layer,S,Cin,Cout", SHAPES)
def test_conv_layer_backward(net224, layer, S, Cin, Cout):
    p, net, params = net224
    B = 3 if S <= 28 else 1
    x = layer_input(layer, B, S, Cin)
    # a ReLU-masked upstream gradient: about half the entries are exactly zero
    dz = si.normal(B * S * S * Cout, seed=200 + layer, stddev=1e-3, bf16_exact=True).reshape(B, S, S, Cout)
    dz = dz * (si.uniform(dz.size, seed=300 + layer).reshape(dz.shape) < 0.5)
    Wt, _ = layer_params(p, net, params, layer)
    xd = torch.from_numpy(x).to(DEV).to(torch.bfloat16)
    dzd = torch.from_numpy(dz).to(DEV).to(torch.bfloat16)
    dw = torch.full((Cout, 3, 3, Cin), float("nan"), dtype=torch.float32, device=DEV)
    db = torch.full((Cout,), float("nan"), dtype=torch.float32, device=DEV)
    dx = None if layer == 1 else torch.full((B, S, S, Cin), float("nan"), dtype=torch.bfloat16, device=DEV)
    p.vgg19_conv_layer_backward(net.handle, layer, xd, dzd, B, dw, db, dx, torch.cuda.current_stream())
    net.sync_status()
    o_dw, o_db = oracle.conv3x3_wgrad(x, dz)
    assert rel_l2(dw.cpu().numpy(), o_dw) <= 1e-3
    assert rel_l2(db.cpu().numpy(), o_db) <= 1e-3
    if dx is not None:
        ref = oracle.round_bf16(oracle.conv3x3_dgrad(dz, Wt))
        assert rel_l2(dx.float().cpu().numpy(), ref) <= 1e-3


@pytest.mark.parametrize("layer,S,Cin,Cout", [(13, 14, 512, 512), (9, 28, 256, 512)])
def test_conv_layer_tail_round_batch100(layer, S, Cin, Cout):
    """At batch 100 the tile count of these layers leaves a last round of CTA pairs less than half full;
    where that saves enough (layer 13 forward and input gradient, layer 9 input gradient) its tiles
    are cut along K over all pairs and summed by a second kernel.  The images in those tiles (the
    last of the batch) and a few from whole rounds are checked against the checker, forward and
    input gradient, and the whole batch against the one-CTA-per-tile kernels."""
    import paper_1810_09868_b200 as p
    B = 100
    params = si.vgg19_params(224, 224, seed=0, bias_std=0.1, bf16_exact=True)
    x = layer_input(layer, B, S, Cin)
    dz = si.normal(B * S * S * Cout, seed=200 + layer, stddev=1e-3, bf16_exact=True).reshape(B, S, S, Cout)
    xd = torch.from_numpy(x).to(DEV).to(torch.bfloat16)
    dzd = torch.from_numpy(dz).to(DEV).to(torch.bfloat16)
    sample = [0, 50, 96, 97, 98, 99]
    outs = {}
    for flags in (0, p.binding.VGG19_FLAG_NO_CTA_PAIRS):
        net = p.Net(224, 224, B, p.VGG19_BF16, params=params, flags=flags)
        y = torch.full((B, S, S, Cout), float("nan"), dtype=torch.bfloat16, device=DEV)
        dx = torch.full((B, S, S, Cin), float("nan"), dtype=torch.bfloat16, device=DEV)
        dw = torch.empty((Cout, 3, 3, Cin), dtype=torch.float32, device=DEV)
        db = torch.empty((Cout,), dtype=torch.float32, device=DEV)
        p.vgg19_conv_layer_forward(net.handle, layer, xd, B, y, None, torch.cuda.current_stream())
        p.vgg19_conv_layer_backward(net.handle, layer, xd, dzd, B, dw, db, dx, torch.cuda.current_stream())
        net.sync_status()
        outs[flags] = (y.float().cpu().numpy(), dx.float().cpu().numpy())
        Wt, b = layer_params(p, net, params, layer)
        net.close()
    y, dx = outs[0]
    assert np.isfinite(y).all() and np.isfinite(dx).all()
    ref_y = oracle.round_bf16(oracle.relu_fwd(oracle.conv3x3_fwd(x[sample], Wt, b)))
    ref_dx = oracle.round_bf16(oracle.conv3x3_dgrad(dz[sample], Wt))
    for row, i in enumerate(sample):
        assert rel_l2(y[i], ref_y[row]) <= 1e-3, i
        assert rel_l2(dx[i], ref_dx[row]) <= 1e-3, i
    # against the single-CTA kernels over the whole batch: rare one-ulp rounding flips only
    assert rel_l2(y, outs[p.binding.VGG19_FLAG_NO_CTA_PAIRS][0]) <= 1e-3
    assert rel_l2(dx, outs[p.binding.VGG19_FLAG_NO_CTA_PAIRS][1]) <= 1e-3


def expected_pool_codes(y):
    """Arg-max code of every 2x2 window of an NHWC activation: 0..3 in the order (0,0), (0,1), (1,0), (1,1),
    the first maximum on ties; 4 where the maximum is not positive."""
    N, H, W, C = y.shape
    w = y.reshape(N, H // 2, 2, W // 2, 2, C).transpose(0, 1, 3, 5, 2, 4).reshape(N, H // 2, W // 2, C, 4)
    code = np.argmax(w, axis=-1).astype(np.uint8)
    code[w.max(axis=-1) <= 0] = 4
    return code


# (layer that ends a block, the layer above the pool or None, H=W of the block-ending layer, its Cin, Cout)
POOLS = [(2, 3, 224, 64, 64), (4, 5, 112, 128, 128), (8, 9, 56, 256, 256), (12, 13, 28, 512, 512), (16, None, 14, 512, 512)]


@pytest.mark.parametrize("below,above,S,Cin,Cout", POOLS)
def test_pool_codes_and_scatter_through_the_pool(net224, below, above, S, Cin, Cout):
    """The block-ending layers record, with the pooled tensor, where each window's maximum sat; the input
    gradient of the layer above the pool is scattered through the pool by those codes (in the kernel's own
    epilogue at the 224x224 and 112x112 blocks).  Codes: against the arg-max of the stored activation.
    Scatter: against the checker's max-pool backward and ReLU backward at that stored activation."""
    p, net, params = net224
    B = 3 if S <= 28 else 1
    x = layer_input(below, B, S, Cin)
    xd = torch.from_numpy(x).to(DEV).to(torch.bfloat16)
    y = torch.empty((B, S, S, Cout), dtype=torch.bfloat16, device=DEV)
    pooled = torch.empty((B, S // 2, S // 2, Cout), dtype=torch.bfloat16, device=DEV)
    code = torch.full((B, S // 2, S // 2, Cout), 255, dtype=torch.uint8, device=DEV)
    st = torch.cuda.current_stream()
    p.vgg19_conv_layer_forward_ex(net.handle, below, xd, B, y, pooled, code, st)
    net.sync_status()
    y_host = y.float().cpu().numpy().astype(np.float64)
    want = expected_pool_codes(y_host)
    got = code.cpu().numpy()
    assert np.array_equal(got, want), f"{(got != want).sum()} of {want.size} codes differ"
    assert (want == 4).any() and all((want == q).any() for q in range(4))
    assert np.array_equal(pooled.float().cpu().numpy(), oracle.maxpool2x2_fwd(y_host))
    if above is None:
        return
    C2 = SHAPES_BY_LAYER[above][2]
    dz = si.normal(B * (S // 2) ** 2 * C2, seed=400 + above, stddev=1e-3, bf16_exact=True).reshape(B, S // 2, S // 2, C2)
    dz = dz * (si.uniform(dz.size, seed=500 + above).reshape(dz.shape) < 0.5)
    dzd = torch.from_numpy(dz).to(DEV).to(torch.bfloat16)
    dfull = torch.full((B, S, S, Cout), float("nan"), dtype=torch.bfloat16, device=DEV)
    p.vgg19_conv_layer_backward_ex(net.handle, above, None, dzd, B, None, None, dfull, None, code, st)
    net.sync_status()
    Wt, _ = layer_params(p, net, params, above)
    low = oracle.round_bf16(oracle.conv3x3_dgrad(dz, Wt))
    ref = oracle.relu_bwd(y_host, oracle.maxpool2x2_bwd(y_host, low))
    g = dfull.float().cpu().numpy()
    assert np.isfinite(g).all()
    assert np.array_equal(g != 0, ref != 0) or rel_l2(g, ref) <= 1e-3
    assert rel_l2(g, ref) <= 1e-3


SHAPES_BY_LAYER = {3: (112, 64, 128), 5: (56, 128, 256), 9: (28, 256, 512), 13: (14, 512, 512)}


@pytest.mark.parametrize("layer,S,Cin,Cout", [(2, 224, 64, 64), (4, 112, 128, 128), (8, 56, 256, 256), (12, 28, 512, 512),
                                              (16, 14, 512, 512)])
def test_block_ending_layers_pool_in_their_epilogue(net224, layer, S, Cin, Cout):
    """Forward-only passes never write the full-resolution output of a block-ending layer: the pooled tensor
    comes out of the convolution's own epilogue (shuffles inside a patch tile at 224x224 and 112x112, a
    max-reduction on global memory at 56x56 and below).  It must equal, bit for bit, the 2x2 max-pool of the
    full-resolution output the same layer writes when asked for it."""
    p, net, params = net224
    B = 3
    x = layer_input(layer, B, S, Cin)
    xd = torch.from_numpy(x).to(DEV).to(torch.bfloat16)
    y = torch.empty((B, S, S, Cout), dtype=torch.bfloat16, device=DEV)
    st = torch.cuda.current_stream()
    p.vgg19_conv_layer_forward(net.handle, layer, xd, B, y, None, st)
    for rep in range(2):
        pooled = torch.full((B, S // 2, S // 2, Cout), float("nan"), dtype=torch.bfloat16, device=DEV)
        p.vgg19_conv_layer_forward_ex(net.handle, layer, xd, B, None, pooled, None, st)
        net.sync_status()
        want = torch.nn.functional.max_pool2d(y.float().permute(0, 3, 1, 2), 2).permute(0, 2, 3, 1)
        assert torch.equal(pooled.float(), want), rep
    Wt, b = layer_params(p, net, params, layer)
    ref = oracle.maxpool2x2_fwd(oracle.round_bf16(oracle.relu_fwd(oracle.conv3x3_fwd(x[:1], Wt, b))))
    assert rel_l2(pooled[:1].float().cpu().numpy(), ref) <= 1e-3


def test_first_block_as_one_kernel(net224):
    """conv1_1 -> conv1_2 (-> pool) in one kernel that never stores conv1_1's activation (what a forward-only
    pass runs): against the checker's two convolutions with the bf16 store between them, and against the two
    separate kernels."""
    p, net, params = net224
    B = 3
    x = si.images(B, 224, 224, seed=1, bf16_exact=True)
    xd = torch.from_numpy(x).to(DEV).to(torch.bfloat16)
    st = torch.cuda.current_stream()
    y2 = torch.full((B, 224, 224, 64), float("nan"), dtype=torch.bfloat16, device=DEV)
    pooled = torch.full((B, 112, 112, 64), float("nan"), dtype=torch.bfloat16, device=DEV)
    p.vgg19_first_block_forward(net.handle, xd, B, y2, pooled, st)
    pooled_only = torch.full((B, 112, 112, 64), float("nan"), dtype=torch.bfloat16, device=DEV)
    p.vgg19_first_block_forward(net.handle, xd, B, None, pooled_only, st)
    net.sync_status()
    # the two separate kernels
    y1 = torch.empty((B, 224, 224, 64), dtype=torch.bfloat16, device=DEV)
    y2_two = torch.empty_like(y2)
    p.vgg19_conv_layer_forward(net.handle, 1, xd, B, y1, None, st)
    p.vgg19_conv_layer_forward(net.handle, 2, y1, B, y2_two, None, st)
    net.sync_status()
    assert torch.isfinite(y2.float()).all()
    same = torch.equal(y2, y2_two)
    print(f"fused first block vs two kernels: {'bit-identical' if same else 'rel-L2 %.2e' % rel_l2(y2.float().cpu().numpy(), y2_two.float().cpu().numpy())}")
    assert same or rel_l2(y2.float().cpu().numpy(), y2_two.float().cpu().numpy()) <= 1e-3
    want_pool = torch.nn.functional.max_pool2d(y2.float().permute(0, 3, 1, 2), 2).permute(0, 2, 3, 1)
    assert torch.equal(pooled.float(), want_pool) and torch.equal(pooled_only, pooled)
    # the checker, on one image (edges and corners of the image included)
    W1, b1 = layer_params(p, net, params, 1)
    W2, b2 = layer_params(p, net, params, 2)
    r1 = oracle.round_bf16(oracle.relu_fwd(oracle.conv3x3_fwd(x[:1], W1, b1)))
    r2 = oracle.round_bf16(oracle.relu_fwd(oracle.conv3x3_fwd(r1, W2, b2)))
    got = y2[:1].float().cpu().numpy()
    assert rel_l2(got, r2) <= 1e-3
    for sl in (np.s_[0, 0, :, :], np.s_[0, -1, :, :], np.s_[0, :, 0, :], np.s_[0, :, -1, :]):
        assert rel_l2(got[sl], r2[sl]) <= 2e-3


def test_forward_pass_with_the_fused_first_block_is_bit_identical(net224):
    """A network created with VGG19_FLAG_FIRST_FUSION runs layers 1 and 2 of a forward-only pass as the one fused
    kernel; the logits must equal, bit for bit, those of the default schedule."""
    p, net, params = net224
    B = 2
    xd = torch.from_numpy(si.images(B, 224, 224, seed=7, bf16_exact=True)).to(DEV).to(torch.bfloat16)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        want = net.forward(xd, stream=s).clone()
    net.sync_status(s)
    fused = p.Net(224, 224, B, p.VGG19_BF16, params=params, flags=p.VGG19_FLAG_FIRST_FUSION, mode=p.VGG19_MODE_FORWARD)
    with torch.cuda.stream(s):
        got = fused.forward(xd, stream=s).clone()
    fused.sync_status(s)
    assert p.vgg19_launch_count(fused.handle, p.VGG19_MODE_FORWARD) == p.vgg19_launch_count(net.handle, p.VGG19_MODE_FORWARD) - 1
    assert torch.equal(got, want)
    fused.close()
