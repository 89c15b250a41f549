"""Parity at the full sizes the benchmark runs: 224x224x3, bf16, batch 1 and
batch 100, in the launch configuration bench.py times (one CUDA graph per
pass, tensor-core kernels).

The fp64 CPU checker needs ~2 s per image forward and ~4 s forward+backward,
so at batch 100 it is applied to sampled images; the rest of the batch is
covered by properties that hold at any size:
  * an image's logits do not depend on which batch it sits in (bit for bit:
    the per-pixel accumulation order does not depend on the batch; the last
    few images of the batch, whose tiles are cut along K to fill the last
    round of CTAs, agree to fp32 rounding order instead);
  * the batch-100 gradient is the mean of the gradients of its ten batch-10
    chunks (the loss is a mean over images);
and the gradient of a sampled chunk is checked against the checker's backward
pass at the forward state the device stored.
Tolerances as in test_gpu_parity.py: 2e-2 relative L2 (bf16 storage, fp32 sums).
"""
import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si
from test_gpu_parity import check_bf16_backward, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
H = W = 224
B = 100


@pytest.fixture(scope="module")
def full():
    import paper_1810_09868_b200 as p
    params = si.vgg19_params(H, W, seed=0, bf16_exact=True)
    images = si.images(B, H, W, seed=1, bf16_exact=True)
    labels = si.labels(B, seed=2)
    net = p.Net(H, W, B, p.VGG19_BF16, params=params)
    x = torch.from_numpy(images).to(DEV).to(torch.bfloat16)
    y = torch.from_numpy(labels).to(DEV)
    yield p, net, params, images, labels, x, y
    net.close()


def top1_agrees(gpu_row, ref_row, bound):
    """Same arg-max, or the checker's margin between the two candidates is within the error bound."""
    g, r = int(np.argmax(gpu_row)), int(np.argmax(ref_row))
    return g == r or abs(ref_row[r] - ref_row[g]) < 2 * bound


def test_config3_forward_batch1(full):
    p, net, params, images, labels, x, y = full
    probs = torch.empty(1, 1000, dtype=torch.float32, device=DEV)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        logits = net.forward(x[:1], probs=probs, stream=s)
    net.sync_status(s)
    p64 = params.astype(np.float64)
    ref = oracle.vgg19_forward(p64, images[:1])
    ref_s = oracle.vgg19_forward(p64, images[:1], storage="bf16")
    got = logits.cpu().numpy()
    assert rel_l2(got, ref) <= 2e-2 and rel_l2(got, ref_s) <= 2e-2
    bound = 2e-2 * np.sqrt(np.mean(ref ** 2))
    assert top1_agrees(got[0], ref[0], bound)
    pr = probs.cpu().numpy()
    assert abs(pr.sum() - 1.0) < 1e-4
    # the softmax of logits this large amplifies a logit error of d into a relative error of ~d
    # in each probability: compare the probabilities the device printed with those of ITS logits
    assert rel_l2(pr, oracle.softmax(got)) <= 1e-4
    print(f"config 3: logits rel-L2 {rel_l2(got, ref):.2e} (unrounded checker), {rel_l2(got, ref_s):.2e} (bf16 storage)")


def test_config4_forward_batch100(full):
    p, net, params, images, labels, x, y = full
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        logits = net.forward(x, stream=s).clone()
    net.sync_status(s)
    got = logits.cpu().numpy()
    assert np.isfinite(got).all()
    p64 = params.astype(np.float64)
    sample = [0, 37, 63, 99]
    ref = oracle.vgg19_forward(p64, images[sample])
    bound = 2e-2 * np.sqrt(np.mean(ref ** 2))
    agree = 0
    for row, i in enumerate(sample):
        assert rel_l2(got[i], ref[row]) <= 2e-2, i
        agree += top1_agrees(got[i], ref[row], bound)
        with torch.cuda.stream(s):
            single = net.forward(x[i:i + 1], stream=s).clone()
        net.sync_status(s)
        if i < 90:
            assert torch.equal(single[0], logits[i]), f"image {i}: logits depend on the batch it sits in"
        else:
            # the last images of a batch of 100 fall into the tail round of the 28x28 and 14x14 layers,
            # whose tiles are summed over K in several pieces: same sums, another fp32 rounding order.
            # Each bf16 store then turns a last-bit difference into a whole bf16 ulp for some elements,
            # so after eight such layers the two results differ like two bf16 implementations do
            # (both are within 2e-2 of the checker, asserted above): bar 1e-2.
            assert rel_l2(single[0].cpu().numpy(), got[i]) <= 1e-2, i
    assert agree == len(sample)
    print(f"config 4: sampled images {sample}, worst logits rel-L2 "
          f"{max(rel_l2(got[i], ref[r]) for r, i in enumerate(sample)):.2e}, top-1 agreement {agree}/{len(sample)}")


def test_config5_backward_batch100(full):
    p, net, params, images, labels, x, y = full
    s = torch.cuda.Stream()
    grads = torch.empty(net.n_params, dtype=torch.float32, device=DEV)
    loss = torch.empty(1, dtype=torch.float32, device=DEV)
    logits = torch.empty(B, 1000, dtype=torch.float32, device=DEV)
    with torch.cuda.stream(s):
        net.backward(x, y, grads=grads, loss=loss, logits=logits, stream=s)
    net.sync_status(s)
    assert torch.isfinite(grads).all()
    # property: mean of the ten batch-10 chunk gradients
    mean = torch.zeros_like(grads)
    mean_loss = 0.0
    g10 = torch.empty_like(grads)
    l10 = torch.empty(1, dtype=torch.float32, device=DEV)
    for c in range(10):
        with torch.cuda.stream(s):
            net.backward(x[10 * c:10 * c + 10], y[10 * c:10 * c + 10], grads=g10, loss=l10, stream=s)
        net.sync_status(s)
        mean += g10 / 10
        mean_loss += float(l10) / 10
    assert abs(float(loss) - mean_loss) <= 1e-4 * abs(mean_loss)
    worst = 0.0
    for off, dims in net.param_slices():
        n = int(np.prod(dims))
        a, b = grads[off:off + n].double(), mean[off:off + n].double()
        e = float((a - b).norm() / b.norm())
        worst = max(worst, e)
        assert e <= 2e-2, (dims, e)
    print(f"config 5: batch-100 gradient vs mean of batch-10 chunk gradients, worst tensor {worst:.2e}")
    # sampled chunk against the checker at the stored forward state
    n_s = 2
    lg = torch.empty(n_s, 1000, dtype=torch.float32, device=DEV)
    with torch.cuda.stream(s):
        net.backward(x[:n_s], y[:n_s], grads=g10, loss=l10, logits=lg, stream=s)
    net.sync_status(s)
    check_bf16_backward(net, params, images[:n_s], labels[:n_s], lg.cpu().numpy(), g10.cpu().numpy(), float(l10))
