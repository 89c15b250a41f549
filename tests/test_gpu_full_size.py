"""Parity at the full sizes the benchmark runs: 224x224x3, bf16, batch 1 and
batch 100, in the launch configuration bench.py times (one CUDA graph per
pass, tensor-core kernels).

The fp64 CPU checker runs on the whole batch (about a third of a second per
image forward and a second and a half backward on a 16-core host):
  * forward: the logits of all 100 images against the checker's, per image,
    with the strict and the near-tie-aware top-1 agreement counted over all
    100; and an image's logits do not depend on which batch it sits in (bit
    for bit: the per-pixel accumulation order does not depend on the batch;
    the last few images of the batch, whose tiles are cut along K to fill the
    last round of CTAs, agree to fp32 rounding order instead);
  * backward: the batch-100 gradient against the checker's backward pass over
    all 100 images at the forward state the device stored for that very pass
    (read back chunk by chunk from the workspace, tail images included); the
    decisions taken on that state against the checker's own on sampled images;
    the batch-100 gradient is the mean of its ten batch-10 chunk gradients.
Tolerances as in test_gpu_parity.py: 2e-2 relative L2 (bf16 storage, fp32 sums).
"""
import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si
from test_gpu_parity import check_bf16_backward, check_decisions, free_running_cosines, rel_l2, FREE_COSINE_MIN

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
    assert int(np.argmax(got[0])) == int(np.argmax(ref[0]))
    pr = probs.cpu().numpy()
    assert abs(pr.sum() - 1.0) < 1e-4
    # the softmax of logits this large amplifies a logit error of d into a relative error of ~d
    # in each probability: compare the probabilities the device printed with those of ITS logits
    assert rel_l2(pr, oracle.softmax(got)) <= 1e-4
    print(f"config 3: logits rel-L2 {rel_l2(got, ref):.2e} (unrounded checker), {rel_l2(got, ref_s):.2e} (bf16 storage)")


def test_config4_forward_batch100_every_image(full):
    p, net, params, images, labels, x, y = full
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        logits = net.forward(x, stream=s).clone()
    net.sync_status(s)
    got = logits.cpu().numpy()
    assert np.isfinite(got).all()
    p64 = params.astype(np.float64)
    ref = np.concatenate([oracle.vgg19_forward(p64, images[i:i + 10]) for i in range(0, B, 10)])
    errs = np.array([rel_l2(got[i], ref[i]) for i in range(B)])
    assert errs.max() <= 2e-2, (int(errs.argmax()), float(errs.max()))
    assert rel_l2(got, ref) <= 2e-2
    # top-1.  These are random weights on noise images: the logits of an image are nearly tied (the
    # checker's margin between its best two classes is often below the 2e-2 error bound on a logit), so
    # the arg-max of several images is decided by rounding.  Counted three ways: strict agreement with
    # the fp64 checker; agreement when a differing arg-max is excused by a checker margin between the
    # two candidates below twice the 2e-2 bound on a logit (both answers are then correct) - this is
    # the reading under which the 99 % bar is asserted; and, as the yardstick for the strict count, how
    # often the checker's own bf16-storage model agrees strictly with its fp64 self.
    bound = 2e-2 * np.sqrt(np.mean(ref ** 2))
    ref_s = np.concatenate([oracle.vgg19_forward(p64, images[i:i + 10], storage="bf16") for i in range(0, B, 10)])
    strict = sum(int(np.argmax(got[i])) == int(np.argmax(ref[i])) for i in range(B))
    excused = sum(top1_agrees(got[i], ref[i], bound) for i in range(B))
    model_strict = sum(int(np.argmax(ref_s[i])) == int(np.argmax(ref[i])) for i in range(B))
    vs_model = sum(int(np.argmax(got[i])) == int(np.argmax(ref_s[i])) for i in range(B))
    margins = [float(abs(ref[i][int(np.argmax(ref[i]))] - ref[i][int(np.argmax(got[i]))]) / bound)
               for i in range(B) if int(np.argmax(got[i])) != int(np.argmax(ref[i]))]
    print(f"config 4: all {B} images, logits rel-L2 worst {errs.max():.2e} median {np.median(errs):.2e}; top-1 strict "
          f"{strict}/{B} (the checker's bf16-storage model against its fp64 self: {model_strict}/{B}; device against "
          f"that model: {vs_model}/{B}), near-ties excused {excused}/{B}; checker margins of the strict "
          f"disagreements, in units of the logit error bound: {[round(m, 2) for m in margins]}")
    assert excused >= 99
    assert strict >= 90 and strict >= model_strict - 3
    assert rel_l2(got, ref_s) <= 2e-2
    # an image's result does not depend on the batch it sits in
    worst_tail = 0.0
    for i in range(B):
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
            e = rel_l2(single[0].cpu().numpy(), got[i])
            worst_tail = max(worst_tail, e)
            assert e <= 1e-2, i
    print(f"config 4: batch-1 logits equal the batch-100 ones bit for bit for images 0..89, tail images within {worst_tail:.2e}")


def stored_state_chunk(p, net, images, logits, lo, hi):
    """The checker's (logits, saved) for images lo..hi-1 of the batch-100 pass, from what the device stored."""
    steps = oracle.vgg19_steps()
    outs, ci, pi, fi = [], 0, 0, 0
    for st in steps:
        if st[0] == "conv":
            idx = ci; ci += 1
        elif st[0] == "pool":
            idx = 16 + pi; pi += 1
        else:
            idx = 21 + fi; fi += 1
        if idx <= 22:
            t = net.saved_tensor(B, p.VGG19_MODE_BACKWARD, idx)[lo:hi].float().cpu().numpy().astype(np.float64)
            outs.append(t.reshape(hi - lo, 4096) if idx >= 21 else t)
        else:
            outs.append(np.asarray(logits[lo:hi], dtype=np.float64))
    return oracle.state_from_outputs(steps, images[lo:hi], outs)


def test_config5_backward_batch100_every_image(full):
    p, net, params, images, labels, x, y = full
    s = torch.cuda.Stream()
    grads = torch.empty(net.n_params, dtype=torch.float32, device=DEV)
    loss = torch.empty(1, dtype=torch.float32, device=DEV)
    logits = torch.empty(B, 1000, dtype=torch.float32, device=DEV)
    with torch.cuda.stream(s):
        net.backward(x, y, grads=grads, loss=loss, logits=logits, stream=s)
    net.sync_status(s)
    assert torch.isfinite(grads).all()
    got_logits = logits.cpu().numpy()
    # the checker differentiates the network, image chunk by image chunk, at the forward state this very
    # batch-100 pass stored (tail images included), and the chunk gradients add up to the batch gradient
    steps = oracle.vgg19_steps()
    p64 = params.astype(np.float64)
    o_grads = np.zeros(p64.size)
    o_loss = 0.0
    decisions_checked = []
    for lo in range(0, B, 4):
        state = stored_state_chunk(p, net, images, got_logits, lo, lo + 4)
        if lo in (0, 48, 96):
            # sampled chunks (start, middle, tail): the device's decisions against the checker's own, and
            # its stored activations against the checker's
            o_logits, o_saved = oracle.forward(steps, p64, images[lo:lo + 4], keep=True, storage="bf16")
            assert rel_l2(got_logits[lo:lo + 4], o_logits) <= 2e-2
            for sd, so in zip(state[1], o_saved):
                if sd[0] in ("conv", "fc"):
                    assert rel_l2(sd[2], so[2]) <= 2e-2, (lo, sd[0])
            decisions_checked.append(check_decisions(state[1], o_saved))
        l, _, _ = oracle.backward(steps, p64, images[lo:lo + 4], labels[lo:lo + 4], n_total=B, grads=o_grads,
                                  storage="bf16", state=state)
        o_loss += l
    assert abs(float(loss) - o_loss) <= 1e-3 * abs(o_loss)
    g = grads.cpu().numpy()
    worst = 0.0
    for off, dims in net.param_slices():
        n = int(np.prod(dims))
        e = rel_l2(g[off:off + n], o_grads[off:off + n])
        worst = max(worst, e)
        assert e <= 2e-2, (dims, e)
    rows = [r for d in decisions_checked for r in d]
    print(f"config 5: batch-100 gradient against the checker over all {B} images at the stored state, worst tensor "
          f"{worst:.2e}; loss {float(loss):.5f} vs {o_loss:.5f}; decisions on images 0-3, 48-51, 96-99: masks differ <= "
          f"{max(f for k, f, _ in rows if k != 'pool'):.2e}, pools <= {max(f for k, f, _ in rows if k == 'pool'):.2e}, "
          f"worst near-tie {max(w for _, _, w in rows):.2e} of rms")
    del o_grads
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
    # free-running: the device's gradient of a batch of 8 (the first and the last four images) against the
    # checker's own pass on them, each side at its own forward state: direction of every tensor
    pick = [0, 1, 2, 3, 96, 97, 98, 99]
    with torch.cuda.stream(s):
        net.backward(x[pick].contiguous(), y[pick].contiguous(), grads=g10, loss=l10, stream=s)
    net.sync_status(s)
    _, own, _ = oracle.vgg19_backward(p64, images[pick], labels[pick], chunk=4, storage="bf16")
    cos = free_running_cosines(net, g10.cpu().numpy(), own)
    print(f"config 5: free-running gradient of 8 images, smallest per-tensor cosine {min(cos):.4f}")
    assert min(cos) >= FREE_COSINE_MIN, cos
