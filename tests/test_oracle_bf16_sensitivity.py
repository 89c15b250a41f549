"""Why bf16 gradients are compared at a given forward state: a measurement made
with the CPU checker alone.

The ReLU masks and the pool arg-maxima of the backward pass (section 7.3) are
integer decisions taken on floating-point values.  With bf16 storage of the
activations, a perturbation of the weights by one part in 10^7 - far below
anything two correct implementations can agree to - is re-amplified to a whole
bf16 ulp at each of the 18 stored layers, flips near-zero pre-activations and
near-tied pooling windows, and each flip switches a whole gradient path on or
off.  In fp64 the same perturbation moves every gradient tensor by ~1e-7.  So
no implementation with bf16 storage can agree with another one to 2e-2 per
gradient tensor when each takes its own decisions; the GPU tests therefore
compare gradients where they are unique (given the stored forward state) and
bound the free-running difference by direction (cosine), not by 2e-2.
"""
import numpy as np

import oracle
import seeded_inputs as si

H = W = 32
B = 5


def per_tensor(flat, shapes):
    out, off = [], 0
    for ws, bs in shapes:
        for s in (ws, bs):
            n = int(np.prod(s))
            out.append(flat[off:off + n])
            off += n
    assert off == flat.size
    return out


def test_a_1e7_weight_perturbation_moves_bf16_storage_gradients_by_percents_but_fp64_ones_not_at_all():
    params = si.vgg19_params(H, W, seed=0, bias_std=0.05, bf16_exact=True).astype(np.float64)
    images = si.images(B, H, W, seed=1, bf16_exact=True)
    labels = si.labels(B, seed=2)
    steps = oracle.vgg19_steps()
    shapes = oracle.param_shapes(steps, H, W, 3)
    noise = np.random.default_rng(0).standard_normal(params.size)
    perturbed = params * (1.0 + 1e-7 * noise)
    moved = {}
    for storage in (None, "bf16"):
        _, g0, _ = oracle.backward(steps, params, images, labels, storage=storage)
        _, g1, _ = oracle.backward(steps, perturbed, images, labels, storage=storage)
        a, b = per_tensor(g0, shapes), per_tensor(g1, shapes)
        rel = [float(np.linalg.norm(u - v) / np.linalg.norm(u)) for u, v in zip(a, b)]
        cos = [float(u @ v / (np.linalg.norm(u) * np.linalg.norm(v))) for u, v in zip(a, b)]
        moved[storage] = (max(rel), float(np.linalg.norm(g0 - g1) / np.linalg.norm(g0)), min(cos))
    # fp64 throughout: the gradient is a smooth function of the weights away from kinks
    assert moved[None][0] < 1e-5
    # bf16 storage: some gradient tensor moves by more than 5 % (measured 21 %), the whole gradient by
    # more than 2e-2 (measured 13 %): the 2e-2 bar cannot hold between two free-running implementations
    assert moved["bf16"][0] > 5e-2
    assert moved["bf16"][1] > 2e-2
    # ... yet the direction of every tensor survives (measured 0.978): that is what can be asserted of a
    # free-running comparison
    assert moved["bf16"][2] > 0.95
