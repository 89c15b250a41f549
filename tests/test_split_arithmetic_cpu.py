"""The arithmetic behind the fp32 configuration's tensor-core path, in numpy (no GPU): a value carried as two fp16
terms keeps 22 bits, three products of the terms stand for the fp32 product to about 2^-21, and why the weights are
scaled by 64 before they are split.  These are the figures the GPU tests' tolerances rest on
(tests/test_gpu_split_fp32.py); the device code is not involved."""
import numpy as np


def split(v):
    v = np.asarray(v, dtype=np.float32)
    hi = v.astype(np.float16)
    lo = (v - hi.astype(np.float32)).astype(np.float16)
    return hi, lo


def test_two_fp16_terms_keep_22_bits_of_values_in_range():
    rng = np.random.default_rng(0)
    v = (rng.standard_normal(200000) * 3.0).astype(np.float32)  # activations of order one
    hi, lo = split(v)
    back = hi.astype(np.float64) + lo.astype(np.float64)
    err = np.abs(back - v.astype(np.float64))
    # 22 bits of the value - or, where the lo term reaches fp16's subnormals (|v| below about 0.25), half of their
    # spacing 2^-24: an absolute 3e-8, nothing beside activations of order one
    assert (err <= np.maximum(2.0 ** -22 * np.abs(v), 2.0 ** -25)).all()
    big = np.abs(v) >= 0.5
    assert (err[big] / np.abs(v[big])).max() <= 2.0 ** -22
    # v - hi is exact in fp32: the first rounding loses nothing that the second term cannot see
    assert np.array_equal((v - hi.astype(np.float32)).astype(np.float64), v.astype(np.float64) - hi.astype(np.float64))


def test_small_weights_need_the_scaling():
    rng = np.random.default_rng(1)
    w = (rng.standard_normal(200000) * 9e-3).astype(np.float32)  # He-normal weights of the first dense layer
    def worst(scale):
        hi, lo = split(w * np.float32(scale))
        back = (hi.astype(np.float64) + lo.astype(np.float64)) / scale
        big = np.abs(w) > 1e-3
        return (np.abs(back - w.astype(np.float64)) / np.abs(w.astype(np.float64)))[big].max()
    assert worst(64.0) <= 2.0 ** -18     # scaled: lo terms are normal numbers (or nearly)
    assert worst(1.0) >= 4 * worst(64.0)  # unscaled: they sink into fp16's subnormals and lose bits


def test_three_products_stand_for_the_fp32_product():
    rng = np.random.default_rng(2)
    K = 4608
    x = np.abs(rng.standard_normal((64, K))).astype(np.float32)
    w = (rng.standard_normal((K, 32)) * 0.02).astype(np.float32)
    xh, xl = split(x)
    wh, wl = split(w * np.float32(64.0))
    f = lambda a: a.astype(np.float64)
    three = (f(xh) @ f(wh) + f(xh) @ f(wl) + f(xl) @ f(wh)) / 64.0   # sums in fp64: the terms alone
    exact = f(x) @ f(w)
    err = np.linalg.norm(three - exact) / np.linalg.norm(exact)
    assert err <= 2e-7   # the split itself is far inside fp32's own rounding of such a sum
    one = (f(xh) @ f(wh)) / 64.0
    assert np.linalg.norm(one - exact) / np.linalg.norm(exact) >= 1e-4  # one fp16 product is not
