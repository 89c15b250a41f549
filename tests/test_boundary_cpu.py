"""Host-side checks that need no GPU: the library loads, exports every entry
point the header declares, and rejects bad configurations before touching CUDA."""
import ctypes
import os
import re

import numpy as np
import pytest

import seeded_inputs as si

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def p():
    import __graft_entry__ as g
    g.build()
    import paper_1810_09868_b200 as pkg
    return pkg


def test_library_exports_every_declared_symbol(p):
    header = open(os.path.join(ROOT, "include", "vgg19_b200.h")).read()
    body = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(vgg19_[a-z_0-9]+)\s*\(", body))
    assert len(declared) >= 20
    lib = p.binding.load()
    missing = [n for n in sorted(declared) if not hasattr(lib, n)]
    assert not missing, missing
    assert declared == set(p.binding.EXPORTS)


def test_bad_configurations_are_rejected_without_a_device(p):
    lib = p.binding.load()
    out = ctypes.c_void_p()
    for (h, w, b, d), code in [((30, 32, 1, 0), p.VGG19_ERR_SHAPE), ((32, 0, 1, 0), p.VGG19_ERR_SHAPE),
                               ((32, 32, 0, 0), p.VGG19_ERR_ARG), ((32, 32, 1, 7), p.VGG19_ERR_ARG)]:
        cfg = p.binding.vgg19_config(h, w, b, d, 0)
        assert lib.vgg19_create(ctypes.byref(cfg), 0, ctypes.byref(out)) == code
        assert out.value is None and p.vgg19_last_error()
    assert lib.vgg19_create(None, 0, ctypes.byref(out)) == p.VGG19_ERR_ARG
    cfg = p.binding.vgg19_config(32, 32, 1, 0, 0)
    assert lib.vgg19_create_from_params(ctypes.byref(cfg), None, ctypes.byref(out)) == p.VGG19_ERR_ARG
    assert lib.vgg19_forward(None, None, 1, None, None, None) == p.VGG19_ERR_ARG
    assert lib.vgg19_workspace_bytes(None, 1, 0) == 0
    lib.vgg19_destroy(None)


def test_seeded_generator_is_reproducible_and_well_distributed():
    a = si.normal(200000, seed=3, stream=1, stddev=2.0)
    assert np.array_equal(a, si.normal(200000, seed=3, stream=1, stddev=2.0))
    assert not np.array_equal(a, si.normal(200000, seed=3, stream=2, stddev=2.0))
    assert abs(a.mean()) < 0.02 and abs(a.std() - 2.0) < 0.02
    u = si.uniform(200000, seed=1)
    assert 0.0 <= u.min() and u.max() < 1.0 and abs(u.mean() - 0.5) < 0.005
    # a prefix of a longer draw is the shorter draw (counter based)
    assert np.array_equal(si.uniform(1000, seed=1), u[:1000])
    lab = si.labels(5000, seed=2)
    assert lab.min() >= 0 and lab.max() < 1000 and len(np.unique(lab)) > 900
    img = si.images(2, 32, 32, seed=1)
    assert img.shape == (2, 32, 32, 3) and -2.0 <= img.min() and img.max() < 2.0
    b = si.normal(1000, seed=3, bf16_exact=True)
    assert np.all((b.view(np.uint32) & 0xFFFF) == 0)
    import torch
    ref = torch.from_numpy(si.normal(1000, seed=3)).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(b, ref)


def test_parameter_layout():
    assert si.vgg19_param_count(224, 224) == 143667240
    assert si.vgg19_param_count(32, 32) == 43003944
    p32 = si.vgg19_params(32, 32, seed=0)
    w1 = p32[:64 * 27]
    assert abs(w1.std() - np.sqrt(2.0 / 27)) < 0.02
    assert np.all(p32[64 * 27:64 * 27 + 64] == 0.0)
    # conv weights do not depend on the input size
    n_conv = 20024384
    p64 = si.vgg19_params(64, 64, seed=0)
    assert np.array_equal(p32[:n_conv], p64[:n_conv])
