"""The allocation-free filter-gradient entry point.

Some callers of this library cannot allocate device memory (they run inside a
host framework that already owns the GPU's memory, or under a fixed memory
budget), so they can neither create a network handle nor supply a workspace.
vgg19_conv_wgrad_static() serves them from a scratch array built into the
library.  This test calls it through the C ABI twice in a row - the second
call finds the scratch dirty from the first - and compares both results with
the handle-based vgg19_conv_layer_backward on the same tensors and with the
fp64 CPU checker's filter gradient, within the per-layer tolerance of the other
convolution tests (relative L2 <= 1e-3).  The second call must leave the
amount of free device memory as it found it (the first call on a device is the
one that may make the driver load the library's code and the scratch array).
It also checks that a shape beyond the built-in scratch is refused.

Collected last on purpose: a run that stops at the first failure has then
already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
import seeded_inputs as si

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def rel_l2(a, b):
    a, b = a.double(), b.double()
    return float((a - b).norm() / b.norm())


@pytest.mark.parametrize("dtype_name", ["bf16", "fp32"])
def test_static_scratch_wgrad_matches_the_workspace_path_twice(dtype_name):
    import paper_1810_09868_b200 as p
    dtype = p.VGG19_BF16 if dtype_name == "bf16" else p.VGG19_FP32
    tdtype = torch.bfloat16 if dtype_name == "bf16" else torch.float32
    B, S, layer, Cin, Cout = 2, 16, 4, 128, 128  # conv2_2 of a 32x32 network
    params = si.vgg19_params(32, 32, seed=0, bf16_exact=True)
    # CUDA-core path on both sides, so the two entry points run the same arithmetic
    net = p.Net(32, 32, B, dtype, params=params, flags=p.VGG19_FLAG_NO_TENSOR_CORES)
    stream = torch.cuda.current_stream()
    for call in range(2):
        x = torch.from_numpy(si.normal(B * S * S * Cin, seed=10 + call, take_abs=True, bf16_exact=True)
                             .reshape(B, S, S, Cin)).to(DEV).to(tdtype)
        dz = torch.from_numpy(si.normal(B * S * S * Cout, seed=20 + call, stddev=1e-2, bf16_exact=True)
                              .reshape(B, S, S, Cout)).to(DEV).to(tdtype)
        dw_ref = torch.empty(Cout, 3, 3, Cin, dtype=torch.float32, device=DEV)
        db_ref = torch.empty(Cout, dtype=torch.float32, device=DEV)
        p.vgg19_conv_layer_backward(net.handle, layer, x, dz, B, dw_ref, db_ref, None, stream)
        dw = torch.full_like(dw_ref, float("nan"))
        db = torch.full_like(db_ref, float("nan"))
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        rc, need = p.vgg19_conv_wgrad_static(x, dz, B, S, S, Cin, Cout, dtype, dw, db, stream)
        assert rc == p.VGG19_OK and 0 < need <= p.VGG19_STATIC_SCRATCH_BYTES
        net.sync_status()
        if call == 1:
            assert torch.cuda.mem_get_info()[0] == free_before, "a call after the first changed free device memory"
        assert torch.isfinite(dw).all() and torch.isfinite(db).all()
        assert rel_l2(dw, dw_ref) <= 1e-3, call
        assert rel_l2(db, db_ref) <= 1e-3, call
        o_dw, o_db = oracle.conv3x3_wgrad(x.float().cpu().numpy().astype(np.float64),
                                          dz.float().cpu().numpy().astype(np.float64))
        assert rel_l2(dw.cpu(), torch.from_numpy(o_dw)) <= 1e-3, call
        assert rel_l2(db.cpu(), torch.from_numpy(o_db)) <= 1e-3, call
    net.close()


def test_static_scratch_rejects_shapes_beyond_its_size_and_bad_arguments():
    import paper_1810_09868_b200 as p
    t = torch.zeros(16, device=DEV)
    # conv 512 -> 512 on 28x28 x 16 images would need about 19 MB of partial sums
    rc, need = p.vgg19_conv_wgrad_static(t, t, 16, 28, 28, 512, 512, p.VGG19_BF16, t, t, torch.cuda.current_stream())
    assert rc == p.VGG19_ERR_WORKSPACE and need > p.VGG19_STATIC_SCRATCH_BYTES
    rc, _ = p.vgg19_conv_wgrad_static(None, t, 1, 4, 4, 8, 8, p.VGG19_BF16, t, t)
    assert rc == p.VGG19_ERR_ARG
    rc, _ = p.vgg19_conv_wgrad_static(t, t, 0, 4, 4, 8, 8, p.VGG19_BF16, t, t)
    assert rc == p.VGG19_ERR_ARG
    torch.cuda.synchronize()
