"""ctypes binding of libvgg19_b200.so: the same entry points as
include/vgg19_b200.h, with argument marshalling only.  Device tensors are
passed as torch CUDA tensors (or raw integer addresses), host buffers as
numpy arrays or torch CPU tensors.  Nothing here computes anything: if the
CUDA library is missing or fails to load, importing the symbols raises.
"""
from __future__ import annotations

import ctypes
import os

from . import build as _build

VGG19_OK = 0
VGG19_ERR_ARG, VGG19_ERR_SHAPE, VGG19_ERR_WORKSPACE = -1, -2, -3
VGG19_ERR_CUDA, VGG19_ERR_DEVICE_TIMEOUT, VGG19_ERR_UNSUPPORTED_ARCH, VGG19_ERR_RANGE = -4, -5, -6, -7
VGG19_FP32, VGG19_BF16 = 0, 1
VGG19_FLAG_NO_GRAPH, VGG19_FLAG_NO_TENSOR_CORES, VGG19_FLAG_NO_CTA_PAIRS, VGG19_FLAG_FIRST_FUSION = 1, 2, 4, 8
VGG19_FLAG_SPLIT_F16 = 16
VGG19_MODE_FORWARD, VGG19_MODE_BACKWARD, VGG19_MODE_TRAIN = 0, 1, 2

EXPORTS = (
    "vgg19_create", "vgg19_create_from_params", "vgg19_destroy", "vgg19_param_count", "vgg19_param_info",
    "vgg19_get_params", "vgg19_set_params", "vgg19_workspace_bytes", "vgg19_bind_workspace",
    "vgg19_forward", "vgg19_backward", "vgg19_sgd_step", "vgg19_train_step", "vgg19_train_steps",
    "vgg19_set_dense_grads_event", "vgg19_io_bytes", "vgg19_forward_host", "vgg19_forward_host_async", "vgg19_backward_host",
    "vgg19_conv_layer_forward", "vgg19_conv_layer_forward_ex", "vgg19_first_block_forward", "vgg19_conv_layer_backward", "vgg19_conv_layer_backward_ex", "vgg19_dense_layer_forward", "vgg19_dense_layer_backward", "vgg19_saved_tensor", "vgg19_conv_wgrad_static", "vgg19_sync_status", "vgg19_selftest_wait_timeout", "vgg19_launch_count",
    "vgg19_describe", "vgg19_last_error",
)


class vgg19_config(ctypes.Structure):
    _fields_ = [("height", ctypes.c_int32), ("width", ctypes.c_int32), ("batch_max", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class Vgg19Error(RuntimeError):
    def __init__(self, code, text):
        super().__init__(f"vgg19 error {code}: {text}")
        self.code = code


_lib = None


def lib_path() -> str:
    return _build.LIB


def load():
    """Load the CUDA library; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise RuntimeError(f"{path} is missing: build it with `python -c 'import __graft_entry__ as g; g.build()'` "
                           "(there is no CPU fallback)")
    L = ctypes.CDLL(path)
    vp, i32, u64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64, ctypes.c_size_t
    cfgp = ctypes.POINTER(vgg19_config)
    sig = {
        "vgg19_create": ([cfgp, u64, ctypes.POINTER(vp)], ctypes.c_int),
        "vgg19_create_from_params": ([cfgp, vp, ctypes.POINTER(vp)], ctypes.c_int),
        "vgg19_destroy": ([vp], None),
        "vgg19_param_count": ([vp, ctypes.POINTER(i32), ctypes.POINTER(sz)], ctypes.c_int),
        "vgg19_param_info": ([vp, i32, ctypes.POINTER(sz), ctypes.POINTER(i32), ctypes.POINTER(ctypes.c_int64)], ctypes.c_int),
        "vgg19_get_params": ([vp, vp], ctypes.c_int),
        "vgg19_set_params": ([vp, vp], ctypes.c_int),
        "vgg19_workspace_bytes": ([vp, i32, i32], sz),
        "vgg19_bind_workspace": ([vp, vp, sz], ctypes.c_int),
        "vgg19_forward": ([vp, vp, i32, vp, vp, vp], ctypes.c_int),
        "vgg19_backward": ([vp, vp, vp, i32, vp, vp, vp, vp], ctypes.c_int),
        "vgg19_sgd_step": ([vp, vp, ctypes.c_float, vp], ctypes.c_int),
        "vgg19_train_step": ([vp, vp, vp, i32, ctypes.c_float, vp, vp], ctypes.c_int),
        "vgg19_train_steps": ([vp, vp, vp, i32, i32, ctypes.c_float, vp, vp], ctypes.c_int),
        "vgg19_set_dense_grads_event": ([vp, vp], ctypes.c_int),
        "vgg19_io_bytes": ([vp, i32, i32], sz),
        "vgg19_forward_host": ([vp, vp, i32, vp, vp, vp], ctypes.c_int),
        "vgg19_forward_host_async": ([vp, vp, i32, vp, vp, vp], ctypes.c_int),
        "vgg19_backward_host": ([vp, vp, vp, i32, vp, vp, vp], ctypes.c_int),
        "vgg19_conv_layer_forward": ([vp, i32, vp, i32, vp, vp, vp], ctypes.c_int),
        "vgg19_conv_layer_backward": ([vp, i32, vp, vp, i32, vp, vp, vp, vp], ctypes.c_int),
        "vgg19_conv_layer_forward_ex": ([vp, i32, vp, i32, vp, vp, vp, vp], ctypes.c_int),
        "vgg19_first_block_forward": ([vp, vp, i32, vp, vp, vp], ctypes.c_int),
        "vgg19_conv_layer_backward_ex": ([vp, i32, vp, vp, i32, vp, vp, vp, vp, vp, vp], ctypes.c_int),
        "vgg19_dense_layer_forward": ([vp, i32, vp, i32, vp, vp, vp], ctypes.c_int),
        "vgg19_dense_layer_backward": ([vp, i32, vp, vp, i32, vp, vp, vp, vp, vp], ctypes.c_int),
        "vgg19_saved_tensor": ([vp, i32, i32, i32, ctypes.POINTER(sz), ctypes.POINTER(ctypes.c_int64)], ctypes.c_int),
        "vgg19_conv_wgrad_static": ([vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, ctypes.POINTER(sz), vp], ctypes.c_int),
        "vgg19_sync_status": ([vp, vp], ctypes.c_int),
        "vgg19_selftest_wait_timeout": ([vp, vp], ctypes.c_int),
        "vgg19_launch_count": ([vp, i32, ctypes.POINTER(i32)], ctypes.c_int),
        "vgg19_describe": ([vp, ctypes.c_char_p, sz], ctypes.c_int),
        "vgg19_last_error": ([vp], ctypes.c_char_p),
    }
    for name, (args, res) in sig.items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = res
    _lib = L
    return L


def _ptr(x):
    """Address of a torch tensor / numpy array / int / None."""
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "data_ptr"):
        return x.data_ptr()
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(type(x))


def _stream(stream):
    if stream is None:
        return None
    return stream if isinstance(stream, int) else stream.cuda_stream


def _check(net, rc):
    if rc != VGG19_OK:
        raise Vgg19Error(rc, load().vgg19_last_error(net).decode())
    return rc


def vgg19_create(height, width, batch_max, dtype, seed, flags=0):
    cfg = vgg19_config(height, width, batch_max, dtype, flags)
    out = ctypes.c_void_p()
    _check(None, load().vgg19_create(ctypes.byref(cfg), seed, ctypes.byref(out)))
    return out.value


def vgg19_create_from_params(height, width, batch_max, dtype, host_params, flags=0):
    cfg = vgg19_config(height, width, batch_max, dtype, flags)
    out = ctypes.c_void_p()
    _check(None, load().vgg19_create_from_params(ctypes.byref(cfg), _ptr(host_params), ctypes.byref(out)))
    return out.value


def vgg19_destroy(net):
    load().vgg19_destroy(net)


def vgg19_param_count(net):
    n, e = ctypes.c_int32(), ctypes.c_size_t()
    _check(net, load().vgg19_param_count(net, ctypes.byref(n), ctypes.byref(e)))
    return n.value, e.value


def vgg19_param_info(net, i):
    off, rank = ctypes.c_size_t(), ctypes.c_int32()
    dims = (ctypes.c_int64 * 4)()
    _check(net, load().vgg19_param_info(net, i, ctypes.byref(off), ctypes.byref(rank), dims))
    return off.value, tuple(dims[:rank.value])


def vgg19_get_params(net, host_params):
    return _check(net, load().vgg19_get_params(net, _ptr(host_params)))


def vgg19_set_params(net, host_params):
    return _check(net, load().vgg19_set_params(net, _ptr(host_params)))


def vgg19_sgd_step(net, grads, lr, stream=None):
    return _check(net, load().vgg19_sgd_step(net, _ptr(grads), float(lr), _stream(stream)))


def vgg19_train_step(net, images, labels, batch, lr, loss=None, stream=None):
    return _check(net, load().vgg19_train_step(net, _ptr(images), _ptr(labels), batch, float(lr), _ptr(loss), _stream(stream)))


def vgg19_train_steps(net, images, labels, batch, steps, lr, losses=None, stream=None):
    return _check(net, load().vgg19_train_steps(net, _ptr(images), _ptr(labels), batch, steps, float(lr), _ptr(losses),
                                                 _stream(stream)))


def vgg19_set_dense_grads_event(net, event):
    """event: a torch.cuda.Event that has been recorded at least once (so that its handle exists), a raw
    cudaEvent_t as an integer, or None."""
    h = None if event is None else (event if isinstance(event, int) else event.cuda_event)
    return _check(net, load().vgg19_set_dense_grads_event(net, h))


def vgg19_workspace_bytes(net, batch, mode):
    return load().vgg19_workspace_bytes(net, batch, mode)


def vgg19_io_bytes(net, batch, mode):
    return load().vgg19_io_bytes(net, batch, mode)


def vgg19_bind_workspace(net, workspace, nbytes):
    return _check(net, load().vgg19_bind_workspace(net, _ptr(workspace), nbytes))


def vgg19_forward(net, images, batch, logits, probs=None, stream=None):
    return _check(net, load().vgg19_forward(net, _ptr(images), batch, _ptr(logits), _ptr(probs), _stream(stream)))


def vgg19_backward(net, images, labels, batch, grads, loss=None, logits=None, stream=None):
    return _check(net, load().vgg19_backward(net, _ptr(images), _ptr(labels), batch, _ptr(grads), _ptr(loss),
                                             _ptr(logits), _stream(stream)))


def vgg19_forward_host(net, host_images, batch, host_logits, host_probs=None, stream=None):
    return _check(net, load().vgg19_forward_host(net, _ptr(host_images), batch, _ptr(host_logits),
                                                  _ptr(host_probs), _stream(stream)))


def vgg19_forward_host_async(net, host_images, batch, host_logits, host_probs=None, stream=None):
    return _check(net, load().vgg19_forward_host_async(net, _ptr(host_images), batch, _ptr(host_logits),
                                                        _ptr(host_probs), _stream(stream)))


def vgg19_backward_host(net, host_images, host_labels, batch, host_grads, host_loss=None, stream=None):
    return _check(net, load().vgg19_backward_host(net, _ptr(host_images), _ptr(host_labels), batch,
                                                   _ptr(host_grads), _ptr(host_loss), _stream(stream)))


def vgg19_conv_layer_forward(net, layer, x, batch, y, pooled=None, stream=None):
    return _check(net, load().vgg19_conv_layer_forward(net, layer, _ptr(x), batch, _ptr(y), _ptr(pooled),
                                                        _stream(stream)))


def vgg19_conv_layer_backward(net, layer, x, dz, batch, dw, db, dx=None, stream=None):
    return _check(net, load().vgg19_conv_layer_backward(net, layer, _ptr(x), _ptr(dz), batch, _ptr(dw), _ptr(db),
                                                         _ptr(dx), _stream(stream)))


def vgg19_dense_layer_forward(net, layer, x, batch, y=None, y_f32=None, stream=None):
    return _check(net, load().vgg19_dense_layer_forward(net, layer, _ptr(x), batch, _ptr(y), _ptr(y_f32), _stream(stream)))


def vgg19_dense_layer_backward(net, layer, x, dy, batch, dw, db, dx=None, relu_mask=None, stream=None):
    return _check(net, load().vgg19_dense_layer_backward(net, layer, _ptr(x), _ptr(dy), batch, _ptr(dw), _ptr(db),
                                                          _ptr(dx), _ptr(relu_mask), _stream(stream)))


def vgg19_conv_layer_forward_ex(net, layer, x, batch, y, pooled=None, pool_code=None, stream=None):
    return _check(net, load().vgg19_conv_layer_forward_ex(net, layer, _ptr(x), batch, _ptr(y), _ptr(pooled),
                                                           _ptr(pool_code), _stream(stream)))


def vgg19_first_block_forward(net, images, batch, y2=None, pooled=None, stream=None):
    return _check(net, load().vgg19_first_block_forward(net, _ptr(images), batch, _ptr(y2), _ptr(pooled), _stream(stream)))


def vgg19_conv_layer_backward_ex(net, layer, x, dz, batch, dw=None, db=None, dx=None, relu_mask=None, pool_code=None,
                                 stream=None):
    return _check(net, load().vgg19_conv_layer_backward_ex(net, layer, _ptr(x), _ptr(dz), batch, _ptr(dw), _ptr(db),
                                                            _ptr(dx), _ptr(relu_mask), _ptr(pool_code), _stream(stream)))


def vgg19_saved_tensor(net, batch, mode, index):
    off = ctypes.c_size_t()
    dims = (ctypes.c_int64 * 4)()
    _check(net, load().vgg19_saved_tensor(net, batch, mode, index, ctypes.byref(off), dims))
    return off.value, tuple(dims)


VGG19_STATIC_SCRATCH_BYTES = 8 << 20


def vgg19_conv_wgrad_static(x, dz, batch, height, width, cin, cout, dtype, dw, db, stream=None):
    """Allocation-free filter/bias gradient; returns (status, scratch bytes the shape needs)."""
    need = ctypes.c_size_t()
    rc = load().vgg19_conv_wgrad_static(_ptr(x), _ptr(dz), batch, height, width, cin, cout, dtype, _ptr(dw), _ptr(db),
                                        ctypes.byref(need), _stream(stream))
    return rc, need.value


def vgg19_sync_status(net, stream=None):
    return _check(net, load().vgg19_sync_status(net, _stream(stream)))


def vgg19_selftest_wait_timeout(net, stream=None):
    return _check(net, load().vgg19_selftest_wait_timeout(net, _stream(stream)))


def vgg19_launch_count(net, mode):
    n = ctypes.c_int32()
    _check(net, load().vgg19_launch_count(net, mode, ctypes.byref(n)))
    return n.value


def vgg19_describe(net):
    need = load().vgg19_describe(net, None, 0)
    buf = ctypes.create_string_buffer(need + 1)
    load().vgg19_describe(net, buf, need + 1)
    return buf.value.decode()


def vgg19_last_error(net=None):
    return load().vgg19_last_error(net).decode()
