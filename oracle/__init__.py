"""TEST INFRASTRUCTURE - not part of the product path.

fp64 CPU checker for the VGG19 forward and backward pass (paper sections 7.2
and 7.3).  The per-operation definitions live in ``vgg19_oracle.c`` (plain
loop nests); this module loads them with ctypes and chains them in the order
the network applies them.  It imports nothing from the CUDA package and the
CUDA package imports nothing from here.

A network is a list of steps acting on an NHWC activation:
    ("conv", Cout)        3x3 conv pad 1 + bias + ReLU
    ("pool",)             2x2 max-pool stride 2
    ("fc", Out, relu)     flatten (h, w, c; c fastest) then dense (+ ReLU)
followed by softmax.  Parameters are one flat fp64 vector: for each conv / fc
step in order, the weight ([Cout,3,3,Cin] or [Out,In]) then the bias.

Parity status: every function is pinned by tests/test_oracle_pins.py; the
whole-network composition has no printed value in the paper to compare with
and is pinned by finite differences on a small network, by the homogeneity of
the bias-free forward pass, and by the analytically vanishing gradient of the
paper's stand-in loss sum(softmax(.)).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "vgg19_oracle.c")
_LIB = os.path.join(_HERE, "libvgg19_oracle.so")
_lib = None

VGG19_CONV = (64, 64, "M", 128, 128, "M", 256, 256, 256, 256, "M",
              512, 512, 512, 512, "M", 512, 512, 512, 512, "M")


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O3", "-fPIC", "-shared", "-fopenmp", "-mavx2", "-mfma", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        d = ctypes.POINTER(ctypes.c_double)
        i32 = ctypes.POINTER(ctypes.c_int32)
        I = ctypes.c_int
        L = ctypes.c_ssize_t
        sig = {
            "oracle_conv3x3_fwd": ([d, d, d, d, I, I, I, I, I], None),
            "oracle_conv3x3_dgrad": ([d, d, d, I, I, I, I, I], None),
            "oracle_conv3x3_wgrad": ([d, d, d, d, I, I, I, I, I], None),
            "oracle_relu_fwd": ([d, d, L], None),
            "oracle_relu_bwd": ([d, d, d, L], None),
            "oracle_maxpool2x2_fwd": ([d, d, I, I, I, I], None),
            "oracle_maxpool2x2_bwd": ([d, d, d, I, I, I, I], None),
            "oracle_dense_fwd": ([d, d, d, d, I, I, I], None),
            "oracle_dense_bwd": ([d, d, d, d, d, d, I, I, I], None),
            "oracle_softmax": ([d, d, I, I], None),
            "oracle_cross_entropy": ([d, i32, I, I, I], ctypes.c_double),
            "oracle_softmax_ce_bwd": ([d, i32, d, I, I, I], None),
            "oracle_softmax_bwd": ([d, d, d, I, I], None),
            "oracle_round_bf16": ([d, L], None),
        }
        for name, (args, res) in sig.items():
            fn = getattr(lib, name)
            fn.argtypes = args
            fn.restype = res
        _lib = lib
    return _lib


def _d(a):
    if a is None:
        return None
    assert a.dtype == np.float64 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _i(a):
    assert a.dtype == np.int32 and a.flags["C_CONTIGUOUS"]
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _c(a):
    return np.ascontiguousarray(a, dtype=np.float64)


# ---------------------------------------------------------------- operations

def conv3x3_fwd(x, W, b=None):
    x, W = _c(x), _c(W)
    N, H, Wd, Cin = x.shape
    Cout = W.shape[0]
    assert W.shape == (Cout, 3, 3, Cin)
    b = None if b is None else _c(b)
    z = np.empty((N, H, Wd, Cout))
    _load().oracle_conv3x3_fwd(_d(x), _d(W), _d(b), _d(z), N, H, Wd, Cin, Cout)
    return z


def conv3x3_dgrad(dz, W):
    dz, W = _c(dz), _c(W)
    N, H, Wd, Cout = dz.shape
    Cin = W.shape[3]
    dx = np.empty((N, H, Wd, Cin))
    _load().oracle_conv3x3_dgrad(_d(dz), _d(W), _d(dx), N, H, Wd, Cin, Cout)
    return dx


def conv3x3_wgrad(x, dz, dW=None, db=None):
    """Returns (dW, db); accumulates into the given arrays when passed."""
    x, dz = _c(x), _c(dz)
    N, H, Wd, Cin = x.shape
    Cout = dz.shape[3]
    if dW is None:
        dW = np.zeros((Cout, 3, 3, Cin))
    if db is None:
        db = np.zeros(Cout)
    _load().oracle_conv3x3_wgrad(_d(x), _d(dz), _d(dW), _d(db), N, H, Wd, Cin, Cout)
    return dW, db


def relu_fwd(z):
    z = _c(z)
    y = np.empty_like(z)
    _load().oracle_relu_fwd(_d(z), _d(y), z.size)
    return y


def relu_bwd(z, dy):
    z, dy = _c(z), _c(dy)
    dz = np.empty_like(z)
    _load().oracle_relu_bwd(_d(z), _d(dy), _d(dz), z.size)
    return dz


def maxpool2x2_fwd(y):
    y = _c(y)
    N, H, Wd, C = y.shape
    p = np.empty((N, H // 2, Wd // 2, C))
    _load().oracle_maxpool2x2_fwd(_d(y), _d(p), N, H, Wd, C)
    return p


def maxpool2x2_bwd(y, dp):
    y, dp = _c(y), _c(dp)
    N, H, Wd, C = y.shape
    dy = np.empty_like(y)
    _load().oracle_maxpool2x2_bwd(_d(y), _d(dp), _d(dy), N, H, Wd, C)
    return dy


def dense_fwd(x, W, b=None):
    x, W = _c(x), _c(W)
    N, In = x.shape
    Out = W.shape[0]
    assert W.shape == (Out, In)
    b = None if b is None else _c(b)
    y = np.empty((N, Out))
    _load().oracle_dense_fwd(_d(x), _d(W), _d(b), _d(y), N, In, Out)
    return y


def dense_bwd(x, W, dy, dW=None, db=None, need_dx=True):
    """Returns (dx, dW, db); accumulates into dW, db when passed."""
    x, W, dy = _c(x), _c(W), _c(dy)
    N, In = x.shape
    Out = W.shape[0]
    dx = np.empty((N, In)) if need_dx else None
    if dW is None:
        dW = np.zeros((Out, In))
    if db is None:
        db = np.zeros(Out)
    _load().oracle_dense_bwd(_d(x), _d(W), _d(dy), _d(dx), _d(dW), _d(db), N, In, Out)
    return dx, dW, db


def softmax(l):
    l = _c(l)
    p = np.empty_like(l)
    _load().oracle_softmax(_d(l), _d(p), l.shape[0], l.shape[1])
    return p


def cross_entropy(l, labels, n_total=None):
    l = _c(l)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    n_total = l.shape[0] if n_total is None else n_total
    return float(_load().oracle_cross_entropy(_d(l), _i(labels), l.shape[0], l.shape[1], n_total))


def softmax_ce_bwd(p, labels, n_total=None):
    p = _c(p)
    labels = np.ascontiguousarray(labels, dtype=np.int32)
    n_total = p.shape[0] if n_total is None else n_total
    dl = np.empty_like(p)
    _load().oracle_softmax_ce_bwd(_d(p), _i(labels), _d(dl), p.shape[0], p.shape[1], n_total)
    return dl


def softmax_bwd(p, g):
    p, g = _c(p), _c(g)
    dl = np.empty_like(p)
    _load().oracle_softmax_bwd(_d(p), _d(g), _d(dl), p.shape[0], p.shape[1])
    return dl


def round_bf16(x):
    """Nearest-bfloat16 (ties to even) of every element, returned as fp64."""
    x = np.array(x, dtype=np.float64, order="C", copy=True)
    _load().oracle_round_bf16(_d(x), x.size)
    return x


def _store(x, storage):
    """Model the storage format of a tensor the configuration keeps in memory:
    exact for fp64, rounded to bf16 for the bf16 configurations."""
    if storage is None:
        return x
    assert storage == "bf16"
    return round_bf16(x)


# ------------------------------------------------------------------ networks

def vgg19_steps():
    """The VGG19 topology (section 7.2; appendix: 16 convolution, 5
    reduce-window, 3 dot, 18 ReLU maxima, one softmax, no rng/dropout)."""
    steps = [("pool",) if v == "M" else ("conv", v) for v in VGG19_CONV]
    steps += [("fc", 4096, True), ("fc", 4096, True), ("fc", 1000, False)]
    return steps


def param_shapes(steps, H, W, Cin=3):
    """[(weight_shape, bias_shape)] for every conv / fc step, in order."""
    shapes = []
    h, w, c = H, W, Cin
    flat = None
    for st in steps:
        if st[0] == "conv":
            shapes.append(((st[1], 3, 3, c), (st[1],)))
            c = st[1]
        elif st[0] == "pool":
            h, w = h // 2, w // 2
        else:
            if flat is None:
                flat = h * w * c
            shapes.append(((st[1], flat), (st[1],)))
            flat = st[1]
    return shapes


def split_params(flat_params, shapes):
    out, off = [], 0
    for ws, bs in shapes:
        nw, nb = int(np.prod(ws)), int(np.prod(bs))
        out.append((flat_params[off:off + nw].reshape(ws), flat_params[off + nw:off + nw + nb]))
        off += nw + nb
    assert off == flat_params.size, (off, flat_params.size)
    return out


def forward(steps, params, images, keep=False, storage=None):
    """Logits [N, classes] (pre-softmax).  With keep=True also returns the
    list of saved tensors the backward pass needs.

    storage=None: every intermediate stays fp64.  storage="bf16": the
    configuration "bf16 activations, fp32 accumulate" - all arithmetic is still
    fp64, but each activation the configuration keeps in memory (the output of
    every conv+ReLU and dense+ReLU) is rounded to bf16 where it is stored, so
    that ReLU masks and pool arg-maxima are decided on the same stored values
    on which the device decides them.  Logits stay unrounded."""
    x = _c(images)
    shapes = param_shapes(steps, x.shape[1], x.shape[2], x.shape[3])
    P = split_params(_c(params), shapes)
    saved, pi = [], 0
    for st in steps:
        if st[0] == "conv":
            Wt, b = P[pi]; pi += 1
            z = conv3x3_fwd(x, Wt, b)
            y = _store(relu_fwd(z), storage)
            saved.append(("conv", x, y))  # y > 0 exactly where z > 0
            x = y
        elif st[0] == "pool":
            p = maxpool2x2_fwd(x)
            saved.append(("pool", x))
            x = p
        else:
            Wt, b = P[pi]; pi += 1
            shp = x.shape
            xf = x.reshape(x.shape[0], -1)
            z = dense_fwd(xf, Wt, b)
            x = _store(relu_fwd(z), storage) if st[2] else z
            saved.append(("fc", xf, x, shp, st[2]))
    return (x, saved) if keep else x


def state_from_outputs(steps, images, outputs):
    """Rebuild the saved forward state from the stored output of every step
    (conv: y after ReLU; pool: pooled tensor; fc: activation, logits for the
    last), e.g. as read back from a device.  Returns (logits, saved) in the
    form forward(keep=True) returns, so that backward() can differentiate the
    network at exactly that state: given the stored activations, the ReLU
    masks and pool arg-maxima are fixed and the gradient is unique."""
    x = _c(images)
    saved = []
    for st, out in zip(steps, outputs):
        out = _c(out)
        if st[0] == "conv":
            saved.append(("conv", x, out))
        elif st[0] == "pool":
            saved.append(("pool", x))
        else:
            saved.append(("fc", x.reshape(x.shape[0], -1), out, x.shape, st[2]))
        x = out
    return x, saved


def backward(steps, params, images, labels=None, n_total=None, grads=None, loss_kind="ce", storage=None,
             state=None):
    """Gradient of the loss with respect to every parameter, flat, in the
    parameter order.  loss_kind "ce": mean cross-entropy of softmax(logits)
    (dlogits = (p - onehot) / n_total).  loss_kind "sum": the paper's
    stand-in sum(softmax(logits)) (section 7.3).  When `grads` is given the
    result is accumulated into it (chunked batches).  With storage="bf16"
    the gradients the configuration keeps in memory between layers (dlogits
    and every activation gradient) are rounded to bf16 where they are stored;
    parameter gradients are never rounded.  With state=(logits, saved) the
    forward pass is not run and the network is differentiated at that given
    forward state.  Returns (loss, grads, logits)."""
    params = _c(params)
    images = _c(images)
    N = images.shape[0]
    n_total = N if n_total is None else n_total
    shapes = param_shapes(steps, images.shape[1], images.shape[2], images.shape[3])
    P = split_params(params, shapes)
    if grads is None:
        grads = np.zeros_like(params)
    G = split_params(grads, shapes)
    if state is None:
        logits, saved = forward(steps, params, images, keep=True, storage=storage)
    else:
        logits, saved = state
    p = softmax(logits)
    if loss_kind == "ce":
        loss = cross_entropy(logits, labels, n_total)
        g = _store(softmax_ce_bwd(p, labels, n_total), storage)
    else:
        loss = float(p.sum())
        g = softmax_bwd(p, np.ones_like(p))
    pi = len(P) - 1
    first_param_step = next(i for i, st in enumerate(steps) if st[0] != "pool")
    for si in range(len(steps) - 1, -1, -1):
        st, sv = steps[si], saved[si]
        if st[0] == "fc":
            _, xf, y, shp, relu = sv
            if relu:
                g = relu_bwd(y, g)
            Wt, _ = P[pi]
            dW, db = G[pi]; pi -= 1
            dx, _, _ = dense_bwd(xf, Wt, g, dW, db, need_dx=si != first_param_step)
            g = None if dx is None else _store(dx.reshape(shp), storage)
        elif st[0] == "pool":
            g = maxpool2x2_bwd(sv[1], g)
        else:
            _, xin, y = sv
            dz = relu_bwd(y, g)
            Wt, _ = P[pi]
            dW, db = G[pi]; pi -= 1
            conv3x3_wgrad(xin, dz, dW, db)
            # the derivative is with respect to the model only: the first
            # layer's input gradient is never needed (47, not 48, convolutions)
            g = _store(conv3x3_dgrad(dz, Wt), storage) if si != first_param_step else None
    return loss, grads, logits


def sgd_step(params, grads, lr):
    """One step of plain gradient descent, w <- w - lr * dL/dw, in fp64.  The paper
    fuses "the training loop" with the two passes (introduction, conclusion) and
    names no optimiser; this is the reading taken."""
    return np.asarray(params, dtype=np.float64).ravel() - float(lr) * np.asarray(grads, dtype=np.float64).ravel()


def vgg19_forward(params, images, storage=None):
    return forward(vgg19_steps(), params, images, storage=storage)


def vgg19_backward(params, images, labels, chunk=4, storage=None):
    """Whole-batch VGG19 loss, gradients and logits, processed `chunk` images
    at a time to bound memory (the loss and gradient are sums over images)."""
    steps = vgg19_steps()
    N = images.shape[0]
    grads = np.zeros(np.asarray(params).size)
    loss, logits = 0.0, []
    for s in range(0, N, chunk):
        l, _, lg = backward(steps, params, images[s:s + chunk], labels[s:s + chunk], n_total=N, grads=grads,
                            storage=storage)
        loss += l
        logits.append(lg)
    return loss, grads, np.concatenate(logits)
