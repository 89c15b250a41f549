"""Seeded synthetic inputs (weights, images, labels) for the VGG19 pass.

Thin ctypes wrapper over ``seeded_inputs.c``.  It contains no arithmetic of
the network: it only produces the numbers that both the CUDA library and the
CPU checker are fed, so that they see identical inputs.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "seeded_inputs.c")
_LIB = os.path.join(_HERE, "libseeded_inputs.so")
_lib = None

N_CLASSES = 1000


def build(force: bool = False) -> str:
    """Compile the generator into its own shared library (gcc, OpenMP)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        f32p = ctypes.POINTER(ctypes.c_float)
        lib.seeded_uniform_f32.argtypes = [f32p, ctypes.c_size_t, ctypes.c_uint64, ctypes.c_uint64,
                                           ctypes.c_double, ctypes.c_double, ctypes.c_int]
        lib.seeded_uniform_f32.restype = None
        lib.seeded_normal_f32.argtypes = [f32p, ctypes.c_size_t, ctypes.c_uint64, ctypes.c_uint64,
                                          ctypes.c_double, ctypes.c_int, ctypes.c_int]
        lib.seeded_normal_f32.restype = None
        lib.seeded_labels_i32.argtypes = [ctypes.POINTER(ctypes.c_int32), ctypes.c_size_t, ctypes.c_uint64,
                                          ctypes.c_uint64, ctypes.c_int32]
        lib.seeded_labels_i32.restype = None
        lib.seeded_vgg19_param_count.argtypes = [ctypes.c_int, ctypes.c_int]
        lib.seeded_vgg19_param_count.restype = ctypes.c_size_t
        lib.seeded_vgg19_params.argtypes = [f32p, ctypes.c_int, ctypes.c_int, ctypes.c_uint64,
                                            ctypes.c_double, ctypes.c_int]
        lib.seeded_vgg19_params.restype = None
        _lib = lib
    return _lib


def _f32p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_float))


def uniform(n: int, seed: int, stream: int = 0, shift: float = 0.0, scale: float = 1.0,
            bf16_exact: bool = False) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)
    _load().seeded_uniform_f32(_f32p(out), n, seed, stream, shift, scale, int(bf16_exact))
    return out


def normal(n: int, seed: int, stream: int = 0, stddev: float = 1.0, take_abs: bool = False,
           bf16_exact: bool = False) -> np.ndarray:
    out = np.empty(n, dtype=np.float32)
    _load().seeded_normal_f32(_f32p(out), n, seed, stream, stddev, int(take_abs), int(bf16_exact))
    return out


def images(batch: int, height: int, width: int, seed: int = 1, bf16_exact: bool = False) -> np.ndarray:
    """[batch, H, W, 3] fp32: u ~ U[0,1) per element, normalised (u - 0.5) / 0.25."""
    return uniform(batch * height * width * 3, seed, 0, 0.5, 4.0, bf16_exact).reshape(batch, height, width, 3)


def labels(batch: int, seed: int = 2) -> np.ndarray:
    out = np.empty(batch, dtype=np.int32)
    _load().seeded_labels_i32(out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), batch, seed, 0, N_CLASSES)
    return out


def vgg19_param_count(height: int, width: int) -> int:
    return int(_load().seeded_vgg19_param_count(height, width))


def vgg19_params(height: int, width: int, seed: int = 0, bias_std: float = 0.0,
                 bf16_exact: bool = False) -> np.ndarray:
    """Flat fp32 VGG19 parameter buffer: layer 1..19, weight then bias."""
    out = np.empty(vgg19_param_count(height, width), dtype=np.float32)
    _load().seeded_vgg19_params(_f32p(out), height, width, seed, bias_std, int(bf16_exact))
    return out
