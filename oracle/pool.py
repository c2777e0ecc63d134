"""TEST INFRASTRUCTURE ONLY -- Python face of the CPU oracle for the pooling nest of Section 6.

Builds ``pool7nl.c`` (plain C, fp64) into ``libpool7nl_oracle.so`` beside this file and exposes it
through ctypes on numpy arrays.  Nothing here may be imported by the CUDA product path; only the
tests, the smoke check and the benchmark's CPU-baseline leg use it.

Array conventions (dense, last subscript fastest): Image [Wi][Hi][C][B] as bf16 bit patterns
(``uint16``), Out [K][H][W][B] in fp64.  ``op`` is ``AVG`` (a + b/(R*S), from 0) or ``MAX``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

from .cnn import Shape

AVG = 0
MAX = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pool7nl.c")
_LIB = os.path.join(_HERE, "libpool7nl_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle if the shared object is missing or older than its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O2", "-fPIC", "-shared", "-std=c11", "-o", _LIB, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    i32 = ctypes.c_int
    dptr = ctypes.POINTER(ctypes.c_double)
    u16p = ctypes.POINTER(ctypes.c_uint16)
    lib.pool7nl_bf16.restype = i32
    lib.pool7nl_bf16.argtypes = [u16p, dptr, dptr] + [i32] * 10
    lib.pool7nl_bf16_at.restype = i32
    lib.pool7nl_bf16_at.argtypes = [u16p, ctypes.POINTER(ctypes.c_int32), ctypes.c_int64, dptr,
                                    dptr] + [i32] * 10
    _lib = lib
    return lib


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _image(image_bits, shp: Shape):
    image_bits = np.ascontiguousarray(image_bits, dtype=np.uint16)
    if image_bits.shape != shp.image_shape:
        raise ValueError(f"Image shape {image_bits.shape} != {shp.image_shape}")
    return image_bits


def pool_bf16(image_bits, shp: Shape, op: int):
    """The whole pooled array.  Returns (Out, Abs); Abs is None for MAX."""
    image_bits = _image(image_bits, shp)
    out = np.empty(shp.out_shape, dtype=np.float64)
    ab = np.empty(shp.out_shape, dtype=np.float64) if op == AVG else None
    rc = _load().pool7nl_bf16(image_bits.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)), _dp(out),
                              _dp(ab) if ab is not None else None, *shp.args(), op)
    if rc != 0:
        raise RuntimeError(f"pool7nl_bf16 failed: {rc}")
    return out, ab


def pool_bf16_at(image_bits, khwb, shp: Shape, op: int):
    """Selected output elements: ``khwb`` is an (n,4) int array of (k,h,w,b).  Returns (Out, Abs)."""
    image_bits = _image(image_bits, shp)
    khwb = np.ascontiguousarray(khwb, dtype=np.int32).reshape(-1, 4)
    n = khwb.shape[0]
    out = np.empty(n, dtype=np.float64)
    ab = np.empty(n, dtype=np.float64)
    rc = _load().pool7nl_bf16_at(image_bits.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16)),
                                 khwb.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                 ctypes.c_int64(n), _dp(out), _dp(ab), *shp.args(), op)
    if rc != 0:
        raise RuntimeError(f"pool7nl_bf16_at failed: {rc}")
    return out, (ab if op == AVG else None)
