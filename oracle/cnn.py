"""TEST INFRASTRUCTURE ONLY -- Python face of the CPU oracle for the seven-nested-loop CNN (Eq. 1).

Builds ``cnn7nl.c`` (plain C, fp64, OpenMP threads) into ``libcnn7nl_oracle.so`` beside this file
and exposes it through ctypes on numpy arrays.  Nothing here may be imported by the CUDA product
path; only the tests, the smoke check and the benchmark's CPU-baseline leg use it.

Array conventions (dense, last subscript fastest):
    Image  [Wi][Hi][C][B], Wi = sw*(W-1)+R, Hi = sh*(H-1)+S
    Filter [K][R][S][C]
    Out    [K][H][W][B]
bf16 values travel as ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "cnn7nl.c")
_LIB = os.path.join(_HERE, "libcnn7nl_oracle.so")
_lib = None


@dataclass(frozen=True)
class Shape:
    """The seven loop bounds and two strides of Eq. 1."""

    B: int
    C: int
    K: int
    W: int
    H: int
    R: int
    S: int
    sw: int = 1
    sh: int = 1

    @property
    def Wi(self) -> int:
        return self.sw * (self.W - 1) + self.R

    @property
    def Hi(self) -> int:
        return self.sh * (self.H - 1) + self.S

    @property
    def image_shape(self):
        return (self.Wi, self.Hi, self.C, self.B)

    @property
    def filter_shape(self):
        return (self.K, self.R, self.S, self.C)

    @property
    def out_shape(self):
        return (self.K, self.H, self.W, self.B)

    @property
    def macs(self) -> int:
        return self.B * self.C * self.K * self.W * self.H * self.R * self.S

    def args(self):
        return (self.B, self.C, self.K, self.W, self.H, self.R, self.S, self.sw, self.sh)


def build(force: bool = False) -> str:
    """Compile the C oracle if the shared object is missing or older than its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["gcc", "-O3", "-march=native", "-fopenmp", "-fPIC", "-shared", "-std=c11",
           "-o", _LIB, _SRC, "-lm"]
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
    nine = [i32] * 9
    lib.cnn7nl_max_threads.restype = i32
    lib.cnn7nl_f64.restype = i32
    lib.cnn7nl_f64.argtypes = [dptr, dptr, dptr, dptr] + nine
    lib.cnn7nl_f64_paper_order.restype = i32
    lib.cnn7nl_f64_paper_order.argtypes = [dptr, dptr, dptr] + nine
    lib.cnn7nl_bf16.restype = i32
    lib.cnn7nl_bf16.argtypes = [u16p, u16p, dptr, dptr] + nine
    lib.cnn7nl_bf16_at.restype = i32
    lib.cnn7nl_bf16_at.argtypes = [u16p, u16p, ctypes.POINTER(ctypes.c_int32), ctypes.c_int64,
                                   dptr, dptr] + nine
    _lib = lib
    return lib


def max_threads() -> int:
    return int(_load().cnn7nl_max_threads())


def _dp(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def _u16(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint16))


def _check_inputs(image, filt, shp: Shape, dtype):
    image = np.ascontiguousarray(image, dtype=dtype)
    filt = np.ascontiguousarray(filt, dtype=dtype)
    if image.shape != shp.image_shape:
        raise ValueError(f"Image shape {image.shape} != {shp.image_shape}")
    if filt.shape != shp.filter_shape:
        raise ValueError(f"Filter shape {filt.shape} != {shp.filter_shape}")
    return image, filt


def cnn_f64(image, filt, shp: Shape, want_abs: bool = True):
    """Eq. 1 on fp64 arrays.  Returns (Out, Abs) with Abs = sum |Image*Filter| (or None)."""
    image, filt = _check_inputs(image, filt, shp, np.float64)
    out = np.empty(shp.out_shape, dtype=np.float64)
    ab = np.empty(shp.out_shape, dtype=np.float64) if want_abs else None
    rc = _load().cnn7nl_f64(_dp(image), _dp(filt), _dp(out), _dp(ab) if want_abs else None,
                            *shp.args())
    if rc != 0:
        raise RuntimeError(f"cnn7nl_f64 failed: {rc}")
    return out, ab


def cnn_f64_paper_order(image, filt, shp: Shape):
    """Eq. 1 with the loops nested in the order the paper lists them (b,c,k,w,h,r,s)."""
    image, filt = _check_inputs(image, filt, shp, np.float64)
    out = np.empty(shp.out_shape, dtype=np.float64)
    rc = _load().cnn7nl_f64_paper_order(_dp(image), _dp(filt), _dp(out), *shp.args())
    if rc != 0:
        raise RuntimeError(f"cnn7nl_f64_paper_order failed: {rc}")
    return out


def cnn_bf16(image_bits, filt_bits, shp: Shape, want_abs: bool = True):
    """Eq. 1 in fp64 on the exact values of bf16 bit patterns (uint16 arrays)."""
    image_bits, filt_bits = _check_inputs(image_bits, filt_bits, shp, np.uint16)
    out = np.empty(shp.out_shape, dtype=np.float64)
    ab = np.empty(shp.out_shape, dtype=np.float64) if want_abs else None
    rc = _load().cnn7nl_bf16(_u16(image_bits), _u16(filt_bits), _dp(out),
                             _dp(ab) if want_abs else None, *shp.args())
    if rc != 0:
        raise RuntimeError(f"cnn7nl_bf16 failed: {rc}")
    return out, ab


def cnn_bf16_at(image_bits, filt_bits, khwb, shp: Shape):
    """Selected output elements: ``khwb`` is an (n,4) int array of (k,h,w,b).  Returns (Out, Abs)."""
    image_bits, filt_bits = _check_inputs(image_bits, filt_bits, shp, np.uint16)
    khwb = np.ascontiguousarray(khwb, dtype=np.int32).reshape(-1, 4)
    n = khwb.shape[0]
    out = np.empty(n, dtype=np.float64)
    ab = np.empty(n, dtype=np.float64)
    rc = _load().cnn7nl_bf16_at(_u16(image_bits), _u16(filt_bits),
                                khwb.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)),
                                ctypes.c_int64(n), _dp(out), _dp(ab), *shp.args())
    if rc != 0:
        raise RuntimeError(f"cnn7nl_bf16_at failed: {rc}")
    return out, ab


def bf16_bits_to_f64(bits):
    """Exact decode of bf16 bit patterns (uint16) to fp64."""
    bits = np.asarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
