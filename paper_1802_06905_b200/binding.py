"""ctypes binding of ``libcconv.so`` -- argument marshalling only; every step runs in the library.

Function names mirror the C ABI (``include/cconv.h``).  Tensors are torch CUDA tensors of dtype
``bfloat16`` in the layouts of Eq. 1 / Section 2:
    Image  [Wi][Hi][C][B], Filter [K][R][S][C], Out [K][H][W][B]   (last subscript fastest).
PyTorch supplies device memory and streams; nothing is computed with it.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.environ.get("CCONV_LIB_PATH") or os.path.join(_HERE, "libcconv.so")
_lib = None

OK = 0
EINVAL, EUNSUPPORTED, ECUDA, EDEVICE_TIMEOUT, ENOMEM, ETOOLARGE = -1, -2, -3, -4, -5, -6
NOALLOC_MAX_SCRATCH_BYTES = 8 * 1024 * 1024
VARIANT_AUTO, VARIANT_SIMT, VARIANT_HALO, VARIANT_STEM, VARIANT_DIRECT = 0, 1, 2, 3, 4
OUT_BF16, OUT_F32 = 0, 1
POOL_AVG, POOL_MAX = 0, 1

EXPORTS = (
    "cconv_lower_bound", "cconv_tiling_lp", "cconv_plan_create", "cconv_plan_info_get",
    "cconv_plan_destroy", "cconv_plan_reserve_accumulate", "cconv_forward_accumulate",
    "cconv_forward_planned", "cconv_forward", "cconv_forward_strided", "cconv_forward_host",
    "cconv_forward_host_async", "cconv_host_wait",
    "cconv_forward_noalloc", "cconv_noalloc_status", "cconv_pool_lower_bound", "cconv_pool_forward",
    "cconv_parallel_lower_bound", "cconv_parallel_partition", "cconv_theorem2_case",
    "cconv_plan_status", "cconv_plan_trace_read", "cconv_stream_order_probe", "cconv_strerror",
    "cconv_last_cuda_error", "cconv_version",
)


class CconvError(RuntimeError):
    def __init__(self, code, where):
        lib = load_library()
        msg = lib.cconv_strerror(code).decode()
        if code == ECUDA:
            msg += ": " + lib.cconv_last_cuda_error().decode()
        super().__init__(f"{where}: {msg} ({code})")
        self.code = code


class PlanInfo(ctypes.Structure):
    _fields_ = [
        ("term", ctypes.c_double * 5), ("bound_words", ctypes.c_double),
        ("bound_argmax", ctypes.c_int), ("M_words", ctypes.c_double),
        ("lp_tile", ctypes.c_double * 9), ("lp_G", ctypes.c_double), ("lp_words", ctypes.c_double),
        ("variant", ctypes.c_int), ("out_dtype", ctypes.c_int),
        ("bb", ctypes.c_int), ("bc", ctypes.c_int), ("bk", ctypes.c_int), ("bw", ctypes.c_int),
        ("bh", ctypes.c_int), ("halo_w", ctypes.c_int), ("halo_h", ctypes.c_int),
        ("stages", ctypes.c_int), ("filter_stages", ctypes.c_int), ("grid", ctypes.c_int),
        ("tiles", ctypes.c_int),
        ("smem_bytes", ctypes.c_int), ("tmem_cols", ctypes.c_int),
        ("tile_words_smem", ctypes.c_double), ("compulsory_words", ctypes.c_double),
        ("tail_h0", ctypes.c_int), ("tail_bb", ctypes.c_int), ("tail_bc", ctypes.c_int),
        ("tail_bw", ctypes.c_int), ("tail_bh", ctypes.c_int), ("tail_tiles", ctypes.c_int),
        ("tail_grid", ctypes.c_int),
        ("scratch_bytes", ctypes.c_double),
        ("run_B", ctypes.c_int), ("run_H", ctypes.c_int), ("bands", ctypes.c_int),
        ("split", ctypes.c_int),
        ("filter_taps", ctypes.c_int),
        ("tile_G", ctypes.c_double), ("tile_G_over_lp_G", ctypes.c_double),
        ("est_cta_cycles", ctypes.c_double), ("est_period_cycles", ctypes.c_double),
        ("wait_variant", ctypes.c_int),
    ]

    def asdict(self):
        out = {}
        for name, _ in self._fields_:
            v = getattr(self, name)
            out[name] = list(v) if hasattr(v, "__len__") else v
        return out


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Load libcconv.so; raises loudly when it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_1802_06905_b200.build` "
            "(nvcc, sm_100a).  There is no CPU fallback.")
    lib = ctypes.CDLL(_LIB_PATH)
    i, d, vp = ctypes.c_int, ctypes.c_double, ctypes.c_void_p
    dp = ctypes.POINTER(ctypes.c_double)
    nine = [i] * 9
    lib.cconv_lower_bound.restype = i
    lib.cconv_lower_bound.argtypes = nine + [d, dp]
    lib.cconv_tiling_lp.restype = i
    lib.cconv_tiling_lp.argtypes = nine + [d, i, dp, dp, dp]
    lib.cconv_plan_create.restype = i
    lib.cconv_plan_create.argtypes = [ctypes.POINTER(vp)] + nine + [i, d, i, i]
    lib.cconv_plan_info_get.restype = i
    lib.cconv_plan_info_get.argtypes = [vp, ctypes.POINTER(PlanInfo)]
    lib.cconv_plan_destroy.restype = None
    lib.cconv_plan_destroy.argtypes = [vp]
    lib.cconv_forward_planned.restype = i
    lib.cconv_forward_planned.argtypes = [vp, vp, vp, vp, vp]
    lib.cconv_plan_reserve_accumulate.restype = i
    lib.cconv_plan_reserve_accumulate.argtypes = [vp]
    lib.cconv_forward_accumulate.restype = i
    lib.cconv_forward_accumulate.argtypes = [vp, vp, vp, vp, vp]
    lib.cconv_forward.restype = i
    lib.cconv_forward.argtypes = [vp, vp, vp] + nine + [i, vp]
    i64p = ctypes.POINTER(ctypes.c_int64)
    lib.cconv_stream_order_probe.restype = i
    lib.cconv_stream_order_probe.argtypes = [vp] * 7 + [i, d, d, i]
    lib.cconv_forward_strided.restype = i
    lib.cconv_forward_strided.argtypes = [vp, i64p, vp, i64p, vp, i64p] + nine + [i, vp]
    lib.cconv_forward_noalloc.restype = i
    lib.cconv_forward_noalloc.argtypes = [vp, vp, vp] + nine + [i, vp, ctypes.POINTER(i)]
    lib.cconv_noalloc_status.restype = i
    lib.cconv_noalloc_status.argtypes = [vp, ctypes.POINTER(i)]
    lib.cconv_forward_host.restype = i
    lib.cconv_forward_host.argtypes = [vp, vp, vp, vp, vp]
    lib.cconv_forward_host_async.restype = i
    lib.cconv_forward_host_async.argtypes = [vp, vp, vp, vp, vp]
    lib.cconv_host_wait.restype = i
    lib.cconv_host_wait.argtypes = [vp, vp]
    lib.cconv_theorem2_case.restype = i
    lib.cconv_theorem2_case.argtypes = [i] * 7 + [d, ctypes.POINTER(i), dp]
    lib.cconv_parallel_lower_bound.restype = i
    lib.cconv_parallel_lower_bound.argtypes = nine + [d, i, i, i, i, dp]
    lib.cconv_parallel_partition.restype = i
    lib.cconv_parallel_partition.argtypes = nine + [d, i, ctypes.POINTER(i), dp]
    lib.cconv_pool_lower_bound.restype = i
    lib.cconv_pool_lower_bound.argtypes = nine + [d, dp]
    lib.cconv_pool_forward.restype = i
    lib.cconv_pool_forward.argtypes = [vp, vp] + nine + [i, i, vp]
    lib.cconv_plan_status.restype = i
    lib.cconv_plan_status.argtypes = [vp, vp, ctypes.POINTER(i)]
    lib.cconv_plan_trace_read.restype = i
    lib.cconv_plan_trace_read.argtypes = [vp, ctypes.POINTER(ctypes.c_ulonglong), i]
    lib.cconv_strerror.restype = ctypes.c_char_p
    lib.cconv_strerror.argtypes = [i]
    lib.cconv_last_cuda_error.restype = ctypes.c_char_p
    lib.cconv_version.restype = i
    _lib = lib
    return lib


def _check(code, where):
    if code != OK:
        raise CconvError(code, where)


def lower_bound(B, C, K, W, H, R, S, sw, sh, M_words):
    """cconv_lower_bound: the five terms of Theorem 1 (host arithmetic inside the library)."""
    t = (ctypes.c_double * 5)()
    _check(load_library().cconv_lower_bound(B, C, K, W, H, R, S, sw, sh, float(M_words), t),
           "cconv_lower_bound")
    return list(t)


def theorem2_case(B, C, K, W, H, R, S, M_words):
    """cconv_theorem2_case: (leaf name as a string such as "2.2.2.1", attainable bound in words)."""
    leaf, alb = ctypes.c_int(), ctypes.c_double()
    _check(load_library().cconv_theorem2_case(B, C, K, W, H, R, S, float(M_words),
                                              ctypes.byref(leaf), ctypes.byref(alb)),
           "cconv_theorem2_case")
    return ".".join(str(leaf.value)), alb.value


def parallel_lower_bound(B, C, K, W, H, R, S, sw, sh, M_words, aB, aK, aH, aW):
    """cconv_parallel_lower_bound: the five terms for an aB x aK x aH x aW cut (Section 8)."""
    t = (ctypes.c_double * 5)()
    _check(load_library().cconv_parallel_lower_bound(B, C, K, W, H, R, S, sw, sh, float(M_words),
                                                     aB, aK, aH, aW, t),
           "cconv_parallel_lower_bound")
    return list(t)


def parallel_partition(B, C, K, W, H, R, S, sw, sh, M_words, p):
    """cconv_parallel_partition: ((aB, aK, aH, aW), bound in words) for p processors."""
    a = (ctypes.c_int * 4)()
    bound = ctypes.c_double()
    _check(load_library().cconv_parallel_partition(B, C, K, W, H, R, S, sw, sh, float(M_words),
                                                   int(p), a, ctypes.byref(bound)),
           "cconv_parallel_partition")
    return tuple(a), bound.value


def pool_lower_bound(B, C, K, W, H, R, S, sw, sh, M_words):
    """cconv_pool_lower_bound: the three terms of the pooling bound (Section 6)."""
    t = (ctypes.c_double * 3)()
    _check(load_library().cconv_pool_lower_bound(B, C, K, W, H, R, S, sw, sh, float(M_words), t),
           "cconv_pool_lower_bound")
    return list(t)


def pool_forward_ptrs(image_ptr, out_ptr, B, C, K, W, H, R, S, sw, sh, op, out_dtype=0, stream=0):
    """cconv_pool_forward on raw device addresses (asynchronous on ``stream``)."""
    _check(load_library().cconv_pool_forward(ctypes.c_void_p(image_ptr), ctypes.c_void_p(out_ptr),
                                             B, C, K, W, H, R, S, sw, sh, int(op), int(out_dtype),
                                             ctypes.c_void_p(stream)), "cconv_pool_forward")


def pool_forward(image, out, B, C, K, W, H, R, S, sw=1, sh=1, op=0, stream=None):
    """cconv_pool_forward on torch CUDA tensors: Image bf16 [Wi][Hi][C][B], Out [K][H][W][B] bf16 or
    fp32 (its dtype selects the output type).  Argument marshalling only."""
    import torch
    Wi, Hi = sw * (W - 1) + R, sh * (H - 1) + S
    if tuple(image.shape) != (Wi, Hi, C, B) or image.dtype != torch.bfloat16:
        raise ValueError(f"Image must be bf16 {(Wi, Hi, C, B)}")
    if tuple(out.shape) != (K, H, W, B) or out.dtype not in (torch.bfloat16, torch.float32):
        raise ValueError(f"Out must be bf16 or fp32 {(K, H, W, B)}")
    if not (image.is_cuda and out.is_cuda and image.is_contiguous() and out.is_contiguous()):
        raise ValueError("dense CUDA tensors are required")
    sp = (stream or torch.cuda.current_stream(image.device)).cuda_stream
    with torch.cuda.device(image.device):
        pool_forward_ptrs(image.data_ptr(), out.data_ptr(), B, C, K, W, H, R, S, sw, sh, op,
                          OUT_F32 if out.dtype == torch.float32 else OUT_BF16, sp)


def stream_order_probe(stream_key, image, filt, out, overlap, sms_by_memory=0.0, sms_by_threads=0.0,
                       sm_count=148):
    """cconv_stream_order_probe: registers a call given as three (lo, hi) byte ranges (None = no such
    array) with the stream-order bookkeeping of ``stream_key`` and returns the hazard bits."""
    def rng(r):
        return (None, None) if r is None else (ctypes.c_void_p(r[0]), ctypes.c_void_p(r[1]))
    (il, ih), (fl, fh), (ol, oh) = rng(image), rng(filt), rng(out)
    rc = load_library().cconv_stream_order_probe(ctypes.c_void_p(stream_key), il, ih, fl, fh, ol, oh,
                                                 int(overlap), float(sms_by_memory), float(sms_by_threads),
                                                 int(sm_count))
    if rc < 0:
        _check(rc, "cconv_stream_order_probe")
    return rc


def tiling_lp(B, C, K, W, H, R, S, sw, sh, M_words, pooling=False):
    """cconv_tiling_lp: (tiles[9], G, words) of the Section-5 LP."""
    t = (ctypes.c_double * 9)()
    G, wd = ctypes.c_double(), ctypes.c_double()
    _check(load_library().cconv_tiling_lp(B, C, K, W, H, R, S, sw, sh, float(M_words),
                                          int(bool(pooling)), t, ctypes.byref(G), ctypes.byref(wd)),
           "cconv_tiling_lp")
    return list(t), G.value, wd.value


def _stream_ptr(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _tensor_args(image, filt, out, dims, out_dtype=OUT_BF16):
    import torch
    B, C, K, W, H, R, S, sw, sh = dims
    exp = ((sw * (W - 1) + R, sh * (H - 1) + S, C, B), (K, R, S, C), (K, H, W, B))
    dts = (torch.bfloat16, torch.bfloat16, torch.float32 if out_dtype == OUT_F32 else torch.bfloat16)
    for name, t, shp, dt in zip(("Image", "Filter", "Out"), (image, filt, out), exp, dts):
        if not (t.is_cuda and t.dtype == dt and t.is_contiguous()):
            raise ValueError(f"{name} must be a contiguous CUDA {dt} tensor")
        if tuple(t.shape) != shp:
            raise ValueError(f"{name} shape {tuple(t.shape)} != {shp}")
    return (ctypes.c_void_p(image.data_ptr()), ctypes.c_void_p(filt.data_ptr()),
            ctypes.c_void_p(out.data_ptr()))


class Plan:
    """Owner of a ``cconv_plan`` handle."""

    def __init__(self, B, C, K, W, H, R, S, sw=1, sh=1, device=0, M_words=0.0,
                 variant=VARIANT_AUTO, out_dtype=OUT_BF16):
        self._lib = load_library()
        self.dims = (B, C, K, W, H, R, S, sw, sh)
        self.out_dtype = int(out_dtype)
        self._h = ctypes.c_void_p()
        _check(self._lib.cconv_plan_create(ctypes.byref(self._h), *self.dims, int(device),
                                           float(M_words), int(variant), self.out_dtype),
               "cconv_plan_create")

    def info(self) -> dict:
        pi = PlanInfo()
        _check(self._lib.cconv_plan_info_get(self._h, ctypes.byref(pi)), "cconv_plan_info_get")
        return pi.asdict()

    def forward(self, image, filt, out, stream=None):
        """cconv_forward_planned on torch CUDA tensors; asynchronous on ``stream``."""
        pi, pf, po = _tensor_args(image, filt, out, self.dims, self.out_dtype)
        _check(self._lib.cconv_forward_planned(self._h, pi, pf, po, _stream_ptr(stream)),
               "cconv_forward_planned")
        return out

    def reserve_accumulate(self):
        """cconv_plan_reserve_accumulate: allocate what forward_accumulate needs (once per plan)."""
        _check(self._lib.cconv_plan_reserve_accumulate(self._h), "cconv_plan_reserve_accumulate")

    def forward_accumulate(self, image, filt, out, stream=None):
        """cconv_forward_accumulate on torch CUDA tensors: out += Eq. 1; asynchronous on ``stream``."""
        pi, pf, po = _tensor_args(image, filt, out, self.dims, self.out_dtype)
        _check(self._lib.cconv_forward_accumulate(self._h, pi, pf, po, _stream_ptr(stream)),
               "cconv_forward_accumulate")
        return out

    def forward_ptrs(self, image_ptr, filt_ptr, out_ptr, stream_ptr):
        """cconv_forward_planned on raw device addresses (the benchmark's inner loop)."""
        return self._lib.cconv_forward_planned(self._h, image_ptr, filt_ptr, out_ptr, stream_ptr)

    def forward_host(self, h_image, h_filt, h_out, stream=None):
        """cconv_forward_host on CPU tensors (pinned for asynchronous copies); synchronises."""
        _check(self._lib.cconv_forward_host(self._h, ctypes.c_void_p(h_image.data_ptr()),
                                            ctypes.c_void_p(h_filt.data_ptr()),
                                            ctypes.c_void_p(h_out.data_ptr()), _stream_ptr(stream)),
               "cconv_forward_host")
        return h_out

    def forward_host_async(self, h_image, h_filt, h_out, stream=None):
        """cconv_forward_host_async on pinned CPU tensors: queues the copies and the kernels and
        returns; ``host_wait`` makes ``h_out`` valid."""
        _check(self._lib.cconv_forward_host_async(self._h, ctypes.c_void_p(h_image.data_ptr()),
                                                  ctypes.c_void_p(h_filt.data_ptr()),
                                                  ctypes.c_void_p(h_out.data_ptr()), _stream_ptr(stream)),
               "cconv_forward_host_async")
        return h_out

    def host_wait(self, stream=None):
        """cconv_host_wait: waits for every queued forward_host_async call; raises on a device status."""
        _check(self._lib.cconv_host_wait(self._h, _stream_ptr(stream)), "cconv_host_wait")

    def status(self, stream=None):
        """cconv_plan_status: synchronises and returns (code, detail bit mask)."""
        detail = ctypes.c_int(0)
        code = self._lib.cconv_plan_status(self._h, _stream_ptr(stream), ctypes.byref(detail))
        return code, detail.value

    def trace(self):
        """cconv_plan_trace_read: (grid, 16) array of device time stamps in ns (empty if off)."""
        import numpy as np
        n = (148 + 16) * 16
        buf = (ctypes.c_ulonglong * n)()
        got = self._lib.cconv_plan_trace_read(self._h, buf, n)
        if got < 0:
            raise CconvError(got, "cconv_plan_trace_read")
        return np.array(buf[:got], dtype=np.uint64).reshape(-1, 16)

    def check(self, stream=None):
        code, detail = self.status(stream)
        if code != OK:
            raise CconvError(code, f"cconv_plan_status (detail={detail:#x})")

    def close(self):
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.cconv_plan_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def conv_forward(image, filt, out, B, C, K, W, H, R, S, sw=1, sh=1, out_dtype=OUT_BF16,
                 stream=None):
    """cconv_forward: plan (cached per shape) and launch; asynchronous on ``stream``."""
    dims = (B, C, K, W, H, R, S, sw, sh)
    pi, pf, po = _tensor_args(image, filt, out, dims, out_dtype)
    _check(load_library().cconv_forward(pi, pf, po, *dims, int(out_dtype), _stream_ptr(stream)),
           "cconv_forward")
    return out


def conv_forward_noalloc(image, filt, out, B, C, K, W, H, R, S, sw=1, sh=1, out_dtype=OUT_BF16,
                         stream=None, sync=False):
    """cconv_forward_noalloc: the tensor-core convolution for callers that may not allocate device
    memory (its scratch is a fixed array inside the library).  ``sync=True`` also synchronises the
    stream and checks the device status word.  Returns the C return code's success as ``out``."""
    dims = (B, C, K, W, H, R, S, sw, sh)
    pi, pf, po = _tensor_args(image, filt, out, dims, out_dtype)
    st = ctypes.c_int(0)
    rc = load_library().cconv_forward_noalloc(pi, pf, po, *dims, int(out_dtype), _stream_ptr(stream),
                                              ctypes.byref(st) if sync else None)
    _check(rc, f"cconv_forward_noalloc (device status {st.value:#x})")
    return out


def noalloc_status(stream=None):
    """cconv_noalloc_status: synchronises, returns (code, detail bit mask) of the asynchronous
    cconv_forward_noalloc calls made so far on the current device, and clears the word."""
    st = ctypes.c_int(0)
    code = load_library().cconv_noalloc_status(_stream_ptr(stream), ctypes.byref(st))
    return code, st.value


def conv_forward_strided(image, filt, out, B, C, K, W, H, R, S, sw=1, sh=1, out_dtype=OUT_BF16,
                         stream=None):
    """cconv_forward_strided on torch CUDA tensors of ANY strides: ``image`` indexed (x, y, c, b),
    ``filt`` (k, r, s, c), ``out`` (k, h, w, b); the strides are taken from the tensors."""
    Wi, Hi = sw * (W - 1) + R, sh * (H - 1) + S
    for name, t, shp in (("Image", image, (Wi, Hi, C, B)), ("Filter", filt, (K, R, S, C)),
                         ("Out", out, (K, H, W, B))):
        if tuple(t.shape) != shp or not t.is_cuda:
            raise ValueError(f"{name}: CUDA tensor of shape {shp} expected, got {tuple(t.shape)}")
    arr = lambda t: (ctypes.c_int64 * 4)(*[int(v) if v > 0 else 1 for v in t.stride()])
    rc = load_library().cconv_forward_strided(
        ctypes.c_void_p(image.data_ptr()), arr(image), ctypes.c_void_p(filt.data_ptr()), arr(filt),
        ctypes.c_void_p(out.data_ptr()), arr(out), B, C, K, W, H, R, S, sw, sh, int(out_dtype),
        _stream_ptr(stream))
    _check(rc, "cconv_forward_strided")
    return out
