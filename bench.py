#!/usr/bin/env python
"""Benchmark of the seven-nested-loop CNN hot path (Eq. 1) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl reference]

One "step" is one pass of the whole hot path (plan lookup, TMA descriptor use, the convolution
kernel) over one batch of seeded synthetic input.  The default workload is the second benchmark
shape (ResNet-style 3x3, B=32, C=K=256, 14x14 outputs).  Its working set (8.6 MB) is far below the
126 MB L2, so the timed loop rotates through enough distinct buffer sets to exceed L2
("l2": "rotating buffer sets" in `config`).  Timing: CUDA events on the launching stream around
exactly K steps, barrier + synchronize on both sides, max over ranks.

Output: ONE JSON line on rank 0 with metric conv TFLOP/s (2*B*C*K*W*H*R*S / time), the roofline
of the dominant kernel, an end-to-end number through the host-buffer entry point, the CPU oracle
timed as a baseline, sampled SM clocks, and per-configuration results for the other shapes.

`--impl reference` times the fp64 CPU oracle (the only "reference implementation" of this paper,
which ships no code) on the host cores, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_1802_06905_b200.synth import CONFIGS, ConvShape, make_inputs  # noqa: E402

METRIC = "conv TFLOP/s & % of roofline; HBM bytes vs paper's lower bound"
L2_BYTES = 126 * 1024 * 1024


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "source": "fallback"}


def dram_traffic_from_profiles(name):
    """Per-launch DRAM bytes of the dominant kernel from a committed ncu summary, or None."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    with open(path) as fh:
        for line in fh:
            parts = line.split()
            if len(parts) >= 2 and parts[0] == name:
                try:
                    return float(parts[1])
                except ValueError:
                    return None
    return None


class ClockSampler:
    """Samples SM clock and throttle reasons while the timed region runs (NVML, else nvidia-smi)."""

    BAD = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40}
    NOTE = {"sw_power_cap": 0x4}

    def __init__(self, index):
        self.index = index
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thr = None
        self._nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nvml = None

    def sample_once(self):
        if self._nvml is not None:
            try:
                n = self._nvml
                self.samples.append(n.nvmlDeviceGetClockInfo(self._h, n.NVML_CLOCK_SM))
                mask = n.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                for k, bit in {**self.BAD, **self.NOTE}.items():
                    if mask & bit:
                        self.reasons.add(k)
                return
            except Exception:
                pass
        try:
            out = subprocess.run(
                ["nvidia-smi", "-i", str(self.index),
                 "--query-gpu=clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
                 "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                 "clocks_event_reasons.sw_power_cap", "--format=csv,noheader,nounits"],
                capture_output=True, text=True, timeout=10).stdout.strip().split(",")
            self.samples.append(float(out[0]))
            self.max_mhz = float(out[1])
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                "sw_power_cap"), out[2:]):
                if v.strip().lower().startswith("active"):
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample_once()
            self._stop.wait(0.005 if self._nvml is not None else 0.2)

    def start(self):
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": float(self.max_mhz) if self.max_mhz else None,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def to_dev(bits, torch, dev):
    return torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(dev)


def time_config(cfg, torch, binding, dev, steps, warmup, dist=None, sampler=None):
    """Device-resident timing of one configuration.  Returns (seconds for `steps`, plan info)."""
    ib, fb = make_inputs(cfg)
    set_bytes = 2 * (cfg.image_words + cfg.filter_words + cfg.out_words)
    nsets = max(2, min(64, -(-int(1.5 * L2_BYTES) // set_bytes)))
    base_i, base_f = to_dev(ib, torch, dev), to_dev(fb, torch, dev)
    imgs = [base_i] + [base_i.clone() for _ in range(nsets - 1)]
    flts = [base_f] + [base_f.clone() for _ in range(nsets - 1)]
    outs = [torch.empty(cfg.out_shape, dtype=torch.bfloat16, device=dev) for _ in range(nsets)]
    plan = binding.Plan(*cfg.dims(), device=dev.index, out_dtype=binding.OUT_BF16)
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    ptrs = [(imgs[i].data_ptr(), flts[i].data_ptr(), outs[i].data_ptr()) for i in range(nsets)]
    for i in range(max(warmup, 3)):
        a, b, c = ptrs[i % nsets]
        rc = plan.forward_ptrs(a, b, c, sp)
        assert rc == 0, rc
    plan.check()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    if sampler:
        sampler.start()
    e0.record(stream)
    for i in range(steps):
        a, b, c = ptrs[i % nsets]
        plan.forward_ptrs(a, b, c, sp)
    e1.record(stream)
    if sampler:
        sampler.sample_once()
    torch.cuda.synchronize()
    if sampler:
        sampler.stop()
    if dist is not None:
        dist.barrier()
    plan.check()
    secs = e0.elapsed_time(e1) * 1e-3
    info = plan.info()
    plan.close()
    return secs, info, nsets


def time_repeats(cfg, torch, binding, dev, launches, repeats=5):
    """Per-configuration table: median over `repeats` of the CUDA-event time of `launches`
    back-to-back forward calls, L2-cold (rotating buffer sets larger than L2) and L2-warm (one
    buffer set), and L2-cold again with the calls captured once into a CUDA graph and replayed.
    Returns (cold seconds per call, warm seconds per call, plan info, graph seconds per call)."""
    ib, fb = make_inputs(cfg)
    set_bytes = 2 * (cfg.image_words + cfg.filter_words + cfg.out_words)
    nsets = max(2, min(64, -(-int(1.5 * L2_BYTES) // set_bytes)))
    base_i, base_f = to_dev(ib, torch, dev), to_dev(fb, torch, dev)
    imgs = [base_i] + [base_i.clone() for _ in range(nsets - 1)]
    flts = [base_f] + [base_f.clone() for _ in range(nsets - 1)]
    outs = [torch.empty(cfg.out_shape, dtype=torch.bfloat16, device=dev) for _ in range(nsets)]
    plan = binding.Plan(*cfg.dims(), device=dev.index, out_dtype=binding.OUT_BF16)
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    ptrs = [(imgs[i].data_ptr(), flts[i].data_ptr(), outs[i].data_ptr()) for i in range(nsets)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    result = []
    for rotate in (True, False):
        times = []
        for rep in range(repeats + 1):            # the first repeat is warm-up
            torch.cuda.synchronize()
            e0.record(stream)
            for i in range(launches):
                a, b, c = ptrs[i % nsets] if rotate else ptrs[0]
                plan.forward_ptrs(a, b, c, sp)
            e1.record(stream)
            torch.cuda.synchronize()
            if rep:
                times.append(e0.elapsed_time(e1) * 1e-3 / launches)
        result.append(float(np.median(times)))
    # the same rotation captured once into a CUDA graph and replayed (no host work per call)
    graph_s = None
    try:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            cap = torch.cuda.current_stream().cuda_stream
            for i in range(launches):
                a, b, c = ptrs[i % nsets]
                plan.forward_ptrs(a, b, c, cap)
        g.replay()
        torch.cuda.synchronize()
        times = []
        for rep in range(repeats):
            e0.record(stream)
            g.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1) * 1e-3 / launches)
        graph_s = float(np.median(times))
        del g
    except RuntimeError:
        graph_s = None
    plan.check()
    info = plan.info()
    plan.close()
    return result[0], result[1], info, graph_s


def time_general_shapes(torch, binding, dev, launches=30, repeats=3):
    """Shapes outside the five benchmark configurations that exercise the planner's other paths:
    tiles split over clusters of 2 or 4 CTAs (few output pixels, long channel loops) and bands of
    output rows standing in for images (B < 8).  Each shape is timed twice, back-to-back calls on one
    buffer set: as planned, and with that path switched off through the planner's diagnostic
    environment variables (read at plan creation)."""
    shapes = [("resnet50_conv5_3x3_b64", (64, 512, 512, 7, 7, 3, 3, 1, 1), "CCONV_FORCE_TILE", "0,0,0,0,0,1"),
              ("deep_7x7_3x3_b16", (16, 1024, 256, 7, 7, 3, 3, 1, 1), "CCONV_FORCE_TILE", "0,0,0,0,0,1"),
              ("deep_7x7_5x5_b8", (8, 512, 512, 7, 7, 5, 5, 1, 1), "CCONV_FORCE_TILE", "0,0,0,0,0,1"),
              ("single_image_56x56_3x3", (1, 256, 256, 56, 56, 3, 3, 1, 1), "CCONV_BANDS", "1")]
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rows = []
    for name, dims, var, off in shapes:
        c = ConvShape(name, *dims)
        ib, fb = make_inputs(c)
        img, flt = to_dev(ib, torch, dev), to_dev(fb, torch, dev)
        out = torch.empty(c.out_shape, dtype=torch.bfloat16, device=dev)
        res = {}
        for label, value in (("planned", None), ("path_off", off)):
            saved = os.environ.get(var)
            if value is None:
                os.environ.pop(var, None)
            else:
                os.environ[var] = value
            try:
                plan = binding.Plan(*dims, device=dev.index, out_dtype=binding.OUT_BF16)
            finally:
                if saved is None:
                    os.environ.pop(var, None)
                else:
                    os.environ[var] = saved
            times = []
            for rep in range(repeats + 1):
                torch.cuda.synchronize()
                e0.record(stream)
                for _ in range(launches):
                    plan.forward_ptrs(img.data_ptr(), flt.data_ptr(), out.data_ptr(), sp)
                e1.record(stream)
                torch.cuda.synchronize()
                if rep:
                    times.append(e0.elapsed_time(e1) * 1e3 / launches)
            plan.check()
            info = plan.info()
            plan.close()
            res[label] = {"us_per_launch": float(np.median(times)), "split": info["split"],
                          "bands": info["bands"], "grid": info["grid"],
                          "tile": [info[k] for k in ("bb", "bw", "bh", "bc")]}
        rows.append({"workload": name, "dims": dict(zip("B C K W H R S sw sh".split(), dims)),
                     "tflops": c.flops / res["planned"]["us_per_launch"] / 1e6, **res})
    return rows


def time_pooling(torch, binding, dev, peaks, launches=50, repeats=5):
    """Pooling (Section 6) rows: median CUDA-event time of back-to-back cconv_pool_forward calls over
    rotating buffer sets larger than L2.  Algorithmic bytes = Image + Out, each moved once; the
    roofline is the measured HBM copy rate."""
    from paper_1802_06905_b200.synth import POOL_SHAPES
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rows = []
    gen = torch.Generator(device="cpu").manual_seed(0x18020690 + 60)
    for name, B, C, K, W, H, R, S, sw, sh in POOL_SHAPES:
        Wi, Hi = sw * (W - 1) + R, sh * (H - 1) + S
        ibytes, obytes = 2 * Wi * Hi * C * B, 2 * K * H * W * B
        nsets = max(2, min(16, -(-int(1.5 * L2_BYTES) // (ibytes + obytes))))
        base = torch.randn((Wi, Hi, C, B), generator=gen).to(torch.bfloat16).to(dev)
        imgs = [base] + [base.clone() for _ in range(nsets - 1)]
        outs = [torch.empty((K, H, W, B), dtype=torch.bfloat16, device=dev) for _ in range(nsets)]
        terms = binding.pool_lower_bound(B, C, K, W, H, R, S, sw, sh, L2_BYTES / 4.0)
        for op, opname in ((binding.POOL_AVG, "avg"), (binding.POOL_MAX, "max")):
            times = []
            for rep in range(repeats + 1):        # the first repeat is warm-up
                torch.cuda.synchronize()
                e0.record(stream)
                for i in range(launches):
                    binding.pool_forward_ptrs(imgs[i % nsets].data_ptr(), outs[i % nsets].data_ptr(),
                                              B, C, K, W, H, R, S, sw, sh, op, binding.OUT_BF16, sp)
                e1.record(stream)
                torch.cuda.synchronize()
                if rep:
                    times.append(e0.elapsed_time(e1) * 1e-3 / launches)
            t = float(np.median(times))
            rows.append({"workload": name, "op": opname,
                         "dims": dict(zip("B C K W H R S sw sh".split(), (B, C, K, W, H, R, S, sw, sh))),
                         "us_per_launch": t * 1e6, "algorithmic_bytes": ibytes + obytes,
                         "gbs": (ibytes + obytes) / t / 1e9,
                         "roofline": {"bound": "hbm", "achieved": (ibytes + obytes) / t / 1e9,
                                      "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                      "frac": (ibytes + obytes) / t / 1e9 / peaks["hbm_gbs"]},
                         "lower_bound_bytes_at_L2": 2.0 * max(terms), "launches": launches})
        del imgs, outs, base
    return rows


def oracle_sample(cfg, budget_s=2.5):
    """The CPU oracle on a bounded k-slice of one configuration: (TFLOP/s, cores, seconds, sample)."""
    from oracle import cnn as ocnn
    ib, fb = make_inputs(cfg)
    threads = ocnn.max_threads()
    k_probe = min(cfg.K, max(1, threads))
    shp = ocnn.Shape(cfg.B, cfg.C, k_probe, cfg.W, cfg.H, cfg.R, cfg.S, cfg.sw, cfg.sh)
    t0 = time.perf_counter()
    ocnn.cnn_bf16(ib, fb[:k_probe], shp)
    t_probe = time.perf_counter() - t0
    k_sub = int(min(cfg.K, max(k_probe, k_probe * budget_s // max(t_probe, 1e-9))))
    shp = ocnn.Shape(cfg.B, cfg.C, k_sub, cfg.W, cfg.H, cfg.R, cfg.S, cfg.sw, cfg.sh)
    t0 = time.perf_counter()
    ocnn.cnn_bf16(ib, fb[:k_sub], shp)
    t = time.perf_counter() - t0
    return {"tflops": 2.0 * shp.macs / t / 1e12, "cores": threads, "seconds": t,
            "sample": f"out-channels 0..{k_sub - 1} of {cfg.K}"}


def time_e2e(cfg, torch, binding, dev, steps):
    """The same metric through the host-buffer entry point: H2D of Image and Filter from pinned
    memory, the kernel, D2H of Out, every step."""
    ib, fb = make_inputs(cfg)
    hi = torch.from_numpy(ib.view(np.int16)).view(torch.bfloat16).pin_memory()
    hf = torch.from_numpy(fb.view(np.int16)).view(torch.bfloat16).pin_memory()
    ho = torch.empty(cfg.out_shape, dtype=torch.bfloat16).pin_memory()
    plan = binding.Plan(*cfg.dims(), device=dev.index, out_dtype=binding.OUT_BF16)
    stream = torch.cuda.current_stream()
    for _ in range(3):
        plan.forward_host(hi, hf, ho, stream)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(steps):
        plan.forward_host(hi, hf, ho, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    secs_sync = e0.elapsed_time(e1) * 1e-3
    # the same steps through the pipelined entry point: every step still copies its Image and Filter
    # in and its Out back, but the copies of neighbouring steps overlap (two staging sets, a copy
    # stream per direction); the wait for the last Out is inside the timed region
    for _ in range(3):
        plan.forward_host_async(hi, hf, ho, stream)
    plan.host_wait(stream)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(steps):
        plan.forward_host_async(hi, hf, ho, stream)
    plan.host_wait(stream)
    e1.record(stream)
    torch.cuda.synchronize()
    secs = e0.elapsed_time(e1) * 1e-3
    plan.close()
    return secs, 2 * (cfg.image_words + cfg.filter_words), 2 * cfg.out_words, secs_sync


def kernels_per_step(info, binding):
    """Kernels of this library launched by one forward call."""
    if info["variant"] == binding.VARIANT_SIMT:
        return 1
    n = 2                                    # Filter packing + convolution
    if info["variant"] == binding.VARIANT_HALO and info["tail_tiles"] > 0:
        n += 1                               # wave-quantisation tail launch
    return n


def write_only_gbs(torch, dev):
    """HBM bandwidth of a write-only stream: cudaMemsetAsync over rotating 256 MB buffers (the CUDA
    runtime that torch has loaded, called through ctypes; torch's own fill kernel reaches only about
    two thirds of this rate and is used only if the runtime cannot be reached).  The copy figure
    in MEASURED_PEAKS.json counts bytes read plus bytes written; a kernel that mostly writes Out is
    bounded by this figure instead."""
    import ctypes
    n = 256 * 1024 * 1024
    bufs = [torch.empty(n, dtype=torch.uint8, device=dev) for _ in range(3)]
    for b in bufs:
        b.zero_()
    stream = torch.cuda.current_stream()
    memset = None
    try:
        rt = ctypes.CDLL("libcudart.so.12")
        rt.cudaMemsetAsync.restype = ctypes.c_int
        rt.cudaMemsetAsync.argtypes = [ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_void_p]
        if rt.cudaMemsetAsync(bufs[0].data_ptr(), 0, n, stream.cuda_stream) == 0:
            memset = rt.cudaMemsetAsync
    except (OSError, AttributeError):
        memset = None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    reps = 12
    for i in range(reps):
        if memset is not None:
            memset(bufs[i % 3].data_ptr(), 0, n, stream.cuda_stream)
        else:
            bufs[i % 3].zero_()
    e1.record(stream)
    torch.cuda.synchronize()
    return n * reps / (e0.elapsed_time(e1) * 1e-3) / 1e9


def roofline_for(cfg, info, secs_per_launch, peaks, binding):
    """Roofline of the dominant kernel: tensor-bound where the tcgen05 kernel ran (dense
    contraction), HBM-bound for the CUDA-core kernel (reported against compulsory bytes)."""
    traffic = dram_traffic_from_profiles(cfg.name)
    if info["variant"] in (binding.VARIANT_HALO, binding.VARIANT_STEM):
        ach = cfg.flops / secs_per_launch / 1e12
        peak = peaks["bf16_tflops"]
        kernel = "cconv_halo_kernel" if info["variant"] == binding.VARIANT_HALO else "cconv_stem_kernel"
        return {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                "frac": ach / peak, "traffic": traffic, "peak_source": peaks["source"],
                "kernel": kernel,
                "duration": "CUDA-event time of one forward call (Filter packing included) "
                            "/ launches; the convolution kernel alone is shorter"}
    byts = 2.0 * info["compulsory_words"]
    ach = byts / secs_per_launch / 1e9
    return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
            "frac": ach / peaks["hbm_gbs"], "traffic": traffic, "peak_source": peaks["source"],
            "kernel": "cconv_simt_kernel"}


def applicable_roofline_seconds(cfg, info, peaks):
    """t_roof = max(flops / bf16 peak, lower-bound bytes at M = L2 / HBM bandwidth)."""
    from paper_1802_06905_b200 import binding
    terms = binding.lower_bound(*cfg.dims(), L2_BYTES / 2)  # the L2 capacity in bf16 words
    lb_bytes = 2.0 * max(terms)
    return max(cfg.flops / (peaks["bf16_tflops"] * 1e12), lb_bytes / (peaks["hbm_gbs"] * 1e9)), lb_bytes


def cpu_baseline(cfg, budget_s=20.0):
    """The oracle as it stands, timed on the host cores on a bounded sample of the workload:
    the first k_sub output channels (a slice of Filter), sized from a short probe."""
    from oracle import cnn as ocnn
    ib, fb = make_inputs(cfg)
    threads = ocnn.max_threads()
    k_probe = min(cfg.K, max(1, threads))
    shp = ocnn.Shape(cfg.B, cfg.C, k_probe, cfg.W, cfg.H, cfg.R, cfg.S, cfg.sw, cfg.sh)
    t0 = time.perf_counter()
    ocnn.cnn_bf16(ib, fb[:k_probe], shp)
    t_probe = time.perf_counter() - t0
    rate = shp.macs / max(t_probe, 1e-9)
    k_sub = int(min(cfg.K, max(k_probe, (budget_s * rate) // (shp.macs // k_probe))))
    shp = ocnn.Shape(cfg.B, cfg.C, k_sub, cfg.W, cfg.H, cfg.R, cfg.S, cfg.sw, cfg.sh)
    passes, t = 0, 0.0
    while passes < 1 or (t < 3.0 and passes < 50):   # a quick workload is timed over several passes
        t0 = time.perf_counter()
        ocnn.cnn_bf16(ib, fb[:k_sub], shp)
        t += time.perf_counter() - t0
        passes += 1
    return {"value": 2.0 * shp.macs * passes / t / 1e12, "unit": "TFLOP/s", "cores": threads,
            "kind": "oracle", "seconds": t,
            "sample": f"output channels 0..{k_sub - 1} of {cfg.K} (all b,h,w,c,r,s), {passes} "
                      f"pass(es), fp64 with the |.| sum"}


def chosen_config(args):
    if args.shape:
        dims = tuple(int(v) for v in args.shape.split(","))
        if len(dims) != 9 or min(dims) <= 0:
            raise SystemExit("--shape wants nine positive integers: B,C,K,W,H,R,S,sw,sh")
        return ConvShape("shape_" + "x".join(str(v) for v in dims), *dims)
    return CONFIGS[args.config]


def run_reference(args):
    """--impl reference: the CPU oracle on host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import cnn as ocnn
    cfg = chosen_config(args)
    ib, fb = make_inputs(cfg)
    threads = ocnn.max_threads()
    total = args.steps + args.warmup
    step_budget = min(0.5, 150.0 / max(total, 1))
    k_probe = min(cfg.K, max(1, threads))
    shp = ocnn.Shape(cfg.B, cfg.C, k_probe, cfg.W, cfg.H, cfg.R, cfg.S, cfg.sw, cfg.sh)
    t0 = time.perf_counter()
    ocnn.cnn_bf16(ib, fb[:k_probe], shp)
    t_probe = time.perf_counter() - t0
    k_sub = int(min(cfg.K, max(1, round(k_probe * step_budget / max(t_probe, 1e-9)))))
    shp = ocnn.Shape(cfg.B, cfg.C, k_sub, cfg.W, cfg.H, cfg.R, cfg.S, cfg.sw, cfg.sh)
    for _ in range(args.warmup):
        ocnn.cnn_bf16(ib, fb[:k_sub], shp)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ocnn.cnn_bf16(ib, fb[:k_sub], shp)
    t = time.perf_counter() - t0
    val = 2.0 * shp.macs * args.steps / t / 1e12
    sample = (f"each step = output channels 0..{k_sub - 1} of {cfg.K} of {cfg.name} "
              f"(all b,h,w,c,r,s), fp64 oracle with the |.| sum")
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": t / max(args.steps, 1) * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "dims": dict(zip("B C K W H R S sw sh".split(), cfg.dims())),
                       "sample": sample},
            "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0,
                    "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--config", type=int, default=1, help="index into the five benchmark shapes")
    ap.add_argument("--shape", default=None,
                    help="B,C,K,W,H,R,S,sw,sh: time this shape instead of a benchmark configuration "
                         "(same input recipe as the default configuration; no profile figures exist for it)")
    ap.add_argument("--impl", default="cconv", choices=["cconv", "reference"])
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the per-configuration table, the e2e leg and the CPU baseline")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    from paper_1802_06905_b200 import binding
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (sm_100a); there is no CPU fallback")
    binding.load_library()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dev = torch.device("cuda", local)
    torch.cuda.set_device(dev)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod

    peaks = measured_peaks()
    cfg = chosen_config(args)
    steps, warmup = max(1, args.steps), max(3, args.warmup)
    sampler = ClockSampler(local)
    secs, info, nsets = time_config(cfg, torch, binding, dev, steps, warmup, dist, sampler)
    if dist is not None:
        t = torch.tensor([secs], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        secs = float(t.item())
    # weak scaling: every rank convolves its own batch of B images with the replicated Filter
    value = world * cfg.flops * steps / secs / 1e12
    per_launch = secs / steps
    roof = roofline_for(cfg, info, per_launch, peaks, binding)
    t_roof, lb_bytes = applicable_roofline_seconds(cfg, info, peaks)

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": per_launch * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name,
                   "dims": dict(zip("B C K W H R S sw sh".split(), cfg.dims())),
                   "l2": f"rotating {nsets} distinct buffer sets ({nsets * 2 * (cfg.image_words + cfg.filter_words + cfg.out_words) / 1e6:.0f} MB > 126 MB L2)",
                   "out_dtype": "bf16", "accumulate": "fp32",
                   "parallelism": f"batch-sharded x{world}, no collective" if world > 1 else "single GPU"},
        "roofline": roof,
        "applicable_roofline": {"t_roof_us": t_roof * 1e6, "frac": t_roof / per_launch,
                                "lower_bound_bytes_at_L2": lb_bytes,
                                "compulsory_bytes": 2.0 * info["compulsory_words"]},
        "plan": {k: info[k] for k in ("variant", "bb", "bc", "bk", "bw", "bh", "halo_w", "halo_h",
                                      "stages", "grid", "tiles", "smem_bytes", "tmem_cols",
                                      "bound_argmax", "bound_words", "lp_words", "tile_words_smem",
                                      "M_words")},
        "clocks": sampler.summary(),
        "gpu_launches": steps * kernels_per_step(info, binding),
    }
    if info["tail_tiles"] > 0:
        line["plan"]["tail"] = {k: info[k] for k in ("tail_h0", "tail_bb", "tail_bw", "tail_bh",
                                                     "tail_bc", "tail_tiles", "tail_grid")}

    if rank == 0 and not args.no_extras:
        e_steps = max(5, min(50, steps))
        e_secs, h2d, d2h, e_sync = time_e2e(cfg, torch, binding, dev, e_steps)
        line["e2e"] = {"value": cfg.flops * e_steps / e_secs / 1e12, "unit": "TFLOP/s",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "ms_per_step": e_secs / e_steps * 1e3, "steps": e_steps,
                       "call": "cconv_forward_host_async per step + one cconv_host_wait (copies of "
                               "neighbouring steps overlap)",
                       "one_call_at_a_time": {"call": "cconv_forward_host (waits every step)",
                                              "value": cfg.flops * e_steps / e_sync / 1e12,
                                              "ms_per_step": e_sync / e_steps * 1e3}}
        if world == 1:
            wgbs = write_only_gbs(torch, dev)
            line["applicable_roofline"]["write_only_stream_gbs"] = wgbs
            rows = []
            for i, c in enumerate(CONFIGS):
                # median of 5 repeats of >= 100 back-to-back calls (20 for the 0.3 ms shape)
                n_i = 100 if c.flops < 1e11 else 20
                cold, warm, info_i, graph_s = time_repeats(c, torch, binding, dev, n_i)
                tr, lbb = applicable_roofline_seconds(c, info_i, peaks)
                m_cta = binding.lower_bound(*c.dims(), info_i["M_words"])
                rows.append({"workload": c.name, "variant": info_i["variant"],
                             "us_per_launch": cold * 1e6, "us_per_launch_l2_warm": warm * 1e6,
                             "us_per_launch_cuda_graph": None if graph_s is None else graph_s * 1e6,
                             "t_write_out_us": 2.0 * c.out_words / (wgbs * 1e9) * 1e6,
                             "tflops": c.flops / cold / 1e12,
                             "tflops_vs_sustained_peak": c.flops / cold / 1e12 /
                                                         peaks["bf16_tflops_sustained"],
                             "t_roof_us": tr * 1e6, "roofline_frac": tr / cold,
                             "roofline_frac_l2_warm": tr / warm,
                             "lower_bound_bytes_at_L2": lbb,
                             "lower_bound_bytes_at_cta_smem": 2.0 * max(m_cta),
                             "planned_bytes_into_smem": 2.0 * info_i["tile_words_smem"],
                             "dram_bytes_ncu": dram_traffic_from_profiles(c.name),
                             "tile": [info_i[k] for k in ("bb", "bw", "bh", "bc", "stages")],
                             "oracle": oracle_sample(c)})
            line["all_configs"] = rows
            line["pooling"] = time_pooling(torch, binding, dev, peaks)
            line["general_shapes"] = time_general_shapes(torch, binding, dev)
            line["cpu_baseline"] = cpu_baseline(cfg)
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
