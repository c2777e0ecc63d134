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


def buffer_sets(cfg, torch, dev, ib, fb):
    """Enough distinct (Image, Filter, Out) sets that 1.5 x L2 of other sets' traffic passes between
    two uses of a set: back-to-back calls read cold inputs, and no Out is rewritten while its lines
    from the last round still sit in L2 (which would save the write-back)."""
    set_bytes = 2 * (cfg.image_words + cfg.filter_words + cfg.out_words)
    nsets = max(3, min(64, 1 - (-int(1.5 * L2_BYTES) // set_bytes)))
    base_i, base_f = to_dev(ib, torch, dev), to_dev(fb, torch, dev)
    imgs = [base_i] + [base_i.clone() for _ in range(nsets - 1)]
    flts = [base_f] + [base_f.clone() for _ in range(nsets - 1)]
    outs = [torch.empty(cfg.out_shape, dtype=torch.bfloat16, device=dev) for _ in range(nsets)]
    ptrs = [(imgs[i].data_ptr(), flts[i].data_ptr(), outs[i].data_ptr()) for i in range(nsets)]
    return (imgs, flts, outs), ptrs, nsets


def time_config(cfg, ib, fb, torch, binding, dev, steps, warmup, repeats, dist=None, sampler=None):
    """Device-resident timing of one configuration: after `warmup` calls, `repeats` timed regions of
    exactly `steps` back-to-back forward calls each (synchronise, event, calls, event, synchronise;
    barrier on both sides with several ranks).  Returns the per-region seconds, plan info, nsets."""
    keep, ptrs, nsets = buffer_sets(cfg, torch, dev, ib, fb)
    plan = binding.Plan(*cfg.dims(), device=dev.index, out_dtype=binding.OUT_BF16)
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    for i in range(max(warmup, 3)):
        a, b, c = ptrs[i % nsets]
        rc = plan.forward_ptrs(a, b, c, sp)
        assert rc == 0, rc
    plan.check()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sampler:
        sampler.start()
    regions = []
    k = 0
    for rep in range(repeats):
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(steps):
            a, b, c = ptrs[k % nsets]
            k += 1
            plan.forward_ptrs(a, b, c, sp)
        e1.record(stream)
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        regions.append(e0.elapsed_time(e1) * 1e-3)
    if sampler:
        sampler.sample_once()
        sampler.stop()
    plan.check()
    info = plan.info()
    plan.close()
    del keep
    return regions, info, nsets


def time_repeats(cfg, torch, binding, dev, launches, repeats=5):
    """Per-configuration table.  Median over `repeats` of the CUDA-event time of `launches`
    back-to-back forward calls over rotating buffer sets larger than L2 (L2-cold); the same rotation
    captured once into a CUDA graph and replayed; and the time of a call that runs alone
    (synchronised on both sides; includes the launch).  Returns a dict of seconds per call."""
    ib, fb = make_inputs(cfg)
    keep, ptrs, nsets = buffer_sets(cfg, torch, dev, ib, fb)
    plan = binding.Plan(*cfg.dims(), device=dev.index, out_dtype=binding.OUT_BF16)
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(dev.index)
    sampler.start()
    times = []
    k = 0
    for rep in range(repeats + 1):            # the first repeat is warm-up
        torch.cuda.synchronize()
        e0.record(stream)
        for i in range(launches):
            a, b, c = ptrs[k % nsets]
            k += 1
            plan.forward_ptrs(a, b, c, sp)
        e1.record(stream)
        torch.cuda.synchronize()
        if rep:
            times.append(e0.elapsed_time(e1) * 1e-3 / launches)
    sampler.sample_once()
    sampler.stop()
    res = {"stream": float(np.median(times)), "graph": None, "alone": None,
           "sm_mhz": sampler.summary()["sm_mhz"], "nsets": nsets}
    alone = []
    for i in range(7):
        a, b, c = ptrs[i % nsets]
        torch.cuda.synchronize()
        e0.record(stream)
        plan.forward_ptrs(a, b, c, sp)
        e1.record(stream)
        torch.cuda.synchronize()
        alone.append(e0.elapsed_time(e1) * 1e-3)
    res["alone"] = float(np.median(alone))
    res["alone_latency_plan"] = None
    if plan.info()["variant"] == binding.VARIANT_DIRECT:
        # the same call on a plan made for one call at a time (what CCONV_OBJECTIVE=latency selects)
        lat_plan = binding.Plan(*cfg.dims(), device=dev.index, variant=binding.VARIANT_HALO,
                                out_dtype=binding.OUT_BF16)
        alone = []
        for i in range(8):
            a, b, c = ptrs[i % nsets]
            torch.cuda.synchronize()
            e0.record(stream)
            lat_plan.forward_ptrs(a, b, c, sp)
            e1.record(stream)
            torch.cuda.synchronize()
            alone.append(e0.elapsed_time(e1) * 1e-3)
        res["alone_latency_plan"] = float(np.median(alone[1:]))
        lat_plan.check()
        lat_plan.close()
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
        res["graph"] = float(np.median(times))
        del g
    except RuntimeError:
        res["graph"] = None
    plan.check()
    info = plan.info()
    plan.close()
    del keep
    return res, info


def time_general_shapes(torch, binding, dev, launches=30, repeats=3):
    """Shapes outside the five benchmark configurations: layers with few output pixels and long
    channel loops, and a single image (B < 8: bands of output rows stand in for images).  Each is
    timed as planned (AUTO) and on the halo kernel (VARIANT_HALO: Filter-packing kernel, tiles split
    over CTA clusters where the planner does so), back-to-back calls over rotating buffer sets."""
    shapes = [("resnet50_conv5_3x3_b64", (64, 512, 512, 7, 7, 3, 3, 1, 1)),
              ("deep_7x7_3x3_b16", (16, 1024, 256, 7, 7, 3, 3, 1, 1)),
              ("deep_7x7_5x5_b8", (8, 512, 512, 7, 7, 5, 5, 1, 1)),
              ("single_image_56x56_3x3", (1, 256, 256, 56, 56, 3, 3, 1, 1))]
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rows = []
    for name, dims in shapes:
        c = ConvShape(name, *dims)
        ib, fb = make_inputs(c)
        keep, ptrs, nsets = buffer_sets(c, torch, dev, ib, fb)
        res = {}
        for label, variant in (("planned", binding.VARIANT_AUTO), ("halo_kernel", binding.VARIANT_HALO)):
            plan = binding.Plan(*dims, device=dev.index, out_dtype=binding.OUT_BF16, variant=variant)
            times = []
            k = 0
            for rep in range(repeats + 1):
                torch.cuda.synchronize()
                e0.record(stream)
                for _ in range(launches):
                    a, b, cc = ptrs[k % nsets]
                    k += 1
                    plan.forward_ptrs(a, b, cc, sp)
                e1.record(stream)
                torch.cuda.synchronize()
                if rep:
                    times.append(e0.elapsed_time(e1) * 1e3 / launches)
            plan.check()
            info = plan.info()
            plan.close()
            res[label] = {"us_per_launch": float(np.median(times)), "variant": info["variant"],
                          "split": info["split"], "bands": info["bands"], "grid": info["grid"],
                          "tile": [info[k2] for k2 in ("bb", "bw", "bh", "bk", "bc")]}
        del keep
        rows.append({"workload": name, "dims": dict(zip("B C K W H R S sw sh".split(), dims)),
                     "tflops": c.flops / res["planned"]["us_per_launch"] / 1e6, **res})
    return rows


def time_pooling(torch, binding, dev, peaks, launches=50, repeats=5, shapes=None, ops=("avg", "max")):
    """Pooling (Section 6) rows: median CUDA-event time of back-to-back cconv_pool_forward calls over
    rotating buffer sets (1.5 x L2 of other sets between two uses of one).  Algorithmic bytes = Image + Out, each moved once; the
    roofline is the measured HBM copy rate."""
    from paper_1802_06905_b200.synth import POOL_SHAPES
    stream = torch.cuda.current_stream()
    sp = stream.cuda_stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    rows = []
    gen = torch.Generator(device="cpu").manual_seed(0x18020690 + 60)
    for name, B, C, K, W, H, R, S, sw, sh in (shapes or POOL_SHAPES):
        Wi, Hi = sw * (W - 1) + R, sh * (H - 1) + S
        ibytes, obytes = 2 * Wi * Hi * C * B, 2 * K * H * W * B
        nsets = max(3, min(16, 1 - (-int(1.5 * L2_BYTES) // (ibytes + obytes))))   # as buffer_sets
        base = torch.randn((Wi, Hi, C, B), generator=gen).to(torch.bfloat16).to(dev)
        imgs = [base] + [base.clone() for _ in range(nsets - 1)]
        outs = [torch.empty((K, H, W, B), dtype=torch.bfloat16, device=dev) for _ in range(nsets)]
        terms = binding.pool_lower_bound(B, C, K, W, H, R, S, sw, sh, L2_BYTES / 4.0)
        for op, opname in ((binding.POOL_AVG, "avg"), (binding.POOL_MAX, "max")):
            if opname not in ops:
                continue
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
    if info["variant"] in (binding.VARIANT_SIMT, binding.VARIANT_DIRECT):
        return 1
    n = 2                                    # Filter packing + convolution
    if info["variant"] == binding.VARIANT_HALO and info["tail_tiles"] > 0:
        n += 1                               # wave-quantisation tail launch
    return n


KERNEL_NAMES = {1: "cconv_simt_kernel", 2: "cconv_halo_kernel", 3: "cconv_stem_kernel",
                4: "cconv_direct_kernel"}


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
    """Roofline of the dominant kernel: tensor-bound where a tcgen05 kernel ran (dense contraction),
    HBM-bound for the CUDA-core kernel (reported against compulsory bytes).  `traffic` is ncu's
    in-kernel DRAM byte count of one call from the committed profile summary (Out still in L2 when
    the kernel ends is written back later and not in it); the compulsory bytes and the paper's bound
    at both memory levels stand beside it."""
    traffic = dram_traffic_from_profiles(cfg.name)
    if info["variant"] != binding.VARIANT_SIMT:
        ach = cfg.flops / secs_per_launch / 1e12
        peak = peaks["bf16_tflops"]
        return {"bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                "frac": ach / peak, "traffic": traffic, "peak_source": peaks["source"],
                # the burst figure is the denominator; the timed loop of a large shape runs for
                # hundreds of milliseconds under the power cap, so the sustained figure stands beside it
                "peak_sustained": peaks["bf16_tflops_sustained"],
                "frac_of_sustained_peak": ach / peaks["bf16_tflops_sustained"],
                "kernel": KERNEL_NAMES[info["variant"]],
                "duration": "CUDA-event time of `steps` back-to-back forward calls / steps, median of "
                            "`repeats` such regions (calls of small shapes overlap on the GPU)"}
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


def make_rank_problem(cfg, world, rank):
    """Several ranks: ONE problem of world*B images, cut over b with the Filter replicated (no
    collective in the forward); rank r gets images [b0, b0+n).  Returns (local shape, Image bits,
    Filter bits, (b0, n), global B)."""
    if world == 1:
        ib, fb = make_inputs(cfg)
        return cfg, ib, fb, (0, cfg.B), cfg.B
    from dataclasses import replace
    from paper_1802_06905_b200 import sharding
    glob = replace(cfg, B=cfg.B * world)
    b0, n = sharding.shard_batch(glob.B, world, rank)
    ib, fb = make_inputs(glob)
    return replace(cfg, B=n), sharding.slice_batch(ib, b0, n), fb, (b0, n), glob.B


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--repeats", type=int, default=25,
                    help="timed regions of `steps` calls each; ms_per_step is the median region / steps")
    ap.add_argument("--config", type=int, default=4,
                    help="index into the five benchmark shapes (default: the largest, cfg5)")
    ap.add_argument("--shape", default=None,
                    help="B,C,K,W,H,R,S,sw,sh: time this shape instead of a benchmark configuration "
                         "(same input recipe as the default configuration; no profile figures exist for it)")
    ap.add_argument("--pool-shape", default=None,
                    help="B,C,K,W,H,R,S,sw,sh: time cconv_pool_forward on this shape only and print its row")
    ap.add_argument("--pool-op", default="avg,max", help="avg, max or avg,max (with --pool-shape)")
    ap.add_argument("--impl", default="cconv", choices=["cconv", "reference"])
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the per-configuration table, the e2e leg and the CPU baseline")
    ap.add_argument("--detail-file", default=os.path.join(ROOT, "gpurun_out", "bench_detail.json"),
                    help="where the long per-configuration / pooling / general-shape tables go")
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
    peaks = measured_peaks()

    if args.pool_shape:
        dims = tuple(int(v) for v in args.pool_shape.split(","))
        rows = time_pooling(torch, binding, dev, peaks, shapes=[("pool_shape",) + dims],
                            ops=tuple(args.pool_op.split(",")))
        print(json.dumps({"pooling": rows}))
        return 0

    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=dev)
        dist = dist_mod

    cfg_named = chosen_config(args)
    cfg, ib, fb, (b0, nb), global_B = make_rank_problem(cfg_named, world, rank)
    steps, warmup, repeats = max(1, args.steps), max(3, args.warmup), max(1, args.repeats)
    sampler = ClockSampler(local)
    regions, info, nsets = time_config(cfg, ib, fb, torch, binding, dev, steps, warmup, repeats, dist,
                                       sampler)
    secs = float(np.median(regions))
    flops_rank = float(cfg.flops)
    flops_all = flops_rank
    if dist is not None:
        t = torch.tensor([secs], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        secs = float(t.item())
        f = torch.tensor([flops_rank], dtype=torch.float64, device=dev)
        dist.all_reduce(f, op=dist.ReduceOp.SUM)
        flops_all = float(f.item())
    # weak scaling: the problem grows with the ranks (world*B images), every rank convolves its
    # shard with the replicated Filter
    value = flops_all * steps / secs / 1e12
    per_launch = secs / steps
    roof = roofline_for(cfg, info, per_launch, peaks, binding)
    t_roof, lb_bytes = applicable_roofline_seconds(cfg, info, peaks)
    m_cta = binding.lower_bound(*cfg.dims(), info["M_words"])
    roof["applicable"] = {"t_roof_us": t_roof * 1e6, "frac": t_roof / per_launch,
                          "rule": "max(flops / bf16 peak, bound bytes at M = L2 / HBM copy rate)"}
    roof["bytes"] = {"compulsory": 2.0 * info["compulsory_words"],
                     "bound_at_M_L2": lb_bytes, "bound_at_M_cta_smem": 2.0 * max(m_cta),
                     "compulsory_over_bound_at_M_cta_smem": 2.0 * info["compulsory_words"] / (2.0 * max(m_cta)),
                     "note": "the kernels move compulsory bytes through HBM (ncu: reads = Image + Filter "
                             "once); the paper's bound is evaluated at the kernel's effective M, the "
                             "shared memory of one CTA, and at M = L2"}

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": steps,
        "warmup": warmup, "ms_per_step": per_launch * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg_named.name,
                   "dims": dict(zip("B C K W H R S sw sh".split(), cfg_named.dims())),
                   "repeats": repeats,
                   "timing": "median over `repeats` regions of exactly `steps` back-to-back calls, each "
                             "bracketed by synchronize (and a barrier with several ranks)",
                   "l2": f"rotating {nsets} distinct buffer sets ({nsets * 2 * (cfg.image_words + cfg.filter_words + cfg.out_words) / 1e6:.0f} MB > 126 MB L2)",
                   "out_dtype": "bf16", "accumulate": "fp32",
                   "parallelism": (f"one problem of {global_B} images cut over b into {world} shards, "
                                   f"Filter replicated, no collective") if world > 1 else "single GPU"},
        "roofline": roof,
        "plan": {k: info[k] for k in ("variant", "bb", "bc", "bk", "bw", "bh", "stages", "filter_stages",
                                      "grid", "tiles", "smem_bytes", "tmem_cols", "bound_argmax",
                                      "tile_G_over_lp_G")},
        "clocks": sampler.summary(),
        "gpu_launches": steps * repeats * kernels_per_step(info, binding),
    }
    if world > 1:
        line["config"]["shard_of_rank0"] = [b0, nb]

    detail = {}
    if rank == 0 and not args.no_extras:
        e_steps = max(5, min(50, steps))
        e_secs, h2d, d2h, e_sync = time_e2e(cfg, torch, binding, dev, e_steps)
        line["e2e"] = {"value": cfg.flops * e_steps / e_secs / 1e12, "unit": "TFLOP/s",
                       "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "ms_per_step": e_secs / e_steps * 1e3, "steps": e_steps,
                       "call": "cconv_forward_host_async per step + one cconv_host_wait",
                       "one_call_at_a_time_ms_per_step": e_sync / e_steps * 1e3}
        if world == 1:
            wgbs = write_only_gbs(torch, dev)
            roof["applicable"]["write_only_stream_gbs"] = wgbs
            per, rows = {}, []
            for c in CONFIGS:
                # Regions of about 4 ms (20 to 1000 calls, sized from the roofline time): calls of the
                # small shapes overlap on the GPU, and a short region would add the drain of its last
                # call, (CTA life - period) / calls, to every call; much longer regions leave the burst
                # regime in which the roofline's denominators were measured (after some 40 ms of
                # continuous work cfg3 settles 17 % lower, as cfg5 does under the power cap).
                t_guess = 1.5 * applicable_roofline_seconds(c, binding.Plan(*c.dims(), device=-1).info(), peaks)[0]
                n_i = int(min(1000, max(20, round(4e-3 / max(t_guess, 4e-6)))))
                res, info_i = time_repeats(c, torch, binding, dev, n_i)
                cold = res["stream"]
                tr, lbb = applicable_roofline_seconds(c, info_i, peaks)
                m_i = binding.lower_bound(*c.dims(), info_i["M_words"])
                tensor = info_i["variant"] != binding.VARIANT_SIMT
                bound = ("launch" if c.flops < 1e7 else
                         "tensor" if c.flops / (peaks["bf16_tflops"] * 1e12) >= lbb / (peaks["hbm_gbs"] * 1e9)
                         else "hbm")
                per[c.name.split("_")[0]] = {
                    "us": round(cold * 1e6, 2),
                    "us_graph": None if res["graph"] is None else round(res["graph"] * 1e6, 2),
                    "us_alone": round(res["alone"] * 1e6, 1),
                    "us_alone_latency_plan": (None if res["alone_latency_plan"] is None
                                              else round(res["alone_latency_plan"] * 1e6, 1)),
                    "tflops": round(c.flops / cold / 1e12, 1), "t_roof_us": round(tr * 1e6, 2),
                    "frac": round(tr / cold, 3), "bound": bound, "kernel": KERNEL_NAMES[info_i["variant"]],
                    "dram_bytes_ncu": dram_traffic_from_profiles(c.name),
                    "compulsory_bytes": 2.0 * info_i["compulsory_words"],
                    "bound_bytes_M_L2": lbb, "bound_bytes_M_cta": 2.0 * max(m_i),
                    "staged_bytes_l2_to_sm": 2.0 * info_i["tile_words_smem"],
                    "sm_mhz": res["sm_mhz"],
                    "tile": [info_i[k] for k in ("bb", "bw", "bh", "bk", "bc")], "grid": info_i["grid"],
                    "G_over_lp_G": round(info_i["tile_G_over_lp_G"], 3) if tensor else None}
                rows.append({"workload": c.name, "plan": info_i, "timing_s": res, "oracle": oracle_sample(c)})
            roof["per_config"] = per
            roof["per_config_note"] = ("us = L2-cold back-to-back calls on one stream, median of 5 regions of "
                                       "about 4 ms (20 to 1000 calls); independent calls of small shapes "
                                       "run side by side on the SMs; us_alone = one call between "
                                       "synchronisations, launch included (us_alone_latency_plan: on a plan "
                                       "made with CCONV_OBJECTIVE=latency); frac = t_roof_us / us")
            pool = time_pooling(torch, binding, dev, peaks)
            roof["pooling"] = {f"{r['workload']}_{r['op']}": {"us": round(r["us_per_launch"], 2),
                                                               "frac_of_hbm_copy": round(r["roofline"]["frac"], 3)}
                               for r in pool}
            detail = {"all_configs": rows, "pooling": pool,
                      "general_shapes": time_general_shapes(torch, binding, dev)}
            roof["general_shapes_us"] = {g["workload"]: [round(g["planned"]["us_per_launch"], 1),
                                                          round(g["halo_kernel"]["us_per_launch"], 1)]
                                         for g in detail["general_shapes"]}
            line["cpu_baseline"] = cpu_baseline(cfg)
    if rank == 0:
        if detail:
            try:
                os.makedirs(os.path.dirname(args.detail_file), exist_ok=True)
                with open(args.detail_file, "w") as fh:
                    json.dump({"line": line, **detail}, fh, indent=1, default=str)
            except OSError:
                pass
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
