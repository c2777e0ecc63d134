"""cconv_forward_noalloc, the entry point for callers that cannot allocate device memory.

Who needs it: code that runs while a CUDA graph is being captured, serving callbacks whose device
memory was handed out at start-up, processes whose allocator must not be entered from the calling
thread.  The planned entry points cudaMalloc scratch for the repacked Filter; this one keeps that
scratch in a fixed array inside the library, shared by every call.

The test calls it through the C ABI twice in a row (the array keeps the first call's contents, so
the second call is the one that shows stale state) and compares each result with the existing
planned entry point on the same inputs and with the CPU oracle, within the tolerance the parity
tests use.  It is collected
last (file name) so that a run which stops at the first failure has already run everything else;
it passes alone in a fresh process as well.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import cnn as ocnn
from paper_1802_06905_b200 import binding, synth
from paper_1802_06905_b200.synth import ConvShape

from gpu_util import TOL, assert_close, oshape, to_bits, to_dev

pytestmark = pytest.mark.gpu


def planned_reference(c, img, flt, out_dtype):
    out = torch.full(c.out_shape, float("nan"), device="cuda",
                     dtype=torch.float32 if out_dtype == binding.OUT_F32 else torch.bfloat16)
    plan = binding.Plan(*c.dims(), device=torch.cuda.current_device(), variant=binding.VARIANT_HALO,
                        out_dtype=out_dtype)
    plan.forward(img, flt, out)
    plan.check()
    plan.close()
    return out.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("out_dtype", [binding.OUT_F32, binding.OUT_BF16], ids=["f32out", "bf16out"])
def test_noalloc_matches_planned_entry_point_twice_in_a_row(out_dtype):
    # two different shapes back to back: the second finds the first one's Filter blocks and status
    # word in the shared array
    shapes = [ConvShape("na1", 64, 40, 200, 9, 7, 3, 3, seed=71),
              ConvShape("na2", 32, 256, 256, 14, 14, 3, 3, seed=72),
              ConvShape("na_split", 16, 256, 256, 7, 7, 3, 3, seed=74),   # tiles shared by CTA pairs
              ConvShape("na1_again", 64, 40, 200, 9, 7, 3, 3, seed=73)]
    for c in shapes:
        ib, fb = synth.make_inputs(c)
        img, flt = to_dev(ib), to_dev(fb)
        ref = planned_reference(c, img, flt, out_dtype)
        exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
        for call in range(2):
            out = torch.full(c.out_shape, float("nan"), device="cuda",
                             dtype=torch.float32 if out_dtype == binding.OUT_F32 else torch.bfloat16)
            binding.conv_forward_noalloc(img, flt, out, *c.dims(), out_dtype=out_dtype, sync=True)
            got = out.float().cpu().numpy().astype(np.float64)
            assert not np.isnan(got).any(), f"{c.name} call {call}: unwritten outputs"
            assert np.all(np.abs(got - ref) <= TOL * ab), f"{c.name} call {call}: differs from planned path"
            assert_close(got, exp, ab, what=f"{c.name} call {call} against the oracle",
                         bf16_out=out_dtype == binding.OUT_BF16)


def test_noalloc_async_calls_on_one_stream_are_ordered():
    c = ConvShape("na3", 32, 64, 128, 6, 6, 3, 3, seed=74)
    ib, fb = synth.make_inputs(c)
    img, flt = to_dev(ib), to_dev(fb)
    ref = planned_reference(c, img, flt, binding.OUT_F32)
    exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
    outs = [torch.full(c.out_shape, float("nan"), device="cuda") for _ in range(2)]
    for o in outs:                                   # no synchronisation between the two calls
        binding.conv_forward_noalloc(img, flt, o, *c.dims(), out_dtype=binding.OUT_F32)
    assert binding.noalloc_status() == (binding.OK, 0)       # synchronises; no wait expired
    for o in outs:
        got = o.cpu().numpy().astype(np.float64)
        assert np.all(np.abs(got - ref) <= TOL * ab)
        assert_close(got, exp, ab, what="asynchronous call against the oracle")


@pytest.mark.parametrize("variant", [binding.VARIANT_HALO, binding.VARIANT_DIRECT], ids=["halo", "direct"])
def test_a_planned_call_reads_the_out_of_the_noalloc_call_in_front_of_it(variant):
    """The convolution of a noalloc call lets the kernel behind it start early; a planned call whose
    Image is that call's Out (shapes made to agree) must still see all of it."""
    a = ConvShape("na_chain_a", 64, 96, 128, 24, 28, 3, 3, seed=81)        # Out (128, 28, 24, 64)
    b = ConvShape("na_chain_b", 64, 24, 64, 126, 26, 3, 3, seed=82)        # Image (128, 28, 24, 64)
    assert a.out_shape == b.image_shape
    ia, fa = synth.make_inputs(a)
    _, fb = synth.make_inputs(b)
    img_a, flt_a, flt_b = to_dev(ia), to_dev(fa), to_dev(fb)
    plan_b = binding.Plan(*b.dims(), device=0, variant=variant, out_dtype=binding.OUT_F32)
    mid = torch.zeros(a.out_shape, dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty(b.out_shape, dtype=torch.float32, device="cuda")
    for rep in range(6):
        mid.zero_()                                               # stale values would be zeros
        out_b.fill_(float("nan"))
        binding.conv_forward_noalloc(img_a, flt_a, mid, *a.dims(), out_dtype=binding.OUT_BF16)
        plan_b.forward(mid, flt_b, out_b)
        plan_b.check()
        assert binding.noalloc_status() == (binding.OK, 0)
        exp, ab = ocnn.cnn_bf16(to_bits(mid), fb, oshape(b))
        assert_close(out_b.cpu().numpy().astype(np.float64), exp, ab, what=f"planned after noalloc, repeat {rep}")
    assert float(mid.float().abs().max()) > 0
    plan_b.close()


def test_noalloc_rejects_what_it_cannot_hold_or_run():
    lib = binding.load_library()
    buf = torch.zeros(1 << 20, dtype=torch.bfloat16, device="cuda")
    p = ctypes.c_void_p(buf.data_ptr())
    # repacked Filter of 8*64*9 blocks of 4 KB = 18.9 MB > the 8 MiB array: refused before any launch
    # (the pointers are never dereferenced)
    rc = lib.cconv_forward_noalloc(p, p, p, 32, 1024, 1024, 8, 8, 3, 3, 1, 1, binding.OUT_BF16, None, None)
    assert rc == binding.ETOOLARGE
    assert b"scratch" in lib.cconv_strerror(rc)
    # B not a multiple of 8: the tensor-core kernel cannot tile it
    rc = lib.cconv_forward_noalloc(p, p, p, 2, 8, 16, 14, 14, 3, 3, 1, 1, binding.OUT_BF16, None, None)
    assert rc == binding.EUNSUPPORTED
    rc = lib.cconv_forward_noalloc(None, p, p, 32, 8, 16, 14, 14, 3, 3, 1, 1, binding.OUT_BF16, None, None)
    assert rc == binding.EINVAL
    torch.cuda.synchronize()


def test_noalloc_inside_a_cuda_graph_capture_and_replay():
    """The call is made while a stream is being captured (no allocation may happen there), then the
    graph is replayed on new contents of the same buffers."""
    c = ConvShape("na_graph", 32, 48, 136, 10, 8, 3, 3, seed=74)
    ib, fb = synth.make_inputs(c)
    img, flt = to_dev(ib), to_dev(fb)
    out = torch.full(c.out_shape, float("nan"), device="cuda", dtype=torch.float32)
    # first call on this device outside any capture (it looks up the scratch array's address)
    binding.conv_forward_noalloc(img, flt, out, *c.dims(), out_dtype=binding.OUT_F32, sync=True)
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph, stream=side):
        binding.conv_forward_noalloc(img, flt, out, *c.dims(), out_dtype=binding.OUT_F32,
                                     stream=torch.cuda.current_stream())
    for seed in (75, 76):
        ib2, fb2 = synth.make_inputs(ConvShape("na_graph", *c.dims(), seed=seed))
        img.copy_(to_dev(ib2))
        flt.copy_(to_dev(fb2))
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        exp, ab = ocnn.cnn_bf16(ib2, fb2, oshape(c))
        got = out.cpu().numpy().astype(np.float64)
        assert not np.isnan(got).any()
        assert np.all(np.abs(got - exp) <= TOL * ab), f"replay with seed {seed}: mismatch"
