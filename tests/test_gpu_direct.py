"""GPU parity and stream-order tests of the direct-Filter tensor-core kernel (variant DIRECT), through
the C ABI, against the fp64 CPU oracle of Eq. 1.  Tolerance: 2e-3 * sum|Image*Filter| per element.

Calls of this variant overlap on the GPU (a call lets its successors start at once and ends only
after its predecessors), so besides parity these tests cover what stream order promises: a call
reads what earlier calls wrote, and does not overwrite what they still read."""
import numpy as np
import pytest
import torch

from oracle import cnn as ocnn
from paper_1802_06905_b200 import binding, synth
from paper_1802_06905_b200.synth import CONFIGS, ConvShape

from gpu_util import assert_close, check_full, oshape, to_bits, to_dev

pytestmark = pytest.mark.gpu

DTYPES = [binding.OUT_F32, binding.OUT_BF16]
DT_IDS = ["f32out", "bf16out"]


def cs(name, B, C, K, W, H, R, S, sw=1, sh=1, seed=4321):
    return ConvShape(name, B, C, K, W, H, R, S, sw, sh, seed=seed)


# force string: bb,bw,bh,kt,bc,tg,i_stages,f_stages,grid (0 = the planner's choice)
FORCED = [
    ("64,2,1,1,64", cs("d_1x1_sw128", 64, 64, 128, 4, 3, 1, 1)),          # 128-byte Filter rows
    ("64,2,1,1,32", cs("d_1x1_sw64", 64, 64, 128, 4, 3, 1, 1)),           # 64-byte Filter rows
    ("64,2,1,1,16", cs("d_1x1_sw32", 64, 32, 128, 4, 3, 1, 1)),           # 32-byte Filter rows
    ("32,3,1,1,32", cs("d_3x3", 32, 32, 128, 6, 5, 3, 3)),
    ("32,3,2,1,64", cs("d_3x3_bh2", 32, 64, 128, 6, 5, 3, 3)),
    ("32,3,2,2,32", cs("d_3x3_k256", 32, 64, 256, 6, 5, 3, 3)),           # two out-channel blocks per CTA
    ("32,3,2,2,32", cs("d_ragged", 40, 72, 200, 7, 5, 3, 3)),             # B, C, K, W, H all ragged
    ("32,2,2,1,16", cs("d_strides", 32, 32, 96, 5, 4, 3, 2, 2, 1)),
    ("32,2,3,1,32", cs("d_bh3", 32, 40, 72, 5, 7, 3, 3)),                 # generic b_h loop
    ("64,1,4,2,16,1", cs("d_5x5", 64, 24, 136, 3, 9, 5, 5)),              # one tap per Filter stage
    ("32,4,1,1,32,4", cs("d_taps_not_a_multiple", 32, 32, 64, 9, 3, 3, 3)),  # 9 taps in stages of 4
    ("32,2,2,1,32,0,2,3,3", cs("d_persistent", 64, 64, 256, 8, 6, 3, 3)),  # 3 CTAs walk 48 tiles: both rings and
                                                                            # both accumulator buffers wrap
    ("64,2,2,1,64,0,0,0,5", cs("d_1x1_s2_view", 64, 128, 136, 6, 5, 1, 1, 2, 2)),  # strided 1x1 view
]


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("force,c", FORCED, ids=[c.name for _, c in FORCED])
def test_direct_forced_tiles(monkeypatch, force, c, out_dtype):
    monkeypatch.setenv("CCONV_FORCE_DIRECT", force)
    info = check_full(c, variant=binding.VARIANT_DIRECT, out_dtype=out_dtype)
    assert info["variant"] == binding.VARIANT_DIRECT and info["scratch_bytes"] == 0
    want = [int(v) for v in force.split(",")]
    assert [info["bb"], info["bw"], info["bh"], info["bk"] // 128, info["bc"]] == want[:5]


PLANNED = [
    cs("dp_14x14_3x3", 32, 256, 256, 14, 14, 3, 3),
    cs("dp_14x14_1x1", 64, 512, 256, 14, 14, 1, 1),
    cs("dp_7x7_3x3", 64, 128, 512, 7, 7, 3, 3),
    cs("dp_7x7_5x5_k200", 32, 48, 200, 7, 6, 5, 5),
    cs("dp_28x28_s2", 32, 64, 128, 14, 13, 3, 3, 2, 2),
    cs("dp_b96", 96, 40, 130, 5, 13, 2, 4, 1, 3),
    cs("dp_1x1_s2", 64, 256, 512, 7, 7, 1, 1, 2, 2),
]


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("c", PLANNED, ids=lambda c: c.name)
def test_direct_planned_tiles(c, out_dtype):
    info = check_full(c, variant=binding.VARIANT_DIRECT, out_dtype=out_dtype)
    assert info["variant"] == binding.VARIANT_DIRECT


def test_auto_takes_the_direct_kernel_for_one_wave_problems_only():
    for c, want in ((CONFIGS[1], binding.VARIANT_DIRECT), (CONFIGS[3], binding.VARIANT_DIRECT),
                    (CONFIGS[4], binding.VARIANT_HALO), (cs("c_odd", 32, 20, 64, 14, 14, 3, 3), binding.VARIANT_HALO)):
        p = binding.Plan(*c.dims(), device=0)
        assert p.info()["variant"] == want, c.name
        p.close()


def test_direct_rejects_what_it_cannot_run():
    h = binding.ctypes.c_void_p()
    lib = binding.load_library()
    for dims in ((12, 16, 64, 6, 6, 3, 3, 1, 1), (32, 20, 64, 6, 6, 3, 3, 1, 1)):   # B % 8, C % 8
        assert lib.cconv_plan_create(binding.ctypes.byref(h), *dims, 0, 0.0, binding.VARIANT_DIRECT,
                                     0) == binding.EUNSUPPORTED


def test_calls_that_overlap_on_the_gpu_keep_every_result():
    """Forty unsynchronised calls over rotating buffers with different Filters: several run side by
    side; every Out must be its own call's result."""
    c = cs("d_stream", 32, 128, 256, 14, 14, 3, 3)
    nset = 5
    ins = [synth.make_inputs(c, seed=900 + i) for i in range(nset)]
    imgs = [to_dev(ib) for ib, _ in ins]
    flts = [to_dev(fb) for _, fb in ins]
    outs = [torch.full(c.out_shape, float("nan"), dtype=torch.float32, device="cuda") for _ in range(40)]
    plan = binding.Plan(*c.dims(), device=0, variant=binding.VARIANT_DIRECT, out_dtype=binding.OUT_F32)
    assert plan.info()["grid"] <= 74        # at least two calls fit the SMs side by side
    for i in range(40):
        plan.forward(imgs[i % nset], flts[(i * 3) % nset], outs[i])
    plan.check()
    exp = {}
    for i in (0, 1, 7, 18, 39):
        key = (i % nset, (i * 3) % nset)
        if key not in exp:
            exp[key] = ocnn.cnn_bf16(ins[key[0]][0], ins[key[1]][1], oshape(c))
        e, ab = exp[key]
        assert_close(outs[i].cpu().numpy().astype(np.float64), e, ab, what=f"call {i}")
    # calls 15 apart use the same (Image, Filter) pair: bit-identical results
    for i in range(25):
        assert torch.equal(outs[i], outs[i + 15])
    plan.close()


def test_out_read_as_image_or_filter_by_a_later_call():
    """Stream order, read after write: call B reads call A's Out as its Image (shapes made to agree),
    call F reads call G's Out as its Filter.  Both must see all of it although the kernels may overlap."""
    a = cs("raw_a", 64, 96, 128, 24, 28, 3, 3)                    # Out (128, 28, 24, 64) bf16
    b = cs("raw_b", 64, 24, 64, 126, 26, 3, 3)                    # Image (128, 28, 24, 64)
    g = cs("raw_g", 64, 256, 128, 4, 5, 3, 3)                     # Out (128, 5, 4, 64) bf16
    f = cs("raw_f", 32, 64, 128, 6, 5, 5, 4)                      # Filter (128, 5, 4, 64)
    assert a.out_shape == b.image_shape and g.out_shape == f.filter_shape
    ia, fa = synth.make_inputs(a)
    _, fb = synth.make_inputs(b)
    ig, fg = synth.make_inputs(g)
    i_f, _ = synth.make_inputs(f)
    img_a, flt_a, flt_b = to_dev(ia), to_dev(fa), to_dev(fb)
    img_g, flt_g, img_f = to_dev(ig), to_dev(fg), to_dev(i_f)
    mk = lambda c, od: binding.Plan(*c.dims(), device=0, variant=binding.VARIANT_DIRECT, out_dtype=od)
    plan_a, plan_g = mk(a, binding.OUT_BF16), mk(g, binding.OUT_BF16)
    plan_b, plan_f = mk(b, binding.OUT_F32), mk(f, binding.OUT_F32)
    mid = torch.zeros(a.out_shape, dtype=torch.bfloat16, device="cuda")
    mid_f = torch.zeros(g.out_shape, dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty(b.out_shape, dtype=torch.float32, device="cuda")
    out_f = torch.empty(f.out_shape, dtype=torch.float32, device="cuda")
    for rep in range(6):
        mid.zero_()                                               # stale values would be zeros
        mid_f.zero_()
        out_b.fill_(float("nan"))
        out_f.fill_(float("nan"))
        plan_a.forward(img_a, flt_a, mid)
        plan_g.forward(img_g, flt_g, mid_f)
        plan_b.forward(mid, flt_b, out_b)
        plan_f.forward(img_f, mid_f, out_f)
        plan_a.forward(img_a, flt_a, mid)                         # write after read: B still reads mid
        for p in (plan_a, plan_b, plan_g, plan_f):
            p.check()
        exp, ab = ocnn.cnn_bf16(to_bits(mid), fb, oshape(b))
        assert_close(out_b.cpu().numpy().astype(np.float64), exp, ab, what=f"Out as Image, repeat {rep}")
        exp, ab = ocnn.cnn_bf16(i_f, to_bits(mid_f), oshape(f))
        assert_close(out_f.cpu().numpy().astype(np.float64), exp, ab, what=f"Out as Filter, repeat {rep}")
    assert float(mid.float().abs().max()) > 0 and float(mid_f.float().abs().max()) > 0
    for p in (plan_a, plan_b, plan_g, plan_f):
        p.close()


def test_a_call_does_not_overwrite_what_an_earlier_call_still_reads():
    """Stream order, write after read and write after write: a long call A reads X; a short call B,
    issued right behind it, writes its Out INTO X (shapes made to agree); then a call C writes the
    same Out as A with another Filter.  A must have read the old X; the final Out must be C's."""
    a = cs("war_a", 64, 512, 256, 14, 14, 3, 3)                  # long; Image (16, 16, 512, 64)
    b = cs("war_b", 64, 32, 16, 512, 16, 1, 1)                   # short; Out (16, 16, 512, 64) bf16
    assert b.out_shape == a.image_shape
    ia, fa = synth.make_inputs(a)
    ib, fb = synth.make_inputs(b)
    _, fa2 = synth.make_inputs(a, seed=5151)
    x = to_dev(ia)
    flt_a, flt_a2, img_b, flt_b = to_dev(fa), to_dev(fa2), to_dev(ib), to_dev(fb)
    plan_a = binding.Plan(*a.dims(), device=0, variant=binding.VARIANT_DIRECT, out_dtype=binding.OUT_F32)
    plan_b = binding.Plan(*b.dims(), device=0, variant=binding.VARIANT_DIRECT, out_dtype=binding.OUT_BF16)
    out_a = torch.empty(a.out_shape, dtype=torch.float32, device="cuda")
    exp_a, ab_a = ocnn.cnn_bf16(ia, fa, oshape(a))
    for rep in range(4):
        x.copy_(to_dev(ia))
        out_a.fill_(float("nan"))
        plan_a.forward(x, flt_a, out_a)
        plan_b.forward(img_b, flt_b, x)                           # overwrites A's Image
        plan_a.check()
        plan_b.check()
        assert_close(out_a.cpu().numpy().astype(np.float64), exp_a, ab_a, what=f"write after read, repeat {rep}")
    exp_b, ab_b = ocnn.cnn_bf16(ib, fb, oshape(b))
    assert_close(ocnn.bf16_bits_to_f64(to_bits(x)), exp_b, ab_b, what="the overwriting call", bf16_out=True)
    # write after write
    x.copy_(to_dev(ia))
    exp_c, ab_c = ocnn.cnn_bf16(ia, fa2, oshape(a))
    for rep in range(4):
        plan_a.forward(x, flt_a, out_a)
        plan_a.forward(x, flt_a2, out_a)
        plan_a.check()
        assert_close(out_a.cpu().numpy().astype(np.float64), exp_c, ab_c, what=f"write after write, repeat {rep}")
    plan_a.close()
    plan_b.close()


def test_direct_and_other_variants_mixed_on_one_stream():
    """Direct calls between halo, stem, CUDA-core and pooling calls, no synchronisation in between,
    each on its own buffers, and one chain in which a halo call reads a direct call's Out."""
    shapes = [(cs("mix_d1", 32, 128, 256, 14, 14, 3, 3), binding.VARIANT_DIRECT),
              (cs("mix_h", 64, 32, 136, 9, 7, 3, 3), binding.VARIANT_HALO),
              (cs("mix_d2", 64, 256, 128, 7, 7, 1, 1), binding.VARIANT_DIRECT),
              (cs("mix_s", 64, 3, 64, 12, 11, 7, 7, 2, 2), binding.VARIANT_STEM),
              (cs("mix_c", 2, 8, 16, 9, 9, 3, 3), binding.VARIANT_SIMT)]
    plans, bufs = [], []
    for c, v in shapes:
        ib, fb = synth.make_inputs(c)
        plans.append(binding.Plan(*c.dims(), device=0, variant=v, out_dtype=binding.OUT_F32))
        bufs.append((ib, fb, to_dev(ib), to_dev(fb),
                     torch.full(c.out_shape, float("nan"), dtype=torch.float32, device="cuda")))
    order = np.random.default_rng(7).integers(0, len(shapes), size=40)
    for i in order:
        _, _, img, flt, out = bufs[i]
        plans[i].forward(img, flt, out)
    for p in plans:
        p.check()
    for (c, _), (ib, fb, _, _, out) in zip(shapes, bufs):
        exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
        assert_close(out.cpu().numpy().astype(np.float64), exp, ab, what=c.name)
    for p in plans:
        p.close()
    # a halo call reading the Out of the direct call in front of it
    a = cs("mixchain_a", 64, 96, 128, 24, 28, 3, 3)
    b = cs("mixchain_b", 64, 24, 64, 126, 26, 3, 3)
    ia, fa = synth.make_inputs(a)
    _, fb = synth.make_inputs(b)
    plan_a = binding.Plan(*a.dims(), device=0, variant=binding.VARIANT_DIRECT, out_dtype=binding.OUT_BF16)
    plan_b = binding.Plan(*b.dims(), device=0, variant=binding.VARIANT_HALO, out_dtype=binding.OUT_F32)
    img_a, flt_a, flt_b = to_dev(ia), to_dev(fa), to_dev(fb)
    mid = torch.zeros(a.out_shape, dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty(b.out_shape, dtype=torch.float32, device="cuda")
    for rep in range(4):
        mid.zero_()
        out_b.fill_(float("nan"))
        plan_a.forward(img_a, flt_a, mid)
        plan_b.forward(mid, flt_b, out_b)
        plan_a.check()
        plan_b.check()
        exp, ab = ocnn.cnn_bf16(to_bits(mid), fb, oshape(b))
        assert_close(out_b.cpu().numpy().astype(np.float64), exp, ab, what=f"halo after direct, repeat {rep}")
    plan_a.close()
    plan_b.close()


def test_a_bounded_wait_that_expires_is_reported_and_the_plan_stays_usable(monkeypatch):
    """Diagnostic switch: the Filter producer of the plan's first call leaves out one stage (nothing
    is in flight for it), so the MMA issuer's wait for that stage runs out.  Every role leaves
    through the normal teardown, the status word carries the MMA-wait bit, and the next call on
    the same plan is correct."""
    c = cs("d_timeout", 32, 64, 128, 6, 5, 3, 3)
    monkeypatch.setenv("CCONV_WAIT_LIMIT_MS", "50")
    monkeypatch.setenv("CCONV_DIAG_SKIP_FILTER_STAGE", "1")
    monkeypatch.setenv("CCONV_FORCE_DIRECT", "32,3,1,1,32,3")
    plan = binding.Plan(*c.dims(), device=0, variant=binding.VARIANT_DIRECT, out_dtype=binding.OUT_F32)
    ib, fb = synth.make_inputs(c)
    img, flt = to_dev(ib), to_dev(fb)
    out = torch.full(c.out_shape, float("nan"), dtype=torch.float32, device="cuda")
    plan.forward(img, flt, out)
    code, detail = plan.status()
    assert code == binding.EDEVICE_TIMEOUT
    assert detail & 2                                   # the MMA issuer waited for a stage that never filled
    code, detail = plan.status()
    assert code == binding.OK and detail == 0           # reading the status clears it
    out.fill_(float("nan"))
    plan.forward(img, flt, out)                         # the switch applies to the first call only
    plan.check()
    exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
    assert_close(out.cpu().numpy().astype(np.float64), exp, ab, what="call after the expired wait")
    plan.close()


def test_cconv_forward_on_two_streams_with_one_shape():
    """cconv_forward keeps a plan per (device, stream, shape): two streams running the same shape at
    once do not share scratch."""
    c = cs("two_streams", 32, 64, 136, 10, 9, 3, 3)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    ins = [synth.make_inputs(c, seed=70 + i) for i in range(2)]
    dev = [(to_dev(ib), to_dev(fb)) for ib, fb in ins]
    outs = [[torch.full(c.out_shape, float("nan"), dtype=torch.float32, device="cuda") for _ in range(8)]
            for _ in range(2)]
    torch.cuda.synchronize()
    for i in range(8):
        for j, st in enumerate((s1, s2)):
            binding.conv_forward(dev[j][0], dev[j][1], outs[j][i], *c.dims(), out_dtype=binding.OUT_F32,
                                 stream=st)
    torch.cuda.synchronize()
    for j in range(2):
        exp, ab = ocnn.cnn_bf16(ins[j][0], ins[j][1], oshape(c))
        for i in (0, 3, 7):
            assert_close(outs[j][i].cpu().numpy().astype(np.float64), exp, ab, what=f"stream {j} call {i}")


def test_a_call_that_has_to_wait_runs_the_halo_tiling_and_stays_in_order():
    """AUTO plans that take the direct kernel keep a halo-kernel plan for calls that conflict with a
    call still in flight (they cannot run beside it, and one call alone finishes sooner on many small
    tiles).  A chain B(A(x)) with a third call that rewrites A's Out while B reads it, repeated
    without synchronisation, must match the oracle whichever kernel each call ran."""
    a = cs("wait_a", 64, 96, 128, 24, 28, 3, 3)                   # Out (128, 28, 24, 64) bf16
    b = cs("wait_b", 64, 24, 64, 126, 26, 3, 3)                   # Image (128, 28, 24, 64)
    assert a.out_shape == b.image_shape
    ia, fa = synth.make_inputs(a)
    _, fb = synth.make_inputs(b)
    fa2 = synth.make_inputs(cs("wait_a2", *a.dims(), seed=991))[1]
    img_a, flt_a, flt_a2, flt_b = to_dev(ia), to_dev(fa), to_dev(fa2), to_dev(fb)
    plan_a = binding.Plan(*a.dims(), device=0, out_dtype=binding.OUT_BF16)
    plan_b = binding.Plan(*b.dims(), device=0, out_dtype=binding.OUT_F32)
    infos = [plan_a.info(), plan_b.info()]
    assert any(i["variant"] == binding.VARIANT_DIRECT for i in infos)
    for i in infos:
        assert i["wait_variant"] == (binding.VARIANT_HALO if i["variant"] == binding.VARIANT_DIRECT
                                     else i["variant"])
    mid = torch.zeros(a.out_shape, dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty(b.out_shape, dtype=torch.float32, device="cuda")
    exp_mid, _ = ocnn.cnn_bf16(ia, fa, oshape(a))
    for rep in range(6):
        mid.zero_()
        out_b.fill_(float("nan"))
        plan_a.forward(img_a, flt_a, mid)                         # independent of what is in flight
        plan_b.forward(mid, flt_b, out_b)                         # read after write: waits
        keep = mid.clone() if rep == 0 else None
        plan_a.forward(img_a, flt_a2, mid)                        # write after read: waits
        plan_a.forward(img_a, flt_a, mid)                         # write after write: waits
        plan_a.check()
        plan_b.check()
        exp, ab = ocnn.cnn_bf16(to_bits(mid), fb, oshape(b))
        assert_close(out_b.cpu().numpy().astype(np.float64), exp, ab, what=f"chain, repeat {rep}")
        got_mid = ocnn.bf16_bits_to_f64(to_bits(mid))
        _, ab_mid = ocnn.cnn_bf16(ia, fa, oshape(a))
        assert_close(got_mid, exp_mid, ab_mid, what=f"rewritten Out, repeat {rep}", bf16_out=True)
        if keep is not None:                                      # (written by the call that did not wait)
            assert_close(ocnn.bf16_bits_to_f64(to_bits(keep)), exp_mid, ab_mid, what="first Out", bf16_out=True)
    plan_a.close()
    plan_b.close()


def test_direct_calls_inside_a_cuda_graph():
    """An AUTO plan that took the direct kernel, captured: three calls on two Out buffers (the third
    has to wait for the first: it runs the plan's halo-kernel tiling), replayed on new contents of the
    same buffers."""
    c = cs("graph_direct", 32, 128, 128, 14, 12, 3, 3)
    ib, fb = synth.make_inputs(c)
    img, flt = to_dev(ib), to_dev(fb)
    outs = [torch.full(c.out_shape, float("nan"), device="cuda", dtype=torch.bfloat16) for _ in range(2)]
    plan = binding.Plan(*c.dims(), device=0, out_dtype=binding.OUT_BF16)
    assert plan.info()["variant"] == binding.VARIANT_DIRECT
    plan.forward(img, flt, outs[0])           # warm-up outside the capture
    plan.check()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph, stream=side):
        plan.forward(img, flt, outs[0])
        plan.forward(img, flt, outs[1])
        plan.forward(img, flt, outs[0])
    for seed in (91, 92):
        ib2, fb2 = synth.make_inputs(ConvShape("graph_direct", *c.dims(), seed=seed))
        img.copy_(to_dev(ib2))
        flt.copy_(to_dev(fb2))
        for o in outs:
            o.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        exp, ab = ocnn.cnn_bf16(ib2, fb2, oshape(c))
        for n, o in enumerate(outs):
            assert_close(ocnn.bf16_bits_to_f64(to_bits(o)), exp, ab, what=f"graph replay, seed {seed}, Out {n}",
                         bf16_out=True)
    plan.check()
    plan.close()


@pytest.mark.parametrize("seed", [1, 2])
def test_random_dependent_sequences_match_their_synchronised_run(seed):
    """Stream order as a property (parity with the oracle is the business of the tests above): 150
    random calls -- convolution A writing one of three buffers, convolution B reading one of them as
    its Image, pooling reading one of them -- issued without synchronisation must leave every buffer
    bit-identical to the same sequence with a synchronisation after every call.  (Which kernel a call
    runs depends only on the sequence of calls, so the two runs take the same decisions.)"""
    import random
    a = cs("seq_a", 64, 96, 128, 24, 28, 3, 3)                    # Out (128, 28, 24, 64) bf16
    b = cs("seq_b", 64, 24, 64, 126, 26, 3, 3)                    # Image (128, 28, 24, 64)
    pool_dims = (64, 24, 4, 63, 13, 4, 4, 2, 2)                   # Image (128, 28, 24, 64), Out (4, 13, 63, 64)
    assert a.out_shape == b.image_shape
    ia = [to_dev(synth.make_inputs(cs("seq_a", *a.dims()[:7], seed=10 + i))[0]) for i in range(2)]
    fa = [to_dev(synth.make_inputs(cs("seq_a", *a.dims()[:7], seed=20 + i))[1]) for i in range(2)]
    fb = [to_dev(synth.make_inputs(cs("seq_b", *b.dims()[:7], seed=30 + i))[1]) for i in range(2)]

    def run(sync):
        rng = random.Random(seed)
        mid = [torch.zeros(a.out_shape, dtype=torch.bfloat16, device="cuda") for _ in range(3)]
        outb = [torch.zeros(b.out_shape, dtype=torch.float32, device="cuda") for _ in range(3)]
        pout = [torch.zeros((4, 13, 63, 64), dtype=torch.bfloat16, device="cuda") for _ in range(2)]
        pa = binding.Plan(*a.dims(), device=0, out_dtype=binding.OUT_BF16)
        pb = binding.Plan(*b.dims(), device=0, out_dtype=binding.OUT_F32)
        for _ in range(150):
            r = rng.random()
            if r < 0.45:
                pa.forward(ia[rng.randrange(2)], fa[rng.randrange(2)], mid[rng.randrange(3)])
            elif r < 0.8:
                pb.forward(mid[rng.randrange(3)], fb[rng.randrange(2)], outb[rng.randrange(3)])
            else:
                binding.pool_forward(mid[rng.randrange(3)], pout[rng.randrange(2)], *pool_dims,
                                     op=binding.POOL_MAX)
            if sync:
                torch.cuda.synchronize()
        pa.check()
        pb.check()
        res = [t.clone() for t in mid + outb + pout]
        pa.close()
        pb.close()
        return res

    for n, (x, y) in enumerate(zip(run(False), run(True))):
        assert torch.equal(x, y), f"buffer {n} differs between the two runs"
