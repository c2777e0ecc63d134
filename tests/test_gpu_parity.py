"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle of Eq. 1,
element by element on the same seeded bf16 inputs.  Tolerance: 2e-3 * sum|Image*Filter|."""
import numpy as np
import pytest
import torch

from oracle import cnn as ocnn
from paper_1802_06905_b200 import binding, synth
from paper_1802_06905_b200.synth import CONFIGS, ConvShape

from gpu_util import assert_close, check_full, oshape, run_gpu, to_bits, to_dev

pytestmark = pytest.mark.gpu

BY = {c.name: c for c in CONFIGS}


def cs(name, B, C, K, W, H, R, S, sw=1, sh=1, seed=1234):
    return ConvShape(name, B, C, K, W, H, R, S, sw, sh, seed=seed)


# ---- the benchmark configurations ----------------------------------------------------------------

DTYPES = [binding.OUT_F32, binding.OUT_BF16]
DT_IDS = ["f32out", "bf16out"]


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("name", ["cfg1_tiny_3x3", "cfg2_resnet_3x3", "cfg3_stem_7x7_s2",
                                  "cfg4_pointwise_1x1"])
def test_config_full_parity(name, out_dtype):
    info = check_full(BY[name], out_dtype=out_dtype)
    if name in ("cfg2_resnet_3x3", "cfg4_pointwise_1x1"):
        assert info["variant"] == binding.VARIANT_DIRECT   # the tensor-core path is the one that ran
    if name == "cfg3_stem_7x7_s2":
        assert info["variant"] == binding.VARIANT_STEM
    # On the benchmark shapes |Out| is far below sum|Image*Filter| (random signs, long contractions),
    # so no element needs the clause that widens the band by the bf16 store's rounding.
    assert info["rounding_clause_only"] == 0


_CFG5_ORACLE = {}


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
def test_config5_full_parity(out_dtype):
    """Every one of the 51.4 M outputs of the largest shape, main launch and tail launch alike,
    against the oracle (about ten seconds of host time, computed once for both Out types)."""
    c = BY["cfg5_large_3x3"]
    ib, fb = synth.make_inputs(c)
    got, info = run_gpu(c, ib, fb, out_dtype=out_dtype)
    assert info["variant"] == binding.VARIANT_HALO and info["tail_tiles"] > 0
    if "exp" not in _CFG5_ORACLE:
        _CFG5_ORACLE["exp"], _CFG5_ORACLE["ab"] = ocnn.cnn_bf16(ib, fb, oshape(c))
    n = assert_close(got, _CFG5_ORACLE["exp"], _CFG5_ORACLE["ab"], "cfg5 full",
                     bf16_out=out_dtype == binding.OUT_BF16)
    assert n == 0


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
def test_config5_sampled_parity(out_dtype):
    """Full size, launch configuration of the benchmark; the oracle evaluates sampled elements one by
    one: 60 000 random (k,h,w,b), plus every element of two (k,h) rows and of the last pixel."""
    c = BY["cfg5_large_3x3"]
    ib, fb = synth.make_inputs(c)
    got, info = run_gpu(c, ib, fb, out_dtype=out_dtype)
    assert info["variant"] == binding.VARIANT_HALO
    rng = np.random.default_rng(55)
    idx = np.stack([rng.integers(0, n, size=60000) for n in c.out_shape], axis=1).astype(np.int32)
    rows = []
    for (k, h) in [(0, 0), (c.K - 1, c.H - 1), (257, 13)]:
        for w in range(c.W):
            for b in range(c.B):
                rows.append((k, h, w, b))
    for k in range(c.K):
        rows.append((k, c.H - 1, c.W - 1, c.B - 1))
    idx = np.concatenate([idx, np.array(rows, dtype=np.int32)])
    exp, ab = ocnn.cnn_bf16_at(ib, fb, idx, oshape(c))
    g = got[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
    assert not np.isnan(got).any()
    assert assert_close(g, exp, ab, "cfg5 sampled", bf16_out=out_dtype == binding.OUT_BF16) == 0


# ---- CUDA-core kernel: odd shapes ------------------------------------------------------------------

SIMT_SHAPES = [
    cs("s1", 1, 1, 1, 1, 1, 1, 1),
    cs("s2", 3, 5, 7, 6, 5, 3, 2, 2, 1),
    cs("s3", 2, 3, 5, 9, 4, 2, 5, 3, 2),          # sw > R: skipped Image columns
    cs("s4", 5, 4, 9, 3, 7, 4, 1, 1, 3),
    cs("s5", 33, 9, 17, 5, 6, 3, 3, 2, 2),
    cs("s6", 2, 8, 16, 14, 14, 3, 3),
    cs("s7", 7, 13, 6, 1, 1, 5, 4),
]


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("c", SIMT_SHAPES, ids=lambda c: c.name)
def test_simt_odd_shapes(c, out_dtype):
    check_full(c, variant=binding.VARIANT_SIMT, out_dtype=out_dtype)


# ---- tensor-core kernel: shapes that span several tiles, ragged tails, padded K and C ----------------

HALO_SHAPES = [
    cs("h_1x1", 64, 64, 128, 4, 4, 1, 1),
    cs("h_3x3", 32, 32, 128, 6, 5, 3, 3),
    cs("h_ragged_w", 32, 16, 64, 9, 7, 3, 3),              # K < 128: zero-filled Filter rows
    cs("h_c_tail", 64, 24, 200, 7, 5, 3, 2),               # C, K not multiples of the blocks
    cs("h_stride2", 32, 16, 96, 10, 9, 3, 3, 2, 2),
    cs("h_stride_mixed", 64, 8, 136, 11, 6, 5, 2, 2, 1),
    cs("h_5x5_s2", 32, 8, 64, 12, 12, 5, 5, 2, 2),
    cs("h_7x7_s2_c3", 64, 3, 64, 20, 18, 7, 7, 2, 2),      # C = 3: zero-padded channel chunk
    cs("h_c_odd", 32, 21, 72, 6, 6, 3, 3),                 # C % 8 != 0: element-wise packing
    cs("h_11x11_s4", 32, 3, 96, 5, 5, 11, 11, 4, 4),       # the worked example's filter: 121 taps
    cs("h_asym", 96, 40, 130, 5, 13, 2, 4, 1, 3),          # B = 3 batch blocks of 32; sh > 1
    cs("h_big_c", 32, 520, 128, 3, 3, 3, 3),               # many channel chunks: ring wraps often
    cs("h_many_tiles", 128, 64, 384, 20, 18, 3, 3),        # more tiles than SMs: persistent loop
    cs("h_1x1_s2", 64, 48, 136, 9, 7, 1, 1, 2, 2),         # 1x1 with strides: strided Image view
    cs("h_1x1_s3x1", 32, 32, 64, 6, 11, 1, 1, 3, 1),
    cs("h_1x1_s1x2", 40, 16, 128, 13, 5, 1, 1, 1, 2),
]


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("c", HALO_SHAPES, ids=lambda c: c.name)
def test_halo_shapes(c, out_dtype):
    info = check_full(c, variant=binding.VARIANT_HALO, out_dtype=out_dtype)
    assert info["variant"] == binding.VARIANT_HALO


# ---- small-C tensor-core kernel: (s,c) folded into the contraction ----------------------------------

STEM_SHAPES = [
    cs("st_c3_7x7_s2", 64, 3, 64, 20, 19, 7, 7, 2, 2),      # two stacked rows (shift sh*C = 6), odd H
    cs("st_c4_k40", 64, 4, 40, 9, 6, 3, 3),                 # ragged W tile; K < 64
    cs("st_c1", 128, 1, 16, 10, 7, 5, 5, 1, 2),             # two batch tiles, one channel, 4 stacked rows
    cs("st_c6_s3", 64, 6, 100, 7, 5, 3, 4, 3, 1),           # K = 100: no stacking; sw = 3
    cs("st_c2_wide", 64, 2, 24, 33, 3, 2, 9, 2, 1),         # S*C = 18; four stacked rows, H = 3
    cs("st_c3_k200", 64, 3, 200, 6, 5, 3, 3),               # two out-channel tiles
    cs("st_c5_h1", 64, 5, 64, 3, 1, 4, 2, 1, 3),            # one output row, W < bw
    cs("st_b32", 32, 3, 64, 9, 8, 7, 7, 2, 2),              # half a batch block (zero padded)
    cs("st_b72", 72, 4, 48, 6, 5, 3, 3),                    # one block + 8 images; 144-byte Out rows
]


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("c", STEM_SHAPES, ids=lambda c: c.name)
def test_stem_shapes(c, out_dtype):
    info = check_full(c, variant=binding.VARIANT_STEM, out_dtype=out_dtype)
    assert info["variant"] == binding.VARIANT_STEM


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
def test_halo_tail_launch(monkeypatch, out_dtype):
    """The wave-quantisation tail: output rows h >= tail_h0 come from a second launch with its own
    tile, running beside the first; every output must still be Eq. 1."""
    monkeypatch.setenv("CCONV_FORCE_TILE", "2,2,16,0,64")      # main: 2 x 2 pixels, 5 rows of tiles
    monkeypatch.setenv("CCONV_FORCE_TAIL", "3,4,1,16,0,64")    # keep 3 rows; rows h >= 6: 4 x 1 pixels
    c = cs("tail", 64, 40, 160, 8, 9, 3, 3)
    info = check_full(c, variant=binding.VARIANT_HALO, out_dtype=out_dtype)
    assert info["tail_h0"] == 6 and info["tail_bw"] == 4 and info["tail_bh"] == 1
    assert info["tiles"] == 2 * 1 * 4 * 3 and info["tail_tiles"] == 2 * 1 * 2 * 3


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("force,c", [
    ("4,2,16,0,32,2", cs("split_3x3", 32, 64, 160, 8, 5, 3, 3)),        # b_h = 2: one output row per CTA
    ("8,1,32,0,32,2", cs("split_w", 32, 128, 128, 13, 3, 3, 3)),        # b_h = 1: pixels split; ragged w
    ("2,2,64,0,64,2", cs("split_1x1", 64, 256, 200, 6, 6, 1, 1)),       # 1x1, K not a multiple of 128
    ("4,1,16,0,64,2", cs("split_s2", 64, 32, 64, 7, 4, 5, 3, 2, 1)),    # stride 2, 5x3 filter
    ("4,1,16,0,32,4", cs("split4_3x3", 32, 128, 160, 7, 5, 3, 3)),      # four CTAs per tile, a quarter of the channels each
    ("2,2,32,0,64,4", cs("split4_b64_bh2", 64, 256, 128, 6, 4, 3, 3)),  # b_h = 2: 256 columns, 64 per CTA
    ("8,2,16,0,8,4", cs("split4_blocks_of_8", 8, 64, 72, 7, 6, 3, 3)),  # batch blocks of 8 images
    ("4,1,32,0,16,2", cs("split2_blocks_of_16", 16, 128, 136, 7, 6, 3, 3)),  # ... and of 16
    ("4,1,16,0,32,4", cs("split4_1x1_s2", 32, 192, 64, 5, 5, 1, 1, 2, 2)),  # strided 1x1 view, 12 chunks: 3 per CTA
], ids=lambda v: v.name if hasattr(v, "name") else None)
def test_halo_split_channels_over_a_cta_pair(monkeypatch, force, c, out_dtype):
    """split = 2 or 4: a cluster of that many CTAs shares each tile, an equal share of the channels
    each; the partial sums cross through distributed shared memory.  Every output must still be
    Eq. 1."""
    monkeypatch.setenv("CCONV_FORCE_TILE", force)
    info = check_full(c, variant=binding.VARIANT_HALO, out_dtype=out_dtype)
    assert info["split"] == int(force.split(",")[5]) and info["grid"] == info["split"] * info["tiles"]


def test_tail_is_planned_for_the_large_config():
    cfg = synth.CONFIGS[4]
    p = binding.Plan(*cfg.dims(), device=0)
    info = p.info()
    p.close()
    assert info["variant"] == binding.VARIANT_HALO
    assert 0 < info["tail_h0"] < cfg.H and info["tail_h0"] % info["bh"] == 0
    assert info["tail_tiles"] <= 148 and info["tiles"] % info["grid"] != 1


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("c", [
    cs("b8", 8, 32, 64, 6, 5, 3, 3),            # a quarter of one batch block
    cs("b24_1x1", 24, 48, 130, 5, 4, 1, 1),     # 24 of 32 images, K and C ragged too
    cs("b40_s2", 40, 16, 32, 7, 6, 3, 5, 2, 1),  # one full block + 8 images
    cs("b72", 72, 64, 128, 4, 9, 3, 3),         # two full blocks + 8 images
], ids=lambda c: c.name)
def test_halo_batch_not_a_multiple_of_the_block(monkeypatch, c, out_dtype):
    """B % 8 == 0 but B % 32 != 0 with blocks of 32 images (forced where the planner would take a
    block of 8): the last batch block is zero padded by the TMA loads and its stores stop at B;
    nothing beyond Out's end may be touched (guard bands in run_gpu)."""
    monkeypatch.setenv("CCONV_FORCE_TILE", "0,0,0,0,32")
    info = check_full(c, variant=binding.VARIANT_HALO, out_dtype=out_dtype)
    assert info["bb"] == 32 and c.B % 32 != 0


@pytest.mark.parametrize("variant,c", [
    (binding.VARIANT_HALO, cs("chain_halo", 64, 64, 256, 20, 18, 3, 3)),     # several tiles per CTA
    (binding.VARIANT_STEM, cs("chain_stem", 64, 3, 64, 40, 38, 7, 7, 2, 2)),
], ids=["halo", "stem"])
def test_back_to_back_calls_with_changing_filters(variant, c):
    """The Filter packing of call n+1 runs while the convolution of call n is still executing (two
    scratch buffers, programmatic dependent launch).  Twelve unsynchronised calls that alternate
    between three Filters and two Images, each into its own Out: every one must be Eq. 1 of ITS
    inputs.  A packing kernel that overwrote a buffer still being read, or a convolution that
    started before its packing kernel finished, would show here."""
    inputs = [synth.make_inputs(c, seed=1000 + i) for i in range(3)]
    imgs = [to_dev(inputs[i][0]) for i in range(2)]
    flts = [to_dev(inputs[i][1]) for i in range(3)]
    exp = {}
    for i in range(2):
        for f in range(3):
            exp[(i, f)] = ocnn.cnn_bf16(inputs[i][0], inputs[f][1], oshape(c))
    plan = binding.Plan(*c.dims(), device=torch.cuda.current_device(), variant=variant,
                        out_dtype=binding.OUT_F32)
    calls = [(n % 2, (n * 2 + n // 3) % 3) for n in range(12)]
    outs = [torch.full(c.out_shape, float("nan"), dtype=torch.float32, device="cuda") for _ in calls]
    for (i, f), o in zip(calls, outs):
        plan.forward(imgs[i], flts[f], o)          # no synchronisation in between
    plan.check()
    plan.close()
    for n, ((i, f), o) in enumerate(zip(calls, outs)):
        e, ab = exp[(i, f)]
        assert_close(o.cpu().numpy().astype(np.float64), e, ab, f"call {n} (image {i}, filter {f})")


def test_random_shapes_tensor_kernels_match_the_cuda_core_kernel():
    """Forty seeded random shapes (batch multiples of 8, 1x1 to 7x7 filters, strides up to 3, ragged
    channel counts, tails, batch padding): whatever kernel the planner picks must agree with the
    CUDA-core kernel to fp32-accumulation noise; every fifth shape is also checked against the
    oracle with the stated tolerance."""
    import random
    rng = random.Random(20260)
    done = 0
    it = 0
    while done < 40:
        it += 1
        B = rng.choice([8, 16, 24, 32, 40, 64, 64, 96, 128])
        R = rng.choice([1, 1, 2, 3, 3, 3, 5, 7])
        S = rng.choice([1, 3, 3, R, R, 4])
        C = rng.choice([1, 3, 4, 8, 16, 24, 32, 48, 64, 100, 128, 192, 256])
        K = rng.choice([8, 16, 40, 64, 100, 128, 160, 256, 300])
        W, H = rng.randint(1, 17), rng.randint(1, 17)
        sw, sh = rng.choice([1, 1, 1, 2, 3]), rng.choice([1, 1, 1, 2])
        c = cs(f"rnd{it}", B, C, K, W, H, R, S, sw, sh)
        if c.macs > 1.5e9:
            continue
        done += 1
        ib, fb = synth.make_inputs(c, seed=7000 + it)
        ref, _ = run_gpu(c, ib, fb, binding.VARIANT_SIMT, binding.OUT_F32)
        got, info = run_gpu(c, ib, fb, binding.VARIANT_AUTO, binding.OUT_F32)
        assert info["variant"] != binding.VARIANT_SIMT, c
        scale = np.abs(ref).max() + 1e-30
        assert np.abs(got - ref).max() <= 2e-5 * scale * np.sqrt(C * R * S), (c, info)
        if done % 5 == 0:
            exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
            assert_close(got, exp, ab, f"{c.name} {c.dims()}")


def test_halo_matches_simt_kernel_on_device():
    c = cs("cross", 64, 48, 160, 9, 8, 3, 3)
    ib, fb = synth.make_inputs(c)
    a, _ = run_gpu(c, ib, fb, binding.VARIANT_HALO)
    b, _ = run_gpu(c, ib, fb, binding.VARIANT_SIMT)
    _, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
    # two fp32 accumulations of the same C*R*S products in different orders
    assert np.all(np.abs(a - b) <= c.C * c.R * c.S * 2.0 ** -23 * ab)


# ---- index pins on the device ---------------------------------------------------------------------------

@pytest.mark.parametrize("variant", [binding.VARIANT_SIMT, binding.VARIANT_HALO])
def test_delta_filter_on_device(variant):
    c = cs("delta", 32, 16, 40, 6, 5, 3, 2, 2, 1)
    ib, _ = synth.make_inputs(c)
    fb = np.zeros(c.filter_shape, dtype=np.uint16)
    k0, r0, s0, c0 = 33, 2, 1, 9
    fb[k0, r0, s0, c0] = 0x3F80                  # 1.0
    got, _ = run_gpu(c, ib, fb, variant, binding.OUT_BF16)
    img = ocnn.bf16_bits_to_f64(ib)
    for h in range(c.H):
        for w in range(c.W):
            np.testing.assert_array_equal(got[k0, h, w, :], img[r0 + c.sw * w, s0 + c.sh * h, c0, :])
    got[k0] = 0
    assert not got.any()


@pytest.mark.parametrize("variant", [binding.VARIANT_SIMT, binding.VARIANT_HALO])
def test_constant_inputs_on_device(variant):
    c = cs("const", 32, 16, 24, 5, 4, 3, 3)
    ib = np.full(c.image_shape, 0x3F00, dtype=np.uint16)     # 0.5
    fb = np.full(c.filter_shape, 0xBE80, dtype=np.uint16)    # -0.25
    for dt in DTYPES:
        got, _ = run_gpu(c, ib, fb, variant, dt)
        np.testing.assert_array_equal(got, np.full(c.out_shape, c.C * c.R * c.S * 0.5 * -0.25))


# ---- the other entry points --------------------------------------------------------------------------------

def test_cconv_forward_cached_plan_and_guard_bands():
    c = BY["cfg1_tiny_3x3"]
    ib, fb = synth.make_inputs(c)
    img, flt = to_dev(ib), to_dev(fb)
    n = int(np.prod(c.out_shape))
    buf = torch.full((n + 256,), -7.0, dtype=torch.bfloat16, device="cuda")
    out = buf[128:128 + n].view(c.out_shape)
    for _ in range(2):                                         # second call hits the plan cache
        binding.conv_forward(img, flt, out, *c.dims())
    torch.cuda.synchronize()
    exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
    assert_close(ocnn.bf16_bits_to_f64(to_bits(out)), exp, ab, "cconv_forward", bf16_out=True)
    assert (buf[:128] == -7.0).all() and (buf[128 + n:] == -7.0).all()   # nothing written outside Out


def test_forward_host_entry_point():
    c = cs("host", 32, 16, 128, 6, 6, 3, 3)
    ib, fb = synth.make_inputs(c)
    hi = torch.from_numpy(ib.view(np.int16)).view(torch.bfloat16).pin_memory()
    hf = torch.from_numpy(fb.view(np.int16)).view(torch.bfloat16).pin_memory()
    ho = torch.empty(c.out_shape, dtype=torch.bfloat16).pin_memory()
    plan = binding.Plan(*c.dims(), device=0)
    plan.forward_host(hi, hf, ho)
    exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
    assert_close(ocnn.bf16_bits_to_f64(to_bits(ho)), exp, ab, "cconv_forward_host", bf16_out=True)
    plan.close()


def test_pipelined_host_calls_keep_every_steps_result():
    """cconv_forward_host_async: six queued steps with different inputs and their own Out buffers
    (two staging sets inside the plan, so sets are re-used twice); each Out must be its own step's."""
    c = cs("host_pipe", 32, 24, 72, 9, 8, 3, 3)
    plan = binding.Plan(*c.dims(), device=0, out_dtype=binding.OUT_BF16)
    steps = []
    for n in range(6):
        ib, fb = synth.make_inputs(ConvShape(c.name, *c.dims(), seed=8600 + n))
        hi = torch.from_numpy(ib.view(np.int16)).view(torch.bfloat16).pin_memory()
        hf = torch.from_numpy(fb.view(np.int16)).view(torch.bfloat16).pin_memory()
        ho = torch.full(c.out_shape, float("nan"), dtype=torch.bfloat16).pin_memory()
        steps.append((ib, fb, hi, hf, ho))
    for _, _, hi, hf, ho in steps:
        plan.forward_host_async(hi, hf, ho)
    plan.host_wait()
    for n, (ib, fb, _, _, ho) in enumerate(steps):
        exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
        assert_close(ocnn.bf16_bits_to_f64(to_bits(ho)), exp, ab, f"pipelined step {n}", bf16_out=True)
    # the synchronous call still works on the same plan afterwards
    ib, fb, hi, hf, ho = steps[0]
    ho.fill_(float("nan"))
    plan.forward_host(hi, hf, ho)
    exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
    assert_close(ocnn.bf16_bits_to_f64(to_bits(ho)), exp, ab, "synchronous call after the pipeline", bf16_out=True)
    plan.close()


def test_misaligned_and_null_pointers_are_rejected_on_the_host():
    c = BY["cfg1_tiny_3x3"]
    plan = binding.Plan(*c.dims(), device=0)
    buf = torch.zeros(1 << 16, dtype=torch.bfloat16, device="cuda")
    p = buf.data_ptr()
    assert plan.forward_ptrs(p + 2, p + 4096, p + 8192, None) == binding.EINVAL
    assert plan.forward_ptrs(None, p + 4096, p + 8192, None) == binding.EINVAL
    plan.close()


def test_repeated_launches_are_deterministic():
    """Every kernel adds its terms in a fixed order: repeated launches of one kernel variant give the
    same bits.  An AUTO plan may run a call that has to wait for the stream's earlier work on its
    second (halo-kernel) tiling, which sums in another order, so for AUTO plans what repeats bit for
    bit is the same sequence of calls."""
    c = BY["cfg2_resnet_3x3"]
    ib, fb = synth.make_inputs(c)
    img, flt = to_dev(ib), to_dev(fb)
    for variant in (binding.VARIANT_DIRECT, binding.VARIANT_HALO):
        plan = binding.Plan(*c.dims(), device=0, variant=variant)
        outs = []
        for _ in range(3):
            out = torch.empty(c.out_shape, dtype=torch.bfloat16, device="cuda")
            plan.forward(img, flt, out)
            outs.append(to_bits(out))
        plan.check()
        np.testing.assert_array_equal(outs[0], outs[1])
        np.testing.assert_array_equal(outs[0], outs[2])
        plan.close()
    plan = binding.Plan(*c.dims(), device=0)
    bufs = [torch.empty(c.out_shape, dtype=torch.bfloat16, device="cuda") for _ in range(2)]
    runs = []
    for _ in range(2):
        torch.cuda.synchronize()
        for _ in range(2):                       # the same sequence twice: a, b, a (waits), b (waits)
            for out in bufs:
                plan.forward(img, flt, out)
        plan.check()
        runs.append([to_bits(out) for out in bufs])
    for x, y in zip(*runs):
        np.testing.assert_array_equal(x, y)
    plan.close()


def test_out_of_one_call_read_as_image_by_the_next_call_on_the_stream():
    """The convolution kernel of a call may start while the previous call's kernel is in its last
    tiles.  If the previous call's Out IS this call's Image (the layouts differ, but shapes can be
    made to agree: (K,H,W,B) of call A = (Wi,Hi,C,B) of call B), call B must still see all of it."""
    a = cs("chain_a", 64, 96, 128, 28, 28, 3, 3)                  # Out (128, 28, 28, 64)
    b = cs("chain_b", 64, 28, 64, 126, 26, 3, 3)                  # Image (128, 28, 28, 64)
    assert a.out_shape == b.image_shape
    ia, fa = synth.make_inputs(a)
    _, fb = synth.make_inputs(b)
    img_a, flt_a, flt_b = to_dev(ia), to_dev(fa), to_dev(fb)
    plan_a = binding.Plan(*a.dims(), device=0, variant=binding.VARIANT_HALO, out_dtype=binding.OUT_BF16)
    plan_b = binding.Plan(*b.dims(), device=0, variant=binding.VARIANT_HALO, out_dtype=binding.OUT_F32)
    mid = torch.zeros(a.out_shape, dtype=torch.bfloat16, device="cuda")
    out_b = torch.empty(b.out_shape, dtype=torch.float32, device="cuda")
    for rep in range(6):
        mid.zero_()                                               # stale values would be zeros
        out_b.fill_(float("nan"))
        plan_a.forward(img_a, flt_a, mid)
        plan_b.forward(mid, flt_b, out_b)
        plan_a.check()
        plan_b.check()
        exp, ab = ocnn.cnn_bf16(to_bits(mid), fb, oshape(b))      # oracle on what call A really wrote
        assert_close(out_b.cpu().numpy().astype(np.float64), exp, ab, what=f"chained call, repeat {rep}")
    # call A itself is checked elsewhere; here only that it wrote something
    assert float(mid.float().abs().max()) > 0
    plan_a.close()
    plan_b.close()


def test_out_of_one_call_read_as_filter_by_the_next_call_on_the_stream():
    """The Filter-packing kernel of a call normally runs beside the previous call's convolution.  If
    the previous call's Out IS this call's Filter ((K,H,W,B) of call A = (K,R,S,C) of call B), the
    packing must wait until all of it has been written."""
    a = cs("fchain_a", 64, 256, 128, 4, 5, 3, 3)                  # Out (128, 5, 4, 64) bf16
    b = cs("fchain_b", 32, 64, 128, 6, 5, 5, 4)                   # Filter (128, 5, 4, 64)
    a3 = cs("fchain_a3", 8, 64, 64, 3, 7, 3, 3)                   # Out (64, 7, 3, 8) bf16
    b3 = cs("fchain_b3", 64, 8, 64, 12, 11, 7, 3, 2, 2)           # Filter (64, 7, 3, 8)
    assert a.out_shape == b.filter_shape and a3.out_shape == b3.filter_shape
    for pa, pb in ((a, b), (a3, b3)):
        ia, fa = synth.make_inputs(pa)
        ib, _ = synth.make_inputs(pb)
        img_a, flt_a, img_b = to_dev(ia), to_dev(fa), to_dev(ib)
        plan_a = binding.Plan(*pa.dims(), device=0, variant=binding.VARIANT_HALO, out_dtype=binding.OUT_BF16)
        plan_b = binding.Plan(*pb.dims(), device=0, variant=binding.VARIANT_HALO, out_dtype=binding.OUT_F32)
        mid = torch.zeros(pa.out_shape, dtype=torch.bfloat16, device="cuda")
        out_b = torch.empty(pb.out_shape, dtype=torch.float32, device="cuda")
        for rep in range(6):
            mid.zero_()                                           # a stale Filter would be zeros
            out_b.fill_(float("nan"))
            plan_a.forward(img_a, flt_a, mid)
            plan_b.forward(img_b, mid, out_b)
            plan_a.check()
            plan_b.check()
            exp, ab = ocnn.cnn_bf16(ib, to_bits(mid), oshape(pb))
            assert_close(out_b.cpu().numpy().astype(np.float64), exp, ab,
                         what=f"{pb.name}: Out as Filter, repeat {rep}")
        assert float(mid.float().abs().max()) > 0
        plan_a.close()
        plan_b.close()


def test_two_plans_with_different_shared_memory_needs_stay_usable():
    """Plans share the kernels: creating a second plan with a smaller tile must not lower the
    shared-memory ceiling the first one needs."""
    big = cs("two_plans_big", 64, 64, 128, 12, 10, 3, 3)
    small = cs("two_plans_small", 32, 16, 64, 4, 3, 1, 1)
    plan_big = binding.Plan(*big.dims(), device=0, variant=binding.VARIANT_HALO, out_dtype=binding.OUT_F32)
    plan_small = binding.Plan(*small.dims(), device=0, variant=binding.VARIANT_HALO, out_dtype=binding.OUT_F32)
    assert plan_small.info()["smem_bytes"] <= plan_big.info()["smem_bytes"]
    for shp, plan in ((big, plan_big), (small, plan_small), (big, plan_big)):
        ib, fb = synth.make_inputs(shp)
        out = torch.full(shp.out_shape, float("nan"), dtype=torch.float32, device="cuda")
        plan.forward(to_dev(ib), to_dev(fb), out)
        plan.check()
        exp, ab = ocnn.cnn_bf16(ib, fb, oshape(shp))
        assert_close(out.cpu().numpy().astype(np.float64), exp, ab, what=shp.name)
    plan_big.close()
    plan_small.close()


def test_planned_forward_and_pooling_inside_a_cuda_graph():
    """Plans allocate at creation only: a planned forward call (packing kernel + convolution,
    programmatic dependent launch) and a pooling call can be captured into a CUDA graph and
    replayed on new contents of the same buffers."""
    from oracle import pool as opool
    c = cs("graph_planned", 64, 32, 128, 12, 9, 3, 3)
    ib, fb = synth.make_inputs(c)
    img, flt = to_dev(ib), to_dev(fb)
    out = torch.full(c.out_shape, float("nan"), device="cuda", dtype=torch.float32)
    # pooling reads the same Image: (Wi, Hi, C, B) -> 2x2 stride-2 windows, channel reduction, 3 planes
    pdims = (c.B, c.C, 3, (c.Wi - 2) // 2 + 1, (c.Hi - 2) // 2 + 1, 2, 2, 2, 2)
    pshape = ocnn.Shape(*pdims)
    pimg = img[:pshape.Wi, :pshape.Hi].contiguous()
    pout = torch.full(pshape.out_shape, float("nan"), device="cuda", dtype=torch.float32)
    plan = binding.Plan(*c.dims(), device=0, variant=binding.VARIANT_HALO, out_dtype=binding.OUT_F32)
    plan.forward(img, flt, out)               # warm-up outside the capture
    plan.check()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph, stream=side):
        plan.forward(img, flt, out)
        binding.pool_forward(pimg, pout, *pdims, op=binding.POOL_MAX)
    for seed in (81, 82):
        ib2, fb2 = synth.make_inputs(ConvShape("graph_planned", *c.dims(), seed=seed))
        img.copy_(to_dev(ib2))
        flt.copy_(to_dev(fb2))
        pimg.copy_(img[:pshape.Wi, :pshape.Hi])
        out.fill_(float("nan"))
        pout.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        exp, ab = ocnn.cnn_bf16(ib2, fb2, oshape(c))
        assert_close(out.cpu().numpy().astype(np.float64), exp, ab, what=f"graph replay, seed {seed}")
        pexp, _ = opool.pool_bf16(to_bits(pimg), pshape, opool.MAX)
        np.testing.assert_array_equal(pout.cpu().numpy().astype(np.float64), pexp)
    plan.check()
    plan.close()


def test_split_banded_and_accumulating_calls_inside_a_cuda_graph():
    """The other launch shapes survive capture too: a cluster launch of four CTAs per tile, a call on
    banded copies (padding kernel, convolution, compaction kernel) and an accumulating call (the
    twin's kernels plus the add kernel), captured once and replayed on new inputs."""
    c4 = cs("graph_split4", 16, 512, 128, 7, 6, 3, 3)
    c1 = cs("graph_bands", 1, 64, 64, 12, 16, 3, 3)
    jobs = []
    for c in (c4, c1):
        ib, fb = synth.make_inputs(c)
        jobs.append([c, to_dev(ib), to_dev(fb),
                     torch.full(c.out_shape, float("nan"), device="cuda", dtype=torch.float32),
                     binding.Plan(*c.dims(), device=0, out_dtype=binding.OUT_F32,
                                  variant=binding.VARIANT_HALO)])
    assert jobs[0][4].info()["split"] == 4 and jobs[1][4].info()["bands"] == 8
    acc = torch.zeros(c4.out_shape, device="cuda", dtype=torch.float32)
    jobs[0][4].reserve_accumulate()
    for c, img, flt, out, plan in jobs:
        plan.forward(img, flt, out)           # warm-up outside the capture
        plan.check()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.graph(graph, stream=side):
        for c, img, flt, out, plan in jobs:
            plan.forward(img, flt, out)
        jobs[0][4].forward_accumulate(jobs[0][1], jobs[0][2], acc)
    for seed in (91, 92):
        exps = []
        for c, img, flt, out, plan in jobs:
            ib2, fb2 = synth.make_inputs(ConvShape(c.name, *c.dims(), seed=seed))
            img.copy_(to_dev(ib2))
            flt.copy_(to_dev(fb2))
            out.fill_(float("nan"))
            exps.append(ocnn.cnn_bf16(ib2, fb2, oshape(c)))
        acc.fill_(2.5)
        graph.replay()
        torch.cuda.synchronize()
        for (c, img, flt, out, plan), (exp, ab) in zip(jobs, exps):
            assert_close(out.cpu().numpy().astype(np.float64), exp, ab, what=f"{c.name}, seed {seed}")
        assert_close(acc.cpu().numpy().astype(np.float64), exps[0][0] + 2.5, exps[0][1] + 2.5,
                     what=f"accumulate in a graph, seed {seed}")
    for job in jobs:
        job[4].check()
        job[4].close()


def test_mixed_plans_and_pooling_back_to_back_without_synchronisation():
    """Sixty calls of five plans (three kernel variants) and a pooling kernel on one stream, in a
    seeded random order, each with its own Filter and Out and no synchronisation in between: every
    kernel may start while its predecessors are still running (programmatic dependent launch), and
    every plan alternates its two scratch buffers.  All sixty results are checked afterwards."""
    from oracle import pool as opool
    rng = np.random.default_rng(1234)
    shapes = [
        (cs("mix_halo_3x3", 64, 32, 136, 9, 7, 3, 3), binding.VARIANT_HALO),
        (cs("mix_halo_1x1", 32, 64, 64, 6, 5, 1, 1, 2, 2), binding.VARIANT_HALO),
        (cs("mix_halo_big", 64, 64, 256, 14, 14, 3, 3), binding.VARIANT_HALO),   # several tiles per CTA
        (cs("mix_stem", 64, 3, 64, 11, 9, 5, 5, 2, 2), binding.VARIANT_STEM),
        (cs("mix_simt", 3, 5, 7, 6, 5, 3, 2), binding.VARIANT_SIMT),
    ]
    plans = [binding.Plan(*c.dims(), device=0, variant=v, out_dtype=binding.OUT_F32) for c, v in shapes]
    images = [to_dev(synth.make_inputs(c)[0]) for c, _ in shapes]
    pool_shape = ocnn.Shape(32, 4, 3, 5, 4, 3, 3, 2, 2)
    pool_bits = synth.make_inputs(ConvShape("mix_pool", *pool_shape.args(), seed=99))[0]
    pool_img = to_dev(pool_bits)
    jobs = []
    for n in range(60):
        i = int(rng.integers(0, len(shapes) + 1))
        if i == len(shapes):
            out = torch.full(pool_shape.out_shape, float("nan"), device="cuda", dtype=torch.float32)
            jobs.append(("pool", None, None, out))
        else:
            c = shapes[i][0]
            fb = synth.make_inputs(ConvShape(c.name, *c.dims(), seed=7000 + n))[1]
            out = torch.full(c.out_shape, float("nan"), device="cuda", dtype=torch.float32)
            jobs.append((i, fb, to_dev(fb), out))
    for kind, _, flt, out in jobs:                       # launch everything, no synchronisation
        if kind == "pool":
            binding.pool_forward(pool_img, out, *pool_shape.args(), op=binding.POOL_AVG)
        else:
            plans[kind].forward(images[kind], flt, out)
    for pl in plans:
        pl.check()
    pexp, pab = opool.pool_bf16(pool_bits, pool_shape, opool.AVG)
    cache = {}
    for n, (kind, fb, _, out) in enumerate(jobs):
        got = out.cpu().numpy().astype(np.float64)
        if kind == "pool":
            assert_close(got, pexp, pab, what=f"job {n}: pooling")
            continue
        c = shapes[kind][0]
        ib = cache.setdefault(kind, synth.make_inputs(c)[0])
        exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
        assert_close(got, exp, ab, what=f"job {n}: {c.name}")
    for pl in plans:
        pl.close()


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("variant,c", [
    (binding.VARIANT_HALO, cs("pad_b3", 3, 24, 72, 7, 6, 3, 3)),
    (binding.VARIANT_HALO, cs("pad_b12_s2", 12, 16, 136, 9, 8, 3, 3, 2, 2)),
    (binding.VARIANT_HALO, cs("pad_b100_1x1", 100, 32, 64, 5, 4, 1, 1)),
    (binding.VARIANT_HALO, cs("pad_b1", 1, 64, 128, 14, 14, 3, 3)),
    (binding.VARIANT_STEM, cs("pad_stem_b5", 5, 3, 64, 12, 11, 7, 7, 2, 2)),
    (binding.VARIANT_STEM, cs("pad_stem_b70", 70, 4, 40, 8, 6, 3, 3)),
], ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_batches_that_are_not_multiples_of_8_on_the_tensor_core_kernels(variant, c, out_dtype):
    info = check_full(c, variant=variant, out_dtype=out_dtype)
    assert info["variant"] == variant


def test_padded_batch_calls_back_to_back_with_changing_inputs():
    c = cs("pad_b2b", 6, 32, 128, 10, 9, 3, 3)
    plan = binding.Plan(*c.dims(), device=0, variant=binding.VARIANT_HALO, out_dtype=binding.OUT_F32)
    jobs = []
    for n in range(6):
        ib, fb = synth.make_inputs(ConvShape(c.name, *c.dims(), seed=8100 + n))
        out = torch.full(c.out_shape, float("nan"), device="cuda", dtype=torch.float32)
        jobs.append((ib, fb, to_dev(ib), to_dev(fb), out))
    for _, _, img, flt, out in jobs:
        plan.forward(img, flt, out)
    plan.check()
    for n, (ib, fb, _, _, out) in enumerate(jobs):
        exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
        assert_close(out.cpu().numpy().astype(np.float64), exp, ab, what=f"padded call {n}")
    plan.close()


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("c", [
    cs("taps_7x1", 32, 40, 136, 9, 8, 7, 1),            # R x 1: four-tap blocks along the filter row
    cs("taps_9x1_bh2", 64, 16, 128, 12, 10, 9, 1),
    cs("taps_1x7", 32, 24, 64, 8, 9, 1, 7),             # 1 x S: four-tap blocks along the filter column
    cs("taps_5x5", 64, 32, 128, 9, 9, 5, 5),
    cs("taps_6x4_s2", 32, 16, 72, 7, 6, 6, 4, 2, 2),
    cs("taps_4x8", 32, 8, 64, 6, 5, 4, 8),
], ids=lambda c: c.name)
def test_filters_that_use_the_four_tap_issue_blocks(c, out_dtype):
    info = check_full(c, variant=binding.VARIANT_HALO, out_dtype=out_dtype)
    assert info["variant"] == binding.VARIANT_HALO


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("c", [
    cs("sb_b8_3x3", 8, 32, 136, 13, 7, 3, 3),              # batch block of 8 images (16-byte rows)
    cs("sb_b8_1x1_s2", 8, 64, 64, 9, 6, 1, 1, 2, 2),
    cs("sb_b16_3x3", 16, 24, 200, 11, 9, 3, 3),            # batch block of 16 images (32-byte swizzle)
    cs("sb_b16_5x5_s2", 16, 16, 64, 8, 8, 5, 5, 2, 2),
    cs("sb_b1_3x3", 1, 48, 128, 30, 9, 3, 3),              # padded to 8: ragged w tile, two rows
    cs("sb_b3_w2", 3, 16, 64, 2, 5, 3, 3),                 # output row narrower than a 4-pixel group
    cs("sb_b12_3x3", 12, 32, 72, 10, 10, 3, 3),            # padded to 16
    cs("sb_b8_many_tiles", 8, 32, 384, 40, 36, 3, 3),      # more tiles than SMs
], ids=lambda c: c.name)
def test_small_batch_blocks(c, out_dtype):
    info = check_full(c, variant=binding.VARIANT_HALO, out_dtype=out_dtype)
    assert info["variant"] == binding.VARIANT_HALO


@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("force,c", [
    ("4,1,16,0,8", cs("sbf_b8_1x1_s2", 8, 64, 64, 9, 6, 1, 1, 2, 2)),      # forced blocks of 8 ...
    ("8,2,16,0,8", cs("sbf_b5_5x2", 5, 16, 72, 10, 7, 5, 2)),
    ("2,2,16,0,16", cs("sbf_b12_3x3", 12, 32, 72, 10, 10, 3, 3)),          # ... and of 16 images
    ("16,1,32,0,16", cs("sbf_b16_1x1", 16, 96, 128, 20, 3, 1, 1)),
], ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_forced_small_batch_blocks(monkeypatch, force, c, out_dtype):
    monkeypatch.setenv("CCONV_FORCE_TILE", force)
    info = check_full(c, variant=binding.VARIANT_HALO, out_dtype=out_dtype)
    assert info["bb"] == int(force.split(",")[4])


# ---- fewer than 8 images: bands of output rows take the place of images -----------------------------
@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("variant,c,bands", [
    (binding.VARIANT_HALO, cs("bands_b1_3x3", 1, 40, 136, 11, 23, 3, 3), 8),        # 8 bands of 3 rows, last one ragged
    (binding.VARIANT_HALO, cs("bands_b1_5x4_s2x3", 1, 16, 64, 9, 17, 5, 4, 2, 3), 6),  # strides; 17 rows = 6 bands of 3
    (binding.VARIANT_HALO, cs("bands_b2_1x1_s2", 2, 64, 72, 7, 9, 1, 1, 2, 2), 3),  # strided 1x1 view of 3-row bands
    (binding.VARIANT_HALO, cs("bands_b3", 3, 24, 128, 10, 8, 3, 3), 2),             # 2 bands x 3 images + 2 zero images
    (binding.VARIANT_HALO, cs("bands_b4_h1", 4, 32, 64, 12, 1, 3, 3), 1),           # one output row: nothing to cut
    (binding.VARIANT_HALO, cs("bands_b1_h5", 1, 32, 64, 6, 5, 3, 3), 5),            # fewer rows than bands wanted
    (binding.VARIANT_HALO, cs("bands_b7", 7, 16, 64, 6, 6, 3, 3), 1),               # 7 images: one band, one zero image
    (binding.VARIANT_STEM, cs("bands_stem_b1", 1, 3, 64, 20, 21, 7, 7, 2, 2), 7),   # 21 rows = 7 bands of 3
    (binding.VARIANT_STEM, cs("bands_stem_b2", 2, 4, 40, 9, 10, 3, 3), 4),
], ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_bands_of_output_rows_stand_in_for_images_when_the_batch_is_below_8(variant, c, bands, out_dtype):
    info = check_full(c, variant=variant, out_dtype=out_dtype)
    assert info["variant"] == variant and info["bands"] == bands
    assert info["run_H"] == -(-c.H // bands) and info["run_B"] == -(-c.B * bands // 8) * 8


def test_banded_calls_back_to_back_with_changing_inputs():
    """The banded copies are plan-owned scratch that every call overwrites: calls queued without
    synchronisation must not see one another's."""
    c = cs("bands_b2b", 1, 32, 128, 12, 19, 3, 3)
    plan = binding.Plan(*c.dims(), device=0, variant=binding.VARIANT_AUTO, out_dtype=binding.OUT_BF16)
    assert plan.info()["variant"] == binding.VARIANT_HALO and plan.info()["bands"] == 7
    jobs = []
    for n in range(5):
        ib, fb = synth.make_inputs(ConvShape(c.name, *c.dims(), seed=8300 + n))
        out = torch.full(c.out_shape, float("nan"), device="cuda", dtype=torch.bfloat16)
        jobs.append((ib, fb, to_dev(ib), to_dev(fb), out))
    for _, _, img, flt, out in jobs:
        plan.forward(img, flt, out)
    plan.check()
    for n, (ib, fb, _, _, out) in enumerate(jobs):
        exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
        assert_close(out.float().cpu().numpy().astype(np.float64), exp, ab, what=f"banded call {n}", bf16_out=True)
    plan.close()


# ---- Eq. 1's "+=" on an Out that already holds values ----------------------------------------------
@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("variant,c", [
    (binding.VARIANT_SIMT, cs("acc_simt", 3, 5, 7, 6, 5, 3, 2)),
    (binding.VARIANT_HALO, cs("acc_halo", 32, 40, 136, 9, 8, 3, 3)),
    (binding.VARIANT_HALO, cs("acc_halo_1x1_s2", 64, 64, 72, 7, 6, 1, 1, 2, 2)),
    (binding.VARIANT_HALO, cs("acc_halo_bands", 1, 32, 64, 10, 13, 3, 3)),
    (binding.VARIANT_STEM, cs("acc_stem", 64, 3, 64, 12, 11, 7, 7, 2, 2)),
], ids=lambda v: v.name if hasattr(v, "name") else str(v))
def test_accumulate_adds_the_convolution_to_what_out_holds(variant, c, out_dtype):
    """Out0 + Conv against Out0 + oracle, twice in a row (Out0 + 2 Conv); the tolerance scales with
    |Out0| + sum|Image*Filter|, and the stored bf16 value may be the rounding of any value inside it."""
    f32 = out_dtype == binding.OUT_F32
    ib, fb = synth.make_inputs(c)
    rng = np.random.default_rng(4400 + c.B)
    out0 = torch.from_numpy(rng.normal(0.0, 3.0, size=c.out_shape).astype(np.float32))
    out = out0.cuda() if f32 else out0.to(torch.bfloat16).cuda()
    start = out.float().cpu().numpy().astype(np.float64)
    plan = binding.Plan(*c.dims(), device=0, variant=variant, out_dtype=out_dtype)
    with pytest.raises(binding.CconvError):
        plan.forward_accumulate(to_dev(ib), to_dev(fb), out)          # nothing reserved yet
    plan.reserve_accumulate()
    plan.reserve_accumulate()                                          # a second call changes nothing
    img, flt = to_dev(ib), to_dev(fb)
    exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
    plan.forward_accumulate(img, flt, out)
    plan.check()
    once = out.float().cpu().numpy().astype(np.float64)
    assert_close(once, start + exp, np.abs(start) + ab, what=f"{c.name}: Out0 + Conv", bf16_out=not f32)
    plan.forward_accumulate(img, flt, out)
    plan.check()
    twice = out.float().cpu().numpy().astype(np.float64)
    assert_close(twice, once + exp, np.abs(once) + ab, what=f"{c.name}: second call", bf16_out=not f32)
    # the plain call still overwrites
    plan.forward(img, flt, out)
    plan.check()
    assert_close(out.float().cpu().numpy().astype(np.float64), exp, ab, what=f"{c.name}: plain",
                 bf16_out=not f32)
    plan.close()


# ---- split tiles chosen by the planner: small grids, long channel loops ------------------------------
@pytest.mark.parametrize("out_dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("c", [
    cs("autosplit_b16_3x3", 16, 256, 256, 7, 7, 3, 3),           # 28 whole tiles -> 56 tiles x 2 CTAs
    cs("autosplit_b32_5x5", 32, 128, 200, 5, 4, 5, 5),           # K padded to 256, ragged w tile
    cs("autosplit_b64_3x3", 64, 256, 128, 6, 5, 3, 3),           # blocks of 64 images, one pixel per tile
    cs("autosplit_b24_s2", 24, 512, 64, 5, 4, 3, 3, 2, 1),       # B % 32 != 0, strides
    cs("autosplit_b40_4x4", 40, 160, 136, 4, 4, 4, 4),           # C = 160: ten 16-channel chunks, five per CTA
    cs("autosplit_b8", 8, 512, 512, 7, 7, 3, 3),                 # batch blocks of 8 images, four CTAs per tile
    cs("autosplit_b16_5x5", 16, 256, 136, 7, 6, 5, 5),
], ids=lambda c: c.name)
def test_planner_splits_channels_over_cta_pairs_on_small_grids(c, out_dtype):
    info = check_full(c, variant=binding.VARIANT_HALO, out_dtype=out_dtype)
    assert info["variant"] == binding.VARIANT_HALO and info["split"] in (2, 4)
    assert info["grid"] == info["split"] * info["tiles"]
