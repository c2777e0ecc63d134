"""Host-side checks of the C-ABI library: it loads without a GPU, exports every declared symbol,
rejects bad arguments, and its planner agrees with the planner oracle.  No compute calls."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import bounds as ob
from paper_1802_06905_b200 import binding
from paper_1802_06905_b200.synth import CONFIGS

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1802_06905_b200 import build
    build.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "cconv.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(cconv_[a-z_0-9]+)\s*\(", hdr))
    assert declared, "no declarations found"
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_strerror_and_version(lib):
    assert lib.cconv_version() >= 100
    assert lib.cconv_strerror(0) == b"ok"
    assert b"invalid" in lib.cconv_strerror(binding.EINVAL)


def test_lower_bound_matches_oracle_terms():
    rng = np.random.default_rng(5)
    for _ in range(100):
        B, C, K, W, H = (int(v) for v in rng.integers(1, 500, size=5))
        R, S = (int(v) for v in rng.integers(1, 12, size=2))
        sw, sh = (int(v) for v in rng.integers(1, 5, size=2))
        M = float(rng.integers(2, 10 ** 6))
        got = binding.lower_bound(B, C, K, W, H, R, S, sw, sh, M)
        exp = ob.theorem1_terms(B, C, K, W, H, R, S, sw, sh, M)
        np.testing.assert_allclose(got, exp, rtol=1e-13)


def test_lower_bound_rejects_bad_arguments(lib):
    t = (ctypes.c_double * 5)()
    assert lib.cconv_lower_bound(0, 1, 1, 1, 1, 1, 1, 1, 1, 10.0, t) == binding.EINVAL
    assert lib.cconv_lower_bound(1, 1, 1, 1, 1, 1, 1, 1, 1, 0.0, t) == binding.EINVAL
    assert lib.cconv_lower_bound(1, 1, 1, 1, 1, 1, 1, 1, 1, 10.0, None) == binding.EINVAL


def lp_shapes():
    shapes = [c.dims() for c in CONFIGS] + [(1000, 3, 96, 55, 55, 11, 11, 4, 4)]
    rng = np.random.default_rng(17)
    for _ in range(60):
        B, C, K = (int(v) for v in rng.integers(1, 400, size=3))
        sw, sh = (int(v) for v in rng.integers(1, 4, size=2))
        R, S = int(rng.integers(1, 4 * sw + 1)), int(rng.integers(1, 4 * sh + 1))
        W, H = int(rng.integers(1, 80)), int(rng.integers(1, 80))
        shapes.append((B, C, K, W, H, R, S, sw, sh))
    return shapes


@pytest.mark.parametrize("dims", lp_shapes(), ids=lambda d: "-".join(map(str, d)))
def test_tiling_lp_objective_matches_oracle(dims):
    """The optimiser is not unique; its objective G (hence the words moved) is."""
    for M in (64.0, 1024.0, 116224.0, 6.0e7):
        tiles, G, words = binding.tiling_lp(*dims, M)
        _, G_o, words_o = ob.tiling_lp(*dims, M)
        assert G == pytest.approx(G_o, rel=1e-7)
        assert words == pytest.approx(words_o, rel=1e-7)
        # feasibility of the library's own point in the block constraints
        bb, bc, bk, bw, bh, r1, r2, s1, s2 = tiles
        B, C, K, W, H, R, S, sw, sh = dims
        tol = 1 + 1e-9
        assert all(t >= 1 / tol for t in tiles)
        assert bb <= B * tol and bc <= C * tol and bk <= K * tol and bw <= W * tol and bh <= H * tol
        assert r2 <= sw * tol and s2 <= sh * tol
        assert r1 <= max(1.0, R / sw) * tol and s1 <= max(1.0, S / sh) * tol
        assert bb * bk * bw * bh <= M * tol
        assert bc * bk * r1 * r2 * s1 * s2 <= M * tol
        for x in (bw, r1):
            for y in (bh, s1):
                assert bb * bc * x * y * r2 * s2 <= M * tol
        assert np.prod(tiles) == pytest.approx(G, rel=1e-9)


def test_pooling_lp_matches_oracle():
    d = CONFIGS[4].dims()
    for M in (512.0, 8192.0):
        _, G, _ = binding.tiling_lp(*d, M, pooling=True)
        assert G == pytest.approx(ob.tiling_lp(*d, M, pooling=True)[1], rel=1e-7)


def test_inspection_plans_are_hardware_legal():
    """device=-1: a plan for a nominal B200, no CUDA call; the chosen tile must fit the SM."""
    for cfg in CONFIGS:
        p = binding.Plan(*cfg.dims(), device=-1)
        info = p.info()
        exp_terms = ob.theorem1_terms(*cfg.dims(), info["M_words"])
        np.testing.assert_allclose(info["term"], exp_terms, rtol=1e-13)
        assert info["bound_argmax"] == int(np.argmax(exp_terms)) + 1
        assert info["lp_words"] == pytest.approx(ob.tiling_lp(*cfg.dims(), info["M_words"])[2], rel=1e-7)
        assert info["compulsory_words"] == cfg.image_words + cfg.filter_words + cfg.out_words
        if info["variant"] == binding.VARIANT_HALO:
            assert cfg.B % 8 == 0
            n = info["bb"] * info["bw"]
            assert n % 16 == 0 and 16 <= n <= 256                      # tcgen05 N rule at M=128
            assert n * info["bh"] <= 512 and info["tmem_cols"] <= 512   # tensor memory
            assert info["smem_bytes"] <= 232448                        # 227 KB
            assert info["stages"] >= 1                                     # Image ring
            assert info["halo_w"] == cfg.sw * (info["bw"] - 1) + cfg.R
            assert info["halo_h"] == cfg.sh * (info["bh"] - 1) + cfg.S
            img_stage = info["halo_w"] * info["halo_h"] * info["bc"] * info["bb"] * 2
            assert info["filter_stages"] >= 2
            assert info["stages"] * img_stage + info["filter_stages"] * 4096 <= info["smem_bytes"]
            units = -(-cfg.C // 16) * cfg.R * cfg.S
            assert info["scratch_bytes"] == -(-cfg.K // 128) * units * 4096
            # wave-quantisation tail: whole rows of main tiles, the rest in one partial wave
            if info["tail_h0"] < cfg.H:
                assert info["tail_h0"] % info["bh"] == 0 and info["tail_h0"] > 0
                per_row = -(-cfg.K // 128) * (cfg.B // info["bb"]) * -(-cfg.W // info["bw"])
                assert info["tiles"] == per_row * (info["tail_h0"] // info["bh"])
                rows = cfg.H - info["tail_h0"]
                assert info["tail_tiles"] == (-(-cfg.K // 128) * (cfg.B // info["tail_bb"]) *
                                              -(-cfg.W // info["tail_bw"]) * -(-rows // info["tail_bh"]))
                assert info["tail_tiles"] <= 148
            else:
                assert info["tail_tiles"] == 0
            # the staged words can never undercut the bound at the shared-memory size
            assert info["tile_words_smem"] >= max(exp_terms) * 0.999 or max(exp_terms) < info["M_words"]
        elif info["variant"] == binding.VARIANT_DIRECT:
            assert cfg.B % 8 == 0 and cfg.C % 8 == 0                   # 16-byte TMA strides
            n = info["bb"] * info["bw"]
            assert n % 16 == 0 and 16 <= n <= 256                      # tcgen05 N rule at M=128
            assert info["bk"] in (128, 256) and info["bc"] in (16, 32, 64)
            kt = info["bk"] // 128
            assert n * info["bh"] * kt <= info["tmem_cols"] <= 512     # tensor memory
            assert info["smem_bytes"] <= 232448                        # 227 KB
            assert info["halo_w"] == cfg.sw * (info["bw"] - 1) + cfg.R
            assert info["halo_h"] == cfg.sh * (info["bh"] - 1) + cfg.S
            img_stage = info["halo_w"] * info["halo_h"] * info["bc"] * info["bb"] * 2
            filt_stage = info["filter_taps"] * info["bk"] * info["bc"] * 2
            assert 1 <= info["filter_taps"] <= cfg.R * cfg.S
            assert info["stages"] >= 1 and info["filter_stages"] >= 2
            assert info["stages"] * img_stage + info["filter_stages"] * filt_stage <= info["smem_bytes"]
            assert info["scratch_bytes"] == 0 and info["tail_tiles"] == 0
            assert info["tiles"] == (-(-cfg.K // info["bk"]) * -(-cfg.B // info["bb"]) *
                                     -(-cfg.W // info["bw"]) * -(-cfg.H // info["bh"]))
            assert info["grid"] == min(info["tiles"], 148)
            assert info["est_cta_cycles"] > 0 and info["est_period_cycles"] > 0
            assert info["tile_G"] == (info["bb"] * info["bc"] * info["bk"] * info["bw"] * info["bh"] *
                                      cfg.R * cfg.S)
            assert info["tile_words_smem"] >= max(exp_terms) * 0.999 or max(exp_terms) < info["M_words"]
        elif info["variant"] == binding.VARIANT_STEM:
            assert cfg.B % 8 == 0 and cfg.C < 8
            assert 1 <= info["bw"] <= 4 and 2 * 64 * info["bw"] <= info["tmem_cols"] <= 512
            assert info["bk"] * info["bh"] <= 128            # stacked output rows share the MMA's M
            assert info["halo_h"] == cfg.sh * (info["bh"] - 1) + cfg.S
            assert info["smem_bytes"] <= 232448 and info["stages"] >= 2
        else:
            assert info["variant"] == binding.VARIANT_SIMT
        # forward on an inspection plan is refused on the host, before any launch
        assert p._lib.cconv_forward_planned(p._h, 16, 16, 16, None) == binding.EINVAL
        # ... and so are reserving for, and making, accumulating calls
        assert p._lib.cconv_plan_reserve_accumulate(p._h) == binding.EINVAL
        assert p._lib.cconv_forward_accumulate(p._h, 32, 32, 32, None) == binding.EINVAL
        p.close()


def test_plan_create_rejects_bad_arguments(lib):
    h = ctypes.c_void_p()
    assert lib.cconv_plan_create(ctypes.byref(h), 0, 8, 8, 4, 4, 3, 3, 1, 1, -1, 0.0, 0, 0) == binding.EINVAL
    assert lib.cconv_plan_create(ctypes.byref(h), 2, 8, 8, 4, 4, 3, 3, 1, 1, -1, 0.0, 7, 0) == binding.EINVAL
    assert lib.cconv_plan_create(None, 2, 8, 8, 4, 4, 3, 3, 1, 1, -1, 0.0, 0, 0) == binding.EINVAL
    assert lib.cconv_plan_create(ctypes.byref(h), 2, 8, 8, 4, 4, 3, 3, 1, 1, -1, 0.0, 0, 5) == binding.EINVAL
    # B not a multiple of 8: the tensor-core variants run on a batch padded to the next multiple of 8
    for B in (2, 36):
        assert lib.cconv_plan_create(ctypes.byref(h), B, 8, 64, 12, 12, 3, 3, 1, 1, -1, 0.0,
                                     binding.VARIANT_HALO, 0) == binding.OK
        lib.cconv_plan_destroy(h)
    # B = 48: a multiple of 8 but not of 32 -> blocks of 32 images, the last one zero padded
    assert lib.cconv_plan_create(ctypes.byref(h), 48, 8, 64, 12, 12, 3, 3, 1, 1, -1, 0.0,
                                 binding.VARIANT_HALO, 0) == binding.OK
    info = binding.PlanInfo()
    assert lib.cconv_plan_info_get(h, ctypes.byref(info)) == binding.OK
    assert info.bb == 32 and info.tiles == 1 * 2 * -(-12 // info.bw) * -(-12 // info.bh)
    lib.cconv_plan_destroy(h)


def test_missing_library_fails_loudly(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "_LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        binding.load_library()


def test_strided_1x1_is_planned_on_a_subsampled_view():
    """A 1x1 filter with strides skips Image pixels: the tile's halo is the tile itself."""
    plan = binding.Plan(64, 1024, 2048, 7, 7, 1, 1, 2, 2, device=-1)
    info = plan.info()
    plan.close()
    assert info["variant"] in (binding.VARIANT_HALO, binding.VARIANT_DIRECT)
    assert info["halo_w"] == info["bw"] and info["halo_h"] == info["bh"]
    plan = binding.Plan(64, 64, 128, 7, 7, 3, 3, 2, 2, device=-1)
    info = plan.info()
    plan.close()
    assert info["halo_w"] == 2 * (info["bw"] - 1) + 3


def test_pool_lower_bound_matches_the_oracle_terms():
    for dims in [(64, 64, 256, 27, 27, 3, 3, 2, 2), (8, 3, 5, 6, 5, 3, 2, 1, 3)]:
        for M in (512.0, 116224.0):
            got = binding.pool_lower_bound(*dims, M)
            exp = ob.pooling_terms(*dims, M)
            assert got == pytest.approx(exp, rel=1e-12)
    lib = binding.load_library()
    t = (ctypes.c_double * 3)()
    assert lib.cconv_pool_lower_bound(0, 1, 1, 1, 1, 1, 1, 1, 1, 4.0, t) == -1
    assert lib.cconv_pool_lower_bound(1, 1, 1, 1, 1, 1, 1, 1, 1, 0.0, t) == -1


def test_parallel_bound_and_partition_match_the_oracle():
    rng = np.random.default_rng(17)
    for _ in range(40):
        B, C, K = (int(v) for v in rng.integers(1, 40, size=3))
        W, H = (int(v) for v in rng.integers(1, 12, size=2))
        R, S = (int(v) for v in rng.integers(1, 6, size=2))
        sw, sh = (int(v) for v in rng.integers(1, 3, size=2))
        M = float(rng.integers(64, 10 ** 5))
        p = int(rng.integers(1, 40))
        a, bound = binding.parallel_partition(B, C, K, W, H, R, S, sw, sh, M, p)
        a_exp, bound_exp = ob.parallel_partition(B, C, K, W, H, R, S, sw, sh, M, p)
        assert a == a_exp
        assert bound == pytest.approx(bound_exp, rel=1e-12)
        got = binding.parallel_lower_bound(B, C, K, W, H, R, S, sw, sh, M, *a)
        assert got == pytest.approx(ob.parallel_terms(B, C, K, W, H, R, S, sw, sh, M, *a), rel=1e-12)
        assert max(got) == pytest.approx(bound, rel=1e-12)
    lib = binding.load_library()
    t = (ctypes.c_double * 5)()
    assert lib.cconv_parallel_lower_bound(4, 4, 4, 4, 4, 1, 1, 1, 1, 64.0, 5, 1, 1, 1, t) == -1  # aB > B
    a = (ctypes.c_int * 4)()
    assert lib.cconv_parallel_partition(4, 4, 4, 4, 4, 1, 1, 1, 1, 64.0, 0, a, None) == -1


def test_batch_sharding_is_the_partition_the_bound_prefers_on_the_benchmark_shapes():
    """Multi-GPU runs shard the batch: for the large shapes the paper's own criterion picks a cut
    without aK (the Image is the big array), and with 8 processors the bound stays at |Out|."""
    for cfg in CONFIGS[1:]:
        dims = cfg.dims()
        a, bound = binding.parallel_partition(*dims, 116224.0, 8)
        one = max(binding.lower_bound(*dims, 116224.0))
        batch_cut = max(binding.parallel_lower_bound(*dims, 116224.0, 8, 1, 1, 1))
        assert batch_cut <= 1.0001 * max(one, 8 * dims[1] * dims[2] * dims[5] * dims[6])
        assert bound <= batch_cut * (1 + 1e-12)


def test_theorem2_leaf_matches_the_oracle_and_the_benchmark_shapes():
    rng = np.random.default_rng(23)
    seen = set()
    for _ in range(400):
        B, C, K = (int(v) for v in rng.integers(1, 300, size=3))
        W, H = (int(v) for v in rng.integers(1, 40, size=2))
        R, S = (int(v) for v in rng.integers(1, 12, size=2))
        M = float(2 ** rng.integers(1, 20))
        leaf, alb = binding.theorem2_case(B, C, K, W, H, R, S, M)
        leaf_exp, alb_exp = ob.theorem2_case(B, C, K, W, H, R, S, M)
        assert leaf == leaf_exp
        assert alb == pytest.approx(alb_exp, rel=1e-12)
        seen.add(leaf)
    assert seen == {"1", "2.1", "2.2.1", "2.2.2.1", "2.2.2.2"}
    # the two leaves no benchmark shape reaches, multiplied out by hand (Theorem 2's tree)
    assert binding.theorem2_case(2, 3, 5, 4, 4, 4, 4, 16.0) == ("2.1", 480.0)
    assert binding.theorem2_case(1, 10, 8, 5, 4, 3, 3, 64.0) == ("2.2.1", 720.0)
    assert binding.theorem2_case(2, 2, 8, 5, 4, 3, 3, 64.0) == ("2.2.2.2", 320.0)
    # the stride-1 benchmark shapes at the shared memory of one CTA
    M = 116224.0
    assert binding.theorem2_case(*CONFIGS[0].dims()[:7], M)[0] == "1"
    assert binding.theorem2_case(*CONFIGS[1].dims()[:7], M)[0] == "2.2.2.1"
    assert binding.theorem2_case(*CONFIGS[3].dims()[:7], M)[0] == "2.2.2.2"
    assert binding.theorem2_case(*CONFIGS[4].dims()[:7], M)[0] == "2.2.2.1"


def test_auto_variant_for_batches_that_are_not_multiples_of_8():
    """Small problems stay on the CUDA-core kernel (a padded batch costs two more kernels); large ones
    take the tensor-core path on a padded batch."""
    small = binding.Plan(2, 8, 16, 14, 14, 3, 3, 1, 1, device=-1)        # the tiny benchmark shape
    assert small.info()["variant"] == binding.VARIANT_SIMT
    small.close()
    big = binding.Plan(1, 64, 64, 14, 14, 3, 3, 1, 1, device=-1)        # 7 M multiply-adds, one image
    assert big.info()["variant"] == binding.VARIANT_HALO
    big.close()
    stem = binding.Plan(20, 3, 64, 56, 56, 7, 7, 2, 2, device=-1)
    assert stem.info()["variant"] == binding.VARIANT_STEM
    stem.close()


def test_random_shapes_plan_to_hardware_legal_tiles():
    """A thousand seeded random shapes (any batch size, filters up to 11x11, strides up to 4): every
    plan for a nominal B200 obeys the limits of the SM, whichever variant AUTO picks."""
    rng = np.random.default_rng(2718)
    seen = {binding.VARIANT_SIMT: 0, binding.VARIANT_HALO: 0, binding.VARIANT_STEM: 0,
            binding.VARIANT_DIRECT: 0}
    for _ in range(1000):
        B = int(rng.choice([1, 2, 3, 8, 12, 16, 24, 32, 40, 64, 100, 128, 256]))
        C = int(rng.choice([1, 3, 4, 7, 8, 16, 24, 48, 64, 100, 128, 256, 512, 1024]))
        K = int(rng.choice([1, 8, 16, 40, 64, 100, 128, 200, 256, 512, 1000]))
        W, H = (int(v) for v in rng.integers(1, 60, size=2))
        R = int(rng.choice([1, 1, 2, 3, 3, 5, 7, 11]))
        S = int(rng.choice([1, 3, R, R, 4]))
        sw, sh = (int(v) for v in rng.choice([1, 1, 2, 3, 4], size=2))
        p = binding.Plan(B, C, K, W, H, R, S, sw, sh, device=-1)
        info = p.info()
        p.close()
        seen[info["variant"]] += 1
        Bp, Hrun = info["run_B"], info["run_H"]   # the batch and rows the tensor-core kernels run
        assert Bp % 8 == 0 and Bp >= B * info["bands"] and Bp - B * info["bands"] < 8
        assert info["bands"] * Hrun >= H > (info["bands"] - 1) * Hrun
        assert (info["bands"] == 1 and Hrun == H) if B >= 8 else info["bands"] <= 8 // B
        if info["variant"] == binding.VARIANT_HALO:
            n = info["bb"] * info["bw"]
            assert info["bb"] in (8, 16, 32, 64) and info["bc"] in (16, 32, 64, 128)
            assert info["bb"] >= 32 or (Bp % info["bb"] == 0 and n % 32 == 0)
            assert n % 16 == 0 and 16 <= n <= 256
            assert n * info["bh"] <= 512 and info["tmem_cols"] in (32, 64, 128, 256, 512)
            assert 117760 <= info["smem_bytes"] <= 232448
            assert 1 <= info["stages"] <= 6 and 2 <= info["filter_stages"] <= 4
            assert 1 <= info["halo_w"] <= 256 and 1 <= info["halo_h"] <= 256
            img_stage = info["halo_w"] * info["halo_h"] * info["bc"] * info["bb"] * 2
            assert info["stages"] * img_stage + info["filter_stages"] * 4096 <= info["smem_bytes"]
            assert 1 <= info["grid"] <= 148 and info["split"] in (1, 2, 4)
            if info["split"] > 1:    # a cluster of two or four CTAs per tile, one wave
                assert info["grid"] == info["split"] * info["tiles"] and R * S >= 9
                assert (n * info["bh"]) % (32 * info["split"]) == 0 and info["tail_h0"] == Hrun
                assert info["split"] == 2 or info["grid"] <= 128
            else:
                assert info["tiles"] >= info["grid"]
            assert info["bw"] <= max(W, 1) + 3 and info["bh"] <= max(Hrun, 1)
            if info["tail_h0"] < Hrun:
                assert 0 < info["tail_h0"] and 1 <= info["tail_tiles"] <= 148
        elif info["variant"] == binding.VARIANT_DIRECT:
            # one wave of large tiles on the caller's own arrays
            n = info["bb"] * info["bw"]
            kt = info["bk"] // 128
            assert B % 8 == 0 and C % 8 == 0 and Bp == B
            assert info["bb"] in (32, 64) and info["bc"] in (16, 32, 64) and kt in (1, 2)
            assert n % 16 == 0 and 16 <= n <= 256
            assert n * info["bh"] * kt <= info["tmem_cols"] <= 512
            assert info["smem_bytes"] <= 232448 and (info["tmem_cols"] <= 256 or info["smem_bytes"] >= 117760)
            assert 1 <= info["halo_w"] <= 256 and 1 <= info["halo_h"] <= 256
            img_stage = info["halo_w"] * info["halo_h"] * info["bc"] * info["bb"] * 2
            filt_stage = info["filter_taps"] * info["bk"] * info["bc"] * 2
            assert info["stages"] * img_stage + info["filter_stages"] * filt_stage <= info["smem_bytes"]
            assert info["tiles"] == info["grid"] <= 148 and info["scratch_bytes"] == 0
        elif info["variant"] == binding.VARIANT_STEM:
            assert C < 8
            assert 1 <= info["bw"] <= 4 and info["bk"] in (32, 64, 128) and info["bk"] * info["bh"] <= 128
            assert 117760 <= info["smem_bytes"] <= 232448 and info["stages"] >= 2
            assert info["tmem_cols"] == 512 and 1 <= info["grid"] <= 148
        else:
            # the CUDA-core kernel is left only with tiny problems whose batch is not a multiple of 8
            assert B % 8 != 0 and B * C * K * W * H * R * S < 4e6 or Bp != B
    assert all(v > 0 for v in seen.values()), seen


def test_planner_split_rule():
    """Tiles are split over clusters of 2 or 4 CTAs only for filters of 9 or more taps with long channel
    loops and few output pixels; the benchmark shapes, 1x1 filters and short loops stay whole; four
    CTAs per tile need 288 units (C*R*S >= 4608)."""
    def split_of(*dims):
        p = binding.Plan(*dims, device=-1, variant=binding.VARIANT_HALO)
        info = p.info()
        p.close()
        return info["split"], info
    for cfg in CONFIGS:
        assert split_of(*cfg.dims())[0] == 1, cfg.name
    assert split_of(64, 512, 512, 7, 7, 3, 3, 1, 1)[0] == 2          # ResNet-50 conv5: 56 tiles x 2
    assert split_of(16, 1024, 256, 7, 7, 3, 3, 1, 1)[0] == 4         # 576 units: a quarter each
    assert split_of(16, 256, 256, 7, 7, 3, 3, 1, 1)[0] == 2          # 144 units: too short for four
    assert split_of(8, 512, 512, 7, 7, 5, 5, 1, 1)[0] == 4
    assert split_of(16, 128, 128, 7, 7, 3, 3, 1, 1)[0] == 1          # 72 units: stays whole
    assert split_of(16, 2048, 512, 7, 7, 1, 1, 1, 1)[0] == 1         # 1x1 filters stay whole
    assert split_of(64, 256, 256, 14, 14, 3, 3, 1, 1)[0] == 1        # enough pixels: whole tiles fill the SMs
    s, info = split_of(32, 1024, 256, 4, 4, 3, 3, 1, 1)
    assert s == 4 and info["grid"] == 4 * info["tiles"] <= 128
