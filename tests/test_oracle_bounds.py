"""Pins for the planner oracle (Theorem 1 terms, the Section-5 tiling LP, Theorem 2).  No GPU.

Expected values are the ones the paper prints for its AlexNet-layer example (read from
tests/golden/fig1_alexnet_layer.txt), identities the paper states, or explicit tilings from the
Appendix-A lemmas -- never outputs of the code under test.
"""
import math
import os

import numpy as np
import pytest

from oracle import bounds as ob
from paper_1802_06905_b200.synth import CONFIGS

GOLD = os.path.join(os.path.dirname(__file__), "golden", "fig1_alexnet_layer.txt")


def load_gold():
    g = {}
    with open(GOLD) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split()
            g[k] = float(v)
    return g


G = load_gold()
ALEX = tuple(int(G[k]) for k in ("B", "C", "K", "W", "H", "R", "S", "sw", "sh"))


def test_terms_are_the_printed_formula():
    B, C, K, W, H, R, S, sw, sh = 2, 3, 5, 7, 11, 4, 6, 2, 3
    M = 100.0
    t = ob.theorem1_terms(B, C, K, W, H, R, S, sw, sh, M)
    assert t[0] == 2 * 5 * 7 * 11
    assert t[1] == 2 * 3 * 2 * 3 * 7 * 11
    assert t[2] == 3 * 5 * 4 * 6
    assert t[3] == pytest.approx(2 * 3 * 5 * 7 * 11 * 24 / 100)
    assert t[4] == pytest.approx(2 * 3 * 5 * 7 * 11 * math.sqrt(24 * 6 / 100))


def test_fig1_term5_tight_up_to_17k_words():
    # term 5 stops being the largest where it meets term 1: M = C^2 R S sw sh = 9*121*16
    Mx = 9 * 121 * 16
    assert abs(Mx - G["term5_tight_up_to_words"]) / G["term5_tight_up_to_words"] < 0.03
    for M, is5 in [(Mx * 0.98, True), (Mx * 1.02, False), (1024, True), (64, True)]:
        _, arg = ob.theorem1_bound(*ALEX, M)
        assert (arg == 5) == is5
    t = ob.theorem1_terms(*ALEX, float(Mx))
    assert t[4] == pytest.approx(t[0], rel=1e-12)


def test_fig1_matmul_reuse_ratio():
    # matmul-level reuse would cost BCKWHRS/sqrt(M); the ratio to term 5 is sqrt(RS/(sw sh)) = 11/4
    M = 1024.0
    B, C, K, W, H, R, S, sw, sh = ALEX
    matmul_like = B * C * K * W * H * R * S / math.sqrt(M)
    t5 = ob.theorem1_terms(*ALEX, M)[4]
    assert matmul_like / t5 == pytest.approx(G["matmul_reuse_ratio"], rel=1e-12)


def test_fig1_tiling_at_1024_words():
    M = G["M"]
    B, C, K, W, H, R, S, sw, sh = ALEX
    printed = [G[k] for k in ("b_b", "b_c", "b_k", "b_w", "b_h", "b_r1", "b_r2", "b_s1", "b_s2")]
    exact = [math.sqrt(M * sh * sw / (R * S)), C, math.sqrt(M * sh * sw / (R * S)), R / sw, S / sh,
             R / sw, 1.0, S / sh, math.sqrt(M * sh * sw / (R * S)) / C]
    for p, e in zip(printed, exact):          # the printed integers are the closed forms rounded
        assert abs(p - e) <= 0.5
    tiles, Gopt, cost = ob.tiling_lp(*ALEX, M)
    # the optimum is not unique but its objective is: compare the product, not the factors
    assert Gopt == pytest.approx(np.prod(exact), rel=1e-6)
    F = B * C * K * W * H * R * S
    assert cost == pytest.approx(F * M / np.prod(exact), rel=1e-6)
    # and that cost is exactly the fifth term
    assert cost == pytest.approx(ob.theorem1_terms(*ALEX, M)[4], rel=1e-6)
    # the printed tiling is feasible for the block constraints
    bb, bc, bk, bw, bh, br1, br2, bs1, bs2 = exact
    assert bb * bk * bw * bh <= M * (1 + 1e-9)
    assert bc * bk * br1 * br2 * bs1 * bs2 <= M * (1 + 1e-9)
    for x in (bw, br1):
        for y in (bh, bs1):
            assert bb * bc * x * y * br2 * bs2 <= M * (1 + 1e-9)


def test_term5_exceeds_term4_iff_RS_lt_M_sw_sh():
    rng = np.random.default_rng(0)
    for _ in range(200):
        B, C, K, W, H = (int(v) for v in rng.integers(1, 40, size=5))
        R, S = (int(v) for v in rng.integers(1, 12, size=2))
        sw, sh = int(rng.integers(1, R + 1)), int(rng.integers(1, S + 1))
        M = float(rng.integers(2, 400))
        t = ob.theorem1_terms(B, C, K, W, H, R, S, sw, sh, M)
        if R * S != M * sw * sh:
            assert (t[4] > t[3]) == (R * S < M * sw * sh)


def test_pointwise_reduces_to_matmul_bound():
    # R=S=1, stride 1: n x n times n x k matmul has bound max(sizes, n^2 k / sqrt(M)) (Section 3)
    n, kk, M = 512, 300, 4096.0
    t = ob.theorem1_terms(B=kk, C=n, K=n, W=1, H=1, R=1, S=1, sw=1, sh=1, M=M)
    assert max(t) == pytest.approx(max(n * n, n * kk, n * n * kk / math.sqrt(M)))
    assert t[4] == pytest.approx(n * n * kk / math.sqrt(M))


def shapes_for_lp():
    shapes = [c.dims() for c in CONFIGS] + [ALEX]
    rng = np.random.default_rng(3)
    for _ in range(40):
        B, C, K = (int(v) for v in rng.integers(1, 300, size=3))
        sw, sh = (int(v) for v in rng.integers(1, 4, size=2))
        R, S = int(rng.integers(sw, 4 * sw + 1)), int(rng.integers(sh, 4 * sh + 1))
        W, H = int(rng.integers(-(-R // sw), 60)), int(rng.integers(-(-S // sh), 60))
        shapes.append((B, C, K, W, H, R, S, sw, sh))
    return shapes


@pytest.mark.parametrize("dims", shapes_for_lp(), ids=lambda d: "-".join(map(str, d)))
def test_lp_cost_equals_bound_when_bound_at_least_M(dims):
    """Section 5.2: the tiling's cost equals the largest of the five terms, except where the bound
    is below M; and it never undercuts any term."""
    for M in (256.0, 1024.0, 8192.0, 116224.0, 2.0 ** 21, 3.0e7):
        lb, _ = ob.theorem1_bound(*dims, M)
        _, _, cost = ob.tiling_lp(*dims, M)
        assert cost >= lb * (1 - 1e-7)
        if lb >= M:
            assert cost == pytest.approx(lb, rel=1e-6)
        else:
            assert cost == pytest.approx(M, rel=1e-6)   # a single round of M words


def test_hbl_lp_optimum_is_two():
    assert ob.hbl_lp_value() == pytest.approx(2.0, abs=1e-9)


def test_theorem2_leaves_for_the_benchmark_shapes():
    M = 116224.0        # words of a 227 KB shared memory
    by = {c.name: c for c in CONFIGS}
    d = by["cfg2_resnet_3x3"]
    assert ob.theorem2_case(d.B, d.C, d.K, d.W, d.H, d.R, d.S, M)[0] == "2.2.2.1"
    d = by["cfg5_large_3x3"]
    leaf, alb = ob.theorem2_case(d.B, d.C, d.K, d.W, d.H, d.R, d.S, M)
    assert leaf == "2.2.2.1"
    assert alb == pytest.approx(ob.theorem1_terms(*d.dims(), M)[4])
    d = by["cfg4_pointwise_1x1"]
    leaf, alb = ob.theorem2_case(d.B, d.C, d.K, d.W, d.H, d.R, d.S, M)
    assert leaf == "2.2.2.2" and alb == d.C * d.H * d.W * d.B
    d = by["cfg1_tiny_3x3"]
    assert ob.theorem2_case(d.B, d.C, d.K, d.W, d.H, d.R, d.S, M)[0] == "1"


def test_theorem2_leaves_21_and_221_by_hand():
    """Theorem 2 (Appendix A), the two leaves no benchmark shape reaches, multiplied out by hand.
    Case 2.1: every array exceeds M and R*S >= M; ALB = K*C*H*W*B*R*S / M.
    Case 2.2.1: R*S < M and M*R*S >= (B*H*W)^2; ALB = K*C*R*S."""
    # B=2 C=3 K=5 W=H=4 R=S=4, M=16: CHWB = 96, KCRS = 240, KHWB = 160, all > 16; RS = 16 >= 16
    leaf, alb = ob.theorem2_case(2, 3, 5, 4, 4, 4, 4, 16.0)
    assert leaf == "2.1" and alb == 480.0            # 5*3*4*4*2*16 / 16
    # one word more of fast memory and R*S < M: (BHW)^2 = 1024 > M*RS = 272, min(C,K) = 3 >= sqrt(17/16)
    leaf, alb = ob.theorem2_case(2, 3, 5, 4, 4, 4, 4, 17.0)
    assert leaf == "2.2.2.1" and alb == pytest.approx(480.0 * math.sqrt(16.0 / 17.0), rel=1e-15)
    # B=1 C=10 K=8 W=5 H=4 R=S=3, M=64: CHWB = 200, KCRS = 720, KHWB = 160, all > 64; RS = 9 < 64;
    # M*RS = 576 >= (BHW)^2 = 400
    leaf, alb = ob.theorem2_case(1, 10, 8, 5, 4, 3, 3, 64.0)
    assert leaf == "2.2.1" and alb == 720.0          # 8*10*3*3
    # two images: (BHW)^2 = 1600 > 576, min(C,K) = 8 >= sqrt(64/9): Case 2.2.2.1, 8*10*40*sqrt(9/64)
    leaf, alb = ob.theorem2_case(2, 10, 8, 5, 4, 3, 3, 64.0)
    assert leaf == "2.2.2.1" and alb == pytest.approx(1200.0, rel=1e-15)
    # ... and with too few channels for that, Case 2.2.2.2: max(KHWB, CHWB) = max(320, 80)
    leaf, alb = ob.theorem2_case(2, 2, 8, 5, 4, 3, 3, 64.0)
    assert leaf == "2.2.2.2" and alb == 320.0
    # an array that fits: Case 1 whatever the rest says (CHWB = 40 <= 64)
    leaf, alb = ob.theorem2_case(1, 2, 8, 5, 4, 3, 3, 64.0)
    assert leaf == "1" and alb == 160.0              # max(40, 144, 160)


def test_case_2221_lemma_tiling_is_admissible_and_attains_term5():
    # Lemma for case 2.2.2.1: bK=bC=sqrt(M/RS), bR=R, bS=S, bH*bW*bB=sqrt(M*RS); G=M^1.5 (RS)^0.5
    d = [c for c in CONFIGS if c.name == "cfg5_large_3x3"][0]
    M = 116224.0
    bK = bC = math.sqrt(M / (d.R * d.S))
    hwb = math.sqrt(M * d.R * d.S)
    assert bK * hwb <= M * (1 + 1e-12) and bC * hwb <= M * (1 + 1e-12)
    assert bK * bC * d.R * d.S <= M * (1 + 1e-12)
    cost = ob.tiling_cost(d.macs, M, [bK, bC, d.R, d.S, hwb])
    assert cost == pytest.approx(ob.theorem1_terms(*d.dims(), M)[4], rel=1e-12)
    # and the general LP (stride 1) finds the same cost
    assert ob.tiling_lp(*d.dims(), M)[2] == pytest.approx(cost, rel=1e-6)


def test_pooling_lp_drops_filter_constraint():
    # Section 6: without the Filter block the tile can only grow
    d = CONFIGS[4]
    M = 8192.0
    g_conv = ob.tiling_lp(*d.dims(), M)[1]
    g_pool = ob.tiling_lp(*d.dims(), M, pooling=True)[1]
    assert g_pool >= g_conv * (1 - 1e-9)


# ---- parallel sketch (Section 8): p processors, output cut into aB x aK x aH x aW blocks ----------

def test_parallel_terms_are_p_times_theorem1_on_the_subproblem():
    # the definition the section starts from: p * (Theorem 1 with B, K, H, W divided by the a's)
    dims = (32, 24, 48, 12, 8, 3, 3, 2, 1)
    B, C, K, W, H, R, S, sw, sh = dims
    M = 4096.0
    for (aB, aK, aH, aW) in [(1, 1, 1, 1), (2, 1, 1, 1), (1, 4, 1, 1), (2, 2, 2, 3), (4, 3, 4, 2)]:
        p = aB * aK * aH * aW
        sub = ob.theorem1_terms(B // aB, C, K // aK, W // aW, H // aH, R, S, sw, sh, M)
        got = ob.parallel_terms(*dims, M, aB, aK, aH, aW)
        np.testing.assert_allclose(got, [p * x for x in sub], rtol=1e-12)
    # one processor: Theorem 1 itself
    assert ob.parallel_terms(*dims, M, 1, 1, 1, 1) == ob.theorem1_terms(*dims, M)


def test_parallel_partition_prefers_the_cut_that_replicates_the_smaller_array():
    M = 116224.0
    # large 3x3 shape (B128 C512 K512 28x28): Filter is 2.4 M words, Image 51 M: cutting the batch
    # in 8 replicates only the Filter (8 * 2.4 M < |Out|), so the bound does not move
    dims = (128, 512, 512, 28, 28, 3, 3, 1, 1)
    one = max(ob.theorem1_terms(*dims, M))
    (aB, aK, aH, aW), bound = ob.parallel_partition(*dims, M, 8)
    assert aK == 1 and aB * aH * aW == 8
    assert bound == pytest.approx(one)
    # cutting the out-channels instead multiplies the Image term: strictly worse once it passes the max
    t_k = ob.parallel_terms(*dims, M, 1, 8, 1, 1)
    assert t_k[1] == pytest.approx(8 * 128 * 512 * 28 * 28) and max(t_k) > bound
    # a huge Filter and a single small image: now the out-channels are what to cut
    dims2 = (1, 64, 4096, 2, 2, 7, 7, 1, 1)
    (aB, aK, aH, aW), _ = ob.parallel_partition(*dims2, 1024.0, 4)
    assert (aB, aK, aH, aW) == (1, 4, 1, 1)


def test_parallel_partition_uses_all_processors_the_output_allows():
    dims = (2, 8, 3, 2, 2, 3, 3, 1, 1)      # only 2*3*2*2 = 24 output blocks exist
    (aB, aK, aH, aW), _ = ob.parallel_partition(*dims, 512.0, 64)
    assert aB * aK * aH * aW == 24
    (aB, aK, aH, aW), _ = ob.parallel_partition(*dims, 512.0, 5)
    assert aB * aK * aH * aW == 4           # 5 is prime and > every extent: 4 is the largest product
