"""Pins for the CPU oracle of Eq. 1 (the seven-nested-loop CNN).  No GPU, no CUDA path.

Every check compares the oracle with something it does not compute itself: index identities
(delta inputs), a pure-Python per-element evaluation, a library matrix product, a closed form,
a different loop nest, linearity, and a library convolution on permuted tensors.
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import cnn as ocnn
from oracle.cnn import Shape
from paper_1802_06905_b200 import synth

ASYM = Shape(B=3, C=2, K=4, W=5, H=3, R=3, S=2, sw=2, sh=1)   # every extent differs
ASYM2 = Shape(B=2, C=3, K=2, W=3, H=4, R=2, S=3, sw=1, sh=3)  # sh > S-1 gaps, sw=1


def rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


@pytest.mark.parametrize("shp", [ASYM, ASYM2])
def test_delta_filter_selects_shifted_image(shp):
    img = rand(shp.image_shape, 1)
    for (k0, r0, s0, c0) in [(1, 2 % shp.R, 1 % shp.S, 1), (0, 0, 0, 0),
                             (shp.K - 1, shp.R - 1, shp.S - 1, shp.C - 1)]:
        f = np.zeros(shp.filter_shape)
        f[k0, r0, s0, c0] = 1.0
        out, ab = ocnn.cnn_f64(img, f, shp)
        for h in range(shp.H):
            for w in range(shp.W):
                np.testing.assert_array_equal(out[k0, h, w, :],
                                              img[r0 + shp.sw * w, s0 + shp.sh * h, c0, :])
                np.testing.assert_array_equal(ab[k0, h, w, :],
                                              np.abs(img[r0 + shp.sw * w, s0 + shp.sh * h, c0, :]))
        mask = np.ones(shp.K, bool)
        mask[k0] = False
        assert not out[mask].any()


@pytest.mark.parametrize("shp", [ASYM, ASYM2])
def test_delta_image_scatters_filter(shp):
    f = rand(shp.filter_shape, 2)
    for (x0, y0, c0, b0) in [(2, 1, 1, 1), (0, 0, 0, 0), (shp.Wi - 1, shp.Hi - 1, shp.C - 1, shp.B - 1)]:
        img = np.zeros(shp.image_shape)
        img[x0, y0, c0, b0] = 1.0
        out, _ = ocnn.cnn_f64(img, f, shp)
        exp = np.zeros(shp.out_shape)
        for h in range(shp.H):
            for w in range(shp.W):
                r, s = x0 - shp.sw * w, y0 - shp.sh * h
                if 0 <= r < shp.R and 0 <= s < shp.S:
                    exp[:, h, w, b0] = f[:, r, s, c0]
        np.testing.assert_array_equal(out, exp)


def brute_force(img, f, shp):
    """Eq. 1 term by term in pure Python with exact-rounded fsum per element."""
    import math
    out = np.zeros(shp.out_shape)
    ab = np.zeros(shp.out_shape)
    for k, h, w, b in itertools.product(range(shp.K), range(shp.H), range(shp.W), range(shp.B)):
        terms = [float(img[r + shp.sw * w][s + shp.sh * h][c][b]) * float(f[k][r][s][c])
                 for c in range(shp.C) for r in range(shp.R) for s in range(shp.S)]
        out[k, h, w, b] = math.fsum(terms)
        ab[k, h, w, b] = math.fsum(abs(t) for t in terms)
    return out, ab


def small_shapes():
    shapes = []
    rng = np.random.default_rng(7)
    for _ in range(24):
        B, C, K, W, H, R, S = (int(v) for v in rng.integers(1, 4, size=7))
        sw, sh = (int(v) for v in rng.integers(1, 4, size=2))
        shapes.append(Shape(B, C, K, W, H, R, S, sw, sh))
    shapes += [Shape(1, 1, 1, 1, 1, 1, 1, 1, 1), Shape(2, 3, 2, 4, 3, 3, 2, 3, 1),
               Shape(3, 2, 3, 2, 4, 1, 4, 2, 3)]
    return shapes


@pytest.mark.parametrize("shp", small_shapes(), ids=lambda s: "-".join(map(str, s.args())))
def test_brute_force_tiny(shp):
    img = rand(shp.image_shape, 11)
    f = rand(shp.filter_shape, 12)
    out, ab = ocnn.cnn_f64(img, f, shp)
    eo, ea = brute_force(img, f, shp)
    n = shp.C * shp.R * shp.S
    assert np.all(np.abs(out - eo) <= n * 2.0 ** -52 * ea + 1e-300)
    assert np.all(np.abs(ab - ea) <= n * 2.0 ** -52 * ea + 1e-300)


def test_pointwise_equals_matrix_product():
    shp = Shape(B=5, C=7, K=6, W=4, H=3, R=1, S=1)
    img = rand(shp.image_shape, 3)
    f = rand(shp.filter_shape, 4)
    out, _ = ocnn.cnn_f64(img, f, shp)
    fm = f[:, 0, 0, :]                      # K x C
    for h in range(shp.H):
        for w in range(shp.W):
            np.testing.assert_allclose(out[:, h, w, :], fm @ img[w, h, :, :], rtol=0, atol=1e-13)


@pytest.mark.parametrize("shp", [ASYM, Shape(4, 8, 3, 5, 6, 3, 3, 1, 1), Shape(2, 3, 4, 6, 5, 7, 7, 2, 2)])
def test_constant_inputs_closed_form(shp):
    a, fv = 0.5, -0.25                       # exactly representable in bf16
    img = np.full(shp.image_shape, a)
    f = np.full(shp.filter_shape, fv)
    out, ab = ocnn.cnn_f64(img, f, shp)
    n = shp.C * shp.R * shp.S
    np.testing.assert_array_equal(out, np.full(shp.out_shape, n * a * fv))
    np.testing.assert_array_equal(ab, np.full(shp.out_shape, n * abs(a * fv)))


@pytest.mark.parametrize("shp", [ASYM, ASYM2, Shape(3, 5, 4, 6, 5, 3, 3, 1, 1)])
def test_loop_order_invariance(shp):
    img = rand(shp.image_shape, 5)
    f = rand(shp.filter_shape, 6)
    out, ab = ocnn.cnn_f64(img, f, shp)
    out2 = ocnn.cnn_f64_paper_order(img, f, shp)
    n = shp.C * shp.R * shp.S
    assert np.all(np.abs(out - out2) <= n * 2.0 ** -52 * ab)
    assert np.abs(out - out2).max() > 0 or n == 1  # the two nests really sum in different orders


def test_linearity():
    shp = ASYM
    i1, i2 = rand(shp.image_shape, 8), rand(shp.image_shape, 9)
    f = rand(shp.filter_shape, 10)
    alpha = 1.75
    lhs, ab = ocnn.cnn_f64(alpha * i1 + i2, f, shp)
    o1, a1 = ocnn.cnn_f64(i1, f, shp)
    o2, a2 = ocnn.cnn_f64(i2, f, shp)
    n = shp.C * shp.R * shp.S
    assert np.all(np.abs(lhs - (alpha * o1 + o2)) <= 4 * n * 2.0 ** -52 * (alpha * a1 + a2))


@pytest.mark.parametrize("shp", [ASYM, ASYM2, Shape(2, 8, 16, 14, 14, 3, 3, 1, 1),
                                 Shape(4, 3, 8, 9, 10, 7, 7, 2, 2), Shape(2, 4, 4, 5, 4, 2, 5, 3, 2)])
def test_against_library_conv2d(shp):
    """torch's fp64 CPU conv2d (cross-correlation, stride (sh,sw), no padding) on permuted views."""
    img = rand(shp.image_shape, 21)
    f = rand(shp.filter_shape, 22)
    out, ab = ocnn.cnn_f64(img, f, shp)
    x = torch.from_numpy(img).permute(3, 2, 1, 0).contiguous()      # [b][c][y][x]
    wgt = torch.from_numpy(f).permute(0, 3, 2, 1).contiguous()      # [k][c][s][r]
    y = torch.nn.functional.conv2d(x, wgt, stride=(shp.sh, shp.sw))  # [b][k][h][w]
    exp = y.permute(1, 2, 3, 0).numpy()                             # [k][h][w][b]
    n = shp.C * shp.R * shp.S
    assert np.all(np.abs(out - exp) <= 4 * n * 2.0 ** -52 * ab)


def test_bf16_front_end_and_sampling_agree_with_f64_core():
    shp = Shape(4, 5, 6, 7, 5, 3, 2, 2, 1)
    cs = synth.ConvShape("t", *shp.args(), image_dist="normal", filter_dist="normal_fan", seed=99)
    ib, fb = synth.make_inputs(cs)
    # decode independently of the oracle's own decoder
    img = synth.bf16_bits_to_f32(ib).astype(np.float64)
    f = synth.bf16_bits_to_f32(fb).astype(np.float64)
    np.testing.assert_array_equal(img, ocnn.bf16_bits_to_f64(ib))
    o1, a1 = ocnn.cnn_f64(img, f, shp)
    o2, a2 = ocnn.cnn_bf16(ib, fb, shp)
    np.testing.assert_array_equal(o1, o2)
    np.testing.assert_array_equal(a1, a2)
    idx = np.array(list(itertools.product(range(shp.K), range(shp.H), range(shp.W), range(shp.B))),
                   dtype=np.int32)
    o3, a3 = ocnn.cnn_bf16_at(ib, fb, idx, shp)
    n = shp.C * shp.R * shp.S
    assert np.all(np.abs(o3 - o1.reshape(-1)) <= n * 2.0 ** -52 * a1.reshape(-1))
    assert np.all(np.abs(a3 - a1.reshape(-1)) <= n * 2.0 ** -52 * a1.reshape(-1))


def test_bf16_rounding_is_nearest_even():
    # 1 + 2^-8 is a tie between 1.0 and 1+2^-7 -> even mantissa (1.0); 1+3*2^-8 ties up to 1+2^-6
    x = np.array([1.0, 1.0 + 2.0 ** -8, 1.0 + 2.0 ** -7, 1.0 + 3 * 2.0 ** -8, -0.3, 3.0e-5],
                 dtype=np.float32)
    bits = synth.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, ref)
    big = np.random.default_rng(0).standard_normal(100000).astype(np.float32)
    np.testing.assert_array_equal(
        synth.f32_to_bf16_bits(big),
        torch.from_numpy(big).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16))


def test_config_shapes_match_the_benchmark_statement():
    exp = {
        "cfg1_tiny_3x3": ((16, 16, 8, 2), (16, 3, 3, 8)),
        "cfg2_resnet_3x3": ((16, 16, 256, 32), (256, 3, 3, 256)),
        "cfg3_stem_7x7_s2": ((229, 229, 3, 64), (64, 7, 7, 3)),
        "cfg4_pointwise_1x1": ((14, 14, 1024, 64), (256, 1, 1, 1024)),
        "cfg5_large_3x3": ((30, 30, 512, 128), (512, 3, 3, 512)),
    }
    for c in synth.CONFIGS:
        assert (c.image_shape, c.filter_shape) == exp[c.name]
