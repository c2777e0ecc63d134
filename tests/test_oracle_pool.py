"""Pins for the CPU oracle of the pooling nest (Section 6).  No GPU, no CUDA path.

Every check compares the oracle with something it does not compute itself: a library pooling
routine on permuted tensors, the (separately pinned) convolution oracle with a constant filter,
closed forms for constant and delta images, and a pure-Python per-element evaluation.
"""
import itertools

import numpy as np
import pytest
import torch

from oracle import bounds as ob
from oracle import cnn as ocnn
from oracle import pool as opool
from oracle.cnn import Shape
from paper_1802_06905_b200 import synth

ASYM = Shape(B=3, C=2, K=4, W=5, H=3, R=3, S=2, sw=2, sh=1)   # every extent differs
ASYM2 = Shape(B=2, C=3, K=2, W=3, H=4, R=2, S=3, sw=1, sh=3)  # sh > S-1: rows that no window reads
ONE_CH = Shape(B=4, C=1, K=1, W=6, H=5, R=3, S=3, sw=2, sh=2)  # the usual per-channel layer


def rand_bits(shape, seed):
    x = np.random.default_rng(seed).standard_normal(shape).astype(np.float32)
    return synth.f32_to_bf16_bits(x)


def values(bits):
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def library_pool(img, shp, op):
    """Per-channel pooling by the library on input[b][c][y][x] = Image[x][y][c][b]: (B,C,H,W)."""
    t = torch.from_numpy(img).permute(3, 2, 1, 0).contiguous()
    fn = torch.nn.functional.avg_pool2d if op == opool.AVG else torch.nn.functional.max_pool2d
    return fn(t, kernel_size=(shp.S, shp.R), stride=(shp.sh, shp.sw)).numpy()


@pytest.mark.parametrize("op", [opool.AVG, opool.MAX])
@pytest.mark.parametrize("shp", [ONE_CH, ASYM, ASYM2])
def test_against_library_pooling_reduced_over_channels(shp, op):
    bits = rand_bits(shp.image_shape, 11)
    out, ab = opool.pool_bf16(bits, shp, op)
    per_channel = library_pool(values(bits), shp, op)            # (B, C, H, W)
    red = per_channel.sum(axis=1) if op == opool.AVG else per_channel.max(axis=1)  # (B, H, W)
    exp = np.transpose(red, (1, 2, 0))                           # (H, W, B)
    for k in range(shp.K):
        if op == opool.AVG:
            np.testing.assert_allclose(out[k], exp, rtol=0, atol=1e-13 * shp.C * shp.R * shp.S)
        else:
            np.testing.assert_array_equal(out[k], exp)
    if op == opool.AVG:
        ab_exp = np.transpose(library_pool(np.abs(values(bits)), shp, op).sum(axis=1), (1, 2, 0))
        np.testing.assert_allclose(ab[0], ab_exp, rtol=0, atol=1e-13 * shp.C * shp.R * shp.S)


@pytest.mark.parametrize("shp", [ASYM, ASYM2])
def test_average_is_the_convolution_with_a_constant_filter(shp):
    bits = rand_bits(shp.image_shape, 12)
    out, _ = opool.pool_bf16(bits, shp, opool.AVG)
    filt = np.full(shp.filter_shape, 1.0 / (shp.R * shp.S))
    conv, _ = ocnn.cnn_f64(values(bits), filt, shp)
    np.testing.assert_allclose(out, conv, rtol=0, atol=1e-13 * shp.C * shp.R * shp.S)


@pytest.mark.parametrize("op", [opool.AVG, opool.MAX])
def test_constant_image_closed_form(op):
    shp = ASYM
    bits = synth.f32_to_bf16_bits(np.full(shp.image_shape, -0.75, dtype=np.float32))
    out, ab = opool.pool_bf16(bits, shp, op)
    if op == opool.AVG:
        # R*S terms of -0.75/(R*S) per channel: C * (-0.75) up to fp64 rounding of the division
        np.testing.assert_allclose(out, shp.C * -0.75, rtol=1e-14)
        np.testing.assert_allclose(ab, shp.C * 0.75, rtol=1e-14)
    else:
        np.testing.assert_array_equal(out, -0.75)   # a wrong start value (0) would show here


@pytest.mark.parametrize("shp", [ASYM, ASYM2])
def test_delta_image_marks_the_windows_that_hold_it(shp):
    for (x0, y0, c0, b0) in [(2, 1, 1, 1), (0, 0, 0, 0), (shp.Wi - 1, shp.Hi - 1, shp.C - 1, shp.B - 1)]:
        img = np.zeros(shp.image_shape, dtype=np.float32)
        img[x0, y0, c0, b0] = 2.0
        bits = synth.f32_to_bf16_bits(img)
        avg, _ = opool.pool_bf16(bits, shp, opool.AVG)
        mx, _ = opool.pool_bf16(bits, shp, opool.MAX)
        exp = np.zeros(shp.out_shape)
        for h in range(shp.H):
            for w in range(shp.W):
                if 0 <= x0 - shp.sw * w < shp.R and 0 <= y0 - shp.sh * h < shp.S:
                    exp[:, h, w, b0] = 1.0
        np.testing.assert_allclose(avg, exp * 2.0 / (shp.R * shp.S), rtol=1e-15)
        np.testing.assert_array_equal(mx, exp * 2.0)


def brute_force(vals, shp, op):
    out = np.empty(shp.out_shape)
    for k, h, w, b in itertools.product(range(shp.K), range(shp.H), range(shp.W), range(shp.B)):
        terms = [vals[r + shp.sw * w][s + shp.sh * h][c][b]
                 for c in range(shp.C) for r in range(shp.R) for s in range(shp.S)]
        out[k, h, w, b] = sum(terms) / (shp.R * shp.S) if op == opool.AVG else max(terms)
    return out


@pytest.mark.parametrize("op", [opool.AVG, opool.MAX])
def test_brute_force_on_tiny_shapes(op):
    for dims in itertools.product([1, 2], [1, 3], [1, 2], [1, 3], [2], [1, 2], [1, 3], [1, 2], [1, 3]):
        shp = Shape(*dims)
        bits = rand_bits(shp.image_shape, 13)
        out, _ = opool.pool_bf16(bits, shp, op)
        exp = brute_force(values(bits).tolist(), shp, op)
        if op == opool.AVG:
            np.testing.assert_allclose(out, exp, rtol=0, atol=1e-13)
        else:
            np.testing.assert_array_equal(out, exp)


@pytest.mark.parametrize("op", [opool.AVG, opool.MAX])
def test_sampled_elements_equal_the_whole_array(op):
    shp = ASYM
    bits = rand_bits(shp.image_shape, 14)
    out, ab = opool.pool_bf16(bits, shp, op)
    idx = np.array(list(itertools.product(range(shp.K), range(shp.H), range(shp.W), range(shp.B))))
    got, gab = opool.pool_bf16_at(bits, idx, shp, op)
    np.testing.assert_allclose(got, out.reshape(-1), rtol=0, atol=1e-14)
    if op == opool.AVG:
        np.testing.assert_allclose(gab, ab.reshape(-1), rtol=0, atol=1e-14)


def test_pooling_bound_terms_and_the_lp_without_the_filter_constraint():
    # Section 6: the bound is max(|Out|, |Image|, F*R*S/M) and the LP of Section 5 without the
    # Filter constraint attains it.  With blocks not clipped by the loop bounds the LP's optimum is
    # G = M^2, so its cost F*R*S*M/G equals the third term.
    dims = (2, 2048, 4096, 4, 4, 3, 3, 1, 1)   # K >= M and C*R*S >= M: no block is clipped
    for M in (1024.0, 2048.0):
        t = ob.pooling_terms(*dims, M)
        assert t[0] == 2 * 4096 * 16 and t[1] == 2 * 2048 * 16
        B, C, K, W, H, R, S, _, _ = dims
        assert t[2] == pytest.approx(B * C * K * W * H * R * S / M)
        _, G, words = ob.tiling_lp(*dims, M, pooling=True)
        assert G == pytest.approx(M * M, rel=1e-6)
        assert words == pytest.approx(max(t), rel=1e-6)
        # with the Filter constraint the same LP cannot do better
        _, G_conv, _ = ob.tiling_lp(*dims, M, pooling=False)
        assert G_conv <= G * (1 + 1e-9)
