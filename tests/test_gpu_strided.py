"""cconv_forward_strided: Eq. 1 on arrays with explicit element strides per subscript.  Section 2 of
the paper defines Image(x, y, c, b), Filter(k, r, s, c) and Out(k, h, w, b) by their subscripts only;
the same values stored row-major (last subscript fastest, the ABI's own layout), column-major (first
subscript fastest) and as windows of larger arrays must give the same result, checked against the
fp64 CPU oracle.  Tolerance: 2e-3 * sum|Image*Filter| per element."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import cnn as ocnn
from paper_1802_06905_b200 import binding, synth
from paper_1802_06905_b200.synth import ConvShape

from gpu_util import assert_close, oshape, to_dev

pytestmark = pytest.mark.gpu


def column_major_like(t):
    """A tensor with the values and shape of `t` whose FIRST subscript is the fastest in memory."""
    rev = torch.empty(tuple(reversed(t.shape)), dtype=t.dtype, device=t.device)
    cm = rev.permute(*reversed(range(t.dim())))
    cm.copy_(t)
    assert cm.stride()[0] == 1 or t.shape[0] == 1
    return cm


SHAPES = [ConvShape("s_3x3", 16, 24, 40, 6, 5, 3, 3, seed=31),
          ConvShape("s_strides", 8, 5, 9, 5, 4, 3, 2, 2, 1, seed=32),
          ConvShape("s_1x1", 64, 32, 16, 4, 3, 1, 1, seed=33)]


@pytest.mark.parametrize("out_dtype", [binding.OUT_F32, binding.OUT_BF16], ids=["f32out", "bf16out"])
@pytest.mark.parametrize("c", SHAPES, ids=lambda c: c.name)
def test_row_major_and_column_major_storage_agree_with_the_oracle(c, out_dtype):
    ib, fb = synth.make_inputs(c)
    exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
    img, flt = to_dev(ib), to_dev(fb)
    odt = torch.float32 if out_dtype == binding.OUT_F32 else torch.bfloat16
    results = {}
    for layout in ("row_major", "column_major", "mixed"):
        out = torch.full(c.out_shape, float("nan"), dtype=odt, device="cuda")
        i2, f2, o2 = img, flt, out
        if layout == "column_major":
            i2, f2, o2 = column_major_like(img), column_major_like(flt), column_major_like(out)
        if layout == "mixed":       # row-major inputs, column-major Out
            o2 = column_major_like(out)
        binding.conv_forward_strided(i2, f2, o2, *c.dims(), out_dtype=out_dtype)
        torch.cuda.synchronize()
        got = o2.float().cpu().numpy().astype(np.float64)
        assert_close(got, exp, ab, what=f"{c.name} {layout}", bf16_out=out_dtype == binding.OUT_BF16)
        results[layout] = got
    # the two CUDA-core runs add the same terms in the same order
    assert np.array_equal(results["column_major"], results["mixed"])


def test_a_window_of_a_larger_image_runs_through_a_strided_tensor_map(monkeypatch):
    """Image = a window of a larger array (x, y and c strides of the parent, images contiguous),
    Filter and Out dense: the tensor-core kernels read it through a tensor map built from the strides.
    The same window copied to a dense array must give bit-identical results on that path (with one
    kernel per plan: a repeated call on the same buffers would otherwise take the plan's second,
    halo-kernel tiling, which sums in another order)."""
    monkeypatch.setenv("CCONV_WAIT_TWIN", "0")
    for c in (ConvShape("win_3x3", 32, 64, 128, 14, 14, 3, 3, seed=41),       # one wave: direct kernel
              ConvShape("win_big", 64, 32, 128, 40, 36, 3, 3, seed=42),      # several waves: halo kernel
              ConvShape("win_1x1_s2", 64, 64, 128, 7, 7, 1, 1, 2, 2, seed=43)):
        ib, fb = synth.make_inputs(c)
        exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
        Wi, Hi = c.image_shape[:2]
        big = torch.randn((Wi + 3, Hi + 2, c.C + 16, c.B), device="cuda").to(torch.bfloat16)
        win = big[2:2 + Wi, 1:1 + Hi, 8:8 + c.C, :]
        win.copy_(to_dev(ib))
        assert not win.is_contiguous() and win.stride(3) == 1
        flt = to_dev(fb)
        out = torch.full(c.out_shape, float("nan"), dtype=torch.float32, device="cuda")
        for rep in range(2):                       # the second call finds the cached plan
            out.fill_(float("nan"))
            binding.conv_forward_strided(win, flt, out, *c.dims(), out_dtype=binding.OUT_F32)
            torch.cuda.synchronize()
            assert_close(out.cpu().numpy().astype(np.float64), exp, ab, what=f"{c.name} window, call {rep}")
        dense = torch.full(c.out_shape, float("nan"), dtype=torch.float32, device="cuda")
        binding.conv_forward(win.contiguous(), flt, dense, *c.dims(), out_dtype=binding.OUT_F32)
        torch.cuda.synchronize()
        assert torch.equal(out, dense), c.name


def test_images_that_are_not_contiguous_take_the_cuda_core_kernel():
    c = ConvShape("s_b_stride2", 8, 16, 24, 5, 4, 3, 3, seed=51)
    ib, fb = synth.make_inputs(c)
    exp, ab = ocnn.cnn_bf16(ib, fb, oshape(c))
    big = torch.zeros(c.image_shape[:3] + (2 * c.B,), dtype=torch.bfloat16, device="cuda")
    img = big[..., ::2]                                   # every other image of the parent
    img.copy_(to_dev(ib))
    out = torch.full(c.out_shape, float("nan"), dtype=torch.float32, device="cuda")
    binding.conv_forward_strided(img, to_dev(fb), out, *c.dims(), out_dtype=binding.OUT_F32)
    torch.cuda.synchronize()
    assert_close(out.cpu().numpy().astype(np.float64), exp, ab, what=c.name)


def test_strided_entry_rejects_bad_arguments():
    lib = binding.load_library()
    buf = torch.zeros(1 << 16, dtype=torch.bfloat16, device="cuda")
    p = ctypes.c_void_p(buf.data_ptr())
    ok = (ctypes.c_int64 * 4)(512, 64, 8, 1)
    zero = (ctypes.c_int64 * 4)(512, 64, 0, 1)
    neg = (ctypes.c_int64 * 4)(512, -64, 8, 1)
    dims = (8, 8, 8, 4, 4, 3, 3, 1, 1)
    assert lib.cconv_forward_strided(p, zero, p, ok, p, ok, *dims, 0, None) == binding.EINVAL
    assert lib.cconv_forward_strided(p, ok, p, neg, p, ok, *dims, 0, None) == binding.EINVAL
    assert lib.cconv_forward_strided(None, ok, p, ok, p, ok, *dims, 0, None) == binding.EINVAL
    assert lib.cconv_forward_strided(p, ok, p, ok, p, None, *dims, 0, None) == binding.EINVAL
    assert lib.cconv_forward_strided(p, ok, p, ok, p, ok, 0, 8, 8, 4, 4, 3, 3, 1, 1, 0, None) == binding.EINVAL
    assert lib.cconv_forward_strided(p, ok, p, ok, p, ok, *dims, 7, None) == binding.EINVAL
    torch.cuda.synchronize()
