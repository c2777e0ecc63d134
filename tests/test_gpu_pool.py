"""GPU parity of the pooling kernel (Section 6) with its CPU oracle, through the C ABI.

Average: |gpu - oracle| <= 2e-3 * (1/(R*S)) * sum|Image| per element (fp32 accumulation, then for
bf16 storage the rounding clause of gpu_util.assert_close).  Max: the stored value must equal the
oracle's exactly (the maximum of bf16 values is one of them; bf16 and fp32 both hold it).
"""
import numpy as np
import pytest
import torch

from gpu_util import assert_close, to_bits, to_dev
from oracle import cnn as ocnn
from oracle import pool as opool
from oracle.cnn import Shape
from paper_1802_06905_b200 import binding, synth

pytestmark = pytest.mark.gpu

OPS = [(binding.POOL_AVG, opool.AVG), (binding.POOL_MAX, opool.MAX)]
OP_IDS = ["avg", "max"]
DTYPES = [torch.bfloat16, torch.float32]
DT_IDS = ["bf16", "f32"]

SHAPES = [
    Shape(B=64, C=16, K=24, W=9, H=7, R=3, S=3, sw=2, sh=2),     # cooperative path, ragged last block
    Shape(B=32, C=1, K=1, W=20, H=11, R=2, S=2, sw=2, sh=2),     # the usual layer: one thread per vector
    Shape(B=8, C=3, K=5, W=6, H=5, R=3, S=2, sw=1, sh=3),        # rows that no window reads (sh > S)
    Shape(B=40, C=7, K=100, W=5, H=4, R=1, S=1, sw=1, sh=1),     # no window: channel reduction only
    Shape(B=6, C=5, K=9, W=7, H=3, R=3, S=3, sw=1, sh=1),        # B % 8 != 0: scalar path
    Shape(B=3, C=40, K=70, W=4, H=4, R=2, S=3, sw=3, sh=1),      # scalar + cooperative + k split
    Shape(B=16, C=64, K=130, W=3, H=2, R=3, S=3, sw=1, sh=1),    # few pixels, many planes: k split
    Shape(B=128, C=2, K=3, W=33, H=17, R=5, S=4, sw=2, sh=3),    # several blocks of 256 vectors
    Shape(B=72, C=1, K=1, W=13, H=9, R=3, S=3, sw=2, sh=2),      # window kernel: 3x3 stride 2, ragged last block
    Shape(B=16, C=1, K=3, W=7, H=6, R=3, S=3, sw=1, sh=3),       # window kernel: overlapping columns, 3 planes
    Shape(B=8, C=1, K=2, W=5, H=40, R=2, S=2, sw=1, sh=1),       # window kernel: 2x2 stride 1
]


def run_pool(shp, bits, op, dtype, poison=True):
    img = to_dev(bits)
    out = torch.empty(shp.out_shape, dtype=dtype, device="cuda")
    if poison:
        out.fill_(float("nan"))
    binding.pool_forward(img, out, *shp.args(), op=op)
    torch.cuda.synchronize()
    if dtype == torch.float32:
        return out.cpu().numpy().astype(np.float64)
    return ocnn.bf16_bits_to_f64(to_bits(out))


@pytest.mark.parametrize("dtype", DTYPES, ids=DT_IDS)
@pytest.mark.parametrize("op", OPS, ids=OP_IDS)
@pytest.mark.parametrize("shp", SHAPES, ids=lambda s: f"B{s.B}C{s.C}K{s.K}W{s.W}H{s.H}R{s.R}S{s.S}s{s.sw}{s.sh}")
def test_pool_parity(shp, op, dtype):
    x = np.random.default_rng(0x18020690 + shp.B * 131 + shp.C).standard_normal(shp.image_shape)
    bits = synth.f32_to_bf16_bits(x.astype(np.float32))
    got = run_pool(shp, bits, op[0], dtype)
    exp, ab = opool.pool_bf16(bits, shp, op[1])
    if op[1] == opool.MAX:
        np.testing.assert_array_equal(got, exp)
    else:
        assert_close(got, exp, ab, what="avg pool", bf16_out=dtype == torch.bfloat16)


@pytest.mark.parametrize("op", OPS, ids=OP_IDS)
def test_pool_large_sampled(op):
    """A ResNet-sized layer (56x56 -> 27x27, 3x3 stride 2, 64 channels in, 256 planes out): sampled
    elements against the oracle, every k-plane equal to plane 0, and no element left unwritten."""
    shp = Shape(B=64, C=64, K=256, W=27, H=27, R=3, S=3, sw=2, sh=2)
    rng = np.random.default_rng(7)
    bits = synth.f32_to_bf16_bits(rng.standard_normal(shp.image_shape).astype(np.float32))
    img = to_dev(bits)
    out = torch.full(shp.out_shape, float("nan"), dtype=torch.bfloat16, device="cuda")
    binding.pool_forward(img, out, *shp.args(), op=op[0])
    torch.cuda.synchronize()
    assert not torch.isnan(out).any()
    assert bool((out == out[0:1]).all())
    idx = np.stack([rng.integers(0, n, 4096) for n in shp.out_shape], axis=1)
    exp, ab = opool.pool_bf16_at(bits, idx, shp, op[1])
    got = ocnn.bf16_bits_to_f64(to_bits(out))[idx[:, 0], idx[:, 1], idx[:, 2], idx[:, 3]]
    if op[1] == opool.MAX:
        np.testing.assert_array_equal(got, exp)
    else:
        assert_close(got, exp, ab, what="avg pool sampled", bf16_out=True)


def test_pool_rejects_bad_arguments():
    img = torch.zeros(3, 3, 1, 8, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(1, 1, 1, 8, dtype=torch.bfloat16, device="cuda")
    lib = binding.load_library()
    args = (8, 1, 1, 1, 1, 3, 3, 1, 1)
    assert lib.cconv_pool_forward(img.data_ptr(), out.data_ptr(), *args, 7, 0, None) == -1      # op
    assert lib.cconv_pool_forward(img.data_ptr(), out.data_ptr(), *args, 0, 5, None) == -1      # dtype
    assert lib.cconv_pool_forward(None, out.data_ptr(), *args, 0, 0, None) == -1
    assert lib.cconv_pool_forward(img.data_ptr() + 2, out.data_ptr(), *args, 0, 0, None) == -1  # alignment
    assert lib.cconv_pool_forward(img.data_ptr(), out.data_ptr(), 8, 0, 1, 1, 1, 3, 3, 1, 1, 0, 0, None) == -1
    assert lib.cconv_pool_forward(img.data_ptr(), out.data_ptr(), *args, 0, 0, None) == 0
    torch.cuda.synchronize()
