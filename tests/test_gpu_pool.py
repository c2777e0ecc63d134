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


def _max_pool_exact(bits, shp):
    exp, _ = opool.pool_bf16(bits, shp, opool.MAX)
    return exp, synth.f32_to_bf16_bits(exp.astype(np.float32))   # a maximum of bf16 values is one of them


def test_pooling_calls_that_overlap_on_the_gpu_keep_stream_order():
    """Pooling calls start before the call in front of them has ended.  Three calls that depend on
    one another, forty times over with no synchronisation: call 2 reads call 1's Out as its Image
    (read after write), call 3 writes into the buffer call 2 still reads (write after read) and
    call 1 of the next round writes over call 3's Out (write after write).  Maxima are exact, so
    every buffer must end up bit-identical to the oracle run in order."""
    s1 = Shape(B=64, C=16, K=24, W=27, H=27, R=3, S=3, sw=2, sh=2)    # Out (24, 27, 27, 64)
    s2 = Shape(B=64, C=27, K=8, W=11, H=13, R=4, S=3, sw=2, sh=2)     # Image (24, 27, 27, 64)
    s3 = Shape(B=64, C=11, K=50, W=3, H=6, R=2, S=3, sw=3, sh=2)      # Image (8, 13, 11, 64) = call 2's Out
    assert s1.out_shape == s2.image_shape and s2.out_shape == s3.image_shape
    rng = np.random.default_rng(0x5EC6)
    xbits = synth.f32_to_bf16_bits(rng.standard_normal(s1.image_shape).astype(np.float32))
    x = to_dev(xbits)
    y = torch.zeros(s1.out_shape, dtype=torch.bfloat16, device="cuda")
    z = torch.zeros(s2.out_shape, dtype=torch.bfloat16, device="cuda")
    n3 = int(np.prod(s3.out_shape))
    y_head = y.view(-1)[:n3].view(s3.out_shape)                        # call 3's Out: the start of y
    for _ in range(40):
        binding.pool_forward(x, y, *s1.args(), op=binding.POOL_MAX)
        binding.pool_forward(y, z, *s2.args(), op=binding.POOL_MAX)
        binding.pool_forward(z, y_head, *s3.args(), op=binding.POOL_MAX)
    torch.cuda.synchronize()
    e1, b1 = _max_pool_exact(xbits, s1)
    e2, b2 = _max_pool_exact(b1, s2)
    e3, _ = _max_pool_exact(b2, s3)
    np.testing.assert_array_equal(ocnn.bf16_bits_to_f64(to_bits(z)), e2)
    got_y = ocnn.bf16_bits_to_f64(to_bits(y)).reshape(-1)
    np.testing.assert_array_equal(got_y[:n3], e3.reshape(-1))
    np.testing.assert_array_equal(got_y[n3:], e1.reshape(-1)[n3:])


def test_pooling_reads_the_out_of_a_convolution_that_may_still_run():
    """Convolution (tensor-core kernel, overlapping its neighbours) -> pooling of its Out -> a
    convolution that overwrites that Out, on one stream without synchronisation."""
    from paper_1802_06905_b200.synth import ConvShape
    c = ConvShape("conv_then_pool", 64, 64, 128, 14, 14, 3, 3, 1, 1, seed=77)   # Out (128, 14, 14, 64)
    ps = Shape(B=64, C=14, K=6, W=42, H=6, R=5, S=4, sw=3, sh=2)                # Image (128, 14, 14, 64)
    assert c.out_shape == ps.image_shape
    ib, fb = synth.make_inputs(c)
    img, flt = to_dev(ib), to_dev(fb)
    flt2 = to_dev(synth.make_inputs(ConvShape("conv_then_pool_2", *c.dims(), seed=78))[1])
    plan = binding.Plan(*c.dims(), device=0, out_dtype=binding.OUT_BF16)
    mid = torch.empty(c.out_shape, dtype=torch.bfloat16, device="cuda")
    pooled = torch.empty(ps.out_shape, dtype=torch.bfloat16, device="cuda")
    for rep in range(8):
        mid.fill_(3.0e30)                                          # a stale read would win every maximum
        plan.forward(img, flt, mid)
        binding.pool_forward(mid, pooled, *ps.args(), op=binding.POOL_MAX)
        keep = pooled.clone()                                      # (an ordinary kernel of another library)
        plan.forward(img, flt2, mid)                               # write after read
        plan.check()
        got_first = ocnn.bf16_bits_to_f64(to_bits(keep))
        assert float(np.abs(got_first).max()) < 1.0e6, f"repeat {rep}: pooling read Out before it was written"
    # the pooled values are maxima of the first convolution's Out; recompute them from what the
    # same plan writes for (img, flt)
    plan.forward(img, flt, mid)
    plan.check()
    exp, _ = opool.pool_bf16(to_bits(mid), ps, opool.MAX)
    np.testing.assert_array_equal(ocnn.bf16_bits_to_f64(to_bits(keep)), exp)
    plan.close()
