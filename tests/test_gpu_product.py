"""GPU parity: block-sparse GEMM and convolution against the CPU oracle, through the C ABI.

Integer paths must match bit for bit.  Float paths: the stated bound is a max relative error of 1e-2
(bf16 inputs, fp32 accumulation), read as max|y - y_ref| / max|y_ref|; the tests also hold the kernels to
the much tighter figure the arithmetic should deliver (see gpu_util.TIGHT)."""
import numpy as np
import pytest

from oracle import ref
from paper_2407_09453_b200 import bsp, synth
from gpu_util import (TIGHT, TOL, gpu_conv, gpu_gemm, gpu_layer, gpu_mask, make_bias, make_case, make_x,
                      rel_err, from_dev)

pytestmark = pytest.mark.gpu


SHAPES = [(8, 8), (4, 16), (16, 4)]


def check(got, want, dtype, out="f32"):
    if dtype == "i8":
        assert got.dtype == np.int32 and np.array_equal(got, want)
        return
    e = rel_err(got, want)
    assert e <= TOL
    if dtype == "f32":                  # TF32 operands; a bf16 output adds its own rounding on top
        tight = TIGHT["tf32"] + (TIGHT["bf16out"] if out == "bf16" else 0.0)
    else:
        tight = TIGHT["bf16out"] if out == "bf16" else TIGHT["f32out"]
    assert e <= tight, e


def run_conv_case(seed, O, I, H, K, bo, bi, dtype, xshape, stride, pad, frac=0.5, out="f32", bias=True):
    W = make_case(seed, O, I, H, K, dtype)
    NBo, NBi = O // bo, I // bi
    gamma = synth.random_gamma(seed + 1, NBo, NBi, int(round(frac * NBo * NBi)))
    X = make_x(seed + 2, xshape, dtype)
    b = make_bias(seed + 3, O, dtype) if bias else None
    lay = gpu_layer(W, gamma, bo, bi, dtype)
    got = gpu_conv(lay, X, b, dtype, stride, pad, out)
    rp, ci, pl = ref.compact(W, gamma, bo, bi)
    want = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, stride, pad)
    check(got, want, dtype, out)
    return got, want


def test_config_fc_64x64_fp32_random_gamma():
    """Single FC layer: O = I = 64, X 64 x 128 (stored [128][64]), fp32, 8x8, exactly 32 of 64 blocks zeroed."""
    O = I = 64
    W = synth.normal(synth.tensor_seed(1, 0, synth.TENSOR_W), (O, 1, 1, I)).astype(np.float32)
    X = synth.normal(synth.tensor_seed(1, 0, synth.TENSOR_X), (128, I)).astype(np.float32)
    b = synth.normal(synth.tensor_seed(1, 0, synth.TENSOR_BIAS), (O,), 0.1).astype(np.float32)
    gamma = synth.random_gamma(synth.tensor_seed(1, 0, synth.TENSOR_GAMMA), 8, 8, 32)
    lay = gpu_layer(W, gamma, 8, 8, "f32")
    got = gpu_gemm(lay, X, b, "f32")
    rp, ci, pl = ref.compact(W, gamma, 8, 8)
    want = ref.gemm(O, I, 8, 8, rp, ci, pl.reshape(-1, 8, 8), X, b)
    check(got, want, "f32")


@pytest.mark.parametrize("dtype", ["bf16", "i8", "f32"])
@pytest.mark.parametrize("bo,bi", SHAPES)
def test_gemm_shapes_and_ragged_pixel_tail(dtype, bo, bi):
    O, I, P = 192, 256, 333                     # 3 panels, ragged last pixel tile
    W = make_case(201, O, I, 1, 1, dtype)
    gamma = synth.random_gamma(202, O // bo, I // bi, (O // bo) * (I // bi) // 2)
    X = make_x(203, (P, I), dtype)
    b = make_bias(204, O, dtype)
    lay = gpu_layer(W, gamma, bo, bi, dtype)
    got = gpu_gemm(lay, X, b, dtype)
    rp, ci, pl = ref.compact(W, gamma, bo, bi)
    want = ref.gemm(O, I, bo, bi, rp, ci, pl.reshape(-1, bo, bi), X, b)
    check(got, want, dtype)


CONV_CASES = [  # H, K, stride, pad, spatial
    (3, 3, (1, 1), (1, 1), (14, 14)), (1, 1, (1, 1), (0, 0), (9, 7)), (3, 3, (2, 2), (1, 1), (15, 15)),
    (1, 1, (2, 2), (0, 0), (14, 14)), (1, 7, (1, 1), (0, 3), (17, 17)), (7, 1, (1, 1), (3, 0), (17, 17)),
    (3, 3, (2, 2), (0, 0), (17, 17)), (5, 5, (1, 2), (2, 1), (11, 13)),
]


@pytest.mark.parametrize("dtype", ["bf16", "i8", "f32"])
@pytest.mark.parametrize("H,K,stride,pad,sp", CONV_CASES)
def test_conv_taps_strides_padding(dtype, H, K, stride, pad, sp):
    run_conv_case(301 + H * 7 + K, 64, 64, H, K, 8, 8, dtype, (3, sp[0], sp[1], 64), stride, pad)


@pytest.mark.parametrize("dtype", ["bf16", "i8"])
def test_gemm_packed_form_of_the_multi_launch_compaction(dtype):
    """8192 blocks: the packed form comes from the count / scan / fill launches, not the one-launch kernel."""
    O, I, P = 512, 1024, 200
    W = make_case(451, O, I, 1, 1, dtype)
    gamma = synth.random_gamma(452, O // 8, I // 8, (O // 8) * (I // 8) // 2)
    X = make_x(453, (P, I), dtype)
    b = make_bias(454, O, dtype)
    lay = gpu_layer(W, gamma, 8, 8, dtype)
    got = gpu_gemm(lay, X, b, dtype)
    rp, ci, pl = ref.compact(W, gamma, 8, 8)
    check(got, ref.gemm(O, I, 8, 8, rp, ci, pl.reshape(-1, 8, 8), X, b), dtype)


@pytest.mark.parametrize("dtype", ["bf16", "i8"])
@pytest.mark.parametrize("bo,bi", [(4, 16), (16, 4)])
def test_conv_other_block_shapes(dtype, bo, bi):
    run_conv_case(401, 96, 80, 3, 3, bo, bi, dtype, (2, 10, 12, 80), (1, 1), (1, 1))


@pytest.mark.parametrize("dtype", ["bf16", "i8"])
def test_conv_channel_counts_off_the_panel_grid(dtype):
    """O = 48 (Inception-like, not a multiple of 64), I = 24, wide image forcing several column tiles."""
    I = 32 if dtype == "i8" else 24                  # int8 rows of X must be multiples of 16 bytes
    run_conv_case(411, 48, I, 3, 3, 8, 8, dtype, (1, 6, 150, I), (1, 1), (1, 1))
    run_conv_case(413, 1000, 64, 1, 1, 8, 8, dtype, (2, 3, 5, 64), (1, 1), (0, 0))


@pytest.mark.parametrize("frac", [0.0, 0.25, 0.75, 1.0])
def test_conv_sparsity_extremes(frac):
    got, want = run_conv_case(421, 128, 128, 3, 3, 8, 8, "i8", (2, 8, 8, 128), (1, 1), (1, 1), frac)
    if frac == 1.0:                              # Gamma == 0: the bias broadcast
        assert np.array_equal(got, np.tile(got[0], (got.shape[0], 1)))


def test_conv_bf16_output_and_no_bias():
    run_conv_case(431, 128, 64, 3, 3, 8, 8, "bf16", (2, 9, 9, 64), (1, 1), (1, 1), out="bf16")
    run_conv_case(433, 64, 64, 1, 1, 8, 8, "bf16", (2, 9, 9, 64), (1, 1), (0, 0), bias=False)


def test_conv_1x1_equals_gemm_bitwise():
    O, I = 128, 192
    W = make_case(441, O, I, 1, 1, "bf16")
    gamma = synth.random_gamma(442, 16, 24, 192)
    X = make_x(443, (4, 8, 8, I), "bf16")
    b = make_bias(444, O, "bf16")
    lay = gpu_layer(W, gamma, 8, 8, "bf16")
    yc = gpu_conv(lay, X, b, "bf16")
    yg = gpu_gemm(lay, X.reshape(-1, I), b, "bf16")
    assert np.array_equal(yc, yg)


def test_config_resnet_conv_3x3_256_bf16_with_l2_gamma():
    """ResNet50-style 3x3 conv: batch 32, 14x14, I = O = 256, stride 1, pad 1, bf16, He-init weights,
    Gamma at 8x8 from the lowest block L2 norms to 50 % (mask -> compact -> conv, all on the GPU)."""
    layer = synth.Layer("cfg2", 256, 256, 3, 3, 32, 14, 14, 1, 1, 1, 1)
    W, X, b = synth.make_layer_tensors(layer, "bf16", config=2)
    g, s, lay, Wd = gpu_mask(W, 8, 8, "bf16", 512)
    want_s = ref.scores(W, 8, 8)
    want_g = ref.mask(want_s, 512)
    assert np.array_equal(s.view(np.uint64), want_s.view(np.uint64)) and np.array_equal(g, want_g)
    lay.compact(Wd)
    lay.check()
    for out in ("f32", "bf16"):
        got = gpu_conv(lay, X, b, "bf16", (1, 1), (1, 1), out)
        rp, ci, pl = ref.compact(W, want_g, 8, 8)
        want = ref.conv2d(W.shape, 8, 8, rp, ci, pl, X, b, (1, 1), (1, 1))
        check(got, want, "bf16", out)


def test_large_int8_vgg_like_layer_sampled_pixels():
    """VGG16-shaped 3x3 int8 layer 128 -> 128 at 112x112, batch 2, 75 % sparsity; sampled pixels, bit exact."""
    layer = synth.Layer("vgg", 128, 128, 3, 3, 2, 112, 112, 1, 1, 1, 1)
    W, X, b = synth.make_layer_tensors(layer, "i8", config=5)
    g, s, lay, Wd = gpu_mask(W, 8, 8, "i8", 192)
    want_g = ref.mask(ref.scores(W, 8, 8), 192)
    assert np.array_equal(g, want_g)
    lay.compact(Wd)
    got = gpu_conv(lay, X, b, "i8", (1, 1), (1, 1))
    P = 2 * 112 * 112
    pix = np.r_[0, 111, 112, P - 1, synth.uniform_int(9, (600,), 0, P - 1)]
    rp, ci, pl = ref.compact(W, want_g, 8, 8)
    want = ref.conv2d(W.shape, 8, 8, rp, ci, pl, X, b, (1, 1), (1, 1), pix=pix)
    assert np.array_equal(got[pix], want)
