"""GPU parity of the product kernel over layer shapes (taps, strides, padding, channel counts off the tile grid, tiles
that span images, long position counts) against the CPU oracle: within tolerance for bf16, bit for bit for int8."""
import numpy as np
import pytest

from oracle import ref
import torch

from paper_2407_09453_b200 import bsp, synth
from gpu_util import gpu_conv, gpu_gemm, gpu_layer, gpu_mask, make_bias, make_case, make_x
from test_gpu_product import check, run_conv_case

pytestmark = pytest.mark.gpu


TC_CASES = [  # O, I, H, K, pad, spatial, batch
    (256, 256, 3, 3, (1, 1), (14, 14), 3), (64, 64, 1, 1, (0, 0), (9, 7), 3), (128, 64, 5, 5, (2, 2), (11, 13), 2),
    (64, 64, 1, 7, (0, 3), (17, 17), 2), (64, 64, 7, 1, (3, 0), (17, 17), 2), (64, 32, 3, 3, (0, 0), (12, 12), 2),
    (48, 24, 3, 3, (1, 1), (6, 150), 1), (1000, 64, 1, 1, (0, 0), (3, 5), 2), (136, 128, 3, 3, (1, 1), (28, 28), 2),
]


@pytest.mark.parametrize("O,I,H,K,pad,sp,batch", TC_CASES)
def test_tc_conv_shapes(O, I, H, K, pad, sp, batch):
    run_conv_case(601 + O + H, O, I, H, K, 8, 8, "bf16", (batch, sp[0], sp[1], I), (1, 1), pad)


STRIDED = [  # O, I, H, K, stride, pad, spatial, batch
    (128, 64, 3, 3, (2, 2), (1, 1), (15, 15), 3), (64, 64, 1, 1, (2, 2), (0, 0), (14, 14), 3),
    (64, 32, 3, 3, (2, 2), (0, 0), (17, 17), 2), (64, 64, 3, 3, (2, 1), (1, 1), (28, 9), 2),
    (256, 128, 3, 3, (2, 2), (1, 1), (56, 56), 1), (64, 32, 5, 5, (2, 2), (2, 2), (30, 30), 1),
    (64, 32, 7, 7, (2, 2), (3, 3), (30, 30), 1), (72, 48, 5, 5, (1, 2), (2, 1), (11, 13), 2),
    (64, 32, 3, 3, (3, 3), (1, 1), (200, 9), 1),       # a tall image at stride 3: the box height is capped by the tensor map's 256-element extent
]


@pytest.mark.parametrize("dtype", ["bf16", "i8", "f32"])
@pytest.mark.parametrize("O,I,H,K,stride,pad,sp,batch", STRIDED)
def test_tc_strided(dtype, O, I, H, K, stride, pad, sp, batch):
    run_conv_case(671 + O + H, O, I, H, K, 8, 8, dtype, (batch, sp[0], sp[1], I), stride, pad)


I8_CASES = [  # O, I, H, K, pad, spatial, batch: I a multiple of 16 (conv) or 32 (1x1) so that the kernel applies
    (128, 128, 3, 3, (1, 1), (14, 14), 3), (64, 64, 1, 1, (0, 0), (9, 7), 3), (72, 48, 5, 5, (2, 2), (11, 13), 2),
    (64, 32, 1, 7, (0, 3), (17, 17), 2), (1000, 64, 1, 1, (0, 0), (3, 5), 2), (136, 16, 3, 3, (1, 1), (28, 28), 2),
]


@pytest.mark.parametrize("O,I,H,K,pad,sp,batch", I8_CASES)
@pytest.mark.parametrize("bo,bi", [(8, 8), (4, 16), (16, 4)])
def test_tc_int8_bit_exact(O, I, H, K, pad, sp, batch, bo, bi):
    if O % bo or I % bi:
        pytest.skip("channels are not a multiple of the block")
    run_conv_case(641 + O + H, O, I, H, K, bo, bi, "i8", (batch, sp[0], sp[1], I), (1, 1), pad)


@pytest.mark.parametrize("frac", [0.0, 0.75, 1.0])
def test_tc_int8_sparsity_extremes(frac):
    run_conv_case(651, 128, 128, 3, 3, 8, 8, "i8", (2, 8, 8, 128), (1, 1), (1, 1), frac)


@pytest.mark.parametrize("bo,bi", [(4, 16), (16, 4)])
def test_tc_other_block_shapes(bo, bi):
    run_conv_case(611, 96, 80, 3, 3, bo, bi, "bf16", (2, 10, 12, 80), (1, 1), (1, 1))


@pytest.mark.parametrize("frac", [0.0, 0.25, 0.75, 1.0])
def test_tc_sparsity_extremes_and_bf16_output(frac):
    run_conv_case(621, 128, 128, 3, 3, 8, 8, "bf16", (2, 8, 8, 128), (1, 1), (1, 1), frac, out="bf16")


@pytest.mark.parametrize("bo,bi", [(8, 8), (4, 16), (16, 4)])
def test_tc_gemm_ragged(bo, bi):
    O, I, P = 192, 256, 333
    W = make_case(631, O, I, 1, 1, "bf16")
    gamma = synth.random_gamma(632, O // bo, I // bi, (O // bo) * (I // bi) // 2)
    X = make_x(633, (P, I), "bf16")
    b = make_bias(634, O, "bf16")
    lay = gpu_layer(W, gamma, bo, bi, "bf16")
    got = gpu_gemm(lay, X, b, "bf16")
    rp, ci, pl = ref.compact(W, gamma, bo, bi)
    want = ref.gemm(O, I, bo, bi, rp, ci, pl.reshape(-1, bo, bi), X, b)
    check(got, want, "bf16")


@pytest.mark.parametrize("dtype", ["bf16", "i8"])
def test_tc_gemm_two_position_tiles_per_cta(dtype):
    """Enough CTAs that a matrix product takes 256 positions per CTA (two accumulator halves); ragged last tile."""
    O, I, P = 1024, 64, 9500
    W = make_case(661, O, I, 1, 1, dtype)
    gamma = synth.random_gamma(662, O // 8, I // 8, (O // 8) * (I // 8) // 2)
    X = make_x(663, (P, I), dtype)
    b = make_bias(664, O, dtype)
    lay = gpu_layer(W, gamma, 8, 8, dtype)
    got = gpu_gemm(lay, X, b, dtype)
    rp, ci, pl = ref.compact(W, gamma, 8, 8)
    check(got, ref.gemm(O, I, 8, 8, rp, ci, pl.reshape(-1, 8, 8), X, b), dtype)


@pytest.mark.parametrize("dtype,frac", [("bf16", 0.5), ("i8", 0.75), ("bf16", 0.0)])
def test_tc_gemm_two_channel_groups_per_cta(dtype, frac):
    """Five channel tiles of 256 with 120 channels in the last, 297 position tiles with a ragged tail: every persistent CTA
    takes ten tiles."""
    O, I, P = 1144, 96, 38000
    W = make_case(681, O, I, 1, 1, dtype)
    NB = (O // 8) * (I // 8)
    gamma = synth.random_gamma(682, O // 8, I // 8, int(NB * frac))
    X = make_x(683, (P, I), dtype)
    b = make_bias(684, O, dtype)
    lay = gpu_layer(W, gamma, 8, 8, dtype)
    got = gpu_gemm(lay, X, b, dtype)
    rp, ci, pl = ref.compact(W, gamma, 8, 8)
    check(got, ref.gemm(O, I, 8, 8, rp, ci, pl.reshape(-1, 8, 8), X, b), dtype)
