"""GPU parity of the fused pair of layers (bsp_conv2d_chain: T = bf16(act(W1 * X + b1)), Y = W2 * T + b2 with T kept on
chip) against the oracle's chain, through the C ABI.

Tolerance.  Both sides round T to bfloat16; the kernel rounds a float32 sum, the oracle a float64 one, so an entry of T
whose exact value lies within the float32 accumulation error (~1e-6 relative for sums of up to 2304 terms) of a rounding
boundary lands on the neighbouring bfloat16 value, one unit in the last place (2^-8 relative) away: measured 4-7 of
10^4 entries.  One such entry moves an output by up to 2^-8 max|T| max|w2|, about 0.013 for max|T| = 5.4 and
max|w2| = 0.6, against largest outputs of 5 to 7: up to 2.5e-3.  The outputs are held to 4e-3 of the largest output
(8e-3 when Y is bfloat16: half a unit in the last place, 2^-9, on top), and in addition the fused call must equal
bit for bit the two separate calls through a bfloat16 tensor in memory, which round T in the same way."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_09453_b200 import bsp, synth
from gpu_util import gpu_layer, make_bias, make_case, make_x, rel_err, to_dev

pytestmark = pytest.mark.gpu


def run_chain(seed, N, L, J, I, O1, O2, H, K, stride, pad, relu, out="f32", bias=True, b1=(8, 8), b2=(8, 8), frac=0.5):
    W1 = make_case(seed, O1, I, H, K, "bf16")
    W2 = make_case(seed + 1, O2, O1, 1, 1, "bf16")
    g1 = synth.random_gamma(seed + 2, O1 // b1[0], I // b1[1], int(frac * (O1 // b1[0]) * (I // b1[1])))
    g2 = synth.random_gamma(seed + 3, O2 // b2[0], O1 // b2[1], int(frac * (O2 // b2[0]) * (O1 // b2[1])))
    X = make_x(seed + 4, (N, L, J, I), "bf16")
    bias1 = make_bias(seed + 5, O1, "bf16") if bias else None
    bias2 = make_bias(seed + 6, O2, "bf16") if bias else None
    l1, l2 = gpu_layer(W1, g1, b1[0], b1[1], "bf16"), gpu_layer(W2, g2, b2[0], b2[1], "bf16")
    M = (L + 2 * pad[0] - H) // stride[0] + 1
    Nw = (J + 2 * pad[1] - K) // stride[1] + 1
    Y = torch.full((N, M, Nw, O2), -7.0, dtype=torch.bfloat16 if out == "bf16" else torch.float32, device="cuda")
    xd = bsp.XDesc(N, L, J, stride[0], stride[1], pad[0], pad[1])
    d1 = None if bias1 is None else torch.from_numpy(bias1).cuda()
    d2 = None if bias2 is None else torch.from_numpy(bias2).cuda()
    bsp.bsp_conv2d_chain(l1.wd, l1.handle(), l2.wd, l2.handle(), xd, to_dev(X, "bf16"), d1, relu, d2, Y, bsp.dtype_code(Y.dtype), l1.ws)
    l1.check()
    got = Y.float().cpu().numpy().reshape(-1, O2)
    want = ref.chain2(W1.shape, b1[0], b1[1], ref.compact(W1, g1, *b1), X, bias1, relu, O2, b2[0], b2[1], ref.compact(W2, g2, *b2),
                      bias2, stride, pad)
    err = rel_err(got, want)
    assert err <= (8e-3 if out == "bf16" else 4e-3), err
    return got, want


@pytest.mark.parametrize("relu", [0, 1])
def test_bottleneck_tail_3x3_then_1x1(relu):
    """The tail of a ResNet bottleneck: 3x3 64 -> 64 with padding, then 1x1 64 -> 256; box tiles with a ragged edge."""
    run_chain(1001, 3, 14, 14, 64, 64, 256, 3, 3, (1, 1), (1, 1), relu)


@pytest.mark.parametrize("O1,O2", [(128, 512), (256, 64), (192, 200), (8, 8), (72, 1000)])
def test_channel_counts(O1, O2):
    """Tensors between the layers of one to four 64-channel chunks (the last one partly filled) and one to eight tiles
    of 128 output channels with a clipped last tile."""
    run_chain(1011, 2, 9, 11, 32, O1, O2, 3, 3, (1, 1), (1, 1), 1)


@pytest.mark.parametrize("H,K,stride,pad", [(1, 1, (1, 1), (0, 0)), (3, 3, (2, 2), (1, 1)), (1, 7, (1, 1), (0, 3)), (5, 5, (1, 1), (0, 0))])
def test_first_layer_taps_strides_padding(H, K, stride, pad):
    run_chain(1021, 2, 17, 17, 48, 64, 128, H, K, stride, pad, 1)


def test_tiles_that_hold_several_small_images():
    """7x7 and 4x4 images: a tile is a box of whole images (two, eight), the last one ragged in the image count."""
    run_chain(1025, 5, 7, 7, 64, 128, 256, 3, 3, (1, 1), (1, 1), 1)
    run_chain(1027, 11, 4, 4, 32, 64, 72, 1, 1, (1, 1), (0, 0), 0)
    run_chain_q8(1029, 5, 7, 7, 64, 128, 256, 3, 3, (1, 1), (1, 1), 1, True)


def test_many_tiles_per_cta_and_long_k():
    """More position tiles than SMs (every CTA takes several: both second accumulators, the tensor buffer and all stages
    are reused) and a first layer of 9 x 4 K-stages."""
    run_chain(1031, 8, 56, 56, 256, 64, 256, 3, 3, (1, 1), (1, 1), 1)


def test_bf16_output_no_bias_other_block_shapes_and_sparsity_extremes():
    run_chain(1041, 2, 12, 12, 64, 128, 256, 3, 3, (1, 1), (1, 1), 1, out="bf16")
    run_chain(1043, 2, 12, 12, 64, 128, 256, 3, 3, (1, 1), (1, 1), 0, bias=False, b1=(4, 16), b2=(16, 4))
    got, _ = run_chain(1045, 1, 10, 10, 32, 64, 128, 3, 3, (1, 1), (1, 1), 1, frac=1.0)     # both layers all zero: Y = b2
    assert np.array_equal(got, np.tile(got[0], (got.shape[0], 1)))
    run_chain(1047, 1, 10, 10, 32, 64, 128, 3, 3, (1, 1), (1, 1), 1, frac=0.0)


@pytest.mark.parametrize("relu", [0, 1])
@pytest.mark.parametrize("N,L,J,I,O1,O2", [(2, 14, 14, 64, 64, 256), (8, 56, 56, 256, 64, 256), (4, 28, 28, 128, 128, 512)])
def test_equals_the_two_separate_calls_bit_for_bit(N, L, J, I, O1, O2, relu):
    """bsp_conv2d with a bfloat16 output, max(., 0) on it, and bsp_conv2d on the result compute the same thing through
    memory, with the same accumulation order and the same rounding of T: the fused call must agree exactly (the large
    cases give every CTA several tiles, so every buffer and barrier is reused)."""
    W1, W2 = make_case(1051, O1, I, 3, 3, "bf16"), make_case(1052, O2, O1, 1, 1, "bf16")
    g1 = synth.random_gamma(1053, O1 // 8, I // 8, (O1 // 8) * (I // 8) // 2)
    g2 = synth.random_gamma(1054, O2 // 8, O1 // 8, (O2 // 8) * (O1 // 8) // 2)
    X = to_dev(make_x(1055, (N, L, J, I), "bf16"), "bf16")
    b1, b2 = torch.from_numpy(make_bias(1056, O1, "bf16")).cuda(), torch.from_numpy(make_bias(1057, O2, "bf16")).cuda()
    l1, l2 = gpu_layer(W1, g1, 8, 8, "bf16"), gpu_layer(W2, g2, 8, 8, "bf16")
    T = torch.empty((N, L, J, O1), dtype=torch.bfloat16, device="cuda")
    Ya = torch.empty((N, L, J, O2), dtype=torch.float32, device="cuda")
    Yb = torch.full_like(Ya, -7.0)
    l1.conv2d(X, b1, T, (1, 1), (1, 1))
    if relu:
        T = torch.clamp_min(T, 0)                      # exact on bfloat16 values
    l2.conv2d(T, b2, Ya)
    bsp.bsp_conv2d_chain(l1.wd, l1.handle(), l2.wd, l2.handle(), bsp.XDesc(N, L, J, 1, 1, 1, 1), X, b1, relu, b2, Yb, bsp.F32, l1.ws)
    l1.check(); l2.check()
    assert torch.equal(Ya, Yb)


def run_chain_q8(seed, N, L, J, I, O1, O2, H, K, stride, pad, relu, int8_out):
    W1 = make_case(seed, O1, I, H, K, "i8")
    W2 = make_case(seed + 1, O2, O1, 1, 1, "i8")
    g1 = synth.random_gamma(seed + 2, O1 // 8, I // 8, (O1 // 8) * (I // 8) // 2)
    g2 = synth.random_gamma(seed + 3, O2 // 8, O1 // 8, (O2 // 8) * (O1 // 8) // 2)
    X = make_x(seed + 4, (N, L, J, I), "i8")
    b1, b2 = make_bias(seed + 5, O1, "i8"), make_bias(seed + 6, O2, "i8")
    # shifts that leave tensors which use the int8 range (sums of H K I / 2 products of magnitude ~ 64^2)
    base1 = int(np.log2(np.sqrt(H * K * I / 2.0) * 5500 / 40))
    s1 = (base1 + synth.uniform_int(seed + 7, (O1,), -1, 1)).astype(np.int32)
    base2 = int(np.log2(np.sqrt(O1 / 2.0) * 64 * 40 / 40))
    s2 = (base2 + synth.uniform_int(seed + 8, (O2,), -1, 1)).astype(np.int32)
    l1, l2 = gpu_layer(W1, g1, 8, 8, "i8"), gpu_layer(W2, g2, 8, 8, "i8")
    M = (L + 2 * pad[0] - H) // stride[0] + 1
    Nw = (J + 2 * pad[1] - K) // stride[1] + 1
    Y = torch.full((N, M, Nw, O2), -7, dtype=torch.int8 if int8_out else torch.int32, device="cuda")
    xd = bsp.XDesc(N, L, J, stride[0], stride[1], pad[0], pad[1])
    dev = lambda a: torch.from_numpy(a).cuda()
    bsp.bsp_conv2d_chain_q8(l1.wd, l1.handle(), l2.wd, l2.handle(), xd, dev(X), dev(b1), dev(s1), relu, dev(b2),
                            dev(s2) if int8_out else None, Y, l1.ws)
    l1.check()
    got = Y.cpu().numpy().reshape(-1, O2)
    want = ref.chain2_q8(W1.shape, 8, 8, ref.compact(W1, g1, 8, 8), X, b1, s1, relu, O2, 8, 8, ref.compact(W2, g2, 8, 8), b2,
                         s2 if int8_out else None, stride, pad)
    assert got.dtype == want.dtype and np.array_equal(got, want)
    T8 = ref.requant_i8(ref.conv2d(W1.shape, 8, 8, *ref.compact(W1, g1, 8, 8), X, b1, stride, pad), s1)
    assert 16 < np.abs(T8).max() and (np.abs(T8) == 127).mean() < 0.2         # the tensor between the layers is neither tiny nor all saturated
    return got


@pytest.mark.parametrize("relu", [0, 1])
@pytest.mark.parametrize("int8_out", [False, True])
def test_int8_chain_bit_exact(relu, int8_out):
    run_chain_q8(1101, 3, 14, 14, 64, 64, 256, 3, 3, (1, 1), (1, 1), relu, int8_out)


@pytest.mark.parametrize("O1,O2,I", [(128, 512, 128), (256, 128, 64), (16, 16, 16), (144, 208, 48)])
def test_int8_chain_channel_counts(O1, O2, I):
    run_chain_q8(1111, 2, 9, 11, I, O1, O2, 3, 3, (1, 1), (1, 1), 1, True)


def test_int8_chain_many_tiles_strides_and_taps():
    run_chain_q8(1121, 8, 56, 56, 64, 64, 128, 3, 3, (1, 1), (1, 1), 1, False)
    run_chain_q8(1123, 2, 35, 35, 32, 96, 64, 3, 3, (2, 2), (0, 0), 0, True)
    run_chain_q8(1125, 2, 17, 17, 128, 128, 192, 1, 7, (1, 1), (0, 3), 1, True)
    run_chain_q8(1127, 4, 28, 28, 256, 64, 256, 1, 1, (1, 1), (0, 0), 1, True)


def test_argument_errors():
    l1 = bsp.SparseLayer(64, 64, 3, 3, 8, 8, torch.bfloat16)
    l3 = bsp.SparseLayer(128, 64, 3, 3, 8, 8, torch.bfloat16)          # not 1x1
    l4 = bsp.SparseLayer(128, 32, 1, 1, 8, 8, torch.bfloat16)          # wrong input channels
    X = torch.zeros((1, 8, 8, 64), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((1, 8, 8, 128), dtype=torch.float32, device="cuda")
    xd = bsp.XDesc(1, 8, 8, 1, 1, 1, 1)
    for bad in (l3, l4):
        with pytest.raises(bsp.BspError) as e:
            bsp.bsp_conv2d_chain(l1.wd, l1.handle(), bad.wd, bad.handle(), xd, X, None, 1, None, Y, bsp.F32, l1.ws)
        assert e.value.status == bsp.ERR_SHAPE
    li = bsp.SparseLayer(64, 64, 3, 3, 8, 8, torch.int8)
    l2 = bsp.SparseLayer(128, 64, 1, 1, 8, 8, torch.bfloat16)
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_conv2d_chain(li.wd, li.handle(), l2.wd, l2.handle(), xd, X, None, 1, None, Y, bsp.F32, l1.ws)
    assert e.value.status == bsp.ERR_DTYPE
