"""GPU parity of the requantising int8 epilogue (bsp_gemm_q8 / bsp_conv2d_q8) against the oracle, bit for bit: the
oracle's exact int32 product, then its requantisation (power-of-two shift per output channel, nearest with halves away
from zero, saturation)."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_09453_b200 import bsp, synth
from gpu_util import gpu_layer, make_bias, make_case, make_x, to_dev

pytestmark = pytest.mark.gpu


def shifts_for(seed, O, lo, hi):
    s = synth.uniform_int(seed, (O,), lo, hi).astype(np.int32)
    s[0], s[1 % O], s[2 % O] = 0, 31, lo          # the extremes: everything saturates, everything rounds to 0 or +-1
    return s


def run_q8(seed, O, I, H, K, xshape, stride, pad, bo=8, bi=8, frac=0.5, gemm=False, bias=True):
    W = make_case(seed, O, I, H, K, "i8")
    gamma = synth.random_gamma(seed + 1, O // bo, I // bi, int(round(frac * (O // bo) * (I // bi))))
    X = make_x(seed + 2, xshape, "i8")
    b = make_bias(seed + 3, O, "i8") if bias else None
    # typical |accumulator| is about 127^2 sqrt(kept terms) / 3: shifts around it keep most outputs inside the int8 range
    terms = max(1.0, (1 - frac) * I * H * K)
    mid = int(np.log2(127 * 127 * np.sqrt(terms) / 3 / 40))
    shift = shifts_for(seed + 4, O, max(0, mid - 2), mid + 2)
    lay = gpu_layer(W, gamma, bo, bi, "i8")
    Xd = to_dev(X, "i8")
    bd = None if b is None else torch.from_numpy(b).cuda()
    sd = torch.from_numpy(shift).cuda()
    rp, ci, pl = ref.compact(W, gamma, bo, bi)
    if gemm:
        Y = torch.full((xshape[0], O), 77, dtype=torch.int8, device="cuda")
        lay.gemm_q8(Xd, bd, sd, Y)
        y32 = ref.gemm(O, I, bo, bi, rp, ci, pl.reshape(-1, bo, bi), X, b)
    else:
        N, L, J, _ = xshape
        M, Nw = ref.out_hw(L, J, H, K, stride[0], stride[1], pad[0], pad[1])
        Y = torch.full((N, M, Nw, O), 77, dtype=torch.int8, device="cuda")
        lay.conv2d_q8(Xd, bd, sd, Y, stride, pad)
        y32 = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, stride, pad)
    lay.check()
    want = ref.requant_i8(y32, shift)
    got = Y.cpu().numpy().reshape(-1, O)
    assert np.array_equal(got, want)
    inside = np.abs(want[:, 3:].astype(np.int32)) < 127
    assert inside.mean() > 0.5                     # the case exercises the rounding, not only the rails


@pytest.mark.parametrize("bo,bi", [(8, 8), (4, 16), (16, 4)])
def test_gemm_q8_block_shapes_ragged(bo, bi):
    run_q8(801, 192, 256, 1, 1, (333, 256), None, None, bo, bi, gemm=True)


@pytest.mark.parametrize("O,P", [(1008, 77), (48, 300), (16, 5), (320, 129)])
def test_gemm_q8_channel_tiles_off_the_grid(O, P):
    """128-channel staging rounds against channel counts that end inside one (O a multiple of 16)."""
    run_q8(811, O, 96, 1, 1, (P, 96), None, None, gemm=True)


@pytest.mark.parametrize("H,K,stride,pad,sp", [(3, 3, (1, 1), (1, 1), (14, 14)), (1, 1, (2, 2), (0, 0), (14, 14)),
                                                (3, 3, (2, 2), (1, 1), (15, 15)), (1, 7, (1, 1), (0, 3), (17, 17))])
def test_conv_q8_taps_strides_padding(H, K, stride, pad, sp):
    run_q8(821 + H + K, 128, 64, H, K, (3, sp[0], sp[1], 64), stride, pad)


def test_conv_q8_no_bias_and_sparsity_extremes():
    run_q8(831, 64, 64, 3, 3, (2, 8, 8, 64), (1, 1), (1, 1), bias=False)
    run_q8(833, 256, 128, 1, 1, (2, 8, 8, 128), (1, 1), (0, 0), frac=0.0)


def test_q8_argument_errors():
    lay = bsp.SparseLayer(64, 64, 1, 1, 8, 8, torch.bfloat16)
    X = torch.zeros((16, 64), dtype=torch.bfloat16, device="cuda")
    Y = torch.zeros((16, 64), dtype=torch.int8, device="cuda")
    s = torch.zeros(64, dtype=torch.int32, device="cuda")
    with pytest.raises(bsp.BspError) as e:
        lay.gemm_q8(X, None, s, Y)
    assert e.value.status == bsp.ERR_DTYPE               # float weights have no 8-bit epilogue
    lay8 = bsp.SparseLayer(72, 64, 1, 1, 8, 8, torch.int8)
    with pytest.raises(bsp.BspError) as e:
        lay8.gemm_q8(torch.zeros((16, 64), dtype=torch.int8, device="cuda"), None, torch.zeros(72, dtype=torch.int32, device="cuda"),
                     torch.zeros((16, 72), dtype=torch.int8, device="cuda"))
    assert e.value.status == bsp.ERR_SHAPE               # 72 int8 channels: rows of Y are not 16-byte multiples
