"""GPU parity of the product kernel on matrix products (bf16, int8 and fp32-as-TF32 1x1 layers: ragged position and
channel tiles, K tails inside a stage, more tiles than SMs, long K, sparsity extremes, bf16 output) against the CPU
oracle, through the C ABI: within tolerance for floats, bit for bit for int8."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_09453_b200 import bsp, synth
import gpu_util
from gpu_util import gpu_conv, gpu_gemm, gpu_layer, make_bias, make_case, make_x
from test_gpu_product import check

pytestmark = pytest.mark.gpu

SHAPES = [(8, 8), (4, 16), (16, 4)]
YT = {"bf16": bsp.F32, "f32": bsp.F32, "i8": bsp.I32}


def run_gemm(seed, O, I, P, bo, bi, dtype, frac=0.5, out="f32", bias=True):
    wd = bsp.wdesc(O, I, 1, 1, bo, bi, gpu_util.TORCH_DT[dtype])
    assert bsp.conv_kernel_name(wd, bsp.XDesc(P, 1, 1, 1, 1, 0, 0)) == "gemm_tc_kernel"
    W = make_case(seed, O, I, 1, 1, dtype)
    NB = (O // bo) * (I // bi)
    gamma = synth.random_gamma(seed + 1, O // bo, I // bi, int(round(frac * NB)))
    X = make_x(seed + 2, (P, I), dtype)
    b = make_bias(seed + 3, O, dtype) if bias else None
    lay = gpu_layer(W, gamma, bo, bi, dtype)
    got = gpu_gemm(lay, X, b, dtype, out)
    rp, ci, pl = ref.compact(W, gamma, bo, bi)
    want = ref.gemm(O, I, bo, bi, rp, ci, pl.reshape(-1, bo, bi), X, b)
    check(got, want, dtype, out)
    return got, want


@pytest.mark.parametrize("dtype", ["bf16", "i8", "f32"])
@pytest.mark.parametrize("bo,bi", SHAPES)
def test_block_shapes_ragged_positions(dtype, bo, bi):
    """O = 192 (one 192-channel tile), three position tiles with a ragged tail, several K-stages."""
    run_gemm(701, 192, 256, 333, bo, bi, dtype)


@pytest.mark.parametrize("dtype,I", [("bf16", 200), ("i8", 208), ("f32", 40), ("bf16", 8), ("i8", 16)])
@pytest.mark.parametrize("bo,bi", [(8, 8), (16, 4)])
def test_k_tail_inside_a_stage(dtype, I, bo, bi):
    """Rows of X that end inside a 128-byte K-stage: the tensor map fills the rest with zeros, the index masks it."""
    run_gemm(711, 128, I, 150, bo, bi, dtype)


@pytest.mark.parametrize("dtype", ["bf16", "i8"])
@pytest.mark.parametrize("O,P", [(1000, 77), (48, 300), (64, 1), (320, 129)])
def test_channel_tiles_off_the_grid(dtype, O, P):
    """O = 1000: four tiles of 256 with 232 channels in the last; O = 48: a 64-channel tile clipped by the store."""
    run_gemm(721, O, 96, P, 8, 8, dtype)


@pytest.mark.parametrize("dtype,O,P", [("bf16", 1024, 5127), ("i8", 512, 20001), ("f32", 256, 40000)])
def test_more_tiles_than_sms(dtype, O, P):
    """Persistent CTAs take two, three or more tiles each: both accumulator buffers and every stage are reused."""
    run_gemm(731, O, 192, P, 8, 8, dtype)


@pytest.mark.parametrize("frac", [0.0, 0.25, 0.75, 1.0])
@pytest.mark.parametrize("dtype", ["bf16", "i8"])
def test_sparsity_extremes(dtype, frac):
    got, _ = run_gemm(741, 256, 512, 260, 8, 8, dtype, frac)
    if frac == 1.0:                              # Gamma == 0: the bias broadcast
        assert np.array_equal(got, np.tile(got[0], (got.shape[0], 1)))


def test_bf16_output_and_no_bias():
    run_gemm(751, 320, 256, 500, 8, 8, "bf16", out="bf16")
    run_gemm(753, 128, 128, 200, 4, 16, "bf16", bias=False)
    run_gemm(755, 128, 128, 200, 8, 8, "f32", out="bf16")


def test_long_k_wraps_the_stage_ring_many_times():
    run_gemm(761, 256, 4096, 130, 8, 8, "bf16")
    run_gemm(763, 64, 8192, 40, 8, 8, "i8", frac=0.75)


def test_conv2d_1x1_equals_gemm_bitwise():
    O, I = 128, 192
    W = make_case(771, O, I, 1, 1, "bf16")
    gamma = synth.random_gamma(772, 16, 24, 192)
    X = make_x(773, (4, 8, 8, I), "bf16")
    b = make_bias(774, O, "bf16")
    lay = gpu_layer(W, gamma, 8, 8, "bf16")
    yc = gpu_conv(lay, X, b, "bf16")
    yg = gpu_gemm(lay, X.reshape(-1, I), b, "bf16")
    assert np.array_equal(yc, yg)


def test_packed_buffer_of_another_layer_is_refused():
    """The kernel compares the packed header with the descriptor before it loads anything: a buffer that bsp_compact
    filled for a different layer latches BSP_ERR_INDEX and leaves Y untouched (a host-made inconsistency: no access
    outside any buffer happens)."""
    W = make_case(781, 128, 128, 1, 1, "bf16")
    gamma = synth.random_gamma(782, 16, 16, 128)
    lay = gpu_layer(W, gamma, 8, 8, "bf16")
    other = bsp.SparseLayer(128, 128, 1, 1, 4, 16, torch.bfloat16)       # same sizes, another block shape
    X = gpu_util.to_dev(make_x(783, (64, 128), "bf16"), "bf16")
    Y = torch.full((64, 128), -7.0, dtype=torch.float32, device="cuda")
    bsp.bsp_conv2d(other.wd, lay.handle(), bsp.XDesc(64, 1, 1, 1, 1, 0, 0), X, None, Y, bsp.F32, lay.ws)
    with pytest.raises(bsp.BspError) as e:
        lay.check()
    assert e.value.status == bsp.ERR_INDEX
    assert bool((Y == -7.0).all())
    lay.check()                                   # the latched status is cleared once read
