"""GPU parity on the layer tables of the workloads: every sparse-eligible ResNet50 layer (bf16), every VGG16 and
InceptionV3-shaped layer (int8, bit exact) and all nine (block shape, sparsity) cells of the 4096 x 4096 x 8192 product.

Each case is the whole call chain through the C ABI: bsp_mask (Gamma compared with the oracle's bit for bit) ->
bsp_compact -> bsp_conv2d / bsp_gemm, at the layer's full channel counts and spatial size and a small batch; the
oracle evaluates a few hundred sampled output positions (image corners, the seams between 128-position tiles, random
ones)."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_09453_b200 import bsp, synth
from gpu_util import gpu_conv, gpu_gemm, gpu_mask
from test_gpu_product import check

pytestmark = pytest.mark.gpu



def sample_positions(layer, seed, n_random=250):
    P, per = layer.P, layer.M * layer.Nw
    fixed = [0, layer.Nw - 1, per - layer.Nw, per - 1, P - per, P - 1, 126, 127, 128, 129, 255, 256, per, per + 1]
    fixed = [p for p in fixed if 0 <= p < P]
    rnd = synth.uniform_int(seed, (n_random,), 0, P - 1)
    return np.unique(np.r_[fixed, rnd]).astype(np.int64)


def run_layer(layer, dtype, frac, cfg, layer_id):
    W, X, b = synth.make_layer_tensors(layer, dtype, config=cfg, layer_id=layer_id)
    NB = (layer.O // 8) * (layer.I // 8)
    n_zero = int(frac * NB + 0.5)
    stride, pad = (layer.stride_h, layer.stride_w), (layer.pad_h, layer.pad_w)
    tdt = torch.int8 if dtype == "i8" else torch.bfloat16
    name = bsp.conv_kernel_name(bsp.wdesc(layer.O, layer.I, layer.H, layer.K, 8, 8, tdt),
                                bsp.XDesc(layer.N, layer.L, layer.J, stride[0], stride[1], pad[0], pad[1]))
    assert name == "gemm_tc_kernel"
    g, s, lay, Wd = gpu_mask(W, 8, 8, dtype, n_zero)
    want_g = ref.mask(ref.scores(W, 8, 8), n_zero)
    assert np.array_equal(g, want_g)
    lay.compact(Wd)
    lay.check()
    got = gpu_conv(lay, X, b, dtype, stride, pad)
    pix = sample_positions(layer, 9000 + layer_id)
    rp, ci, pl = ref.compact(W, want_g, 8, 8)
    want = ref.conv2d(W.shape, 8, 8, rp, ci, pl, X, b, stride, pad, pix=pix)
    check(got[pix], want, dtype)


RESNET = synth.resnet50_layers(batch=3)


@pytest.mark.parametrize("idx", range(len(RESNET)), ids=[l.name for l in RESNET])
def test_resnet50_layer_bf16_8x8_half_sparse(idx):
    run_layer(RESNET[idx], "bf16", 0.5, 4, idx)


INT8_LAYERS = synth.vgg16_layers(batch=2) + synth.inception_v3_layers(batch=2)


@pytest.mark.parametrize("frac", [0.5, 0.75])
@pytest.mark.parametrize("idx", range(len(INT8_LAYERS)), ids=[l.name for l in INT8_LAYERS])
def test_vgg16_inceptionv3_layer_int8_bit_exact(idx, frac):
    run_layer(INT8_LAYERS[idx], "i8", frac, 5, idx)


@pytest.fixture(scope="module")
def gemm_4096():
    O = I = 4096
    P = 8192
    W = synth.round_to_bf16(synth.normal(synth.tensor_seed(3, 0, 0), (O, 1, 1, I), 1 / 64.0).astype(np.float32))
    X = synth.round_to_bf16(synth.normal(synth.tensor_seed(3, 0, 1), (P, I)).astype(np.float32))
    b = synth.normal(synth.tensor_seed(3, 0, 2), (O,), 0.1).astype(np.float32)
    return W, X, b


@pytest.mark.parametrize("frac", [0.25, 0.5, 0.75])
@pytest.mark.parametrize("bo,bi", [(8, 8), (4, 16), (16, 4)])
def test_gemm_4096_every_block_shape_and_sparsity(gemm_4096, bo, bi, frac):
    """O = I = 4096, P = 8192, bf16, magnitude Gamma over the layer: 40 sampled rows of Y against the oracle."""
    W, X, b = gemm_4096
    O, P = 4096, 8192
    NB = (O // bo) * (O // bi)
    assert bsp.conv_kernel_name(bsp.wdesc(O, O, 1, 1, bo, bi, torch.bfloat16), bsp.XDesc(P, 1, 1, 1, 1, 0, 0)) == "gemm_tc_kernel"
    g, s, lay, Wd = gpu_mask(W, bo, bi, "bf16", int(frac * NB))
    want_g = ref.mask(ref.scores(W, bo, bi), int(frac * NB))
    assert np.array_equal(g, want_g)
    lay.compact(Wd)
    lay.check()
    got = gpu_gemm(lay, X, b, "bf16")
    pix = np.r_[0, 127, 128, 255, 256, P - 1, synth.uniform_int(7 + bo, (34,), 0, P - 1)]
    rp, ci, pl = ref.compact(W, want_g, bo, bi)
    want = ref.gemm(O, O, bo, bi, rp, ci, pl.reshape(-1, bo, bi), X, b, pix=pix)
    check(got[pix], want, "bf16")
    assert np.isfinite(got).all()


FULL_BF16 = {l.name: l for l in synth.resnet50_layers(batch=64)}
FULL_I8 = {l.name: l for l in synth.vgg16_layers(batch=32) + synth.inception_v3_layers(batch=32)}


@pytest.mark.parametrize("name", ["c2.3x3.64-64", "c3.1x1.256-512.s2", "c5.1x1.512-2048"])
def test_resnet50_layers_at_the_batch_the_benchmark_times(name):
    """Batch 64, as in the benchmark's layer pass: thousands of tiles per launch, every CTA takes many."""
    run_layer(FULL_BF16[name], "bf16", 0.5, 4, 900 + len(name))


@pytest.mark.parametrize("name", ["vgg.64-64@224", "vgg.256-256@56", "inc17.1x7.128-128"])
def test_int8_layers_at_the_batch_the_benchmark_times(name):
    """Batch 32: the 224 x 224 layer is 1.6 million positions (64-byte rows of input channels), bit exact on the samples."""
    run_layer(FULL_I8[name], "i8", 0.5, 5, 950 + len(name))
