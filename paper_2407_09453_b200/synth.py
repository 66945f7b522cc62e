"""Seeded synthetic tensors for the block-sparse operator Y = W*X + b.

This module only draws numbers and rounds them to their storage type.  It holds none of the
method's arithmetic (no scores, masks, compaction or products), so that the CPU oracle and the
CUDA path can both be fed from it without sharing any computation.

Generator: a counter-based splitmix64 stream (Steele, Lea, Flood 2014): element ``i`` of a stream
with seed ``s`` is ``mix(s + (i + 1) * 0x9E3779B97F4A7C15)``.  Uniform reals take the top 53 bits,
normals come from the Box-Muller transform of two consecutive stream elements.

The layer-shape tables list convolution shapes of the public ResNet50, VGG16 and InceptionV3
architectures (the paper's three models, Section "Experiments"); only shapes are used, weights
and activations are random.
"""
from __future__ import annotations

import dataclasses
import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
BASE_SEED = 0x24070945

TENSOR_W, TENSOR_X, TENSOR_BIAS, TENSOR_GAMMA = 0, 1, 2, 3


def tensor_seed(config: int, layer: int, tensor_id: int) -> int:
    """Seed of one tensor: a fixed base xor (config, layer, tensor) packed in decimal."""
    return BASE_SEED ^ (config * 1000 + layer * 10 + tensor_id)


def splitmix64(seed: int, n: int, offset: int = 0) -> np.ndarray:
    """Elements offset .. offset+n-1 of the splitmix64 stream of ``seed`` as uint64."""
    with np.errstate(over="ignore"):
        idx = np.arange(offset + 1, offset + n + 1, dtype=np.uint64)
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + idx * _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    return z


def uniform01(seed: int, n: int, offset: int = 0) -> np.ndarray:
    """n doubles in the open interval (0, 1)."""
    bits = splitmix64(seed, n, offset) >> np.uint64(11)
    return (bits.astype(np.float64) + 0.5) * (1.0 / 9007199254740992.0)


def normal(seed: int, shape, sigma: float = 1.0, chunk: int = 1 << 22) -> np.ndarray:
    """float64 N(0, sigma^2) tensor: Box-Muller on stream elements (2i, 2i+1) for element i."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float64)
    for lo in range(0, n, chunk):
        m = min(chunk, n - lo)
        u = uniform01(seed, 2 * m, 2 * lo)
        r = np.sqrt(-2.0 * np.log(u[0::2]))
        out[lo:lo + m] = r * np.cos(2.0 * np.pi * u[1::2])
    return (out * sigma).reshape(shape)


def uniform_int(seed: int, shape, lo: int, hi: int) -> np.ndarray:
    """int64 tensor, uniform on the closed range [lo, hi] (modulo reduction of the 64-bit word)."""
    n = int(np.prod(shape))
    span = np.uint64(hi - lo + 1)
    return ((splitmix64(seed, n) % span).astype(np.int64) + lo).reshape(shape)


def shuffled(seed: int, n: int) -> np.ndarray:
    """A permutation of 0..n-1 by Fisher-Yates, driven by the splitmix64 stream."""
    perm = np.arange(n, dtype=np.int64)
    r = splitmix64(seed, max(n - 1, 0))
    for k, i in enumerate(range(n - 1, 0, -1)):
        j = int(r[k] % np.uint64(i + 1))
        perm[i], perm[j] = perm[j], perm[i]
    return perm


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float values to the nearest bfloat16 (ties to even); result held as float32."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32).astype(np.uint64)
    u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def bf16_bits(a_f32: np.ndarray) -> np.ndarray:
    """The 16-bit patterns (uint16) of float32 values that are exactly representable in bf16."""
    u = np.ascontiguousarray(a_f32, dtype=np.float32).view(np.uint32)
    return (u >> np.uint32(16)).astype(np.uint16)


def bf16_from_bits(bits_u16: np.ndarray) -> np.ndarray:
    """float32 values of bf16 bit patterns."""
    return (bits_u16.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclasses.dataclass(frozen=True)
class Layer:
    """One layer Y = W*X + b in the paper's notation (Introduction): W is O x H x K x I."""
    name: str
    O: int
    I: int
    H: int
    K: int
    N: int          # batch (GEMM: number of columns P of X)
    L: int          # input height
    J: int          # input width
    stride_h: int = 1
    stride_w: int = 1
    pad_h: int = 0
    pad_w: int = 0
    count: int = 1  # how many times the shape occurs in the network

    @property
    def M(self) -> int:
        return (self.L + 2 * self.pad_h - self.H) // self.stride_h + 1

    @property
    def Nw(self) -> int:
        return (self.J + 2 * self.pad_w - self.K) // self.stride_w + 1

    @property
    def P(self) -> int:
        return self.N * self.M * self.Nw

    def dense_flops(self) -> int:
        return 2 * self.P * self.O * self.I * self.H * self.K


def fc(name, O, I, P, count=1) -> Layer:
    return Layer(name, O, I, 1, 1, P, 1, 1, count=count)


def conv(name, I, O, k, size, stride=1, pad=None, batch=1, count=1, kh=None, kw=None,
         pad_h=None, pad_w=None) -> Layer:
    kh = k if kh is None else kh
    kw = k if kw is None else kw
    if pad is None:
        pad = 0
    ph = (pad if pad_h is None else pad_h)
    pw = (pad if pad_w is None else pad_w)
    return Layer(name, O, I, kh, kw, batch, size, size, stride, stride, ph, pw, count)


def resnet50_layers(batch: int = 64):
    """Sparse-eligible layers of ResNet50 (stride on the 3x3 of each bottleneck); stem excluded."""
    b = batch
    L = [
        conv("c2.1x1.64-64", 64, 64, 1, 56, batch=b, count=1),
        conv("c2.1x1.64-256", 64, 256, 1, 56, batch=b, count=4),
        conv("c2.1x1.256-64", 256, 64, 1, 56, batch=b, count=2),
        conv("c2.3x3.64-64", 64, 64, 3, 56, pad=1, batch=b, count=3),
        conv("c3.1x1.256-128", 256, 128, 1, 56, batch=b, count=1),
        conv("c3.3x3.128-128.s2", 128, 128, 3, 56, stride=2, pad=1, batch=b, count=1),
        conv("c3.1x1.128-512", 128, 512, 1, 28, batch=b, count=4),
        conv("c3.1x1.256-512.s2", 256, 512, 1, 56, stride=2, batch=b, count=1),
        conv("c3.1x1.512-128", 512, 128, 1, 28, batch=b, count=3),
        conv("c3.3x3.128-128", 128, 128, 3, 28, pad=1, batch=b, count=3),
        conv("c4.1x1.512-256", 512, 256, 1, 28, batch=b, count=1),
        conv("c4.3x3.256-256.s2", 256, 256, 3, 28, stride=2, pad=1, batch=b, count=1),
        conv("c4.1x1.256-1024", 256, 1024, 1, 14, batch=b, count=6),
        conv("c4.1x1.512-1024.s2", 512, 1024, 1, 28, stride=2, batch=b, count=1),
        conv("c4.1x1.1024-256", 1024, 256, 1, 14, batch=b, count=5),
        conv("c4.3x3.256-256", 256, 256, 3, 14, pad=1, batch=b, count=5),
        conv("c5.1x1.1024-512", 1024, 512, 1, 14, batch=b, count=1),
        conv("c5.3x3.512-512.s2", 512, 512, 3, 14, stride=2, pad=1, batch=b, count=1),
        conv("c5.1x1.512-2048", 512, 2048, 1, 7, batch=b, count=3),
        conv("c5.1x1.1024-2048.s2", 1024, 2048, 1, 14, stride=2, batch=b, count=1),
        conv("c5.1x1.2048-512", 2048, 512, 1, 7, batch=b, count=2),
        conv("c5.3x3.512-512", 512, 512, 3, 7, pad=1, batch=b, count=2),
        fc("fc.2048-1000", 1000, 2048, b, count=1),
    ]
    return L


def vgg16_layers(batch: int = 32):
    """3x3 convolutions of VGG16 except the first (3 input channels)."""
    b = batch
    return [
        conv("vgg.64-64@224", 64, 64, 3, 224, pad=1, batch=b),
        conv("vgg.64-128@112", 64, 128, 3, 112, pad=1, batch=b),
        conv("vgg.128-128@112", 128, 128, 3, 112, pad=1, batch=b),
        conv("vgg.128-256@56", 128, 256, 3, 56, pad=1, batch=b),
        conv("vgg.256-256@56", 256, 256, 3, 56, pad=1, batch=b, count=2),
        conv("vgg.256-512@28", 256, 512, 3, 28, pad=1, batch=b),
        conv("vgg.512-512@28", 512, 512, 3, 28, pad=1, batch=b, count=2),
        conv("vgg.512-512@14", 512, 512, 3, 14, pad=1, batch=b, count=3),
    ]


def inception_v3_layers(batch: int = 32):
    """InceptionV3-shaped branches at 35x35, 17x17 and 8x8 (1x1, 3x3, 1x7, 7x1)."""
    b = batch
    return [
        conv("inc35.1x1.192-64", 192, 64, 1, 35, batch=b),
        conv("inc35.1x1.256-48", 256, 48, 1, 35, batch=b),
        conv("inc35.1x1.288-64", 288, 64, 1, 35, batch=b),
        conv("inc35.3x3.64-96", 64, 96, 3, 35, pad=1, batch=b),
        conv("inc35.3x3.96-96", 96, 96, 3, 35, pad=1, batch=b),
        conv("inc35.3x3.288-384.s2", 288, 384, 3, 35, stride=2, batch=b),
        conv("inc35.3x3.96-96.s2", 96, 96, 3, 35, stride=2, batch=b),
        conv("inc17.1x1.768-192", 768, 192, 1, 17, batch=b),
        conv("inc17.1x1.768-128", 768, 128, 1, 17, batch=b),
        conv("inc17.1x7.128-128", 128, 128, 0, 17, batch=b, kh=1, kw=7, pad_h=0, pad_w=3),
        conv("inc17.7x1.128-192", 128, 192, 0, 17, batch=b, kh=7, kw=1, pad_h=3, pad_w=0),
        conv("inc17.1x7.160-160", 160, 160, 0, 17, batch=b, kh=1, kw=7, pad_h=0, pad_w=3),
        conv("inc17.7x1.192-192", 192, 192, 0, 17, batch=b, kh=7, kw=1, pad_h=3, pad_w=0),
        conv("inc17.3x3.192-320.s2", 192, 320, 3, 17, stride=2, batch=b),
        conv("inc17.3x3.192-192.s2", 192, 192, 3, 17, stride=2, batch=b),
        conv("inc8.1x1.1280-320", 1280, 320, 1, 8, batch=b),
        conv("inc8.1x1.2048-384", 2048, 384, 1, 8, batch=b),
        conv("inc8.1x1.2048-448", 2048, 448, 1, 8, batch=b),
        conv("inc8.1x1.2048-192", 2048, 192, 1, 8, batch=b),
        conv("inc8.3x3.448-384", 448, 384, 3, 8, pad=1, batch=b),
    ]


def make_layer_tensors(layer: Layer, dtype: str, config: int = 0, layer_id: int = 0,
                       w_sigma: float | None = None, bias: bool = True):
    """W [O][H][K][I], X [N][L][J][I], bias [O] for one layer.

    dtype "bf16": values rounded to bf16 and returned as float32; "f32": float32;
    "i8": int8 uniform in [-127, 127] with an int32 bias uniform in [-2^15, 2^15].
    Float weights are He-initialised N(0, 2 / (H K I)) unless ``w_sigma`` is given.
    """
    wshape = (layer.O, layer.H, layer.K, layer.I)
    xshape = (layer.N, layer.L, layer.J, layer.I)
    sw = tensor_seed(config, layer_id, TENSOR_W)
    sx = tensor_seed(config, layer_id, TENSOR_X)
    sb = tensor_seed(config, layer_id, TENSOR_BIAS)
    if dtype == "i8":
        W = uniform_int(sw, wshape, -127, 127).astype(np.int8)
        X = uniform_int(sx, xshape, -127, 127).astype(np.int8)
        b = uniform_int(sb, (layer.O,), -(1 << 15), 1 << 15).astype(np.int32) if bias else None
        return W, X, b
    if w_sigma is None:
        w_sigma = float(np.sqrt(2.0 / (layer.H * layer.K * layer.I)))
    W = normal(sw, wshape, w_sigma).astype(np.float32)
    X = normal(sx, xshape, 1.0).astype(np.float32)
    b = normal(sb, (layer.O,), 0.1).astype(np.float32) if bias else None
    if dtype == "bf16":
        W, X = round_to_bf16(W), round_to_bf16(X)
    elif dtype != "f32":
        raise ValueError(dtype)
    return W, X, b


def random_gamma(seed: int, NBo: int, NBi: int, n_zero: int) -> np.ndarray:
    """A 0/1 mask with exactly n_zero zeros at uniformly random block positions."""
    g = np.ones(NBo * NBi, dtype=np.uint8)
    g[shuffled(seed, NBo * NBi)[:n_zero]] = 0
    return g.reshape(NBo, NBi)
