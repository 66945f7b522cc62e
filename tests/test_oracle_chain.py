"""Pins for the oracle's bfloat16 rounding and the two-layer chain with a bfloat16 tensor in between (CPU only)."""
import numpy as np
import pytest

from oracle import ref
from paper_2407_09453_b200 import synth


def bf16_by_bits(v32: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even of float32 values to bfloat16 through their bit patterns (an independent route: integer
    arithmetic on the encoding instead of frexp / ldexp on the value)."""
    u = np.ascontiguousarray(v32, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def test_round_bf16_hand_worked_values():
    """8 significant bits, ties to the even mantissa: 1 + 2^-8 lies half way between 1 and 1 + 2^-7 -> 1 (even);
    1 + 3 * 2^-8 lies half way between 1 + 2^-7 (odd) and 1 + 2^-6 (even) -> 1 + 2^-6."""
    v = np.array([1.0, 1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, 1 + 2.0 ** -8 + 2.0 ** -30, -(1 + 2.0 ** -8), 0.0, 255.5, 0.3],
                 dtype=np.float64)
    want = np.array([1.0, 1.0, 1 + 2.0 ** -6, 1 + 2.0 ** -7, -1.0, 0.0, 256.0, 0.30078125], dtype=np.float32)
    assert np.array_equal(ref.round_bf16(v), want)


def test_round_bf16_against_the_bit_pattern_route_and_its_properties():
    v = synth.normal(801, (20000,)).astype(np.float32) * np.exp2(synth.uniform_int(802, (20000,), -20, 20)).astype(np.float32)
    got = ref.round_bf16(v.astype(np.float64))
    assert np.array_equal(got, bf16_by_bits(v))
    assert np.array_equal(ref.round_bf16(got.astype(np.float64)), got)                    # idempotent
    assert np.all(np.abs(got.astype(np.float64) - v) <= np.abs(v.astype(np.float64)) * 2.0 ** -8)
    s = np.sort(v.astype(np.float64))
    assert np.all(np.diff(ref.round_bf16(s)) >= 0)                                         # monotone
    # float64 inputs that are NOT float32 values: a single rounding, not float64 -> float32 -> bfloat16
    x = np.array([1 + 2.0 ** -8 + 2.0 ** -40, 1 + 2.0 ** -8 - 2.0 ** -40])                # float32 would round both to the tie
    assert np.array_equal(ref.round_bf16(x), np.array([1 + 2.0 ** -7, 1.0], dtype=np.float32))


def make_chain(seed, N, L, J, I, O1, O2, H, K):
    W1 = synth.round_to_bf16(synth.normal(seed, (O1, H, K, I), np.sqrt(2.0 / (H * K * I))).astype(np.float32))
    W2 = synth.round_to_bf16(synth.normal(seed + 1, (O2, 1, 1, O1), np.sqrt(2.0 / O1)).astype(np.float32))
    X = synth.round_to_bf16(synth.normal(seed + 2, (N, L, J, I)).astype(np.float32))
    b1 = synth.normal(seed + 3, (O1,), 0.1).astype(np.float32)
    b2 = synth.normal(seed + 4, (O2,), 0.1).astype(np.float32)
    g1 = synth.random_gamma(seed + 5, O1 // 8, I // 8, (O1 // 8) * (I // 8) // 2)
    g2 = synth.random_gamma(seed + 6, O2 // 8, O1 // 8, (O2 // 8) * (O1 // 8) // 2)
    return W1, W2, X, b1, b2, g1, g2


@pytest.mark.parametrize("relu", [0, 1])
@pytest.mark.parametrize("H,K,stride,pad", [(3, 3, (1, 1), (1, 1)), (1, 1, (1, 1), (0, 0)), (3, 3, (2, 2), (1, 1))])
def test_chain_equals_two_dense_numpy_layers_with_a_bf16_tensor_between(H, K, stride, pad, relu):
    """The plain definition: dense masked layer one (the pinned dense reference), max(., 0), rounding through the
    bit-pattern route, dense masked layer two as a numpy matrix product."""
    W1, W2, X, b1, b2, g1, g2 = make_chain(811, 2, 9, 7, 16, 24, 40, H, K)
    got = ref.chain2(W1.shape, 8, 8, ref.compact(W1, g1, 8, 8), X, b1, relu, 40, 8, 8, ref.compact(W2, g2, 8, 8), b2, stride, pad)
    T = ref.dense_conv2d(ref.apply_mask(W1, g1, 8, 8), X, b1, stride, pad)
    if relu:
        T = np.maximum(T, 0.0)
    Tb = bf16_by_bits(T.astype(np.float32)).astype(np.float64)      # (these sizes never meet a float64 / float32 double-rounding tie)
    want = Tb.reshape(-1, 24) @ ref.apply_mask(W2, g2, 8, 8)[:, 0, 0, :].astype(np.float64).T + b2.astype(np.float64)
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    # leaving out the rounding, the activation or the first bias must show
    raw = ref.dense_conv2d(ref.apply_mask(W1, g1, 8, 8), X, b1, stride, pad).reshape(-1, 24)
    plain = raw @ ref.apply_mask(W2, g2, 8, 8)[:, 0, 0, :].astype(np.float64).T + b2.astype(np.float64)
    assert not np.allclose(got, plain, rtol=1e-6, atol=1e-6)


def test_chain_with_an_identity_second_layer_returns_the_rounded_tensor():
    W1, _, X, b1, _, g1, _ = make_chain(821, 1, 6, 6, 16, 16, 16, 3, 3)
    W2 = np.eye(16, dtype=np.float32).reshape(16, 1, 1, 16)
    g2 = np.ones((2, 2), dtype=np.uint8)
    got = ref.chain2(W1.shape, 8, 8, ref.compact(W1, g1, 8, 8), X, b1, 1, 16, 8, 8, ref.compact(W2, g2, 8, 8), None, (1, 1), (1, 1))
    T = np.maximum(ref.conv2d(W1.shape, 8, 8, *ref.compact(W1, g1, 8, 8), X, b1, (1, 1), (1, 1)), 0.0)
    assert np.array_equal(got, ref.round_bf16(T).astype(np.float64))
    assert np.all(got >= 0.0)


@pytest.mark.parametrize("relu,with_shift2", [(0, False), (1, False), (1, True)])
def test_int8_chain_equals_integer_numpy_layers(relu, with_shift2):
    """The 8-bit chain against plain integer numpy: dense masked layer one (the pinned dense reference), the
    rounding shift written out with exact rationals, max(., 0), an int64 matrix product for layer two."""
    from fractions import Fraction
    N, L, J, I, O1, O2 = 2, 7, 6, 16, 16, 24
    W1 = synth.uniform_int(831, (O1, 3, 3, I), -127, 127).astype(np.int8)
    W2 = synth.uniform_int(832, (O2, 1, 1, O1), -127, 127).astype(np.int8)
    X = synth.uniform_int(833, (N, L, J, I), -127, 127).astype(np.int8)
    b1 = synth.uniform_int(834, (O1,), -(1 << 15), 1 << 15).astype(np.int32)
    b2 = synth.uniform_int(835, (O2,), -(1 << 15), 1 << 15).astype(np.int32)
    s1 = synth.uniform_int(836, (O1,), 9, 13).astype(np.int32)
    s2 = synth.uniform_int(837, (O2,), 8, 12).astype(np.int32) if with_shift2 else None
    g1 = synth.random_gamma(838, O1 // 8, I // 8, 2)
    g2 = synth.random_gamma(839, O2 // 8, O1 // 8, 3)
    got = ref.chain2_q8(W1.shape, 8, 8, ref.compact(W1, g1, 8, 8), X, b1, s1, relu, O2, 8, 8, ref.compact(W2, g2, 8, 8), b2, s2, (1, 1), (1, 1))

    def rq(v, sh):                                        # nearest integer of v / 2^sh, halves away from zero, saturated
        out = np.empty(v.shape, dtype=np.int64)
        for idx in np.ndindex(*v.shape):
            f = Fraction(int(v[idx]), 1 << int(sh[idx[-1]]))
            q = int(abs(f) + Fraction(1, 2))               # floor(|f| + 1/2)
            out[idx] = max(-128, min(127, q if f >= 0 else -q))
        return out

    T = ref.dense_conv2d(ref.apply_mask(W1, g1, 8, 8), X, b1, (1, 1), (1, 1)).astype(np.int64).reshape(-1, O1)
    T8 = rq(T, s1)
    if relu:
        T8 = np.maximum(T8, 0)
    Y = T8 @ ref.apply_mask(W2, g2, 8, 8)[:, 0, 0, :].astype(np.int64).T + b2.astype(np.int64)
    want = rq(Y, s2) if with_shift2 else Y
    assert np.array_equal(got.astype(np.int64), want)
    assert got.dtype == (np.int8 if with_shift2 else np.int32)
    if not with_shift2:
        assert np.abs(T8).max() == 127 or np.abs(T8).max() > 20          # the shifts leave a tensor that uses the int8 range
