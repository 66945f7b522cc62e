"""Pins for the oracle's block-sparse GEMM and convolution (CPU only)."""
import os

import numpy as np
import pytest
from scipy.signal import correlate2d

from oracle import ref
from paper_2407_09453_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def sparse_setup(seed, O, I, H, K, bo, bi, dtype, frac_zero=0.5):
    NBo, NBi = O // bo, I // bi
    if dtype == "i8":
        W = synth.uniform_int(seed, (O, H, K, I), -127, 127).astype(np.int8)
    else:
        W = synth.normal(seed, (O, H, K, I)).astype(np.float32)
    gamma = synth.random_gamma(seed + 1, NBo, NBi, int(round(frac_zero * NBo * NBi)))
    return W, gamma, ref.compact(W, gamma, bo, bi)


def scipy_dense_conv(W, X, bias, stride, pad):
    """Dense cross-correlation through scipy.signal.correlate2d, one (o, i) plane pair at a time."""
    O, H, K, I = W.shape
    N, L, J, _ = X.shape
    M, Nw = ref.out_hw(L, J, H, K, stride[0], stride[1], pad[0], pad[1])
    Y = np.zeros((N, M, Nw, O))
    Xp = np.pad(X.astype(np.float64), ((0, 0), (pad[0], pad[0]), (pad[1], pad[1]), (0, 0)))
    for n in range(N):
        for o in range(O):
            acc = np.zeros((Xp.shape[1] - H + 1, Xp.shape[2] - K + 1))
            for i in range(I):
                acc += correlate2d(Xp[n, :, :, i], W[o, :, :, i].astype(np.float64), mode="valid")
            Y[n, :, :, o] = acc[::stride[0], ::stride[1]][:M, :Nw]
    if bias is not None:
        Y += bias.astype(np.float64)
    return Y.reshape(-1, O)


@pytest.mark.parametrize("bo,bi", [(8, 8), (4, 16), (16, 4)])
def test_gemm_equals_dense_matmul_of_masked_weights(bo, bi):
    O, I, P = 48, 64, 37
    W, gamma, (rp, ci, pl) = sparse_setup(41, O, I, 1, 1, bo, bi, "f32")
    X = synth.normal(43, (P, I)).astype(np.float32)
    b = synth.normal(44, (O,), 0.1).astype(np.float32)
    Y = ref.gemm(O, I, bo, bi, rp, ci, pl, X, b)
    Wm = ref.apply_mask(W, gamma, bo, bi)[:, 0, 0, :].astype(np.float64)
    want = X.astype(np.float64) @ Wm.T + b.astype(np.float64)
    assert np.allclose(Y, want, rtol=1e-12, atol=1e-12)
    # a dropped block or a transposed payload would show here
    assert not np.allclose(Y, X.astype(np.float64) @ W[:, 0, 0, :].astype(np.float64).T + b, atol=1e-3)


def test_gemm_int8_exact_and_pixel_subset():
    O, I, P, bo, bi = 32, 64, 50, 8, 8
    W, gamma, (rp, ci, pl) = sparse_setup(47, O, I, 1, 1, bo, bi, "i8")
    X = synth.uniform_int(48, (P, I), -127, 127).astype(np.int8)
    b = synth.uniform_int(49, (O,), -(1 << 15), 1 << 15).astype(np.int32)
    Y = ref.gemm(O, I, bo, bi, rp, ci, pl, X, b)
    want = X.astype(np.int64) @ ref.apply_mask(W, gamma, bo, bi)[:, 0, 0, :].astype(np.int64).T + b
    assert Y.dtype == np.int32 and np.array_equal(Y, want)
    pix = np.array([49, 0, 7, 7, 23])
    assert np.array_equal(ref.gemm(O, I, bo, bi, rp, ci, pl, X, b, pix=pix), want[pix])


def test_paper_2x2_block_product_example():
    """Section "Block Sparsity in a Matrix": C0=A1 B2, C1=A0 B1, C2=A3 B2, C3=A2 B1."""
    rules = {}
    for line in open(os.path.join(GOLD, "matmul_2x2_example.txt")):
        if line.strip() and not line.startswith("#"):
            c, a, b = line.split()
            rules[int(c[1])] = (int(a[1]), int(b[1]))
    n = 8
    A = synth.normal(51, (2 * n, 2 * n)).astype(np.float32)
    Bblk = {1: synth.normal(52, (n, n)).astype(np.float32), 2: synth.normal(53, (n, n)).astype(np.float32)}
    B = np.zeros((2 * n, 2 * n), dtype=np.float32)
    B[:n, n:], B[n:, :n] = Bblk[1], Bblk[2]
    Ablk = {0: A[:n, :n], 1: A[:n, n:], 2: A[n:, :n], 3: A[n:, n:]}
    # our operator: Y[p][o] = sum_i Wbar[o][i] X[p][i] = (X Wbar^T)[p][o]; with Wbar = B^T, X = A: Y = A B
    Wbar = np.ascontiguousarray(B.T).reshape(2 * n, 1, 1, 2 * n)
    gamma = np.array([[0, 1], [1, 0]], dtype=np.uint8)
    rp, ci, pl = ref.compact(Wbar, gamma, n, n)
    assert list(rp) == [0, 1, 2] and list(ci) == [1, 0]
    Y = ref.gemm(2 * n, 2 * n, n, n, rp, ci, pl, A)
    Cgot = {0: Y[:n, :n], 1: Y[:n, n:], 2: Y[n:, :n], 3: Y[n:, n:]}
    for c, (a, b) in rules.items():
        want = Ablk[a].astype(np.float64) @ Bblk[b].astype(np.float64)
        assert np.allclose(Cgot[c], want, rtol=1e-12, atol=1e-12)


def test_gemm_identity_blocks_copy_rows_of_x():
    bo = bi = 8
    O, I, P = 16, 24, 5
    W = np.zeros((O, 1, 1, I), dtype=np.float32)
    gamma = np.zeros((2, 3), dtype=np.uint8)
    gamma[0, 2] = gamma[1, 0] = 1
    W[0:8, 0, 0, 16:24] = np.eye(8)
    W[8:16, 0, 0, 0:8] = np.eye(8)
    rp, ci, pl = ref.compact(W, gamma, bo, bi)
    X = synth.normal(57, (P, I)).astype(np.float32)
    Y = ref.gemm(O, I, bo, bi, rp, ci, pl, X)
    assert np.array_equal(Y[:, 0:8], X[:, 16:24].astype(np.float64))
    assert np.array_equal(Y[:, 8:16], X[:, 0:8].astype(np.float64))


CONV_CASES = [  # H, K, stride, pad
    (1, 1, (1, 1), (0, 0)), (3, 3, (1, 1), (1, 1)), (3, 3, (2, 2), (1, 1)), (3, 3, (2, 2), (0, 0)),
    (1, 7, (1, 1), (0, 3)), (7, 1, (1, 1), (3, 0)), (3, 3, (1, 2), (3, 0)), (1, 1, (2, 2), (0, 0)),
]


@pytest.mark.parametrize("H,K,stride,pad", CONV_CASES)
def test_conv_equals_scipy_dense_correlation_of_masked_weights(H, K, stride, pad):
    O, I, bo, bi = 16, 16, 8, 8
    W, gamma, (rp, ci, pl) = sparse_setup(61 + H * 10 + K, O, I, H, K, bo, bi, "f32")
    X = synth.normal(63, (2, 6, 7, I)).astype(np.float32)
    b = synth.normal(64, (O,), 0.1).astype(np.float32)
    Y = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, stride, pad)
    Wm = ref.apply_mask(W, gamma, bo, bi)
    want = scipy_dense_conv(Wm, X, b, stride, pad)
    assert Y.shape == want.shape
    assert np.allclose(Y, want, rtol=1e-11, atol=1e-11)
    # the oracle's own textbook dense loop agrees too, and a flipped kernel would not
    assert np.allclose(ref.dense_conv2d(Wm, X, b, stride, pad), want, rtol=1e-11, atol=1e-11)
    if H * K > 1:
        flipped = scipy_dense_conv(Wm[:, ::-1, ::-1, :], X, b, stride, pad)
        assert not np.allclose(Y, flipped, atol=1e-3)


def brute_conv(Wm, X, bias, stride, pad):
    O, H, K, I = Wm.shape
    N, L, J, _ = X.shape
    M, Nw = ref.out_hw(L, J, H, K, stride[0], stride[1], pad[0], pad[1])
    Y = np.zeros((N, M, Nw, O), dtype=np.int64)
    for n in range(N):
        for y in range(M):
            for x in range(Nw):
                for o in range(O):
                    acc = int(bias[o])
                    for h in range(H):
                        for k in range(K):
                            yi, xi = y * stride[0] + h - pad[0], x * stride[1] + k - pad[1]
                            if 0 <= yi < L and 0 <= xi < J:
                                acc += int(np.dot(Wm[o, h, k].astype(np.int64), X[n, yi, xi].astype(np.int64)))
                    Y[n, y, x, o] = acc
    return Y.reshape(-1, O)


@pytest.mark.parametrize("bo,bi", [(8, 8), (4, 16), (16, 4)])
@pytest.mark.parametrize("H,K,stride,pad", [(3, 3, (1, 1), (1, 1)), (3, 3, (2, 2), (1, 1)), (1, 7, (1, 1), (0, 3))])
def test_conv_int8_brute_force_tiny(bo, bi, H, K, stride, pad):
    O = I = 16
    W, gamma, (rp, ci, pl) = sparse_setup(71, O, I, H, K, bo, bi, "i8")
    X = synth.uniform_int(73, (1, 5, 5, I), -127, 127).astype(np.int8)
    b = synth.uniform_int(74, (O,), -(1 << 15), 1 << 15).astype(np.int32)
    Y = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, stride, pad)
    want = brute_conv(ref.apply_mask(W, gamma, bo, bi), X, b, stride, pad)
    assert Y.dtype == np.int32 and np.array_equal(Y, want)
    assert np.array_equal(ref.dense_conv2d(ref.apply_mask(W, gamma, bo, bi), X, b, stride, pad), want)


def test_conv_1x1_equals_gemm_and_subset():
    O, I, bo, bi = 32, 48, 4, 16
    W, gamma, (rp, ci, pl) = sparse_setup(81, O, I, 1, 1, bo, bi, "f32")
    X = synth.normal(83, (3, 4, 5, I)).astype(np.float32)
    b = synth.normal(84, (O,), 0.1).astype(np.float32)
    Yc = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b)
    Yg = ref.gemm(O, I, bo, bi, rp, ci, pl.reshape(-1, bo, bi), X.reshape(-1, I), b)
    assert np.array_equal(Yc, Yg)
    pix = np.array([59, 3, 17])
    assert np.array_equal(ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, pix=pix), Yc[pix])


def test_conv_delta_kernel_is_a_shifted_zero_padded_copy():
    """One tap at (h,k)=(0,2) with identity channels: Y[n,y,x,:] = X[n, y-1, x+1, 8:16] (pad 1, no flip)."""
    bo = bi = 8
    O, I, H, K = 8, 16, 3, 3
    W = np.zeros((O, H, K, I), dtype=np.float32)
    W[:, 0, 2, 8:16] = np.eye(8)
    gamma = np.array([[0, 1]], dtype=np.uint8)
    rp, ci, pl = ref.compact(W, gamma, bo, bi)
    X = synth.normal(91, (1, 5, 6, I)).astype(np.float32)
    Y = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, None, (1, 1), (1, 1)).reshape(5, 6, 8)
    want = np.zeros((5, 6, 8))
    want[1:, :5, :] = X[0, :4, 1:, 8:16]
    assert np.array_equal(Y, want)
    # stride 2, pad 0: Y[y,x] = X[2y, 2x+2]
    Y2 = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, None, (2, 2), (0, 0)).reshape(2, 2, 8)
    assert np.array_equal(Y2, X[0, 0:3:2, 2:5:2, 8:16].astype(np.float64))


def test_bias_only_and_linearity():
    bo = bi = 8
    O, I = 16, 16
    W, gamma, _ = sparse_setup(95, O, I, 3, 3, bo, bi, "i8")
    X = synth.uniform_int(96, (1, 4, 4, I), -127, 127).astype(np.int8)
    b = synth.uniform_int(97, (O,), -1000, 1000).astype(np.int32)
    rp0, ci0, pl0 = ref.compact(W, np.zeros_like(gamma), bo, bi)
    Y0 = ref.conv2d(W.shape, bo, bi, rp0, ci0, pl0, X, b, (1, 1), (1, 1))
    assert np.array_equal(Y0, np.tile(b, (16, 1)))                       # Gamma == 0: bias broadcast
    rp, ci, pl = ref.compact(W, gamma, bo, bi)
    Yb = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, (1, 1), (1, 1))
    Yn = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, None, (1, 1), (1, 1))
    assert np.array_equal(Yb - Yn, np.tile(b, (16, 1)))


def test_int8_overflow_is_reported():
    bo = bi = 8
    W = np.full((8, 1, 1, 8), 127, dtype=np.int8)
    rp, ci, pl = ref.compact(W, np.ones((1, 1), np.uint8), bo, bi)
    X = np.full((1, 8), 127, dtype=np.int8)
    b = np.full(8, 2**31 - 1, dtype=np.int32)
    with pytest.raises(RuntimeError):
        ref.gemm(8, 8, bo, bi, rp, ci, pl.reshape(-1, 8, 8), X, b)


def test_gemm_f32_sampled_rows_against_numpy():
    """The sampled-rows branch of the float product (the one the large GPU cases lean on): listed rows, in the listed
    order and with repeats, equal the same rows of the full result bit for bit, and numpy's matmul of Gamma (.) W on
    those rows of X to rounding."""
    O, I, P, bo, bi = 64, 96, 41, 16, 4
    W, gamma, (rp, ci, pl) = sparse_setup(301, O, I, 1, 1, bo, bi, "f32")
    X = synth.normal(303, (P, I)).astype(np.float32)
    b = synth.normal(304, (O,), 0.1).astype(np.float32)
    pix = np.array([40, 0, 13, 13, 7, 39])
    full = ref.gemm(O, I, bo, bi, rp, ci, pl, X, b)
    sub = ref.gemm(O, I, bo, bi, rp, ci, pl, X, b, pix=pix)
    assert sub.shape == (len(pix), O) and np.array_equal(sub, full[pix])
    Wm = ref.apply_mask(W, gamma, bo, bi)[:, 0, 0, :].astype(np.float64)
    assert np.allclose(sub, X[pix].astype(np.float64) @ Wm.T + b, rtol=1e-12, atol=1e-12)
    # a subset taken from the wrong rows (an off-by-one in the position list) must not pass
    assert not np.allclose(sub, X[(pix + 1) % P].astype(np.float64) @ Wm.T + b, atol=1e-3)


@pytest.mark.parametrize("stride,pad", [((1, 1), (1, 1)), ((2, 2), (1, 1)), ((1, 2), (0, 1))])
def test_conv_int8_sampled_positions_against_brute_force(stride, pad):
    """The sampled-positions branch of the int8 convolution: positions across images, on the border (padding) and
    inside, against the pure-Python brute force of the same positions and against the full result."""
    O, I, H, K, bo, bi = 16, 32, 3, 3, 8, 8
    W, gamma, (rp, ci, pl) = sparse_setup(311, O, I, H, K, bo, bi, "i8")
    X = synth.uniform_int(313, (2, 6, 7, I), -127, 127).astype(np.int8)
    b = synth.uniform_int(314, (O,), -(1 << 15), 1 << 15).astype(np.int32)
    M, Nw = ref.out_hw(6, 7, H, K, stride[0], stride[1], pad[0], pad[1])
    P = 2 * M * Nw
    pix = np.array([P - 1, 0, Nw - 1, Nw, M * Nw, M * Nw + Nw + 1, 5, 5])
    want = brute_conv(ref.apply_mask(W, gamma, bo, bi), X, b, stride, pad)
    sub = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, stride, pad, pix=pix)
    assert sub.dtype == np.int32 and np.array_equal(sub, want[pix])
    assert np.array_equal(sub, ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, stride, pad)[pix])


def test_conv_f32_sampled_positions_against_scipy():
    O, I, H, K, bo, bi = 16, 16, 3, 3, 4, 16
    W, gamma, (rp, ci, pl) = sparse_setup(321, O, I, H, K, bo, bi, "f32")
    X = synth.normal(323, (2, 5, 6, I)).astype(np.float32)
    b = synth.normal(324, (O,), 0.1).astype(np.float32)
    want = scipy_dense_conv(ref.apply_mask(W, gamma, bo, bi), X, b, (1, 1), (1, 1))
    pix = np.array([59, 0, 5, 6, 30, 31])
    sub = ref.conv2d(W.shape, bo, bi, rp, ci, pl, X, b, (1, 1), (1, 1), pix=pix)
    assert np.allclose(sub, want[pix], rtol=1e-12, atol=1e-12)
