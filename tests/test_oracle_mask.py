"""Pins for the oracle's block scores, Gamma selection and compaction (CPU only)."""
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import ref
from paper_2407_09453_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def read_kv(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = int(v)
    return out


def test_block_index_example_from_paper():
    """Introduction, after Eq. (1): Gamma(W-bar, 4x16)[1,2] covers rows 4..7, columns 32..47."""
    g = read_kv("block_index_example.txt")
    bo, bi = g["bo"], g["bi"]
    O, I, H, K = 16, 64, 2, 3
    W = np.ones((O, H, K, I), dtype=np.float32)
    gamma = np.ones((O // bo, I // bi), dtype=np.uint8)
    gamma[g["l"], g["iota"]] = 0
    Wm = ref.apply_mask(W, gamma, bo, bi)
    zero = np.argwhere(Wm[:, 0, 0, :] == 0)
    assert zero[:, 0].min() == g["i_lo"] and zero[:, 0].max() == g["i_hi"]
    assert zero[:, 1].min() == g["j_lo"] and zero[:, 1].max() == g["j_hi"]
    assert len(zero) == bo * bi
    assert (Wm == 0).sum() == bo * bi * H * K          # the H x K taps hide inside the entry
    # scores: a single large weight inside the block makes that block the top score
    W2 = np.zeros((O, H, K, I), dtype=np.float32)
    W2[g["i_lo"] + 1, 1, 2, g["j_hi"]] = 3.0
    s = ref.scores(W2, bo, bi)
    assert np.unravel_index(np.argmax(s), s.shape) == (g["l"], g["iota"]) and s.max() == 9.0
    # compaction: keeping only that block returns exactly that slice of W
    Wr = synth.normal(5, (O, H, K, I)).astype(np.float32)
    only = np.zeros_like(gamma)
    only[g["l"], g["iota"]] = 1
    row_ptr, col_idx, payload = ref.compact(Wr, only, bo, bi)
    assert list(col_idx) == [g["iota"]] and list(row_ptr) == [0, 0, 1, 1, 1]
    want = Wr[g["i_lo"]:g["i_hi"] + 1, :, :, g["j_lo"]:g["j_hi"] + 1]
    assert np.array_equal(payload[0], want)


@pytest.mark.parametrize("bo,bi", [(8, 8), (4, 16), (16, 4)])
def test_scores_int8_closed_form_and_numpy(bo, bi):
    O, I, H, K = 32, 48, 3, 2
    W = np.full((O, H, K, I), 127, dtype=np.int8)
    s = ref.scores(W, bo, bi)
    assert s.dtype == np.int64 and np.all(s == 16129 * bo * H * K * bi)
    W = synth.uniform_int(7, (O, H, K, I), -127, 127).astype(np.int8)
    s = ref.scores(W, bo, bi)
    w64 = W.astype(np.int64).reshape(O // bo, bo, H, K, I // bi, bi)
    assert np.array_equal(s, (w64 * w64).sum(axis=(1, 2, 3, 5)))
    assert np.array_equal(ref.scores(W, bo, bi, ref.NORM_L1), np.abs(w64).sum(axis=(1, 2, 3, 5)))


def test_scores_float_within_one_ulp_of_exact_rational_sum():
    bo, bi, H, K = 8, 8, 3, 3
    W = synth.round_to_bf16(synth.normal(11, (16, H, K, 16), 0.05).astype(np.float32))
    s = ref.scores(W, bo, bi)
    for l in range(2):
        for j in range(2):
            blk = W[l * bo:(l + 1) * bo, :, :, j * bi:(j + 1) * bi].ravel()
            exact = sum(Fraction(float(v)) ** 2 for v in blk)
            got = Fraction(float(s[l, j]))
            assert abs(got - exact) <= Fraction(float(np.spacing(s[l, j]))) * 40   # 576 adds, tiny bound
            assert abs(float(got - exact)) <= 1e-13 * float(exact)
    # same numbers from numpy in another summation order agree to rounding
    w = W.astype(np.float64).reshape(2, bo, H, K, 2, bi)
    assert np.allclose(s, (w * w).sum(axis=(1, 2, 3, 5)), rtol=1e-13, atol=0)


def test_scores_float_summation_order_is_rows_then_blockrow():
    """The stated order (per output row over (h,k,c), then over rows) is observable in rounding."""
    bo, bi = 8, 8
    W = synth.normal(3, (8, 1, 1, 8), 1.0).astype(np.float32)
    s = ref.scores(W, bo, bi)[0, 0]
    w = W.astype(np.float64)[:, 0, 0, :]
    total = 0.0
    for r in range(8):
        pr = 0.0
        for c in range(8):
            pr += w[r, c] * w[r, c]
        total += pr
    assert s == total


def test_scores_l1_and_variance_against_numpy():
    bo, bi, H, K = 4, 16, 2, 2
    W = synth.normal(13, (8, H, K, 32)).astype(np.float32)
    w = W.astype(np.float64).reshape(2, bo, H, K, 2, bi)
    assert np.allclose(ref.scores(W, bo, bi, ref.NORM_L1), np.abs(w).sum(axis=(1, 2, 3, 5)), rtol=1e-13)
    blocks = w.transpose(0, 4, 1, 2, 3, 5).reshape(2, 2, -1)
    assert np.allclose(ref.scores(W, bo, bi, ref.NORM_VAR), blocks.var(axis=2), rtol=1e-12)


@pytest.mark.parametrize("scope", [ref.SCOPE_LAYER, ref.SCOPE_ROW])
def test_mask_counts_eq2_and_order(scope):
    NBo, NBi = 12, 20
    s = synth.normal(17, (NBo, NBi)) ** 2
    n_zero = 100 if scope == ref.SCOPE_LAYER else 7
    g = ref.mask(s, n_zero, scope)
    assert set(np.unique(g)) <= {0, 1}
    if scope == ref.SCOPE_LAYER:
        assert int((g == 0).sum()) == n_zero                       # Eq. (2): exact count of zeros
        assert s[g == 0].max() <= s[g == 1].min()
        order = np.lexsort((np.arange(s.size), s.ravel()))         # numpy's own sort as the pin
        want = np.ones(s.size, np.uint8)
        want[order[:n_zero]] = 0
        assert np.array_equal(g.ravel(), want)
    else:
        assert np.all((g == 0).sum(axis=1) == n_zero)              # Eq. (2) for every row of Gamma
        for l in range(NBo):
            assert s[l][g[l] == 0].max() <= s[l][g[l] == 1].min()


def test_mask_ties_by_index_and_extremes():
    s = np.ones((4, 8), dtype=np.float64)
    g = ref.mask(s, 13)
    assert np.array_equal(g.ravel(), np.r_[np.zeros(13, np.uint8), np.ones(19, np.uint8)])
    si = np.array([[5, 3, 5, 3, 9, 3, 5, 0]], dtype=np.int64)
    assert list(ref.mask(si, 3).ravel()) == [1, 0, 1, 0, 1, 1, 1, 0]       # 0, then the first two 3s
    assert list(ref.mask(si, 5).ravel()) == [0, 0, 1, 0, 1, 0, 1, 0]       # + third 3, first 5
    assert ref.mask(si, 0).all() and not ref.mask(si, 8).any()


def test_mask_planted_small_blocks_are_the_ones_zeroed():
    bo = bi = 8
    O, I, H, K = 64, 64, 3, 3
    W = synth.normal(19, (O, H, K, I)).astype(np.float32)
    planted = synth.shuffled(23, 64)[:20]
    for b in planted:
        l, j = divmod(int(b), 8)
        W[l * 8:(l + 1) * 8, :, :, j * 8:(j + 1) * 8] *= 1e-3
    g = ref.mask(ref.scores(W, bo, bi), 20)
    assert sorted(np.flatnonzero(g.ravel() == 0)) == sorted(int(b) for b in planted)


@pytest.mark.parametrize("bo,bi", [(8, 8), (4, 16), (16, 4)])
def test_compact_round_trip_and_invariants(bo, bi):
    O, I, H, K = 32, 64, 3, 2
    W = synth.uniform_int(29, (O, H, K, I), -127, 127).astype(np.int8)
    NBo, NBi = O // bo, I // bi
    gamma = synth.random_gamma(31, NBo, NBi, (NBo * NBi) // 2)
    row_ptr, col_idx, payload = ref.compact(W, gamma, bo, bi)
    nnz = NBo * NBi - (NBo * NBi) // 2
    assert row_ptr[0] == 0 and row_ptr[-1] == nnz == len(col_idx) and np.all(np.diff(row_ptr) >= 0)
    assert np.array_equal(np.diff(row_ptr), gamma.sum(axis=1))
    back = np.zeros_like(W)
    for l in range(NBo):
        cols = col_idx[row_ptr[l]:row_ptr[l + 1]]
        assert np.all(np.diff(cols) > 0)
        for n, j in zip(range(row_ptr[l], row_ptr[l + 1]), cols):
            back[l * bo:(l + 1) * bo, :, :, j * bi:(j + 1) * bi] = payload[n]
    assert np.array_equal(back, ref.apply_mask(W, gamma, bo, bi))          # bitwise round trip
    # Gamma == 1: a pure re-tiling; Gamma == 0: nothing stored
    rp, ci, pl = ref.compact(W, np.ones_like(gamma), bo, bi)
    assert len(ci) == NBo * NBi and np.array_equal(ci.reshape(NBo, NBi), np.tile(np.arange(NBi), (NBo, 1)))
    assert np.array_equal(pl.reshape(NBo, NBi, bo, H, K, bi).transpose(0, 2, 3, 4, 1, 5).reshape(W.shape), W)
    rp, ci, pl = ref.compact(W, np.zeros_like(gamma), bo, bi)
    assert len(ci) == 0 and not rp.any()
