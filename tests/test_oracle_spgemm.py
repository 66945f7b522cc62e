"""Pins for the oracle's block-sparse x block-sparse product and relative index (CPU only)."""
import numpy as np
import pytest

from oracle import ref
from paper_2407_09453_b200 import synth


def compact_matrix(seed, rows, cols, kb, frac_zero):
    W = synth.normal(seed, (rows, 1, 1, cols)).astype(np.float32)
    gamma = synth.random_gamma(seed + 1, rows // kb, cols // kb, int(round(frac_zero * (rows // kb) * (cols // kb))))
    return W, gamma, ref.compact(W, gamma, kb, kb)


@pytest.mark.parametrize("kb", [8, 4, 16])
@pytest.mark.parametrize("fa,fb", [(0.5, 0.5), (0.0, 0.75), (0.9, 0.1)])
def test_spgemm_equals_dense_product_of_masked_matrices(kb, fa, fb):
    """The plain definition: C = (Gamma . A)(Omega . B)^t as a dense numpy product."""
    A, ga, ca = compact_matrix(601, 6 * kb, 10 * kb, kb, fa)
    B, gb, cb = compact_matrix(611, 5 * kb, 10 * kb, kb, fb)
    Cm = ref.spgemm(kb, ca, cb)
    Am = ref.apply_mask(A, ga, kb, kb)[:, 0, 0, :].astype(np.float64)
    Bm = ref.apply_mask(B, gb, kb, kb)[:, 0, 0, :].astype(np.float64)
    assert np.allclose(Cm, Am @ Bm.T, rtol=1e-12, atol=1e-12)
    if 0 < fa < 1:          # dropping the masks, or forgetting the transpose of B, must show
        assert not np.allclose(Cm, A[:, 0, 0, :].astype(np.float64) @ B[:, 0, 0, :].astype(np.float64).T, atol=1e-3)


def test_paper_two_by_two_example_with_a_sparse_second_operand():
    """The matrix example of Section "Block Sparsity in a Matrix": C = A [[0, B1], [B2, 0]] gives C0 = A1 B2, C1 = A0 B1,
    C2 = A3 B2, C3 = A2 B1.  Here the second operand is passed as rows of its transpose: row 0 of B^t holds B2^t at
    column 1, row 1 holds B1^t at column 0."""
    kb = 8
    A = synth.normal(621, (2 * kb, 2 * kb)).astype(np.float32)
    B1 = synth.normal(622, (kb, kb)).astype(np.float32)
    B2 = synth.normal(623, (kb, kb)).astype(np.float32)
    a = (np.array([0, 2, 4]), np.array([0, 1, 0, 1]),
         np.stack([A[:kb, :kb], A[:kb, kb:], A[kb:, :kb], A[kb:, kb:]]))
    bt = (np.array([0, 1, 2]), np.array([1, 0]), np.stack([B2.T, B1.T]))
    Cm = ref.spgemm(kb, a, bt)
    A0, A1, A2, A3 = [x.astype(np.float64) for x in (A[:kb, :kb], A[:kb, kb:], A[kb:, :kb], A[kb:, kb:])]
    want = np.block([[A1 @ B2, A0 @ B1], [A3 @ B2, A2 @ B1]])
    assert np.allclose(Cm, want, rtol=1e-12, atol=1e-12)


def test_spgemm_rows_without_common_columns_give_zero_blocks():
    kb = 8
    eye = np.eye(kb, dtype=np.float32)
    a = (np.array([0, 2, 2]), np.array([0, 3]), np.stack([eye, 2 * eye]))
    b = (np.array([0, 1, 3]), np.array([1, 0, 3]), np.stack([eye, 3 * eye, 5 * eye]))
    Cm = ref.spgemm(kb, a, b)
    want = np.zeros((2 * kb, 2 * kb))
    want[:kb, kb:] = (1 * 3 + 2 * 5) * np.eye(kb)          # row 0 of A meets row 1 of B at columns 0 and 3
    assert np.array_equal(Cm, want)


def test_relative_index_round_trip_and_values():
    row_ptr = np.array([0, 3, 3, 5, 6], dtype=np.int32)
    col = np.array([2, 5, 6, 0, 9, 4], dtype=np.int32)
    rel = ref.index_to_relative(row_ptr, col)
    assert rel.tolist() == [2, 3, 1, 0, 9, 4]               # worked by hand: first of a row absolute, then distances
    assert np.array_equal(ref.index_from_relative(row_ptr, rel), col)
    W, gamma, (rp, ci, pl) = compact_matrix(631, 64, 256, 8, 0.6)
    rel = ref.index_to_relative(rp, ci)
    assert np.array_equal(ref.index_from_relative(rp, rel), ci)
    for l in range(len(rp) - 1):                            # against numpy: diff within a row, cumsum back
        seg = ci[rp[l]:rp[l + 1]]
        if seg.size:
            assert np.array_equal(rel[rp[l]:rp[l + 1]], np.r_[seg[0], np.diff(seg)])
            assert np.all(rel[rp[l] + 1:rp[l + 1]] >= 1)
