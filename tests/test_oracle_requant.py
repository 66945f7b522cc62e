"""Pins for the oracle's requantising epilogue (CPU only): hand-worked values, an exact rational restatement, a floating
point restatement, and the properties that a wrong rounding mode, sign handling or saturation would break."""
import os
from fractions import Fraction

import numpy as np

from oracle import ref
from paper_2407_09453_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "requant_examples.txt")


def test_hand_worked_examples():
    rows = [tuple(int(t) for t in ln.split()) for ln in open(GOLD) if ln.strip() and not ln.startswith("#")]
    assert len(rows) >= 30
    for v, s, want in rows:
        got = int(ref.requant_i8(np.array([[v]], dtype=np.int32), np.array([s], dtype=np.int32))[0, 0])
        assert got == want, (v, s, got, want)


def exact_round_half_away(v: int, s: int) -> int:
    q = Fraction(v, 1 << s)
    n = int(abs(q) + Fraction(1, 2))            # floor(|q| + 1/2)
    n = -n if q < 0 else n
    return max(-128, min(127, n))


def test_against_exact_rationals_and_float64():
    O = 24
    shift = synth.uniform_int(501, (O,), 0, 31).astype(np.int32)
    shift[:4] = [0, 1, 31, 8]
    y = synth.uniform_int(502, (64, O), -(1 << 31), (1 << 31) - 1).astype(np.int64)
    y[1] = (synth.uniform_int(503, (O,), -300, 300)) << shift          # values near the int8 range after the shift
    y[2] = y[1] + (np.int64(1) << np.maximum(shift - 1, 0))             # exact halves
    y[3] = y[1] - (np.int64(1) << np.maximum(shift - 1, 0))
    y = np.clip(y, -(1 << 31), (1 << 31) - 1).astype(np.int32)
    got = ref.requant_i8(y, shift)
    want = np.array([[exact_round_half_away(int(y[p, o]), int(shift[o])) for o in range(O)] for p in range(y.shape[0])])
    assert np.array_equal(got, want)
    # float64 restatement (|v| < 2^31 and a power-of-two divisor: every step is exact)
    f = y.astype(np.float64) / np.exp2(shift.astype(np.float64))
    fl = np.clip(np.sign(f) * np.floor(np.abs(f) + 0.5), -128, 127)
    assert np.array_equal(got, fl.astype(np.int8))
    # round half to even or half up (toward +infinity) differ on the planted halves
    assert not np.array_equal(fl, np.clip(np.rint(f), -128, 127))
    assert not np.array_equal(fl, np.clip(np.floor(f + 0.5), -128, 127))


def test_properties():
    shift = np.array([0, 3, 9], dtype=np.int32)
    v = np.arange(-70000, 70000, 7, dtype=np.int32)
    y = np.repeat(v[:, None], 3, axis=1)
    q = ref.requant_i8(y, shift).astype(np.int64)
    assert np.all(np.diff(q, axis=0) >= 0)                              # monotone in the value
    inside = np.abs(q) < 127
    assert np.array_equal(q[inside], -ref.requant_i8(-y, shift).astype(np.int64)[inside])    # odd, away from the rails
    assert q.min() == -128 and q.max() == 127
    err = np.abs(q[:, 1] * 8 - v)[np.abs(q[:, 1]) < 127]
    assert err.max() <= 4                                              # within half a step of the scaled value
    bad = np.array([32], dtype=np.int32)
    try:
        ref.requant_i8(np.zeros((1, 1), dtype=np.int32), bad)
        assert False
    except RuntimeError:
        pass
